// Exact multi-class top-k selection and ordered stream compaction by one thread-block
// cluster (8 CTAs) per problem.  Used by the per-event key-token top-k, the
// event-weighted top-k of the prefill pruning step and the KV TOPK policy.
//
// Ordering: item i outranks item j when its score is larger, or equal with i < j.
//
// A problem is a row of positions [0, S); the positions [vis_start, vis_start + n) are
// scored items, every other position is always kept.  CTA r of the cluster owns a
// contiguous slice of positions and caches the keys and classes of its items in shared
// memory, so the global arrays are read once and the work of a sweep is spread over
// eight SMs.
//
// The n best of a class are found by narrowing a key range instead of sorting.
// Scores map to order-preserving 32-bit keys.  A pass cuts the current range [lo, hi]
// of a class into NB equal buckets and histograms the class's items that fall inside
// (shared-memory counters per CTA); CTA r then adds up, over the cluster's eight
// histograms, the r-th eighth of the buckets (distributed shared memory) and every CTA
// walks the eight slice totals and the one slice that holds the n-th best.  All CTAs
// read the same numbers and take the same decision, so nothing is broadcast.  The
// first range is the [min, max] of the keys present: real score distributions spread
// over many buckets and two or three passes reach a single key value; a pass stops
// early when every item of the kept bucket is taken anyway.  Only when equal scores
// straddle the cut does a second search run, over ~index among the items equal to the
// threshold (lower index wins).  Histogram and slice buffers alternate between passes,
// which leaves two cluster barriers per pass.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace metok {

namespace cg = cooperative_groups;

constexpr int kSelCluster = 8;
constexpr int kSelThreads = 1024;      // upper bound; small problems run with fewer (select_threads)
constexpr int kSelBatch = 8;           // loads in flight per thread

struct SelectSmem {
    // search state, identical in every CTA of the cluster
    uint32_t lo[METOK_MAX_GROUPS], hi[METOK_MAX_GROUPS];   // current key range of the search
    uint32_t thr[METOK_MAX_GROUPS];                        // kept: key > thr, or key == thr and ...
    uint32_t thr2[METOK_MAX_GROUPS];                       // ... (no tie split, or ~index >= thr2)
    int need[METOK_MAX_GROUPS];                            // items still to take inside [lo, hi]
    int shift[METOK_MAX_GROUPS];                           // bucket width = 1 << shift
    int taken[METOK_MAX_GROUPS];                           // clamped budget (what the class keeps)
    unsigned char live[METOK_MAX_GROUPS];                  // search still running
    unsigned char tie[METOK_MAX_GROUPS];                   // equal scores straddle the cut
    unsigned char mode[METOK_MAX_GROUPS];                  // 0 keep none, 1 keep all, 2 threshold
    // what the other CTAs of the cluster read from this one
    uint32_t x_min, x_max;                                 // key range of this CTA's items
    int x_cnt;                                             // positions this CTA keeps
    int slice_tot[2][METOK_MAX_GROUPS];                    // totals of this CTA's merged bucket slice
    // CTA-local scratch
    int warp_tot[32];
    uint32_t red_min[32], red_max[32];
    int pass_ctr;
};

// Dynamic shared memory of a selection kernel.
struct SelectLayout {
    int nb_log2;          // buckets per class and pass = 1 << nb_log2
    int cache_cap;        // items whose key/class a CTA can cache
    size_t hist_off, merged_off, keys_off, cls_off, bytes;
};

inline SelectLayout select_layout(int G, long long items_per_cta) {
    SelectLayout L;
    L.nb_log2 = G <= 4 ? 11 : G <= 8 ? 10 : G <= 16 ? 9 : 8;
    const size_t hist = ((size_t)G << L.nb_log2) * sizeof(uint32_t);
    L.hist_off = 0;
    L.merged_off = 2 * hist;
    L.keys_off = L.merged_off + 2 * hist / kSelCluster;
    const size_t room = (size_t)200 * 1024 - L.keys_off;
    long long cap = (long long)(room / 5) & ~15LL;
    if (items_per_cta < cap) cap = (items_per_cta + 15) & ~15LL;
    L.cache_cap = (int)cap;
    L.cls_off = L.keys_off + (size_t)L.cache_cap * 4;
    L.bytes = L.cls_off + (size_t)L.cache_cap;
    return L;
}

struct SelItem { int cls; uint32_t key; };

// Visits j = tid, tid + nthr, ... < m.  The loads of kSelBatch items are issued before
// the first of them is used.
template <typename LoadF, typename BodyF>
__device__ __forceinline__ void batched_items(int m, LoadF load, BodyF body) {
    const int nthr = blockDim.x;
    for (int base = threadIdx.x; base < m; base += nthr * kSelBatch) {
        SelItem it[kSelBatch];
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = base + u * nthr;
            if (j < m) it[u] = load(j);
        }
#pragma unroll
        for (int u = 0; u < kSelBatch; ++u) {
            const int j = base + u * nthr;
            if (j < m) body(j, it[u]);
        }
    }
}

__device__ __forceinline__ int range_shift(uint32_t lo, uint32_t hi, int nb_log2) {
    const uint32_t width = hi - lo;
    const int bits = width ? 32 - __clz(width) : 0;
    return bits > nb_log2 ? bits - nb_log2 : 0;
}

__device__ __forceinline__ bool is_selected(const SelectSmem& sm, int g, uint32_t key, int i) {
    const int mode = sm.mode[g];
    if (mode != 2) return mode == 1;
    const uint32_t t = sm.thr[g];
    if (key != t) return key > t;
    return !sm.tie[g] || ~(uint32_t)i >= sm.thr2[g];
}

// Everything a selection needs to know about this CTA's share of the problem.
struct SelectCtx {
    cg::cluster_group cl;
    int rank;                 // CTA rank in the cluster
    int G, nb_log2;
    int item_lo, m;           // this CTA's items are the global items [item_lo, item_lo + m)
    bool cached;
    uint32_t* hist;           // [2][G << nb_log2]
    uint32_t* merged;         // [2][(G << nb_log2) / kSelCluster]
    uint32_t* keys;           // [cache_cap]
    unsigned char* cls;       // [cache_cap], 255 = takes no part
    __device__ SelectCtx() : cl(cg::this_cluster()) {}
};

// Narrows the key range of every live class until it is decided.  get(j) -> class (or
// -1) and key of local item j among the candidates of this stage.  kIndexStage: the
// search runs over ~index among threshold-equal items and writes thr2; otherwise the
// first pass also yields the class populations, against which the budgets are clamped.
template <bool kIndexStage, typename GetF>
__device__ void select_refine(SelectCtx& cx, GetF get, const int* budget, SelectSmem& sm) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
    const int G = cx.G, NB = 1 << cx.nb_log2, SL = NB / kSelCluster;
    for (int pass = 0; pass < 40; ++pass) {
        int any_live = 0;
        for (int g = 0; g < G; ++g) any_live |= sm.live[g];
        if (!any_live) break;
        const int buf = sm.pass_ctr & 1;
        uint32_t* hist = cx.hist + (size_t)buf * G * NB;
        uint32_t* merged = cx.merged + (size_t)buf * G * SL;
        for (int b = tid; b < G * NB; b += nthr) hist[b] = 0u;
        __syncthreads();
        if (tid == 0) sm.pass_ctr += 1;
        batched_items(cx.m, get, [&](int, const SelItem& it) {
            const int g = it.cls;
            if (g >= 0 && sm.live[g]) {
                const uint32_t lo = sm.lo[g];
                if (it.key >= lo && it.key <= sm.hi[g]) atomicAdd(&hist[g * NB + (int)((it.key - lo) >> sm.shift[g])], 1u);
            }
        });
        cx.cl.sync();                                   // every CTA's histogram of this pass is complete
        // this CTA adds up its eighth of the buckets over the cluster
        for (int idx = tid; idx < G * SL; idx += nthr) {
            const int g = idx / SL, b = idx - g * SL;
            uint32_t* mine = &hist[g * NB + cx.rank * SL + b];
            uint32_t s = 0;
#pragma unroll
            for (int c = 0; c < kSelCluster; ++c) s += *cx.cl.map_shared_rank(mine, c);
            merged[idx] = s;
        }
        __syncthreads();
        for (int g = warp; g < G; g += nwarps) {
            int s = 0;
            for (int b = lane; b < SL; b += 32) s += (int)merged[g * SL + b];
            s = warp_sum_int(s);
            if (lane == 0) sm.slice_tot[buf][g] = s;
        }
        cx.cl.sync();                                   // merged slices and their totals are visible
        // one warp per class: walk the slices from the top, then the buckets of one slice
        const int c2 = SL >> 5;                         // buckets per lane inside a slice (SL >= 32)
        for (int g = warp; g < G; g += nwarps) {
            if (!sm.live[g]) continue;
            // lane l < 8 looks at slice 7 - l (highest keys first)
            int s = 0;
            if (lane < kSelCluster) s = *cx.cl.map_shared_rank(&sm.slice_tot[buf][g], kSelCluster - 1 - lane);
            int incl = s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += v;
            }
            const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
            int need = sm.need[g];
            if (!kIndexStage && pass == 0) {
                int b = budget[g];
                b = b < total ? b : total;              // a budget above the population keeps everything
                if (lane == 0) sm.taken[g] = b > 0 ? b : 0;
                if (b <= 0 || b >= total) {
                    if (lane == 0) { sm.mode[g] = b <= 0 ? 0 : 1; sm.live[g] = 0; }
                    continue;
                }
                need = b;
            }
            const unsigned hit = __ballot_sync(0xFFFFFFFFu, (incl - s) < need && need <= incl);
            const int hl = __ffs(hit) - 1;              // exactly one lane
            const int slice = kSelCluster - 1 - hl;
            const int above = __shfl_sync(0xFFFFFFFFu, incl - s, hl);   // items in higher slices
            const uint32_t* mslice = cx.cl.map_shared_rank(&merged[g * SL], slice);
            const int top = SL - lane * c2;             // this lane owns buckets [top - c2, top) of the slice
            int hv[8];                                  // c2 <= 8: one remote read per bucket, kept for the walk
            int t = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                hv[q] = q < c2 ? (int)mslice[top - 1 - q] : 0;
                t += hv[q];
            }
            int incl2 = t;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, incl2, o);
                if (lane >= o) incl2 += v;
            }
            const int need2 = need - above;
            const int excl2 = incl2 - t;
            if (excl2 < need2 && need2 <= incl2) {      // exactly one lane
                int cum = excl2, b = top - 1, hb = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (q < c2 && cum + hb < need2) {       // hb: bucket looked at last; move on while it falls short
                        cum += hb;
                        hb = hv[q];
                        b = top - 1 - q;
                    }
                }
                const int sh = sm.shift[g];
                const uint32_t lo = sm.lo[g], hi = sm.hi[g];
                const uint32_t new_lo = lo + ((uint32_t)(slice * SL + b) << sh);
                const uint32_t span = sh ? ((1u << sh) - 1u) : 0u;
                const uint32_t new_hi = new_lo + ((hi - new_lo) < span ? (hi - new_lo) : span);
                const int rem = need2 - cum;            // items to take inside the bucket
                if (hb == rem || sh == 0) {
                    if (kIndexStage) {
                        sm.thr2[g] = new_lo;
                    } else {
                        sm.thr[g] = new_lo;
                        sm.mode[g] = 2;
                        sm.tie[g] = hb != rem;          // a single key value holds more items than it may give
                        sm.need[g] = rem;
                    }
                    sm.live[g] = 0;
                } else {
                    sm.lo[g] = new_lo;
                    sm.hi[g] = new_hi;
                    sm.need[g] = rem;
                    sm.shift[g] = range_shift(new_lo, new_hi, cx.nb_log2);
                }
            }
        }
        __syncthreads();
    }
}

// Decides, for every class g in [0, G), which min(budget[g], population) items it keeps.
// cls(i) -> class in [0,G) or -1 (item takes no part); val(i) -> score; i is the global
// item index.  n = number of items of the whole problem.  `budget` is in shared memory.
// After the call, in every CTA: item i of class g is kept <=> is_selected(sm, g, key, i),
// and item_at(cx, j, cls, val) returns class and key of local item j.
template <typename ClsF, typename ValF>
__device__ __forceinline__ SelItem item_at(const SelectCtx& cx, int j, ClsF cls, ValF val) {
    if (cx.cached) {
        const int c = cx.cls[j];
        return SelItem{c == 255 ? -1 : c, cx.keys[j]};
    }
    return SelItem{cls(cx.item_lo + j), float_key(val(cx.item_lo + j))};
}

template <typename ClsF, typename ValF>
__device__ void cluster_select(SelectCtx& cx, int n, ClsF cls, ValF val, const int* budget, SelectSmem& sm) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
    const int G = cx.G;
    // load this CTA's items once: key range, and the cache
    uint32_t mn = 0xFFFFFFFFu, mx = 0u;
    batched_items(cx.m, [&](int j) { return SelItem{cls(cx.item_lo + j), float_key(val(cx.item_lo + j))}; },
                  [&](int j, const SelItem& it) {
                      if (cx.cached) {
                          cx.keys[j] = it.key;
                          cx.cls[j] = it.cls < 0 ? (unsigned char)255 : (unsigned char)it.cls;
                      }
                      if (it.cls >= 0) {
                          mn = it.key < mn ? it.key : mn;
                          mx = it.key > mx ? it.key : mx;
                      }
                  });
    mn = __reduce_min_sync(0xFFFFFFFFu, mn);
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    if (lane == 0) { sm.red_min[warp] = mn; sm.red_max[warp] = mx; }
    __syncthreads();
    if (warp == 0) {
        mn = lane < nwarps ? sm.red_min[lane] : 0xFFFFFFFFu;
        mx = lane < nwarps ? sm.red_max[lane] : 0u;
        mn = __reduce_min_sync(0xFFFFFFFFu, mn);
        mx = __reduce_max_sync(0xFFFFFFFFu, mx);
        if (lane == 0) { sm.x_min = mn; sm.x_max = mx; sm.pass_ctr = 0; }
    }
    cx.cl.sync();                                       // every CTA's key range is visible
    if (warp == 0) {
        mn = lane < kSelCluster ? *cx.cl.map_shared_rank(&sm.x_min, lane) : 0xFFFFFFFFu;
        mx = lane < kSelCluster ? *cx.cl.map_shared_rank(&sm.x_max, lane) : 0u;
        mn = __reduce_min_sync(0xFFFFFFFFu, mn);
        mx = __reduce_max_sync(0xFFFFFFFFu, mx);
        const bool empty = mn > mx;                     // no item takes part at all
        for (int g = lane; g < G; g += 32) {
            sm.lo[g] = mn;
            sm.hi[g] = mx;
            sm.shift[g] = empty ? 0 : range_shift(mn, mx, cx.nb_log2);
            sm.need[g] = 0;
            sm.taken[g] = 0;
            sm.thr[g] = 0u;
            sm.thr2[g] = 0u;
            sm.tie[g] = 0;
            sm.mode[g] = 0;
            sm.live[g] = empty ? 0 : 1;
        }
    }
    __syncthreads();
    select_refine<false>(cx, [&](int j) { return item_at(cx, j, cls, val); }, budget, sm);

    // equal scores on both sides of the cut: among the items equal to the threshold, the
    // sm.need[g] lowest indices are kept -- the same search over ~index
    int any_tie = 0;
    for (int g = 0; g < G; ++g) any_tie |= sm.tie[g];
    if (any_tie) {
        __syncthreads();
        for (int g = tid; g < G; g += nthr) {
            if (sm.tie[g]) {
                sm.lo[g] = ~(uint32_t)(n - 1);
                sm.hi[g] = 0xFFFFFFFFu;
                sm.shift[g] = range_shift(sm.lo[g], sm.hi[g], cx.nb_log2);
                sm.live[g] = 1;
            }
        }
        __syncthreads();
        select_refine<true>(cx, [&](int j) {
            const SelItem it = item_at(cx, j, cls, val);
            const bool c = it.cls >= 0 && sm.tie[it.cls] && it.key == sm.thr[it.cls];
            return SelItem{c ? it.cls : -1, ~(uint32_t)(cx.item_lo + j)};
        }, budget, sm);
    }
    __syncthreads();
}

// Ordered compaction over the cluster: emit(u, rank) for every flagged position u of this
// CTA's slice [p_lo, p_hi), rank = number of flagged positions before u in the whole
// problem.  Warps own contiguous ranges (counted first, written in a second sweep);
// flag(u) is evaluated twice and must be pure.  Returns the total over the cluster.
// Ends with a cluster barrier: no CTA leaves while another may still read its memory.
template <typename FlagF, typename EmitF>
__device__ int cluster_compact(SelectCtx& cx, int p_lo, int p_hi, FlagF flag, EmitF emit, SelectSmem& sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = blockDim.x >> 5;
    const int n = p_hi - p_lo;
    const int per_w = (((n + nwarps - 1) / nwarps) + 31) & ~31;
    const int lo = p_lo + (warp * per_w < n ? warp * per_w : n);
    const int hi = lo + per_w < p_hi ? lo + per_w : p_hi;
    constexpr int U = 4;                                // flags of 4 x 32 positions are fetched together
    int cnt = 0;
    for (int b = lo; b < hi; b += 32 * U) {
        bool f[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = b + u * 32 + lane;
            f[u] = i < hi && flag(i);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) cnt += __popc(__ballot_sync(0xFFFFFFFFu, f[u]));
    }
    if (lane == 0) sm.warp_tot[warp] = cnt;
    __syncthreads();
    int run = 0, mine = 0;
    for (int w = 0; w < nwarps; ++w) {
        const int c = sm.warp_tot[w];
        if (w < warp) run += c;
        mine += c;
    }
    if (tid == 0) sm.x_cnt = mine;
    cx.cl.sync();                                       // every CTA's count is visible
    int total = 0;
#pragma unroll
    for (int c = 0; c < kSelCluster; ++c) {
        const int v = *cx.cl.map_shared_rank(&sm.x_cnt, c);
        if (c < cx.rank) run += v;
        total += v;
    }
    for (int b = lo; b < hi; b += 32 * U) {
        bool f[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = b + u * 32 + lane;
            f[u] = i < hi && flag(i);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned bal = __ballot_sync(0xFFFFFFFFu, f[u]);
            if (f[u]) emit(b + u * 32 + lane, run + __popc(bal & ((1u << lane) - 1u)));
            run += __popc(bal);
        }
    }
    cx.cl.sync();
    return total;
}

// Slice of positions [0, S) that CTA `rank` owns: whole multiples of 32.
__device__ __forceinline__ void select_slice(int S, int rank, int* p_lo, int* p_hi) {
    const int per = (((S + kSelCluster - 1) / kSelCluster) + 31) & ~31;
    const int lo = rank * per < S ? rank * per : S;
    *p_lo = lo;
    *p_hi = lo + per < S ? lo + per : S;
}

// Threads per CTA: a sweep costs every warp its instructions whether or not it has items,
// so a CTA gets no more threads than about 8 items each.
inline int select_threads(long long items_per_cta) {
    return items_per_cta <= 2048 ? 256 : items_per_cta <= 4096 ? 512 : kSelThreads;
}

inline long long select_items_per_cta(long long S) {
    return ((((S + kSelCluster - 1) / kSelCluster) + 31) / 32) * 32;
}

}  // namespace metok
