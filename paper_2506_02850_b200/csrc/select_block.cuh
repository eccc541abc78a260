// Exact multi-class top-k by ONE CTA of 1024 threads, for problems whose keys fit its
// shared memory (up to about 30 K items).  Used by the class-wise top-k of the pruning
// levels, the K/V lists and the per-event key-token selection; select.cuh has the cluster
// version for larger problems.  That one spends most of its time in cluster barriers;
// here a step costs a __syncthreads, and what is left is the instruction count of the
// sweeps over the items, which one SM has to execute alone -- so the sweeps handle four
// items per thread with 16-byte shared-memory accesses and a few instructions per item.
//
// Every item gets a 64-bit key (score key << 32 | ~index): unique, and larger <=> ranks
// higher (higher score, lower index on equal scores).  A pass cuts the current key range
// of a class into NB buckets, histograms the class's items in the range, and a warp finds
// the bucket that holds the n-th best (lane block sums, then the 32-bucket chunk inside
// the block).  If that bucket has at most kBsCand items they are collected and the n-th
// best among them is found by counting, for each, how many outrank it: the threshold is
// then exact, ties included.  Otherwise the range narrows to the bucket and the pass
// repeats; unique keys guarantee that this ends.  In the first pass every class has the
// same range [min, max] of the score keys, so its two sweeps work on the 32-bit keys;
// typical inputs need no other pass.  The kept items are marked in a bit mask (one
// sweep; the eight lanes that share a word combine their bits by shuffles) and counted
// per 32-item word; the caller writes them out in order.
#pragma once

#include "common.cuh"

namespace metok {

constexpr int kBsThreads = 1024;
constexpr int kBsCand = 128;

struct BlockSelSmem {
    unsigned long long lo[METOK_MAX_GROUPS], hi[METOK_MAX_GROUPS];   // key range of the search
    unsigned long long thr[METOK_MAX_GROUPS];                        // kept: key >= thr (mode 2)
    int shift[METOK_MAX_GROUPS];                                     // bucket width = 1 << shift
    int need[METOK_MAX_GROUPS];                                      // items still to take inside [lo, hi]
    int cand_n[METOK_MAX_GROUPS];
    int first_bucket[METOK_MAX_GROUPS];                              // first pass: bucket to collect, or -1
    unsigned char state[METOK_MAX_GROUPS];                           // 0 done, 1 searching, 2 collecting candidates
    unsigned char mode[METOK_MAX_GROUPS];                            // 0 keep none, 1 keep all, 2 threshold
    uint32_t red_min[32], red_max[32];
    int warp_tot[32];
    int busy;
};

struct BlockSelLayout {
    int nb_log2;
    size_t hist_off, cand_off, keys_off, cls_off, bytes;
    bool fits;
};

inline BlockSelLayout block_sel_layout(int G, long long n_items, long long S) {
    BlockSelLayout L;
    L.nb_log2 = G <= 8 ? 11 : G <= 16 ? 10 : G <= 32 ? 9 : 8;
    L.hist_off = 0;                                          // later the position mask and the word offsets
    const size_t hist_words = (size_t)G << L.nb_log2;
    L.cand_off = hist_words * sizeof(uint32_t);
    L.keys_off = L.cand_off + (size_t)G * kBsCand * sizeof(unsigned long long);
    const size_t n4 = (size_t)((n_items + 3) & ~3LL);
    L.cls_off = L.keys_off + n4 * sizeof(uint32_t);
    L.bytes = L.cls_off + n4;
    (void)S;
    L.fits = L.bytes <= (size_t)200 * 1024 && 2 * (size_t)((n_items + 31) / 32) <= hist_words;
    return L;
}

__device__ __forceinline__ int range_shift64(unsigned long long lo, unsigned long long hi, int nb_log2) {
    const unsigned long long width = hi - lo;
    const int bits = width ? 64 - __clzll((long long)width) : 0;
    return bits > nb_log2 ? bits - nb_log2 : 0;
}

__device__ __forceinline__ unsigned long long item_key64(uint32_t key, int i) {
    return ((unsigned long long)key << 32) | (unsigned long long)(~(uint32_t)i);
}

// One warp per live class: the bucket that holds the need-th best counted from the top, then
// either "collect its items" (state 2) or "search inside it" (state stays 1, sm.busy set).
__device__ inline void block_sel_walk(BlockSelSmem& sm, const uint32_t* hist, int G, int nb_log2, bool first,
                               const int* __restrict__ budgets) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int nwarps = kBsThreads / 32;
    const int NB = 1 << nb_log2;
    for (int g = warp; g < G; g += nwarps) {
        if (sm.state[g] != 1) continue;
        const uint32_t* h = hist + g * NB;
        const int BL = NB >> 5;                             // buckets per lane block (8 .. 64); lane 0 has the top block
        const int top = NB - lane * BL;                     // this lane's block is [top - BL, top)
        int t = 0;
        for (int i = 0; i < BL; ++i) t += (int)h[top - BL + ((i + lane) & (BL - 1))];   // rotated start: no bank conflicts
        int incl = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        int need = sm.need[g];
        if (first) {
            int b = budgets[g];
            b = b < total ? b : total;                      // a budget above the population keeps everything
            if (b <= 0 || b >= total) {
                if (lane == 0) { sm.mode[g] = b <= 0 ? 0 : 1; sm.state[g] = 0; }
                continue;
            }
            need = b;
        }
        const unsigned hit = __ballot_sync(0xFFFFFFFFu, (incl - t) < need && need <= incl);
        const int hl = __ffs(hit) - 1;                      // exactly one lane
        const int above = __shfl_sync(0xFFFFFFFFu, incl - t, hl);
        const int btop = NB - hl * BL;                      // the block [btop - BL, btop), in chunks of 32 from the top
        int cum = above, bucket = -1, hb = 0;
        for (int c0 = 0; c0 < BL && bucket < 0; c0 += 32) {
            const int v = (c0 + lane < BL) ? (int)h[btop - 1 - c0 - lane] : 0;
            int inc2 = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int w = __shfl_up_sync(0xFFFFFFFFu, inc2, o);
                if (lane >= o) inc2 += w;
            }
            const unsigned hit2 = __ballot_sync(0xFFFFFFFFu, cum + inc2 - v < need && need <= cum + inc2);
            if (hit2) {
                const int l2 = __ffs(hit2) - 1;
                bucket = btop - 1 - c0 - l2;
                hb = __shfl_sync(0xFFFFFFFFu, v, l2);
                cum += __shfl_sync(0xFFFFFFFFu, inc2 - v, l2);
            } else {
                cum += __shfl_sync(0xFFFFFFFFu, inc2, 31);
            }
        }
        if (lane == 0) {
            const int sh = sm.shift[g];
            const unsigned long long lo = sm.lo[g], hi = sm.hi[g];
            const unsigned long long new_lo = lo + ((unsigned long long)bucket << sh);
            const unsigned long long span = sh ? ((1ull << sh) - 1ull) : 0ull;
            const unsigned long long new_hi = (hi - new_lo) < span ? hi : new_lo + span;
            sm.lo[g] = new_lo;
            sm.hi[g] = new_hi;
            sm.need[g] = need - cum;                        // items to take inside the bucket
            if (hb <= kBsCand) {
                sm.state[g] = 2;
                sm.first_bucket[g] = bucket;
            } else {
                sm.shift[g] = range_shift64(new_lo, new_hi, nb_log2);
                sm.busy = 1;
            }
        }
    }
}

// Classes in state 2: the need-th best of the collected items, by counting.
__device__ inline void block_sel_resolve(BlockSelSmem& sm, const unsigned long long* cand, int G) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int nwarps = kBsThreads / 32;
    for (int g = warp; g < G; g += nwarps) {
        if (sm.state[g] != 2) continue;
        const int n = sm.cand_n[g], need = sm.need[g];
        const unsigned long long* c_g = cand + g * kBsCand;
        for (int i = lane; i < n; i += 32) {
            const unsigned long long c = c_g[i];
            int above = 0;
            for (int j = 0; j < n; ++j) above += c_g[j] > c;
            if (above == need - 1) { sm.thr[g] = c; sm.mode[g] = 2; }
        }
        __syncwarp();
        if (lane == 0) { sm.state[g] = 0; sm.first_bucket[g] = -1; }
    }
}

// Everything up to the ordered compaction: after the call mask[w] has one bit per item (kept or
// not), woff[w] the number of kept items before word w, and `kept` is their total.
// `sc` / `token_group` (may be null: one class) are the n items' scores and classes, `budgets`
// the G class budgets.  The keys are no longer needed afterwards: their memory is free.
struct BlockSelView {
    uint32_t* mask;
    int* woff;
    uint32_t* keys;
    int kept;
};

// kOne: a single class and no class array (token_group is null): the class bytes are neither
// loaded, stored nor read back.
template <bool kOne>
__device__ __forceinline__ BlockSelView block_sel_run(BlockSelSmem& sm, unsigned char* sel_dyn, const BlockSelLayout& lay,
                                                      const float* __restrict__ sc,
                                                      const int32_t* __restrict__ token_group, int n_vis, int G,
                                                      const int* __restrict__ budgets) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nb_log2 = lay.nb_log2, NB = 1 << nb_log2;
    uint32_t* hist = reinterpret_cast<uint32_t*>(sel_dyn + lay.hist_off);
    unsigned long long* cand = reinterpret_cast<unsigned long long*>(sel_dyn + lay.cand_off);
    uint32_t* keys = reinterpret_cast<uint32_t*>(sel_dyn + lay.keys_off);
    unsigned char* cls = sel_dyn + lay.cls_off;
    const int n4 = (n_vis + 3) >> 2;                         // items are handled four at a time
    // the class bytes of quad q (255 = takes no part) and the class of item j
    auto cls4 = [&](int q) -> uint32_t {
        if (!kOne) return reinterpret_cast<const uint32_t*>(cls)[q];
        const int left = n_vis - q * 4;                      // items of the quad that exist
        return left >= 4 ? 0u : 0xFFFFFFFFu << (8 * left);
    };
    auto cls1 = [&](int j) -> int { return kOne ? 0 : (int)cls[j]; };

    // sweep 1: the items, once: keys and classes into shared memory, and the key range
    for (int b = tid; b < G * NB; b += kBsThreads) hist[b] = 0u;
    uint32_t mn = 0xFFFFFFFFu, mx = 0u;
    const bool vec = (reinterpret_cast<uintptr_t>(sc) & 15) == 0 &&
                     (!token_group || (reinterpret_cast<uintptr_t>(token_group) & 15) == 0);
    constexpr int kLd = 6;                                   // quads whose loads are in flight together
    for (int q0 = tid; q0 < n4; q0 += kBsThreads * kLd) {
        float v[kLd][4];
        int g[kLd][4];
#pragma unroll
        for (int w = 0; w < kLd; ++w) {
            const int q = q0 + w * kBsThreads;
            if (q < n4) {
                if (vec && q * 4 + 3 < n_vis) {
                    const float4 f = *reinterpret_cast<const float4*>(sc + q * 4);
                    v[w][0] = f.x; v[w][1] = f.y; v[w][2] = f.z; v[w][3] = f.w;
                    if (!kOne && token_group) {
                        const int4 t = *reinterpret_cast<const int4*>(token_group + q * 4);
                        g[w][0] = t.x; g[w][1] = t.y; g[w][2] = t.z; g[w][3] = t.w;
                    } else {
                        g[w][0] = g[w][1] = g[w][2] = g[w][3] = 0;
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int j = q * 4 + u;
                        v[w][u] = j < n_vis ? sc[j] : 0.f;
                        g[w][u] = j < n_vis ? (!kOne && token_group ? token_group[j] : 0) : -1;
                    }
                }
            }
        }
#pragma unroll
        for (int w = 0; w < kLd; ++w) {
            const int q = q0 + w * kBsThreads;
            if (q < n4) {
                uint32_t k4[4], c4 = 0u;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    k4[u] = float_key(v[w][u]);
                    const bool in = g[w][u] >= 0 && g[w][u] < G;
                    c4 |= (in ? (uint32_t)g[w][u] : 255u) << (8 * u);
                    if (in) {
                        mn = k4[u] < mn ? k4[u] : mn;
                        mx = k4[u] > mx ? k4[u] : mx;
                    }
                }
                reinterpret_cast<uint4*>(keys)[q] = make_uint4(k4[0], k4[1], k4[2], k4[3]);
                if (!kOne) reinterpret_cast<uint32_t*>(cls)[q] = c4;
            }
        }
    }
    mn = __reduce_min_sync(0xFFFFFFFFu, mn);
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    if (lane == 0) { sm.red_min[warp] = mn; sm.red_max[warp] = mx; }
    __syncthreads();
    mn = sm.red_min[lane];
    mx = sm.red_max[lane];
    mn = __reduce_min_sync(0xFFFFFFFFu, mn);
    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
    const bool empty = mn > mx;                              // no item takes part at all
    const int sh0 = empty ? 0 : ((mx - mn) ? max(0, 32 - __clz(mx - mn) - nb_log2) : 0);
    for (int g = tid; g < G; g += kBsThreads) {
        sm.lo[g] = (unsigned long long)mn << 32;
        sm.hi[g] = ((unsigned long long)mx << 32) | 0xFFFFFFFFull;
        sm.shift[g] = sh0 + 32;
        sm.need[g] = 0;
        sm.cand_n[g] = 0;
        sm.first_bucket[g] = -1;
        sm.thr[g] = 0ull;
        sm.mode[g] = 0;
        sm.state[g] = empty ? 0 : 1;
    }
    if (tid == 0) sm.busy = 0;
    const int nwords = (n_vis + 31) >> 5;
    uint32_t* mask = hist;                                   // the mask takes the histograms' place when they are done
    int* woff = reinterpret_cast<int*>(hist) + nwords;
    bool fast = false;
    __syncthreads();
    if (!empty) {
        // first pass: every class has the range [mn, mx]; sweep 2 histograms bucket (key - mn) >> sh0
        for (int q = tid; q < n4; q += kBsThreads) {
            const uint4 k = reinterpret_cast<const uint4*>(keys)[q];
            const uint32_t c4 = cls4(q);
            const uint32_t k4[4] = {k.x, k.y, k.z, k.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t g = (c4 >> (8 * u)) & 255u;
                if (g != 255u) atomicAdd(&hist[(g << nb_log2) + ((k4[u] - mn) >> sh0)], 1u);
            }
        }
        __syncthreads();
        block_sel_walk(sm, hist, G, nb_log2, true, budgets);
        __syncthreads();
        if (!sm.busy) {
            // Every class is decided or has its cut inside a small bucket: ONE more sweep marks the
            // items above the bucket as kept and collects the items inside it; the few of those
            // that make the cut get their bits afterwards.  A class that keeps everything has the
            // bucket -1 (every item is above it), one that keeps nothing the largest int.
            fast = true;
            for (int g = tid; g < G; g += kBsThreads)
                if (sm.state[g] != 2) sm.first_bucket[g] = sm.mode[g] == 1 ? -1 : 0x7FFFFFFF;
            __syncthreads();
            for (int q0 = 0; q0 < n4; q0 += kBsThreads) {
                const int q = q0 + tid;
                uint32_t nib = 0u;
                if (q < n4) {
                    const uint4 k = reinterpret_cast<const uint4*>(keys)[q];
                    const uint32_t c4 = cls4(q);
                    const uint32_t k4[4] = {k.x, k.y, k.z, k.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t g = (c4 >> (8 * u)) & 255u;
                        if (g != 255u) {
                            const int b = (int)((k4[u] - mn) >> sh0), fb = sm.first_bucket[g];
                            nib |= (b > fb ? 1u : 0u) << u;
                            if (b == fb) cand[g * kBsCand + atomicAdd(&sm.cand_n[g], 1)] = item_key64(k4[u], q * 4 + u);
                        }
                    }
                }
                uint32_t word = nib << (4 * (lane & 7));
                word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
                word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
                word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
                if ((lane & 7) == 0 && (q >> 3) < nwords) mask[q >> 3] = word;   // over the histograms: they are done
            }
            __syncthreads();
            block_sel_resolve(sm, cand, G);
            __syncthreads();
            for (int idx = tid; idx < G * kBsCand; idx += kBsThreads) {
                const int g = idx / kBsCand, j = idx - g * kBsCand;
                if (j < sm.cand_n[g] && sm.mode[g] == 2 && cand[idx] >= sm.thr[g]) {
                    const uint32_t i = ~(uint32_t)(cand[idx] & 0xFFFFFFFFull);
                    atomicOr(&mask[i >> 5], 1u << (i & 31u));
                }
            }
        } else {
            // sweep 3: the items of the buckets to collect
            for (int q = tid; q < n4; q += kBsThreads) {
                const uint4 k = reinterpret_cast<const uint4*>(keys)[q];
                const uint32_t c4 = cls4(q);
                const uint32_t k4[4] = {k.x, k.y, k.z, k.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t g = (c4 >> (8 * u)) & 255u;
                    if (g != 255u && (int)((k4[u] - mn) >> sh0) == sm.first_bucket[g])
                        cand[g * kBsCand + atomicAdd(&sm.cand_n[g], 1)] = item_key64(k4[u], q * 4 + u);
                }
            }
            __syncthreads();
            block_sel_resolve(sm, cand, G);
            __syncthreads();
        }
    }
    if (!fast) {
    // classes whose first bucket held more than kBsCand items (many equal or near-equal scores)
    for (int pass = 1; pass < 16 && sm.busy; ++pass) {
        for (int b = tid; b < G * NB; b += kBsThreads) hist[b] = 0u;
        __syncthreads();
        if (tid == 0) sm.busy = 0;
        for (int j = tid; j < n_vis; j += kBsThreads) {
            const int g = cls1(j);
            if (g != 255 && sm.state[g] == 1) {
                const unsigned long long c = item_key64(keys[j], j);
                const unsigned long long lo = sm.lo[g];
                if (c >= lo && c <= sm.hi[g]) atomicAdd(&hist[g * NB + (int)((c - lo) >> sm.shift[g])], 1u);
            }
        }
        __syncthreads();
        block_sel_walk(sm, hist, G, nb_log2, false, budgets);
        __syncthreads();
        for (int j = tid; j < n_vis; j += kBsThreads) {
            const int g = cls1(j);
            if (g != 255 && sm.state[g] == 2) {
                const unsigned long long c = item_key64(keys[j], j);
                if (c >= sm.lo[g] && c <= sm.hi[g]) cand[g * kBsCand + atomicAdd(&sm.cand_n[g], 1)] = c;
            }
        }
        __syncthreads();
        block_sel_resolve(sm, cand, G);
        __syncthreads();
    }

    // one threshold per class covers all three modes: keep none = above every key, keep all = 0
    for (int g = tid; g < G; g += kBsThreads) {
        const int mode = sm.mode[g];
        if (mode != 2) sm.thr[g] = mode == 1 ? 0ull : 0xFFFFFFFFFFFFFFFFull;
    }
    // sweep 4: one bit per item (kept or not), 32 items per word.  A thread decides its four
    // items; the eight lanes that share a word combine their bits with three shuffles.
    __syncthreads();
    for (int q0 = 0; q0 < n4; q0 += kBsThreads) {
        const int q = q0 + tid;
        uint32_t nib = 0u;
        if (q < n4) {
            const uint4 k = reinterpret_cast<const uint4*>(keys)[q];
            const uint32_t c4 = cls4(q);
            const uint32_t k4[4] = {k.x, k.y, k.z, k.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t g = (c4 >> (8 * u)) & 255u;
                if (g != 255u) {
                    const uint2 t = *reinterpret_cast<const uint2*>(&sm.thr[g]);   // .x = ~index part, .y = score key
                    const bool f = k4[u] > t.y || (k4[u] == t.y && ~(uint32_t)(q * 4 + u) >= t.x);
                    nib |= (f ? 1u : 0u) << u;
                }
            }
        }
        uint32_t word = nib << (4 * (lane & 7));
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
        if ((lane & 7) == 0 && (q >> 3) < nwords) mask[q >> 3] = word;
    }
    }
    __syncthreads();
    // exclusive offsets of the words: a thread per word, the warps' totals scanned by warp 0
    int kept = 0;
    for (int w0 = 0; w0 < nwords; w0 += kBsThreads) {
        const int w = w0 + tid;
        const int cnt = w < nwords ? __popc(mask[w]) : 0;
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) sm.warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const int t = sm.warp_tot[lane];
            int ti = t;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, ti, o);
                if (lane >= o) ti += v;
            }
            sm.warp_tot[lane] = ti - t;                      // exclusive
            if (lane == 31) sm.busy = ti;                    // total of this round of words
        }
        __syncthreads();
        if (w < nwords) woff[w] = kept + sm.warp_tot[warp] + incl - cnt;
        kept += sm.busy;
        __syncthreads();
    }
    BlockSelView view;
    view.mask = mask;
    view.woff = woff;
    view.keys = keys;
    view.kept = kept;
    return view;
}

}  // namespace metok
