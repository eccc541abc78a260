// metok_kv_compact: per-layer keep lists (section 3.3 policy, top-k policy, or given)
// and the in-place, order-preserving gather of K and V rows.
//
// In-place safety.  Row i receives old row keep[i] with keep ascending, hence
// keep[i] >= i, and after the call only rows [0, n) matter (n = list length).
//
// Fast path.  A source row at or beyond n is never written by anybody, so it can be
// read at any time.  Only the first h rows of the list, h = #{i : keep[i] < n}, have
// their source inside the destination region.  Those h rows are first copied to a
// staging area in the workspace (one kernel), then every row is written from its
// source or from the staging area (a second kernel) -- no ordering inside either
// kernel, any number of CTAs per slab.  With a keep ratio r about r*n rows are staged.
//
// General path (h larger than the staging area: lists that keep most rows).  Rows are
// moved in rounds of consecutive destination rows; a round's sources all lie at or
// beyond the round's first destination row, so
//   * a round only has to finish READING before any of its rows are WRITTEN, and
//   * later rounds' sources are never touched by earlier rounds' writes, so the
//     next round can be prefetched before the current one is stored.
// One thread-block cluster owns one (layer, K|V, head) slab; the read->write
// ordering inside a round is a hardware cluster barrier (no spinning on memory).
#include <cooperative_groups.h>

#include "common.cuh"
#include "launchers.h"

namespace cg = cooperative_groups;

namespace metok {

constexpr int kKvCluster = 4;        // CTAs per slab
constexpr int kKvThreads = 256;
constexpr int kKvUnroll = 4;         // 16-byte chunks per thread per round
constexpr int kKvMaxLayersPerLaunch = 64;

struct KvPtrs {
    void* k[kKvMaxLayersPerLaunch];
    void* v[kKvMaxLayersPerLaunch];
};

// PAPER policy lists: layers below l1 keep everything, the others drop the visual span.
__global__ void __launch_bounds__(256)
kv_paper_lists_kernel(int S_cur, int vis_start, int n_vis, int l1, int32_t* __restrict__ keep_idx,
                      int32_t* __restrict__ keep_len, int32_t* __restrict__ new_len) {
    const int layer = blockIdx.x;
    int32_t* keep = keep_idx + (size_t)layer * S_cur;
    int n;
    if (layer < l1) {
        for (int i = threadIdx.x; i < S_cur; i += blockDim.x) keep[i] = i;
        n = S_cur;
    } else {
        for (int i = threadIdx.x; i < vis_start; i += blockDim.x) keep[i] = i;
        const int tail = S_cur - (vis_start + n_vis);
        for (int i = threadIdx.x; i < tail; i += blockDim.x) keep[vis_start + i] = vis_start + n_vis + i;
        n = vis_start + tail;
    }
    if (threadIdx.x == 0) { keep_len[layer] = n; new_len[layer] = n; }
}

// GIVEN policy: the caller's lists are checked before anything is indexed through them.  One CTA
// per layer reads only the list itself: 0 <= length <= S_cur, entries strictly ascending inside
// [0, S_cur).  valid[layer] says whether the layer may be compacted; a layer with a bad list is
// left untouched and reports S_cur rows.
__global__ void __launch_bounds__(256)
kv_check_lists_kernel(int S_cur, const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ keep_len,
                      int32_t* __restrict__ new_len, int32_t* __restrict__ valid) {
    __shared__ int s_bad;
    const int layer = blockIdx.x;
    const int n = keep_len[layer];
    if (threadIdx.x == 0) s_bad = (n < 0 || n > S_cur) ? 1 : 0;
    __syncthreads();
    if (!s_bad) {
        const int32_t* keep = keep_idx + (size_t)layer * S_cur;
        int bad = 0;
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int v = keep[i];
            const int prev = i > 0 ? keep[i - 1] : -1;
            bad |= (v <= prev) | (v >= S_cur);           // prev >= -1, so v > prev also gives v >= 0
        }
        if (bad) s_bad = 1;                               // same value from every writer
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        valid[layer] = s_bad ? 0 : 1;
        new_len[layer] = s_bad ? S_cur : n;
    }
}

// ---- fast path ------------------------------------------------------------------
constexpr int kKvFastThreads = 256;
constexpr int kKvFastUnroll = 8;          // 16-byte chunks in flight per thread
constexpr int kKvStageSplit = 2;          // CTAs per slab in the staging kernel
constexpr int kKvCopySplit = 4;           // CTAs per slab in the copy kernel
constexpr size_t kKvStageBudget = (size_t)128 << 20;   // bytes of workspace the staging area may take

// First index of the ascending list keep[0..n) whose value is >= n; whole warp, 32-ary search.
__device__ __forceinline__ int warp_lower_bound(const int32_t* __restrict__ keep, int n, int lane) {
    int lo = 0, hi = n;                                   // answer in [lo, hi]
    while (hi > lo) {
        const int step = (hi - lo + 31) / 32;
        const int idx = lo + lane * step;
        const bool ge = idx < hi ? keep[idx] >= n : true;
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, ge);
        const int f = bal ? __ffs(bal) - 1 : 32;          // first probe that is >= n; 32: none was
        const int new_hi = f < 32 ? min(hi, lo + f * step) : hi;   // keep[new_hi] >= n (or new_hi == hi)
        const int new_lo = f > 0 ? lo + (f - 1) * step + 1 : lo;   // the probe before it was < n
        hi = new_hi;
        lo = new_lo;
    }
    return lo;
}

struct SlabId { int ll, which, head; };
__device__ __forceinline__ SlabId slab_of(int slab, int Hkv) {
    SlabId s;
    s.head = slab % Hkv;
    s.which = (slab / Hkv) & 1;
    s.ll = slab / (2 * Hkv);
    return s;
}

// Copies the rows whose source lies inside the destination region to the staging area and
// records h per layer (-1: too many for the staging area, the general path takes the layer).
__global__ void __launch_bounds__(kKvFastThreads)
kv_stage_kernel(KvPtrs ptrs, int layer0, int Hkv, int S_cap, int S_cur, int row_chunks,
                const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ keep_len, int stage_rows,
                int32_t* __restrict__ haz, uint4* __restrict__ stage, const int32_t* __restrict__ valid,
                int n_layers, int32_t* __restrict__ status) {
    grid_dep_wait();
    __shared__ int s_h;
    const SlabId id = slab_of(blockIdx.y, Hkv);
    const int layer = layer0 + id.ll;
    const bool lead = blockIdx.x == 0 && id.which == 0 && id.head == 0 && threadIdx.x == 0;   // one thread per layer
    // the call's status word: a rejected list (GIVEN policy) is an invalid argument
    if (layer0 == 0 && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        int st = METOK_OK;
        if (valid)
            for (int l = 0; l < n_layers; ++l)
                if (!valid[l]) st = METOK_ERR_INVALID_ARG;
        *status = st;
    }
    if (valid && !valid[layer]) {                          // nothing is indexed through a rejected list
        if (lead) haz[layer] = -2;
        return;
    }
    const int32_t* keep = keep_idx + (size_t)layer * S_cur;
    const int n = keep_len[layer];
    if (threadIdx.x < 32) {
        const int h = (n > 0 && n < S_cur) ? warp_lower_bound(keep, n, threadIdx.x) : 0;
        if (threadIdx.x == 0) s_h = h;
    }
    __syncthreads();
    const int h = s_h;
    const bool fast = h <= stage_rows;
    if (lead) haz[layer] = fast ? h : -1;
    if (!fast || h == 0) return;
    const uint4* base = reinterpret_cast<const uint4*>(id.which ? ptrs.v[id.ll] : ptrs.k[id.ll]) +
                        (size_t)id.head * S_cap * row_chunks;
    uint4* dst = stage + ((size_t)(layer * 2 + id.which) * Hkv + id.head) * (size_t)stage_rows * row_chunks;
    const int total = h * row_chunks;
    for (int gc = blockIdx.x * kKvFastThreads + threadIdx.x; gc < total; gc += kKvStageSplit * kKvFastThreads) {
        const int i = gc / row_chunks, c = gc - i * row_chunks;
        const int src = keep[i];
        if (src != i) dst[gc] = base[(size_t)src * row_chunks + c];
    }
}

// Every kept row from its source (at or beyond the new length: never written) or from the
// staging area.
__global__ void __launch_bounds__(kKvFastThreads)
kv_copy_kernel(KvPtrs ptrs, int layer0, int Hkv, int S_cap, int S_cur, int row_chunks,
               const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ keep_len, int stage_rows,
               const int32_t* __restrict__ haz, const uint4* __restrict__ stage) {
    grid_dep_wait();
    const SlabId id = slab_of(blockIdx.y, Hkv);
    const int layer = layer0 + id.ll;
    const int h = haz[layer];
    const int n = keep_len[layer];
    if (h < 0 || n >= S_cur) return;
    const int32_t* keep = keep_idx + (size_t)layer * S_cur;
    uint4* base = reinterpret_cast<uint4*>(id.which ? ptrs.v[id.ll] : ptrs.k[id.ll]) +
                  (size_t)id.head * S_cap * row_chunks;
    const uint4* stg = stage + ((size_t)(layer * 2 + id.which) * Hkv + id.head) * (size_t)stage_rows * row_chunks;
    const int total = n * row_chunks;
    constexpr int kStep = kKvFastThreads * kKvFastUnroll;
    for (int g0 = blockIdx.x * kStep; g0 < total; g0 += kKvCopySplit * kStep) {
        uint4 v[kKvFastUnroll];
        int at[kKvFastUnroll];                            // destination chunk, -1: nothing to store
#pragma unroll
        for (int u = 0; u < kKvFastUnroll; ++u) {
            const int gc = g0 + u * kKvFastThreads + threadIdx.x;
            at[u] = -1;
            if (gc < total) {
                const int i = gc / row_chunks, c = gc - i * row_chunks;
                const int src = keep[i];
                if (src != i) {
                    v[u] = i < h ? stg[gc] : base[(size_t)src * row_chunks + c];
                    at[u] = gc;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kKvFastUnroll; ++u)
            if (at[u] >= 0) base[at[u]] = v[u];
    }
}

// ---- general path -----------------------------------------------------------------
__global__ void __cluster_dims__(kKvCluster, 1, 1) __launch_bounds__(kKvThreads)
kv_gather_kernel(KvPtrs ptrs, int layer0, int Hkv, int S_cap, int S_cur, int row_chunks,
                 const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ keep_len,
                 const int32_t* __restrict__ haz) {
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int slab = blockIdx.x / kKvCluster;            // (layer_local, which, head)
    const int head = slab % Hkv;
    const int which = (slab / Hkv) & 1;
    const int ll = slab / (2 * Hkv);
    if (haz[layer0 + ll] != -1) return;                  // the fast path took this layer, or its list was rejected (uniform per cluster)
    uint4* base = reinterpret_cast<uint4*>(which ? ptrs.v[ll] : ptrs.k[ll]) + (size_t)head * S_cap * row_chunks;
    const int32_t* keep = keep_idx + (size_t)(layer0 + ll) * S_cur;
    const int n = keep_len[layer0 + ll];
    if (n >= S_cur) return;                              // nothing dropped: every row stays (uniform per cluster)
    const long long total = (long long)n * row_chunks;
    constexpr int kPerCta = kKvThreads * kKvUnroll;
    const long long per_round = (long long)kKvCluster * kPerCta;
    const int rounds = (int)((total + per_round - 1) / per_round);

    struct Buf {
        uint4 v[kKvUnroll];
        int row[kKvUnroll];      // -1: nothing to store
        int c[kKvUnroll];
    } b0, b1;

    auto issue = [&](int r, Buf& b) {
#pragma unroll
        for (int u = 0; u < kKvUnroll; ++u) {
            const long long gc = ((long long)r * kKvCluster + crank) * kPerCta + u * kKvThreads + threadIdx.x;
            b.row[u] = -1;
            if (gc < total) {
                const int i = (int)(gc / row_chunks);
                const int c = (int)(gc % row_chunks);
                const int src = keep[i];
                if (src != i) {
                    b.v[u] = base[(size_t)src * row_chunks + c];
                    b.row[u] = i;
                    b.c[u] = c;
                }
            }
        }
    };
    auto store = [&](const Buf& b) {
#pragma unroll
        for (int u = 0; u < kKvUnroll; ++u)
            if (b.row[u] >= 0) base[(size_t)b.row[u] * row_chunks + b.c[u]] = b.v[u];
    };
    if (rounds > 0) issue(0, b0);
    for (int r = 0; r < rounds; r += 2) {
        cluster.sync();                                  // every CTA has read round r
        if (r + 1 < rounds) issue(r + 1, b1);            // its sources lie beyond round r's rows
        store(b0);
        if (r + 1 < rounds) {
            cluster.sync();
            if (r + 2 < rounds) issue(r + 2, b0);
            store(b1);
        }
    }
}

struct KvWs {
    int32_t* status;          // device status word, first in the workspace
    int32_t* haz;
    int32_t* valid;           // GIVEN policy: per layer, whether the caller's list passed the check
    uint4* stage;
    int stage_rows;
};
static KvWs carve_kv(Carver& cv, int L, int Hkv, int S_cur, int row_chunks) {
    KvWs w;
    w.status = cv.take<int32_t>(64);
    w.haz = cv.take<int32_t>((size_t)L);
    w.valid = cv.take<int32_t>((size_t)L);
    const size_t per_row = (size_t)L * 2 * Hkv * row_chunks * sizeof(uint4);
    size_t rows = kKvStageBudget / per_row;
    if (rows > (size_t)S_cur) rows = (size_t)S_cur;
    w.stage_rows = (int)rows;
    w.stage = cv.take<uint4>((size_t)L * 2 * Hkv * rows * row_chunks);
    return w;
}

}  // namespace metok

using namespace metok;

extern "C" size_t metok_kv_compact_workspace_bytes(int dtype, int L, int Hkv, int S_cur, int dh, int policy,
                                                   int n_vis) {
    (void)policy; (void)n_vis;
    if (L < 1 || Hkv < 1 || S_cur < 1 || dh < 1) return 0;
    const int eb = dtype == METOK_F32 ? 4 : 2;
    const int row_chunks = (int)((long long)dh * eb / 16);
    if (row_chunks < 1) return 0;
    Carver cv(nullptr);
    carve_kv(cv, L, Hkv, S_cur, row_chunks);
    return cv.total();
}

extern "C" int metok_kv_compact(void* const* k_layers, void* const* v_layers, int dtype, int L, int Hkv, int S_cap,
                                int S_cur, int dh, int policy, int l1, double keep_ratio, int vis_start, int n_vis,
                                const float* scores, int scores_per_layer, int32_t* keep_idx, int32_t* keep_len,
                                int32_t* new_len, void* ws, size_t ws_bytes, void* stream) {
    if (!k_layers || !v_layers || !keep_idx || !keep_len || !new_len) return METOK_ERR_INVALID_ARG;
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (L < 1 || Hkv < 1 || S_cap < 1 || S_cur < 1 || S_cur > S_cap || dh < 1) return METOK_ERR_INVALID_ARG;
    if (policy != METOK_KV_PAPER && policy != METOK_KV_TOPK && policy != METOK_KV_GIVEN) return METOK_ERR_INVALID_ARG;
    if (vis_start < 0 || n_vis < 0 || (long long)vis_start + n_vis > S_cur) return METOK_ERR_INVALID_ARG;
    if (policy == METOK_KV_PAPER && l1 < 0) return METOK_ERR_INVALID_ARG;
    if (policy == METOK_KV_TOPK && (!scores || !(keep_ratio >= 0.0 && keep_ratio <= 1.0) || n_vis < 1))
        return METOK_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        if (!k_layers[l] || !v_layers[l] || !aligned16(k_layers[l]) || !aligned16(v_layers[l]))
            return METOK_ERR_INVALID_ARG;
    }
    const int eb = dtype == METOK_F32 ? 4 : 2;
    if (((long long)dh * eb) % 16 != 0) return METOK_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < metok_kv_compact_workspace_bytes(dtype, L, Hkv, S_cur, dh, policy, n_vis) || !aligned16(ws))
        return METOK_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int row_chunks = (int)((long long)dh * eb / 16);
    Carver cv(ws);
    const KvWs w = carve_kv(cv, L, Hkv, S_cur, row_chunks);

    // an upper bound, known on the host, of the length of every list that drops anything
    // (-1: not known); lists that keep all rows cause no copying
    int kept_bound = -1;
    if (policy == METOK_KV_PAPER) {
        kept_bound = S_cur - n_vis;
        {
            METOK_TIMED("kv_paper_lists_kernel", st);
            kv_paper_lists_kernel<<<L, 256, 0, st>>>(S_cur, vis_start, n_vis, l1, keep_idx, keep_len, new_len);
        }
        METOK_LAUNCH_CHECK();
    } else if (policy == METOK_KV_TOPK) {
        int32_t budget = ceilq(keep_ratio * (double)n_vis);
        if (budget > n_vis) budget = n_vis;
        // shared scores give the same list in every layer: select once, write it L times
        const int problems = scores_per_layer ? L : 1;
        const int rc = launch_class_topk(scores, scores_per_layer ? (size_t)n_vis : 0, nullptr, n_vis, 1, &budget,
                                         S_cur, vis_start, keep_idx, (size_t)S_cur, scores_per_layer ? 1 : L,
                                         keep_len, new_len, problems, st);
        if (rc != METOK_OK) return rc;
        kept_bound = budget + (S_cur - n_vis);
    } else {
        {
            METOK_TIMED("kv_check_lists_kernel", st);
            kv_check_lists_kernel<<<L, 256, 0, st>>>(S_cur, keep_idx, keep_len, new_len, w.valid);
        }
        METOK_LAUNCH_CHECK();
    }
    const int32_t* valid = policy == METOK_KV_GIVEN ? w.valid : nullptr;
    for (int l0 = 0; l0 < L; l0 += kKvMaxLayersPerLaunch) {
        const int nl = (L - l0) < kKvMaxLayersPerLaunch ? (L - l0) : kKvMaxLayersPerLaunch;
        KvPtrs ptrs;
        for (int l = 0; l < kKvMaxLayersPerLaunch; ++l) {
            ptrs.k[l] = l < nl ? k_layers[l0 + l] : nullptr;
            ptrs.v[l] = l < nl ? v_layers[l0 + l] : nullptr;
        }
        const int slabs = nl * 2 * Hkv;
        {
            METOK_TIMED("kv_stage_kernel", st);
            launch_chained(kv_stage_kernel, dim3(dim3(kKvStageSplit, slabs)), dim3(kKvFastThreads), 0, st, 
                ptrs, l0, Hkv, S_cap, S_cur, row_chunks, keep_idx, keep_len, w.stage_rows, w.haz, w.stage, valid, L,
                w.status);
        }
        METOK_LAUNCH_CHECK();
        {
            METOK_TIMED("kv_copy_kernel", st);
            launch_chained(kv_copy_kernel, dim3(dim3(kKvCopySplit, slabs)), dim3(kKvFastThreads), 0, st, 
                ptrs, l0, Hkv, S_cap, S_cur, row_chunks, keep_idx, keep_len, w.stage_rows, w.haz, w.stage);
        }
        METOK_LAUNCH_CHECK();
        // h <= list length: when every list is known to fit the staging area, no layer takes the general path
        if (kept_bound < 0 || kept_bound > w.stage_rows) {
            {
                METOK_TIMED("kv_gather_kernel", st);
                kv_gather_kernel<<<slabs * kKvCluster, kKvThreads, 0, st>>>(ptrs, l0, Hkv, S_cap, S_cur, row_chunks,
                                                                        keep_idx, keep_len, w.haz);
            }
            METOK_LAUNCH_CHECK();
        }
    }
    return METOK_OK;
}
