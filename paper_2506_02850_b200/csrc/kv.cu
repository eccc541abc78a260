// metok_kv_compact: per-layer keep lists (section 3.3 policy, top-k policy, or given)
// and the in-place, order-preserving gather of K and V rows.
//
// In-place safety.  Row i receives old row keep[i] with keep ascending, hence
// keep[i] >= i.  Rows are moved in rounds of consecutive destination rows; a
// round's sources all lie at or beyond the round's first destination row, so
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

// One keep list serves every layer: rows 1..L-1 of keep_idx and the lengths are copies of row 0.
__global__ void __launch_bounds__(256)
kv_broadcast_list_kernel(int32_t* __restrict__ keep_idx, int S_cur, int32_t* __restrict__ keep_len,
                         int32_t* __restrict__ new_len) {
    const int layer = blockIdx.y + 1;
    const int n = keep_len[0];
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) keep_idx[(size_t)layer * S_cur + i] = keep_idx[i];
    if (i == 0) { keep_len[layer] = n; new_len[layer] = n; }
}

__global__ void copy_len_kernel(const int32_t* __restrict__ a, int32_t* __restrict__ b, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) b[i] = a[i];
}

__global__ void __cluster_dims__(kKvCluster, 1, 1) __launch_bounds__(kKvThreads)
kv_gather_kernel(KvPtrs ptrs, int layer0, int Hkv, int S_cap, int S_cur, int row_chunks,
                 const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ keep_len) {
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int slab = blockIdx.x / kKvCluster;            // (layer_local, which, head)
    const int head = slab % Hkv;
    const int which = (slab / Hkv) & 1;
    const int ll = slab / (2 * Hkv);
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

}  // namespace metok

using namespace metok;

extern "C" size_t metok_kv_compact_workspace_bytes(int dtype, int L, int Hkv, int S_cur, int dh, int policy,
                                                   int n_vis) {
    (void)dtype; (void)L; (void)Hkv; (void)S_cur; (void)dh; (void)policy; (void)n_vis;
    return 256;   // no scratch is needed today; a non-zero size keeps the calling convention uniform
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
    if (!ws || ws_bytes < metok_kv_compact_workspace_bytes(dtype, L, Hkv, S_cur, dh, policy, n_vis))
        return METOK_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    if (policy == METOK_KV_PAPER) {
        {
            METOK_TIMED("kv_paper_lists_kernel", st);
            kv_paper_lists_kernel<<<L, 256, 0, st>>>(S_cur, vis_start, n_vis, l1, keep_idx, keep_len, new_len);
        }
        METOK_LAUNCH_CHECK();
    } else if (policy == METOK_KV_TOPK) {
        int32_t budget = ceilq(keep_ratio * (double)n_vis);
        if (budget > n_vis) budget = n_vis;
        // shared scores give the same list in every layer: select once, then copy
        const int problems = scores_per_layer ? L : 1;
        const int rc = launch_class_topk(scores, scores_per_layer ? (size_t)n_vis : 0, nullptr, n_vis, 1, &budget,
                                         S_cur, vis_start, keep_idx, (size_t)S_cur, keep_len, new_len, problems, st);
        if (rc != METOK_OK) return rc;
        if (problems < L) {
            const int kept = budget + (S_cur - n_vis);
            {
                METOK_TIMED("kv_broadcast_list_kernel", st);
                kv_broadcast_list_kernel<<<dim3(ceil_div(kept > 0 ? kept : 1, 256), L - 1), 256, 0, st>>>(
                    keep_idx, S_cur, keep_len, new_len);
            }
            METOK_LAUNCH_CHECK();
        }
    } else {
        {
            METOK_TIMED("copy_len_kernel", st);
            copy_len_kernel<<<ceil_div(L, 256), 256, 0, st>>>(keep_len, new_len, L);
        }
        METOK_LAUNCH_CHECK();
    }
    const int row_chunks = (int)((long long)dh * eb / 16);
    for (int l0 = 0; l0 < L; l0 += kKvMaxLayersPerLaunch) {
        const int nl = (L - l0) < kKvMaxLayersPerLaunch ? (L - l0) : kKvMaxLayersPerLaunch;
        KvPtrs ptrs;
        for (int l = 0; l < kKvMaxLayersPerLaunch; ++l) {
            ptrs.k[l] = l < nl ? k_layers[l0 + l] : nullptr;
            ptrs.v[l] = l < nl ? v_layers[l0 + l] : nullptr;
        }
        const int grid = nl * 2 * Hkv * kKvCluster;
        {
            METOK_TIMED("kv_gather_kernel", st);
            kv_gather_kernel<<<grid, kKvThreads, 0, st>>>(ptrs, l0, Hkv, S_cap, S_cur, row_chunks, keep_idx, keep_len);
        }
        METOK_LAUNCH_CHECK();
    }
    return METOK_OK;
}
