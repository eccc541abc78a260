// metok_prefill_prune: text->visual attention scores at a pruning layer, class-wise
// top-k under the Eq. 6/7 budgets, and compaction of the surviving hidden states.
#include <cstdlib>

#include "common.cuh"
#include "select.cuh"
#include "select_block.cuh"
#include "launchers.h"
#include "sm100.cuh"

namespace metok {

// --------------------------------------------------------------------------- //
// Attention scores, generic CUDA-core path.
//
// Per KV head g the rep = Hq/Hkv query heads of the group form R = rep*Lt rows
// (row r = local head * Lt + q) that all multiply the same K[g].  The softmax
// normaliser of a row needs every visible key, the column sums need the
// normaliser, and the R x S probability matrix is never stored: pass 1 computes
// per-row running (max, sum) over a split of the columns, pass 2 recomputes the
// logits, normalises, and sums each column over the rows of the tile.
// Everything is reduced in a fixed order (no float atomics).
// --------------------------------------------------------------------------- //
constexpr int kAtTM = 64, kAtTN = 64;
constexpr int kAtLD = 65;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegInf = -3.0e38f;   // finite stand-in: keeps (m_old - m_new) free of inf - inf

struct AttnDims {
    int Hq, Hkv, Lt, S, dh, vis_start, n_vis, rep, R, nrt, nsplit, tiles_n;
    float scale_log2;
};

template <typename T>
__device__ __forceinline__ void load_tile_transposed(const T* __restrict__ base, int row0, int row_end, int dh,
                                                     float* __restrict__ dst /*[dh][kAtLD]*/) {
    constexpr int VN = Vec16<T>::N;
    const int cpr = dh / VN;
    for (int c = threadIdx.x; c < kAtTM * cpr; c += blockDim.x) {
        const int r = c / cpr, ch = c % cpr;
        float v[VN];
        const int row = row0 + r;
        if (row < row_end) Vec16<T>::load(base + (size_t)row * dh + ch * VN, v);
        else Vec16<T>::zero(v);
#pragma unroll
        for (int q = 0; q < VN; ++q) dst[(ch * VN + q) * kAtLD + r] = v[q];
    }
}

__device__ __forceinline__ void tile_logits(const float* __restrict__ Qs, const float* __restrict__ Ks, int dh,
                                            int ty, int tx, float (&acc)[4][4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
    for (int kk = 0; kk < dh; ++kk) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = Qs[kk * kAtLD + ty + 16 * i];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Ks[kk * kAtLD + tx + 16 * j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
attn_stats_kernel(const T* __restrict__ q_text, const T* __restrict__ k_all, AttnDims dm,
                  float* __restrict__ part_m, float* __restrict__ part_l) {
    extern __shared__ float smem[];
    float* Qs = smem;
    float* Ks = smem + dm.dh * kAtLD;
    const int split = blockIdx.x, rt = blockIdx.y, g = blockIdx.z;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const T* Qg = q_text + (size_t)g * dm.R * dm.dh;
    const T* Kg = k_all + (size_t)g * dm.S * dm.dh;
    const int text_start = dm.S - dm.Lt;
    load_tile_transposed<T>(Qg, rt * kAtTM, dm.R, dm.dh, Qs);

    int limit[4];
    float m_run[4], l_run[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = rt * kAtTM + ty + 16 * i;
        limit[i] = r < dm.R ? text_start + (r % dm.Lt) : -1;    // last visible key
        m_run[i] = kNegInf;
        l_run[i] = 0.f;
    }
    const int per = (dm.tiles_n + dm.nsplit - 1) / dm.nsplit;
    const int t_lo = split * per, t_hi = min(dm.tiles_n, t_lo + per);
    for (int tn = t_lo; tn < t_hi; ++tn) {
        __syncthreads();
        load_tile_transposed<T>(Kg, tn * kAtTN, dm.S, dm.dh, Ks);
        __syncthreads();
        float acc[4][4];
        tile_logits(Qs, Ks, dm.dh, ty, tx, acc);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float tmax = kNegInf;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int u = tn * kAtTN + tx + 16 * j;
                acc[i][j] = (u <= limit[i]) ? acc[i][j] * dm.scale_log2 : kNegInf;
                tmax = fmaxf(tmax, acc[i][j]);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, o));
            const float m_new = fmaxf(m_run[i], tmax);
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) s += (acc[i][j] > kNegInf) ? exp2f(acc[i][j] - m_new) : 0.f;
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
            l_run[i] = l_run[i] * exp2f(m_run[i] - m_new) + s;
            m_run[i] = m_new;
        }
    }
    if (tx == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = rt * kAtTM + ty + 16 * i;
            if (r < dm.R) {
                const size_t o = ((size_t)g * dm.nsplit + split) * dm.R + r;
                part_m[o] = m_run[i];
                part_l[o] = l_run[i];
            }
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
attn_colsum_kernel(const T* __restrict__ q_text, const T* __restrict__ k_all, AttnDims dm,
                   const float* __restrict__ part_m, const float* __restrict__ part_l,
                   float* __restrict__ part_col) {
    extern __shared__ float smem[];
    float* Qs = smem;
    float* Ks = smem + dm.dh * kAtLD;
    __shared__ float s_M[kAtTM], s_invZ[kAtTM];
    __shared__ float s_col[8][kAtTN];
    const int split = blockIdx.x, rt = blockIdx.y, g = blockIdx.z;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15, warp = tid >> 5;
    const T* Qg = q_text + (size_t)g * dm.R * dm.dh;
    const T* Kg = k_all + (size_t)g * dm.S * dm.dh;
    const int text_start = dm.S - dm.Lt;
    load_tile_transposed<T>(Qg, rt * kAtTM, dm.R, dm.dh, Qs);
    if (tid < kAtTM) {
        const int r = rt * kAtTM + tid;
        float M = kNegInf, Z = 0.f;
        if (r < dm.R) {
            for (int s = 0; s < dm.nsplit; ++s) M = fmaxf(M, part_m[((size_t)g * dm.nsplit + s) * dm.R + r]);
            for (int s = 0; s < dm.nsplit; ++s) {
                const size_t o = ((size_t)g * dm.nsplit + s) * dm.R + r;
                Z += part_l[o] * exp2f(part_m[o] - M);
            }
        }
        s_M[tid] = M;
        s_invZ[tid] = Z > 0.f ? 1.0f / Z : 0.f;
    }
    __syncthreads();
    int limit[4];
    float rM[4], rI[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int rl = ty + 16 * i;
        const int r = rt * kAtTM + rl;
        limit[i] = r < dm.R ? text_start + (r % dm.Lt) : -1;
        rM[i] = s_M[rl];
        rI[i] = s_invZ[rl];
    }
    const int per = (dm.tiles_n + dm.nsplit - 1) / dm.nsplit;
    const int t_lo = split * per, t_hi = min(dm.tiles_n, t_lo + per);
    const int vis_end = dm.vis_start + dm.n_vis;
    for (int tn = t_lo; tn < t_hi; ++tn) {
        const int u0 = tn * kAtTN;
        if (u0 >= vis_end || u0 + kAtTN <= dm.vis_start) continue;     // no visual column in this tile
        __syncthreads();
        load_tile_transposed<T>(Kg, u0, dm.S, dm.dh, Ks);
        __syncthreads();
        float acc[4][4];
        tile_logits(Qs, Ks, dm.dh, ty, tx, acc);
        float cs[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int u = u0 + tx + 16 * j;
            float c = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                c += (u <= limit[i]) ? exp2f(acc[i][j] * dm.scale_log2 - rM[i]) * rI[i] : 0.f;
            c += __shfl_xor_sync(0xFFFFFFFFu, c, 16);            // the warp's two row groups
            cs[j] = c;
        }
        if ((tid & 31) < 16) {
#pragma unroll
            for (int j = 0; j < 4; ++j) s_col[warp][tx + 16 * j] = cs[j];
        }
        __syncthreads();
        if (tid < kAtTN) {
            const int u = u0 + tid;
            if (u >= dm.vis_start && u < vis_end) {
                float c = 0.f;
#pragma unroll
                for (int w = 0; w < 8; ++w) c += s_col[w][tid];
                part_col[((size_t)g * dm.nrt + rt) * dm.n_vis + (u - dm.vis_start)] = c;
            }
        }
    }
}

__global__ void __launch_bounds__(256)
attn_score_reduce_kernel(const float* __restrict__ part_col, int nparts, int n_vis, float inv_rows,
                         float* __restrict__ scores) {
    grid_dep_wait();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n_vis) return;
    float a = 0.f;
    int p = 0;
    for (; p + 8 <= nparts; p += 8) {                          // eight loads in flight, added in plane order
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = part_col[(size_t)(p + u) * n_vis + j];
#pragma unroll
        for (int u = 0; u < 8; ++u) a += v[u];
    }
    for (; p < nparts; ++p) a += part_col[(size_t)p * n_vis + j];
    scores[j] = a * inv_rows;
}

// --------------------------------------------------------------------------- //
// Class-wise top-k + ordered keep list.  One CTA per problem (blockIdx.x): the
// prefill step launches one, the KV TOPK policy one per layer.
// --------------------------------------------------------------------------- //
struct TopkBudgets { int v[METOK_MAX_GROUPS]; };

__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads)
class_topk_kernel(const float* __restrict__ scores, size_t score_stride, const int32_t* __restrict__ token_group,
                  int n_vis, int G, SelectLayout lay, TopkBudgets budgets, int S, int vis_start,
                  int32_t* __restrict__ keep_idx, size_t keep_stride, int replicas,
                  int32_t* __restrict__ count_a, int32_t* __restrict__ count_b) {
    __shared__ SelectSmem sm;
    __shared__ int s_budget[METOK_MAX_GROUPS];
    extern __shared__ __align__(16) unsigned char sel_dyn[];
    const int problem = blockIdx.x / kSelCluster;
    const float* sc = scores + (size_t)problem * score_stride;
    int32_t* keep = keep_idx + (size_t)problem * keep_stride;
    const int vis_end = vis_start + n_vis;
    SelectCtx cx;
    cx.rank = (int)cx.cl.block_rank();
    cx.G = G;
    cx.nb_log2 = lay.nb_log2;
    int p_lo, p_hi;
    select_slice(S, cx.rank, &p_lo, &p_hi);
    const int v_lo = max(p_lo, vis_start), v_hi = min(p_hi, vis_end);   // scored positions of this slice
    cx.item_lo = v_lo - vis_start;
    cx.m = v_hi > v_lo ? v_hi - v_lo : 0;
    cx.cached = cx.m <= lay.cache_cap;
    cx.hist = reinterpret_cast<uint32_t*>(sel_dyn + lay.hist_off);
    cx.merged = reinterpret_cast<uint32_t*>(sel_dyn + lay.merged_off);
    cx.keys = reinterpret_cast<uint32_t*>(sel_dyn + lay.keys_off);
    cx.cls = sel_dyn + lay.cls_off;
    for (int g = threadIdx.x; g < G; g += blockDim.x) s_budget[g] = budgets.v[g];
    __syncthreads();
    auto cls = [=](int i) {
        if (!token_group) return 0;
        const int g = token_group[i];
        return (g >= 0 && g < G) ? g : -1;
    };
    auto val = [=](int i) { return sc[i]; };
    cluster_select(cx, n_vis, cls, val, s_budget, sm);
    auto flag = [&](int u) {
        if (u < vis_start || u >= vis_end) return true;
        const int i = u - vis_start;
        const SelItem it = item_at(cx, i - cx.item_lo, cls, val);
        return it.cls >= 0 && is_selected(sm, it.cls, it.key, i);
    };
    // one list may serve several layers: `replicas` copies, keep_stride apart
    auto emit = [&](int u, int rank) {
        for (int r = 0; r < replicas; ++r) keep[(size_t)r * keep_stride + rank] = u;
    };
    const int total = cluster_compact(cx, p_lo, p_hi, flag, emit, sm);
    if (cx.rank == 0) {
        for (int r = threadIdx.x; r < replicas; r += blockDim.x) {
            if (count_a) count_a[problem + r] = total;
            if (count_b) count_b[problem + r] = total;
        }
    }
}

template <bool kOne>                     // kOne: one class and no class array
__global__ void __launch_bounds__(kBsThreads, 1)
block_topk_kernel(const float* __restrict__ scores, size_t score_stride, const int32_t* __restrict__ token_group,
                  int n_vis, int G, BlockSelLayout lay, TopkBudgets budgets, int S, int vis_start,
                  int32_t* __restrict__ keep_idx, size_t keep_stride, int replicas,
                  int32_t* __restrict__ count_a, int32_t* __restrict__ count_b) {
    grid_dep_wait();
    __shared__ BlockSelSmem sm;
    extern __shared__ __align__(16) unsigned char sel_dyn[];
    const int problem = blockIdx.x;
    const float* sc = scores + (size_t)problem * score_stride;
    int32_t* keep = keep_idx + (size_t)problem * keep_stride;
    const int tid = threadIdx.x;
    const BlockSelView sel = block_sel_run<kOne>(sm, sel_dyn, lay, sc, kOne ? nullptr : token_group, n_vis, G, budgets.v);
    const uint32_t* mask = sel.mask;
    const int* woff = sel.woff;
    const int kept = sel.kept;
    const int n4 = (n_vis + 3) >> 2;
    const int vis_end = vis_start + n_vis;
    // The kept positions in order.  Positions before and after the visual span are always kept;
    // the kept visual items are first packed in shared memory (over the keys, which the masks
    // have replaced) so that the list leaves in whole coalesced stores.
    // One list may serve several layers: `replicas` copies, keep_stride apart.
    int32_t* packed = reinterpret_cast<int32_t*>(sel.keys);
    for (int q = tid; q < n4; q += kBsThreads) {
        const uint32_t m = mask[q >> 3];
        const int sh = (q & 7) * 4;
        const uint32_t nib = (m >> sh) & 15u;
        int rank = woff[q >> 3] + __popc(m & ((1u << sh) - 1u));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if ((nib >> u) & 1u) packed[rank++] = vis_start + q * 4 + u;
        }
    }
    __syncthreads();
    const int total = vis_start + kept + (S - vis_end);
    for (int i = tid; i < total; i += kBsThreads) {
        const int v = i < vis_start ? i : i < vis_start + kept ? packed[i - vis_start] : vis_end + (i - vis_start - kept);
        for (int r = 0; r < replicas; ++r) keep[(size_t)r * keep_stride + i] = v;
    }
    for (int r = tid; r < replicas; r += kBsThreads) {
        if (count_a) count_a[problem + r] = total;
        if (count_b) count_b[problem + r] = total;
    }
}

int launch_class_topk(const float* scores, size_t score_stride, const int32_t* token_group, int n_vis, int G,
                      const int32_t* budgets_host, int S, int vis_start, int32_t* keep_idx, size_t keep_stride,
                      int replicas, int32_t* count_a, int32_t* count_b, int problems, cudaStream_t st) {
    TopkBudgets b;
    for (int g = 0; g < METOK_MAX_GROUPS; ++g) b.v[g] = g < G ? budgets_host[g] : 0;
    // problems whose keys fit one CTA's shared memory skip the cluster and its barriers
    const BlockSelLayout bl = block_sel_layout(G, n_vis, S);
    if (bl.fits) {
        auto kernel = (G == 1 && !token_group) ? block_topk_kernel<true> : block_topk_kernel<false>;
        if (bl.bytes > 32 * 1024)
            METOK_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bl.bytes));
        {
            METOK_TIMED("class_topk_kernel", st);
            launch_chained(kernel, dim3(problems), dim3(kBsThreads), bl.bytes, st, scores, score_stride, token_group, n_vis, G, bl, b, S,
                                                           vis_start, keep_idx, keep_stride, replicas, count_a, count_b);
        }
        METOK_LAUNCH_CHECK();
        return METOK_OK;
    }
    const SelectLayout lay = select_layout(G, select_items_per_cta((long long)S));
    const int nthreads = select_threads(select_items_per_cta((long long)S));
    if (lay.bytes > 32 * 1024)                        // static + dynamic beyond 48 KiB needs the opt-in
        METOK_CUDA_TRY(cudaFuncSetAttribute(class_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)lay.bytes));
    {
        METOK_TIMED("class_topk_kernel", st);
        class_topk_kernel<<<problems * kSelCluster, nthreads, lay.bytes, st>>>(
            scores, score_stride, token_group, n_vis, G, lay, b, S, vis_start, keep_idx, keep_stride, replicas,
            count_a, count_b);
    }
    METOK_LAUNCH_CHECK();
    return METOK_OK;
}

// --------------------------------------------------------------------------- //
// hidden_out[i] = hidden[keep_idx[i]], i < *S_out.  Rows are whole 16-byte chunks.
// The gather is driven by the copy engine: one thread per CTA moves (row, 8 KiB segment)
// items global -> shared -> global with bulk copies, kGbStages items in flight; no registers
// or warps are spent on the data.
constexpr int kGbStages = 4;
constexpr uint32_t kGbSegBytes = 8192;
constexpr size_t kGbSmemBytes = (size_t)kGbStages * kGbSegBytes + 128;

__global__ void __launch_bounds__(32)
gather_rows_bulk_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst,
                        const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ n_rows,
                        uint32_t row_bytes, int src_rows, int32_t* __restrict__ status) {
    grid_dep_wait();
    using namespace sm100;
    extern __shared__ uint8_t gb_dyn[];
    __shared__ __align__(8) uint64_t s_bar[kGbStages];
    __shared__ int s_abort;
    if (threadIdx.x != 0) return;
    const uint32_t stage0 = (smem_u32(gb_dyn) + 127u) & ~127u;
    for (int j = 0; j < kGbStages; ++j) mbar_init(smem_u32(&s_bar[j]), 1);
    s_abort = 0;
    mbar_fence_init();
    const int nseg = (int)((row_bytes + kGbSegBytes - 1) / kGbSegBytes);
    const long long items = (long long)(*n_rows) * nseg;
    const long long first = blockIdx.x, stride = gridDim.x;
    const long long mine = first < items ? (items - first + stride - 1) / stride : 0;   // items of this CTA
    auto issue_load = [&](long long k) {
        const long long it = first + k * stride;
        const int i = (int)(it / nseg), sg = (int)(it - (long long)i * nseg);
        const uint32_t off = (uint32_t)sg * kGbSegBytes;
        const uint32_t bytes = min(kGbSegBytes, row_bytes - off);
        const uint32_t bar = smem_u32(&s_bar[k % kGbStages]);
        mbar_arrive_expect_tx(bar, bytes);
        const long long row = dbg_bound(keep_idx[i], src_rows, status);
        if (!(dbg_withhold(status, kDbgGatherRows) && blockIdx.x == 0 && k == 0))   // debug builds: one copy never sent
            bulk_load(stage0 + (uint32_t)(k % kGbStages) * kGbSegBytes, src + (size_t)row * row_bytes + off, bytes, bar);
    };
    volatile int* abort_flag = &s_abort;
    for (long long k = 0; k < mine && k < kGbStages; ++k) issue_load(k);
    bool ok = true;
    for (long long k = 0; k < mine; ++k) {
        const int s = (int)(k % kGbStages);
        if (!mbar_wait(smem_u32(&s_bar[s]), (uint32_t)(k / kGbStages) & 1u, abort_flag)) { ok = false; break; }
        const long long it = first + k * stride;
        const int i = (int)(it / nseg), sg = (int)(it - (long long)i * nseg);
        const uint32_t off = (uint32_t)sg * kGbSegBytes;
        const uint32_t bytes = min(kGbSegBytes, row_bytes - off);
        fence_proxy_async();
        bulk_store(dst + (size_t)i * row_bytes + off, stage0 + (uint32_t)s * kGbSegBytes, bytes);
        bulk_commit();
        // the stage of the item before this one is free once its store has read it
        if (k >= 1 && k - 1 + kGbStages < mine) {
            bulk_wait_read<1>();
            issue_load(k - 1 + kGbStages);
        }
    }
    bulk_wait_all();
    if (!ok) {
        // loads still in flight must land before the shared memory goes away
        for (int j = 0; j < kGbStages; ++j) mbar_wait(smem_u32(&s_bar[j]), 0u, abort_flag);
        *status = METOK_ERR_TIMEOUT;
    }
}

int launch_gather_rows_bulk(const void* src, void* dst, const int32_t* idx, const int32_t* n_rows, size_t row_bytes,
                            int src_rows, int32_t* status, const char* timer_name, cudaStream_t st) {
    METOK_CUDA_TRY(cudaFuncSetAttribute(gather_rows_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)kGbSmemBytes));
    {
        METOK_TIMED(timer_name, st);
        launch_chained(gather_rows_bulk_kernel, dim3(kNumSMs * 6), dim3(32), kGbSmemBytes, st, 
            reinterpret_cast<const uint8_t*>(src), reinterpret_cast<uint8_t*>(dst), idx, n_rows, (uint32_t)row_bytes,
            src_rows, status);
    }
    METOK_LAUNCH_CHECK();
    return METOK_OK;
}

static AttnDims make_dims(int Hq, int Hkv, int Lt, int S, int dh, int vis_start, int n_vis, float scale) {
    AttnDims dm;
    dm.Hq = Hq; dm.Hkv = Hkv; dm.Lt = Lt; dm.S = S; dm.dh = dh; dm.vis_start = vis_start; dm.n_vis = n_vis;
    dm.rep = Hq / Hkv;
    dm.R = dm.rep * Lt;
    dm.nrt = ceil_div(dm.R, kAtTM);
    dm.tiles_n = ceil_div(S, kAtTN);
    int ns = ceil_div(4 * kNumSMs, dm.nrt * Hkv);
    if (ns > dm.tiles_n) ns = dm.tiles_n;
    if (ns < 1) ns = 1;
    if (ns > 64) ns = 64;
    dm.nsplit = ns;
    dm.scale_log2 = scale * kLog2e;
    return dm;
}

// The tensor-core scoring path takes bf16 with head dim 64 or 128; METOK_DEBUG_FORCE_SIMT=1 in
// the environment selects the CUDA-core kernels (debugging aid).
static bool use_mma_attn(int dtype, int dh) {
    static const bool force_simt = [] { const char* e = getenv("METOK_DEBUG_FORCE_SIMT"); return e && e[0] == '1'; }();
    return !force_simt && dtype == METOK_BF16 && (dh == 64 || dh == 128);
}

struct PrefillWs {
    int32_t* status;          // device status word, first in the workspace
    float *part_m, *part_l, *part_col;
    int n_planes;
};
static PrefillWs carve_prefill(Carver& cv, const AttnDims& dm, bool mma) {
    PrefillWs w;
    w.status = cv.take<int32_t>(64);
    if (mma) {
        size_t n_ml, n_col;
        attn_mma_workspace(dm.Hq, dm.Hkv, dm.Lt, dm.S, dm.n_vis, &n_ml, &n_col, &w.n_planes);
        w.part_m = cv.take<float>(n_ml);
        w.part_l = cv.take<float>(n_ml);
        w.part_col = cv.take<float>(n_col);
    } else {
        w.part_m = cv.take<float>((size_t)dm.Hkv * dm.nsplit * dm.R);
        w.part_l = cv.take<float>((size_t)dm.Hkv * dm.nsplit * dm.R);
        w.part_col = cv.take<float>((size_t)dm.Hkv * dm.nrt * dm.n_vis);
        w.n_planes = dm.Hkv * dm.nrt;
    }
    return w;
}

static int launch_score_reduce(const PrefillWs& w, const AttnDims& dm, float inv_rows, float* scores, cudaStream_t st) {
    {
        METOK_TIMED("attn_score_reduce_kernel", st);
        launch_chained(attn_score_reduce_kernel, dim3(ceil_div(dm.n_vis, 256)), dim3(256), 0, st, w.part_col, w.n_planes,
                       dm.n_vis, inv_rows, scores);
    }
    METOK_LAUNCH_CHECK();
    return METOK_OK;
}

template <typename T>
static int launch_attn_scores(const void* q_text, const void* k_all, const AttnDims& dm, const PrefillWs& w,
                              float inv_rows, float* scores, cudaStream_t st) {
    const size_t smem = (size_t)2 * dm.dh * kAtLD * sizeof(float);
    METOK_CUDA_TRY(cudaFuncSetAttribute(attn_stats_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    METOK_CUDA_TRY(cudaFuncSetAttribute(attn_colsum_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid(dm.nsplit, dm.nrt, dm.Hkv);
    {
        METOK_TIMED("attn_stats_kernel", st);
        attn_stats_kernel<T><<<grid, 256, smem, st>>>(reinterpret_cast<const T*>(q_text), reinterpret_cast<const T*>(k_all),
                                                  dm, w.part_m, w.part_l);
    }
    METOK_LAUNCH_CHECK();
    {
        METOK_TIMED("attn_colsum_kernel", st);
        attn_colsum_kernel<T><<<grid, 256, smem, st>>>(reinterpret_cast<const T*>(q_text),
                                                   reinterpret_cast<const T*>(k_all), dm, w.part_m, w.part_l,
                                                   w.part_col);
    }
    METOK_LAUNCH_CHECK();
    return launch_score_reduce(w, dm, inv_rows, scores, st);
}

}  // namespace metok

using namespace metok;

// a5 as the calls run it: the status word cleared, then the two passes and the plane sum;
// scores[j] = inv_rows * (sum over this call's heads and text queries of the probabilities).
static int run_attention_scores(const void* q_text, const void* k_all, int dtype, const AttnDims& dm,
                                const PrefillWs& w, float softmax_scale, float inv_rows, float* scores,
                                cudaStream_t st) {
    const bool mma = use_mma_attn(dtype, dm.dh);
    if (!mma) METOK_CUDA_TRY(cudaMemsetAsync(w.status, 0, sizeof(int32_t), st));   // else attn_stats_mma_kernel clears it
    if (mma) {
        const int rc = launch_attn_scores_mma(q_text, k_all, dm.Hq, dm.Hkv, dm.Lt, dm.S, dm.dh, dm.vis_start, dm.n_vis,
                                              softmax_scale, w.part_m, w.part_l, w.part_col, w.status, st);
        return rc == METOK_OK ? launch_score_reduce(w, dm, inv_rows, scores, st) : rc;
    }
    return dtype == METOK_F32 ? launch_attn_scores<float>(q_text, k_all, dm, w, inv_rows, scores, st)
                              : launch_attn_scores<__nv_bfloat16>(q_text, k_all, dm, w, inv_rows, scores, st);
}

extern "C" size_t metok_prefill_prune_workspace_bytes(int dtype, int Hq, int Hkv, int Lt, int S, int dh, int n_vis) {
    if (Hq < 1 || Hkv < 1 || Lt < 1 || S < 1 || dh < 1 || n_vis < 1 || Hq % Hkv) return 0;
    AttnDims dm = make_dims(Hq, Hkv, Lt, S, dh, 0, n_vis, 1.f);
    Carver cv(nullptr);
    carve_prefill(cv, dm, use_mma_attn(dtype, dh));
    return cv.total();
}

// Every check of metok_prefill_prune that needs no device: arguments, shapes, alignment, workspace.
static int validate_prefill_prune(const void* q_text, const void* k_all, const void* hidden, int dtype, int Hq,
                                  int Hkv, int Lt, int S, int dh, int D, int vis_start, int n_vis,
                                  const int32_t* token_group, int G, const int32_t* group_budget,
                                  float softmax_scale, const float* scores, const int32_t* keep_idx,
                                  const int32_t* S_out, const void* hidden_out, const void* ws, size_t ws_bytes) {
    if (!q_text || !k_all || !token_group || !group_budget || !scores || !keep_idx || !S_out)
        return METOK_ERR_INVALID_ARG;
    if ((hidden == nullptr) != (hidden_out == nullptr)) return METOK_ERR_INVALID_ARG;
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (Hq < 1 || Hkv < 1 || Lt < 1 || S < 1 || dh < 1 || n_vis < 1 || (hidden && D < 1)) return METOK_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || Lt > S) return METOK_ERR_INVALID_ARG;
    if (vis_start < 0 || (long long)vis_start + n_vis > (long long)S - Lt) return METOK_ERR_INVALID_ARG;
    if (G < 1 || G > METOK_MAX_GROUPS) return METOK_ERR_INVALID_ARG;
    for (int g = 0; g < G; ++g)
        if (group_budget[g] < 0) return METOK_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f)) return METOK_ERR_INVALID_ARG;
    if (!aligned16(q_text) || !aligned16(k_all) || (hidden && (!aligned16(hidden) || !aligned16(hidden_out))))
        return METOK_ERR_INVALID_ARG;
    const int eb = dtype == METOK_F32 ? 4 : 2;
    if (dtype == METOK_BF16 && dh != 64 && dh != 128) return METOK_ERR_UNSUPPORTED;
    if (dtype == METOK_F32 && (dh > 128 || dh % 4 != 0)) return METOK_ERR_UNSUPPORTED;
    if (hidden && ((long long)D * eb) % 16 != 0) return METOK_ERR_UNSUPPORTED;
    const size_t need = metok_prefill_prune_workspace_bytes(dtype, Hq, Hkv, Lt, S, dh, n_vis);
    if (!ws || ws_bytes < need || !aligned16(ws)) return METOK_ERR_WORKSPACE;
    return METOK_OK;
}

extern "C" int metok_prefill_prune(const void* q_text, const void* k_all, const void* hidden, int dtype, int Hq,
                                   int Hkv, int Lt, int S, int dh, int D, int vis_start, int n_vis,
                                   const int32_t* token_group, int G, const int32_t* group_budget,
                                   float softmax_scale, float* scores, int32_t* keep_idx, int32_t* S_out,
                                   void* hidden_out, void* ws, size_t ws_bytes, void* stream) {
    const int vrc = validate_prefill_prune(q_text, k_all, hidden, dtype, Hq, Hkv, Lt, S, dh, D, vis_start, n_vis,
                                           token_group, G, group_budget, softmax_scale, scores, keep_idx, S_out,
                                           hidden_out, ws, ws_bytes);
    if (vrc != METOK_OK) return vrc;
    const int eb = dtype == METOK_F32 ? 4 : 2;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    AttnDims dm = make_dims(Hq, Hkv, Lt, S, dh, vis_start, n_vis, softmax_scale);
    Carver cv(ws);
    PrefillWs w = carve_prefill(cv, dm, use_mma_attn(dtype, dh));
    int rc = debug_arm(w.status, st);
    if (rc != METOK_OK) return rc;
    rc = run_attention_scores(q_text, k_all, dtype, dm, w, softmax_scale, 1.0f / (float)(Hq * Lt), scores, st);
    if (rc != METOK_OK) return rc;
    rc = launch_class_topk(scores, 0, token_group, n_vis, G, group_budget, S, vis_start, keep_idx, 0, 1, S_out,
                           nullptr, 1, st);
    if (rc != METOK_OK) return rc;
    if (hidden) {
        rc = launch_gather_rows_bulk(hidden, hidden_out, keep_idx, S_out, (size_t)D * eb, S, w.status, "gather_rows_kernel",
                                     st);
        if (rc != METOK_OK) return rc;
    }
    return METOK_OK;
}

extern "C" int metok_attention_scores(const void* q_text, const void* k_all, int dtype, int Hq, int Hkv, int Lt, int S,
                                      int dh, int vis_start, int n_vis, float softmax_scale, int rows_total,
                                      float* scores, void* ws, size_t ws_bytes, void* stream) {
    if (!q_text || !k_all || !scores) return METOK_ERR_INVALID_ARG;
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (Hq < 1 || Hkv < 1 || Lt < 1 || S < 1 || dh < 1 || n_vis < 1) return METOK_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || Lt > S) return METOK_ERR_INVALID_ARG;
    if (vis_start < 0 || (long long)vis_start + n_vis > (long long)S - Lt) return METOK_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || !aligned16(q_text) || !aligned16(k_all)) return METOK_ERR_INVALID_ARG;
    if (rows_total != 0 && (long long)rows_total < (long long)Hq * Lt) return METOK_ERR_INVALID_ARG;
    if (dtype == METOK_BF16 && dh != 64 && dh != 128) return METOK_ERR_UNSUPPORTED;
    if (dtype == METOK_F32 && (dh > 128 || dh % 4 != 0)) return METOK_ERR_UNSUPPORTED;
    const size_t need = metok_prefill_prune_workspace_bytes(dtype, Hq, Hkv, Lt, S, dh, n_vis);
    if (!ws || ws_bytes < need || !aligned16(ws)) return METOK_ERR_WORKSPACE;
    AttnDims dm = make_dims(Hq, Hkv, Lt, S, dh, vis_start, n_vis, softmax_scale);
    Carver cv(ws);
    PrefillWs w = carve_prefill(cv, dm, use_mma_attn(dtype, dh));
    const float inv_rows = 1.0f / (float)(rows_total ? rows_total : Hq * Lt);
    if (const int rc = debug_arm(w.status, reinterpret_cast<cudaStream_t>(stream))) return rc;
    return run_attention_scores(q_text, k_all, dtype, dm, w, softmax_scale, inv_rows, scores,
                                reinterpret_cast<cudaStream_t>(stream));
}

extern "C" size_t metok_prune_by_scores_workspace_bytes(void) { return 1024; }

extern "C" int metok_prune_by_scores(const float* scores, const void* hidden, int dtype, int S, int D, int vis_start,
                                     int n_vis, const int32_t* token_group, int G, const int32_t* group_budget,
                                     int32_t* keep_idx, int32_t* S_out, void* hidden_out, void* ws, size_t ws_bytes,
                                     void* stream) {
    if (!scores || !token_group || !group_budget || !keep_idx || !S_out) return METOK_ERR_INVALID_ARG;
    if ((hidden == nullptr) != (hidden_out == nullptr)) return METOK_ERR_INVALID_ARG;
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (S < 1 || n_vis < 1 || (hidden && D < 1)) return METOK_ERR_INVALID_ARG;
    if (vis_start < 0 || (long long)vis_start + n_vis > (long long)S) return METOK_ERR_INVALID_ARG;
    if (G < 1 || G > METOK_MAX_GROUPS) return METOK_ERR_INVALID_ARG;
    for (int g = 0; g < G; ++g)
        if (group_budget[g] < 0) return METOK_ERR_INVALID_ARG;
    if (hidden && (!aligned16(hidden) || !aligned16(hidden_out))) return METOK_ERR_INVALID_ARG;
    const int eb = dtype == METOK_F32 ? 4 : 2;
    if (hidden && ((long long)D * eb) % 16 != 0) return METOK_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < metok_prune_by_scores_workspace_bytes() || !aligned16(ws)) return METOK_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int32_t* status = reinterpret_cast<int32_t*>(ws);
    METOK_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    int rc = debug_arm(status, st);
    if (rc != METOK_OK) return rc;
    rc = launch_class_topk(scores, 0, token_group, n_vis, G, group_budget, S, vis_start, keep_idx, 0, 1, S_out,
                               nullptr, 1, st);
    if (rc != METOK_OK) return rc;
    if (hidden)
        rc = launch_gather_rows_bulk(hidden, hidden_out, keep_idx, S_out, (size_t)D * eb, S, status, "gather_rows_kernel", st);
    return rc;
}

extern "C" int metok_retention_budgets(double alpha, double r, int stage, const int32_t* N0, int32_t* budget) {
    if (!N0 || !budget) return METOK_ERR_INVALID_ARG;
    if (!(alpha > 0.0 && alpha <= 1.0) || !(r > 0.0 && r <= 1.0)) return METOK_ERR_INVALID_ARG;
    if (stage < 0 || stage > 3 || N0[0] < 0 || N0[1] < 0) return METOK_ERR_INVALID_ARG;
    double rk, rn;
    switch (stage) {
        case 0: rk = 1.0; rn = 1.0; break;
        case 1: rk = r; rn = alpha * r; break;
        case 2: rk = r * r; rn = 0.0; break;
        default: rk = 0.0; rn = 0.0; break;
    }
    int bk = ceilq(rk * (double)N0[0]), bn = ceilq(rn * (double)N0[1]);
    budget[0] = bk < N0[0] ? bk : N0[0];
    budget[1] = bn < N0[1] ? bn : N0[1];
    return METOK_OK;
}

// --------------------------------------------------------------------------- //
// The pruning levels chained on the device.
// --------------------------------------------------------------------------- //
namespace metok {

// One CTA: origin[i] = i, and the class counts of the first level against the caller's N0.
__global__ void __launch_bounds__(1024)
schedule_init_kernel(const int32_t* __restrict__ token_group, int n_vis, int n0_key, int n0_nonkey,
                     int32_t* __restrict__ origin, int32_t* __restrict__ status) {
    __shared__ int s_cnt[2];
    if (threadIdx.x < 2) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    int c0 = 0, c1 = 0;
    for (int i = threadIdx.x; i < n_vis; i += blockDim.x) {
        origin[i] = i;
        const int g = token_group[i];
        c0 += g == 0;
        c1 += g == 1;
    }
    c0 = warp_sum_int(c0);
    c1 = warp_sum_int(c1);
    if ((threadIdx.x & 31) == 0) { atomicAdd(&s_cnt[0], c0); atomicAdd(&s_cnt[1], c1); }
    __syncthreads();
    if (threadIdx.x == 0)
        *status = (s_cnt[0] == n0_key && s_cnt[1] == n0_nonkey && s_cnt[0] + s_cnt[1] == n_vis) ? METOK_OK
                                                                                                 : METOK_ERR_INVALID_ARG;
}

// Class and origin of the i-th surviving visual token: the keep list holds every position before
// the visual span, so its entry vis_start + i is that token's position at the level before.
__global__ void __launch_bounds__(256)
schedule_propagate_kernel(const int32_t* __restrict__ keep_idx, int vis_start, int n_cur, int n_next,
                          const int32_t* __restrict__ group, const int32_t* __restrict__ origin,
                          int32_t* __restrict__ group_next, int32_t* __restrict__ origin_next,
                          const int32_t* __restrict__ level_status, int32_t* __restrict__ status) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    // a level that gave up on a wait leaves its code in its own status word, which the next level
    // clears: the first failure is kept in the caller's
    if (i == 0 && *level_status != METOK_OK && *status == METOK_OK) *status = *level_status;
    if (i >= n_next) return;
    int j = keep_idx[vis_start + i] - vis_start;
    j = j < 0 ? 0 : (j >= n_cur ? n_cur - 1 : j);            // only reached with a wrong N0 (status says so)
    group_next[i] = group[j];
    origin_next[i] = origin[j];
}

}  // namespace metok

namespace metok {
struct KvListSrc { const int32_t* keep_idx[4]; const int32_t* S_out[4]; int S_in[4]; };   // per layer group
// Layer l of group g (the pruning layers at or below it: g of them) holds the rows of level g's input;
// its list is the keep list recorded by level g + 1, or everything when no level follows.
__global__ void __launch_bounds__(256)
schedule_kv_lists_kernel(KvListSrc src, const int32_t* __restrict__ layer_group, int stride,
                         int32_t* __restrict__ kv_keep_idx, int32_t* __restrict__ kv_keep_len) {
    const int layer = blockIdx.x;
    const int g = layer_group[layer];
    int32_t* out = kv_keep_idx + (size_t)layer * stride;
    const int32_t* keep = src.keep_idx[g];
    const int n = keep ? *src.S_out[g] : src.S_in[g];
    for (int i = threadIdx.x; i < n; i += blockDim.x) out[i] = keep ? keep[i] : i;
    if (threadIdx.x == 0) kv_keep_len[layer] = n;
}
}  // namespace metok

extern "C" int metok_prune_schedule_kv_lists(const metok_prune_level* levels, int n_levels, const int32_t* level_layer,
                                             int L, int S, int n_vis, double alpha, double r, const int32_t* N0,
                                             int32_t* kv_keep_idx, int32_t* kv_keep_len, int32_t* kv_S_cur,
                                             void* ws, size_t ws_bytes, void* stream) {
    if (!levels || !level_layer || !N0 || !kv_keep_idx || !kv_keep_len || !kv_S_cur) return METOK_ERR_INVALID_ARG;
    if (L < 1 || S < 1 || n_vis < 1 || n_vis > S) return METOK_ERR_INVALID_ARG;
    int32_t sizes[4];
    const int rc = metok_prune_schedule_sizes(n_levels, alpha, r, N0, sizes);
    if (rc != METOK_OK) return rc;
    if (sizes[0] != n_vis) return METOK_ERR_INVALID_ARG;
    for (int s = 0; s < n_levels; ++s) {
        if (!levels[s].keep_idx || !levels[s].S_out) return METOK_ERR_INVALID_ARG;
        if (level_layer[s] < 0 || (s > 0 && level_layer[s] <= level_layer[s - 1])) return METOK_ERR_INVALID_ARG;
    }
    if (!ws || ws_bytes < (size_t)L * sizeof(int32_t) || !aligned16(ws)) return METOK_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    metok::KvListSrc src;
    for (int g = 0; g < 4; ++g) {
        src.keep_idx[g] = g < n_levels ? levels[g].keep_idx : nullptr;
        src.S_out[g] = g < n_levels ? levels[g].S_out : nullptr;
        src.S_in[g] = g <= n_levels ? S - n_vis + sizes[g] : 0;
    }
    // the group of every layer, known on the host
    int32_t group_host[1024];
    if (L > 1024) return METOK_ERR_UNSUPPORTED;
    for (int l = 0; l < L; ++l) {
        int g = 0;
        while (g < n_levels && level_layer[g] <= l) ++g;
        group_host[l] = g;
        kv_S_cur[l] = src.S_in[g];
    }
    int32_t* group_dev = reinterpret_cast<int32_t*>(ws);
    METOK_CUDA_TRY(cudaMemcpyAsync(group_dev, group_host, (size_t)L * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    {
        METOK_TIMED("schedule_kv_lists_kernel", st);
        metok::schedule_kv_lists_kernel<<<L, 256, 0, st>>>(src, group_dev, S, kv_keep_idx, kv_keep_len);
    }
    METOK_LAUNCH_CHECK();
    return METOK_OK;
}

extern "C" int metok_prune_schedule_sizes(int n_levels, double alpha, double r, const int32_t* N0,
                                          int32_t* n_vis_of_level) {
    if (!N0 || !n_vis_of_level || n_levels < 1 || n_levels > 3) return METOK_ERR_INVALID_ARG;
    for (int s = 0; s <= n_levels; ++s) {
        int32_t b[2];
        const int rc = metok_retention_budgets(alpha, r, s, N0, b);
        if (rc != METOK_OK) return rc;
        n_vis_of_level[s] = b[0] + b[1];
    }
    return METOK_OK;
}

extern "C" size_t metok_prefill_prune_schedule_workspace_bytes(int n_levels, int dtype, int Hq, int Hkv, int Lt, int S,
                                                               int dh, int n_vis, double alpha, double r,
                                                               const int32_t* N0) {
    int32_t sizes[4];
    if (metok_prune_schedule_sizes(n_levels, alpha, r, N0, sizes) != METOK_OK || sizes[0] != n_vis) return 0;
    size_t need = 0;
    for (int s = 0; s < n_levels; ++s) {
        const size_t b = metok_prefill_prune_workspace_bytes(dtype, Hq, Hkv, Lt, S - n_vis + sizes[s], dh, sizes[s]);
        if (b == 0) return 0;
        need = b > need ? b : need;
    }
    return need;
}

extern "C" int metok_prefill_prune_schedule(const metok_prune_level* levels, int n_levels, int dtype, int Hq, int Hkv,
                                            int Lt, int S, int dh, int D, int vis_start, int n_vis, double alpha,
                                            double r, const int32_t* N0, float softmax_scale, int32_t* status,
                                            void* ws, size_t ws_bytes, void* stream) {
    if (!levels || !N0 || !status) return METOK_ERR_INVALID_ARG;
    int32_t sizes[4];
    int rc = metok_prune_schedule_sizes(n_levels, alpha, r, N0, sizes);
    if (rc != METOK_OK) return rc;
    if (sizes[0] != n_vis || n_vis < 1) return METOK_ERR_INVALID_ARG;
    for (int s = 0; s < n_levels; ++s) {
        if (sizes[s] < 1) return METOK_ERR_INVALID_ARG;
        if (!levels[s].token_group || !levels[s].origin) return METOK_ERR_INVALID_ARG;
    }
    // every level's arguments, shapes and workspace are checked before the first launch
    for (int s = 0; s < n_levels; ++s) {
        const metok_prune_level& lv = levels[s];
        int32_t budget[2];
        rc = metok_retention_budgets(alpha, r, s + 1, N0, budget);
        if (rc != METOK_OK) return rc;
        rc = validate_prefill_prune(lv.q_text, lv.k_all, lv.hidden, dtype, Hq, Hkv, Lt, S - n_vis + sizes[s], dh, D,
                                    vis_start, sizes[s], lv.token_group, 2, budget, softmax_scale, lv.scores,
                                    lv.keep_idx, lv.S_out, lv.hidden_out, ws, ws_bytes);
        if (rc != METOK_OK) return rc;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    {
        METOK_TIMED("schedule_init_kernel", st);
        schedule_init_kernel<<<1, 1024, 0, st>>>(levels[0].token_group, n_vis, N0[0], N0[1], levels[0].origin, status);
    }
    METOK_LAUNCH_CHECK();
    for (int s = 0; s < n_levels; ++s) {
        const metok_prune_level& lv = levels[s];
        int32_t budget[2];
        rc = metok_retention_budgets(alpha, r, s + 1, N0, budget);
        if (rc != METOK_OK) return rc;
        const int S_s = S - n_vis + sizes[s];
        rc = metok_prefill_prune(lv.q_text, lv.k_all, lv.hidden, dtype, Hq, Hkv, Lt, S_s, dh, D, vis_start, sizes[s],
                                 lv.token_group, 2, budget, softmax_scale, lv.scores, lv.keep_idx, lv.S_out,
                                 lv.hidden_out, ws, ws_bytes, stream);
        if (rc != METOK_OK) return rc;
        // the level's status word (start of the workspace, cleared again by the next level) is folded
        // into the caller's; this kernel also hands classes and origins to the next level
        const bool more = s + 1 < n_levels;
        const metok_prune_level& nx = levels[more ? s + 1 : s];
        {
            METOK_TIMED("schedule_propagate_kernel", st);
            schedule_propagate_kernel<<<more ? ceil_div(sizes[s + 1], 256) : 1, 256, 0, st>>>(
                lv.keep_idx, vis_start, sizes[s], more ? sizes[s + 1] : 0, lv.token_group, lv.origin, nx.token_group,
                nx.origin, reinterpret_cast<const int32_t*>(ws), status);
        }
        METOK_LAUNCH_CHECK();
    }
    return METOK_OK;
}
