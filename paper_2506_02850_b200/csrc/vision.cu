// metok_compress_vision: text relevance and key events (Eq. 5), per-event key-token
// top-k, merge-assign of the remaining tokens and averaging.
#include <algorithm>
#include <cstdlib>

#include "common.cuh"
#include "select.cuh"
#include "select_block.cuh"
#include "sm100.cuh"
#include "launchers.h"

namespace metok {

// --------------------------------------------------------------------------- //
// token_score[j] = <x_j, t> / (max(|x_j|, eps) * max(|t|, eps)); also 1/max(|x_j|, eps).
// One warp per token row, 16-byte loads, four chunks in flight per lane.
// --------------------------------------------------------------------------- //
template <typename T>
__global__ void __launch_bounds__(256)
tok_score_kernel(const T* __restrict__ feats, const T* __restrict__ text, int Nv, int d,
                 float* __restrict__ token_score, float* __restrict__ inv_norm) {
    constexpr int VN = Vec16<T>::N;
    extern __shared__ float s_t[];                 // [d]
    __shared__ float s_red[8];
    __shared__ float s_tn;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nchunk = d / VN;
    // t is stored in planes of 4 floats per chunk so that a lane's 16-byte reads
    // of consecutive chunks are bank-conflict free
    for (int i = tid; i < d; i += 256) {
        const int c = i / VN, q = i % VN;
        s_t[(q >> 2) * (nchunk * 4) + c * 4 + (q & 3)] = to_float(text[i]);
    }
    __syncthreads();
    float a = 0.f;
    for (int i = tid; i < d; i += 256) a = fmaf(s_t[i], s_t[i], a);
    a = warp_sum(a);
    if (lane == 0) s_red[warp] = a;
    __syncthreads();
    if (tid == 0) {
        float s = 0.f;
        for (int w = 0; w < 8; ++w) s += s_red[w];
        s_tn = fmaxf(sqrtf(s), kEps);
    }
    __syncthreads();
    const float tn = s_tn;
    // rows from the last one down: the pass before this one (segmentation) streams V upwards
    // and leaves its tail in L2
    for (int rr = blockIdx.x * 8 + warp; rr < Nv; rr += gridDim.x * 8) {
        const int row = Nv - 1 - rr;
        const T* x = feats + (size_t)row * d;
        float nn = 0.f, dt = 0.f;
        constexpr int U = 8;                        // 16-byte chunks in flight per lane
        for (int c0 = 0; c0 < nchunk; c0 += 32 * U) {
            uint4 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int c = c0 + u * 32 + lane;
                raw[u] = c < nchunk ? __ldg(reinterpret_cast<const uint4*>(x) + c) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < nchunk) {
                    float v[VN];
                    if constexpr (sizeof(T) == 4) {
                        v[0] = __uint_as_float(raw[u].x); v[1] = __uint_as_float(raw[u].y);
                        v[2] = __uint_as_float(raw[u].z); v[3] = __uint_as_float(raw[u].w);
                    } else {
                        const uint32_t w[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            v[2 * i]     = __uint_as_float(w[i] << 16);
                            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
                        }
                    }
#pragma unroll
                    for (int h = 0; h < VN / 4; ++h) {
                        const float4 tt = reinterpret_cast<const float4*>(s_t + h * (nchunk * 4))[c];
                        nn = fmaf(v[4 * h + 0], v[4 * h + 0], nn);
                        dt = fmaf(v[4 * h + 0], tt.x, dt);
                        nn = fmaf(v[4 * h + 1], v[4 * h + 1], nn);
                        dt = fmaf(v[4 * h + 1], tt.y, dt);
                        nn = fmaf(v[4 * h + 2], v[4 * h + 2], nn);
                        dt = fmaf(v[4 * h + 2], tt.z, dt);
                        nn = fmaf(v[4 * h + 3], v[4 * h + 3], nn);
                        dt = fmaf(v[4 * h + 3], tt.w, dt);
                    }
                }
            }
        }
        nn = warp_sum(nn);
        dt = warp_sum(dt);
        if (lane == 0) {
            const float n = fmaxf(sqrtf(nn), kEps);
            token_score[row] = dt / (n * tn);
            inv_norm[row] = 1.0f / n;
        }
    }
}

// Index e with off[e] <= t < off[e+1] in an ascending offset array off[0..k].
__device__ __forceinline__ int find_event(const int32_t* __restrict__ off, int k, int t) {
    int lo = 0, hi = k;                     // off[lo] <= t < off[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (off[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// Event scores, key events, per-event token budgets and output offsets.  One CTA.
struct PlanParams {
    int Tn, N, k, n_key_events, event_agg, mode, tile_rows, chunk_cols;
    int grid, s1, s2, s1_nonkey, s2_nonkey;     // POOL: side of the token grid and the four strides
    double keep_key, keep_nonkey, beta;
    const uint8_t* key_given;                   // the caller's key events, or null
    const uint8_t* key_frames_given;            // POOL: the caller's key frames, or null
};

// The workspace regions that later kernels of the call expect cleared: written here, at the start of
// the call's first kernel, instead of by separate memset nodes (each costs the chain a launch).
struct PlanClears {
    void* zero_a; size_t zero_a_bytes;      // packed argmax per token (tensor-core path), may be null
    void* zero_b; size_t zero_b_bytes;      // member bits, member counts, long-list counters
    void* ones;   size_t ones_bytes;        // output -> long-list index, all bits set = none
    int32_t* status;                        // device status word
};
// part `part` of `parts` of the fill; p 16-byte aligned, bytes % 4 == 0
__device__ __forceinline__ void block_fill(void* p, size_t bytes, uint32_t word, int part, int parts) {
    if (!p) return;
    uint4* q = reinterpret_cast<uint4*>(p);
    const size_t n16 = bytes / 16;
    for (size_t i = (size_t)part * blockDim.x + threadIdx.x; i < n16; i += (size_t)parts * blockDim.x)
        q[i] = make_uint4(word, word, word, word);
    uint32_t* t = reinterpret_cast<uint32_t*>(q + n16);
    if (part == 0)
        for (size_t i = threadIdx.x; i < (bytes - n16 * 16) / 4; i += blockDim.x) t[i] = word;
}
constexpr int kPlanFillCtas = 8;

__global__ void __launch_bounds__(1024)
event_plan_kernel(const float* __restrict__ token_score, float* __restrict__ frame_score,
                  const int32_t* __restrict__ event_offsets, PlanParams pp,
                  float* __restrict__ event_score, uint8_t* __restrict__ event_is_key,
                  int32_t* __restrict__ ev_lo, int32_t* __restrict__ ev_budget, int32_t* __restrict__ ev_out_off,
                  int32_t* __restrict__ ev_tile_off, int32_t* __restrict__ ev_unit_off,
                  int32_t* __restrict__ frame_ev, int32_t* __restrict__ frame_stride,
                  int32_t* __restrict__ frame_off, int32_t* __restrict__ n_out, PlanClears clr) {
    grid_dep_wait();
    extern __shared__ float s_score[];      // [k]
    if (blockIdx.x > 0) {                   // CTAs 1 .. kPlanFillCtas only clear; CTA 0 plans
        block_fill(clr.zero_a, clr.zero_a_bytes, 0u, (int)blockIdx.x - 1, kPlanFillCtas);
        block_fill(clr.zero_b, clr.zero_b_bytes, 0u, (int)blockIdx.x - 1, kPlanFillCtas);
        block_fill(clr.ones, clr.ones_bytes, 0xFFFFFFFFu, (int)blockIdx.x - 1, kPlanFillCtas);
        return;
    }
    if (threadIdx.x == 0) *clr.status = 0;
    __shared__ int s_scan[1024];
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int k = pp.k, Tn = pp.Tn;
    // frame_score[f] = mean of the frame's N token scores; eight lanes per frame (a lane's loads are
    // independent), fixed shuffle tree; the scores stay in shared memory for the event loops below
    float* s_frame = s_score + k;           // [Tn]
    int* s_evlo = reinterpret_cast<int*>(s_frame + Tn);     // [k] first frame of the event, clamped
    int* s_evhi = s_evlo + k;                                // [k] one past its last frame
    int* s_bud = s_evhi + k;                                 // [k] budget of the event
    unsigned char* s_key = reinterpret_cast<unsigned char*>(s_bud + k);   // [k]
    for (int f0 = 0; f0 < Tn; f0 += nthr >> 3) {
        const int f = f0 + (tid >> 3), part = tid & 7;
        float s = 0.f;
        if (f < Tn) {
            constexpr int kB = 6;                           // loads in flight; the additions keep their order
            for (int p0 = part; p0 < pp.N; p0 += 8 * kB) {
                float x[kB];
#pragma unroll
                for (int u = 0; u < kB; ++u) x[u] = p0 + 8 * u < pp.N ? token_score[(size_t)f * pp.N + p0 + 8 * u] : 0.f;
#pragma unroll
                for (int u = 0; u < kB; ++u)
                    if (p0 + 8 * u < pp.N) s += x[u];
            }
        }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (f < Tn && part == 0) {
            s_frame[f] = s / (float)pp.N;
            frame_score[f] = s_frame[f];
        }
    }
    __syncthreads();
    for (int e = tid; e < k; e += nthr) {
        int lo = min(max(event_offsets[e], 0), Tn);
        int hi = min(max(event_offsets[e + 1], lo), Tn);
        ev_lo[e] = lo;
        if (e == k - 1) ev_lo[k] = hi;
        s_evlo[e] = lo;
        s_evhi[e] = hi;
        float s;
        if (hi <= lo) {
            s = -3.0e38f;
        } else if (pp.event_agg == METOK_AGG_MEAN) {
            float a = 0.f;
            for (int f = lo; f < hi; ++f) a += s_frame[f];
            s = a / (float)(hi - lo);
        } else {
            float a = s_frame[lo];
            for (int f = lo + 1; f < hi; ++f) a = fmaxf(a, s_frame[f]);
            s = a;
        }
        s_score[e] = s;
        event_score[e] = s;
    }
    __syncthreads();
    for (int e = tid; e < k; e += nthr) {
        const float v = s_score[e];
        int rank = 0;
        for (int j = 0; j < k; ++j) {
            const float w = s_score[j];
            rank += (w > v) || (w == v && j < e);
        }
        const bool key = pp.key_given ? pp.key_given[e] != 0 : rank < pp.n_key_events;
        event_is_key[e] = (uint8_t)key;
        s_key[e] = (unsigned char)key;
    }
    __syncthreads();
    if (pp.mode == METOK_MODE_TOPK_MERGE) {
        for (int e = tid; e < k; e += nthr) {
            const int m = (s_evhi[e] - s_evlo[e]) * pp.N;
            const double ratio = s_key[e] ? pp.keep_key : pp.keep_nonkey;
            const double c = ratio * (double)m - 1e-9;
            long long b = (long long)c;
            if ((double)b < c) b += 1;
            if (b < 1) b = 1;
            if (b > m) b = m;
            ev_budget[e] = (int)b;
            s_bud[e] = (int)b;
        }
        __syncthreads();
        if (tid == 0) {                                     // everything it reads is in shared memory
            int slots = 0, tiles = 0, units = 0;
            for (int e = 0; e < k; ++e) {
                ev_out_off[e] = slots;
                ev_tile_off[e] = tiles;
                ev_unit_off[e] = units;
                slots += s_bud[e];
                const int t = ((s_evhi[e] - s_evlo[e]) * pp.N + pp.tile_rows - 1) / pp.tile_rows;
                tiles += t;
                units += t * ((s_bud[e] + pp.chunk_cols - 1) / pp.chunk_cols);   // row tiles x key chunks
            }
            ev_out_off[k] = slots;
            ev_tile_off[k] = tiles;
            ev_unit_off[k] = units;
            *n_out = slots;
        }
    } else {
        // Algorithm 1: key frames = the ceil(beta * len) best-scored frames of every event (ties to the
        // lower frame); a frame's stride follows from its event's and its own class; the pooled
        // frames are laid out in temporal order.
        for (int f = tid; f < Tn; f += nthr) frame_ev[f] = 0;
        __syncthreads();
        for (int e = tid; e < k; e += nthr) {
            const int lo = min(max(event_offsets[e], 0), Tn);
            const int hi = min(max(event_offsets[e + 1], lo), Tn);
            for (int f = lo; f < hi; ++f) frame_ev[f] = e;
        }
        __syncthreads();
        for (int f = tid; f < Tn; f += nthr) {
            const int e = frame_ev[f];
            const int lo = min(max(event_offsets[e], 0), Tn);
            const int hi = min(max(event_offsets[e + 1], lo), Tn);
            const int len = hi - lo;
            const double c = pp.beta * (double)len - 1e-9;
            long long nk = (long long)c;
            if ((double)nk < c) nk += 1;
            if (nk < 1) nk = 1;
            if (nk > len) nk = len;
            const float v = s_frame[f];
            int rank = 0;
            for (int j = lo; j < hi; ++j) {
                const float w = s_frame[j];
                rank += (w > v) || (w == v && j < f);
            }
            const bool key_frame = pp.key_frames_given ? pp.key_frames_given[f] != 0 : rank < (int)nk;
            frame_stride[f] = event_is_key[e] ? (key_frame ? pp.s1 : pp.s2) : (key_frame ? pp.s1_nonkey : pp.s2_nonkey);
        }
        __syncthreads();
        // exclusive scan of the pooled sizes: contiguous ranges per thread, then a scan of the range totals
        const int per = (Tn + nthr - 1) / nthr;
        const int lo = min(Tn, tid * per), hi = min(Tn, lo + per);
        int local = 0;
        for (int f = lo; f < hi; ++f) {
            const int go = (pp.grid + frame_stride[f] - 1) / frame_stride[f];
            local += go * go;
        }
        s_scan[tid] = local;
        __syncthreads();
        for (int off = 1; off < nthr; off <<= 1) {
            const int v = (tid >= off) ? s_scan[tid - off] : 0;
            __syncthreads();
            s_scan[tid] += v;
            __syncthreads();
        }
        int run = s_scan[tid] - local;
        for (int f = lo; f < hi; ++f) {
            frame_off[f] = run;
            const int go = (pp.grid + frame_stride[f] - 1) / frame_stride[f];
            run += go * go;
        }
        if (tid == nthr - 1) { frame_off[Tn] = s_scan[tid]; *n_out = s_scan[tid]; }
    }
}

// --------------------------------------------------------------------------- //
// Adaptive pooling (Algorithm 1): one CTA per output token = one window of one frame's
// G x G token grid, window = stride, edge windows clipped to the grid.  The window's
// cells are added in row-major order in fp32 (two rows of V in flight per thread),
// divided by their number and rounded once.
// --------------------------------------------------------------------------- //
constexpr int kPoolThreads = 128;
constexpr int kPoolChunks = 4;

template <typename T>
__global__ void __launch_bounds__(kPoolThreads)
pool_kernel(const T* __restrict__ feats, int d, int N, int G, int Tn, const int32_t* __restrict__ frame_off,
            const int32_t* __restrict__ frame_stride, const int32_t* __restrict__ frame_ev,
            const int32_t* __restrict__ n_out, T* __restrict__ out_feats, int32_t* __restrict__ out_src,
            int32_t* __restrict__ out_event, int32_t* __restrict__ out_members, int32_t* __restrict__ assign) {
    constexpr int VN = Vec16<T>::N;
    const int o = blockIdx.x;
    if (o >= *n_out) return;
    const int f = find_event(frame_off, Tn, o);
    const int w = o - frame_off[f];
    const int s = frame_stride[f];
    const int go = (G + s - 1) / s;
    const int r0 = (w / go) * s, r1 = min(G, r0 + s);
    const int c0 = (w % go) * s, c1 = min(G, c0 + s);
    const int wc = c1 - c0, cells = (r1 - r0) * wc;
    const int tid = threadIdx.x;
    const int nchunk = d / VN;
    const size_t frame_base = (size_t)f * N;
    auto cell_token = [&](int i) { return frame_base + (size_t)(r0 + i / wc) * G + (c0 + i % wc); };
    for (int cb = 0; cb < nchunk; cb += kPoolThreads * kPoolChunks) {
        float acc[kPoolChunks][VN];
#pragma unroll
        for (int u = 0; u < kPoolChunks; ++u) Vec16<T>::zero(acc[u]);
        int i = 0;
        for (; i + 1 < cells; i += 2) {
            const T* x0 = feats + cell_token(i) * d;
            const T* x1 = feats + cell_token(i + 1) * d;
            float v0[kPoolChunks][VN], v1[kPoolChunks][VN];
#pragma unroll
            for (int u = 0; u < kPoolChunks; ++u) {
                const int ch = cb + u * kPoolThreads + tid;
                if (ch < nchunk) {
                    Vec16<T>::load(x0 + (size_t)ch * VN, v0[u]);
                    Vec16<T>::load(x1 + (size_t)ch * VN, v1[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < kPoolChunks; ++u) {
                const int ch = cb + u * kPoolThreads + tid;
                if (ch < nchunk) {
#pragma unroll
                    for (int q = 0; q < VN; ++q) acc[u][q] = (acc[u][q] + v0[u][q]) + v1[u][q];
                }
            }
        }
        if (i < cells) {
            const T* x0 = feats + cell_token(i) * d;
#pragma unroll
            for (int u = 0; u < kPoolChunks; ++u) {
                const int ch = cb + u * kPoolThreads + tid;
                if (ch < nchunk) {
                    float v0[VN];
                    Vec16<T>::load(x0 + (size_t)ch * VN, v0);
#pragma unroll
                    for (int q = 0; q < VN; ++q) acc[u][q] += v0[q];
                }
            }
        }
        const float inv = 1.0f / (float)cells;
#pragma unroll
        for (int u = 0; u < kPoolChunks; ++u) {
            const int ch = cb + u * kPoolThreads + tid;
            if (ch < nchunk) {
                T* dst = out_feats + (size_t)o * d + (size_t)ch * VN;
                alignas(16) T tmp[VN];
#pragma unroll
                for (int q = 0; q < VN; ++q) from_float(tmp[q], acc[u][q] * inv);
                *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(tmp);
            }
        }
    }
    for (int i = tid; i < cells; i += kPoolThreads) assign[cell_token(i)] = o;
    if (tid == 0) {
        out_src[o] = (int32_t)cell_token(0);
        out_event[o] = frame_ev[f];
        out_members[o] = cells;
    }
}

// Per-event key-token top-k: one cluster per event.
__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads)
event_topk_kernel(const float* __restrict__ token_score, const int32_t* __restrict__ ev_lo, int N,
                  const int32_t* __restrict__ ev_budget, const int32_t* __restrict__ ev_out_off, SelectLayout lay,
                  uint8_t* __restrict__ is_key, int32_t* __restrict__ out_src, int32_t* __restrict__ out_event,
                  int32_t* __restrict__ assign) {
    __shared__ SelectSmem sm;
    __shared__ int s_budget[1];
    extern __shared__ __align__(16) unsigned char sel_dyn[];
    const int e = blockIdx.x / kSelCluster;
    const int lo = ev_lo[e] * N, hi = ev_lo[e + 1] * N;
    const int n = hi - lo;
    if (n <= 0) return;                                   // the whole cluster leaves together
    SelectCtx cx;
    cx.rank = (int)cx.cl.block_rank();
    cx.G = 1;
    cx.nb_log2 = lay.nb_log2;
    int p_lo, p_hi;
    select_slice(n, cx.rank, &p_lo, &p_hi);
    cx.item_lo = p_lo;
    cx.m = p_hi - p_lo;
    cx.cached = cx.m <= lay.cache_cap;
    cx.hist = reinterpret_cast<uint32_t*>(sel_dyn + lay.hist_off);
    cx.merged = reinterpret_cast<uint32_t*>(sel_dyn + lay.merged_off);
    cx.keys = reinterpret_cast<uint32_t*>(sel_dyn + lay.keys_off);
    cx.cls = sel_dyn + lay.cls_off;
    if (threadIdx.x == 0) s_budget[0] = ev_budget[e];
    __syncthreads();
    const float* s = token_score + lo;
    auto cls = [](int) { return 0; };
    auto val = [s](int i) { return s[i]; };
    cluster_select(cx, n, cls, val, s_budget, sm);
    const int slot0 = ev_out_off[e];
    auto flag = [&](int i) { return is_selected(sm, 0, item_at(cx, i - p_lo, cls, val).key, i); };
    auto emit = [&](int i, int rank) {
        const int slot = slot0 + rank;
        out_src[slot] = lo + i;
        out_event[slot] = e;
        assign[lo + i] = slot;
    };
    for (int i = p_lo + threadIdx.x; i < p_hi; i += blockDim.x) is_key[lo + i] = flag(i) ? 1 : 0;
    cluster_compact(cx, p_lo, p_hi, flag, emit, sm);
}

// The same by one CTA per event, when the largest event a segmentation can produce fits a
// CTA's shared memory (select_block.cuh): no cluster barriers.
__global__ void __launch_bounds__(kBsThreads, 1)
event_block_topk_kernel(const float* __restrict__ token_score, const int32_t* __restrict__ ev_lo, int N,
                        const int32_t* __restrict__ ev_budget, const int32_t* __restrict__ ev_out_off,
                        BlockSelLayout lay, uint8_t* __restrict__ is_key, int32_t* __restrict__ out_src,
                        int32_t* __restrict__ out_event, int32_t* __restrict__ assign) {
    grid_dep_wait();
    __shared__ BlockSelSmem sm;
    __shared__ int s_budget[1];
    extern __shared__ __align__(16) unsigned char sel_dyn[];
    const int e = blockIdx.x;
    const int lo = ev_lo[e] * N, hi = ev_lo[e + 1] * N;
    const int n = hi - lo;
    if (n <= 0) return;
    const int tid = threadIdx.x;
    if (tid == 0) s_budget[0] = ev_budget[e];
    __syncthreads();
    const BlockSelView sel = block_sel_run<true>(sm, sel_dyn, lay, token_score + lo, nullptr, n, 1, s_budget);
    const int slot0 = ev_out_off[e];
    const int n4 = (n + 3) >> 2;
    for (int q = tid; q < n4; q += kBsThreads) {
        const uint32_t m = sel.mask[q >> 3];
        const int sh = (q & 7) * 4;
        const uint32_t nib = (m >> sh) & 15u;
        int slot = slot0 + sel.woff[q >> 3] + __popc(m & ((1u << sh) - 1u));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = q * 4 + u;
            if (i < n) {
                const bool key = (nib >> u) & 1u;
                is_key[lo + i] = key ? 1 : 0;
                if (key) {
                    out_src[slot] = lo + i;
                    out_event[slot] = e;
                    assign[lo + i] = slot;
                    ++slot;
                }
            }
        }
    }
}

// --------------------------------------------------------------------------- //
// Merge-assign, generic CUDA-core path (fp32 inputs, and any shape the tensor-core
// path does not take).  CTA = 64 token rows of one event; loops over the event's
// key tokens 64 at a time; fp32 accumulate; fused row argmax of dot * inv_norm(key).
// --------------------------------------------------------------------------- //
constexpr int kMergeTM = 64, kMergeTN = 64, kMergeTK = 32;


template <typename T>
__global__ void __launch_bounds__(256)
merge_assign_simt_kernel(const T* __restrict__ feats, int d, int N, const int32_t* __restrict__ ev_lo, int k,
                         const int32_t* __restrict__ ev_out_off, const int32_t* __restrict__ ev_tile_off,
                         const int32_t* __restrict__ out_src, const float* __restrict__ inv_norm,
                         const uint8_t* __restrict__ is_key, int32_t* __restrict__ assign) {
    constexpr int VN = Vec16<T>::N;
    constexpr int CPR = kMergeTK / VN;      // 16-byte chunks per tile row
    constexpr int LD = kMergeTM + 1;
    __shared__ float As[kMergeTK][LD];
    __shared__ float Bs[kMergeTK][LD];
    __shared__ int s_src[kMergeTN];
    __shared__ float s_inv[kMergeTN];
    const int t = blockIdx.x;
    if (t >= ev_tile_off[k]) return;
    const int e = find_event(ev_tile_off, k, t);
    const int row0 = ev_lo[e] * N + (t - ev_tile_off[e]) * kMergeTM;
    const int row_end = ev_lo[e + 1] * N;
    const int s0 = ev_out_off[e], s1 = ev_out_off[e + 1];
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;

    float best_v[4];
    int best_s[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { best_v[i] = -3.4e38f; best_s[i] = 0x7FFFFFFF; }

    for (int n0 = s0; n0 < s1; n0 += kMergeTN) {
        __syncthreads();
        if (tid < kMergeTN) {
            const int slot = n0 + tid;
            const int src = slot < s1 ? out_src[slot] : -1;
            s_src[tid] = src;
            s_inv[tid] = src >= 0 ? inv_norm[src] : 0.f;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        for (int k0 = 0; k0 < d; k0 += kMergeTK) {
            for (int c = tid; c < kMergeTM * CPR; c += 256) {
                const int r = c / CPR, ch = c % CPR;
                const int kk = k0 + ch * VN;
                float va[VN], vb[VN];
                const int row = row0 + r;
                if (row < row_end && kk < d) Vec16<T>::load(feats + (size_t)row * d + kk, va);
                else Vec16<T>::zero(va);
                const int src = s_src[r];
                if (src >= 0 && kk < d) Vec16<T>::load(feats + (size_t)src * d + kk, vb);
                else Vec16<T>::zero(vb);
#pragma unroll
                for (int q = 0; q < VN; ++q) {
                    As[ch * VN + q][r] = va[q];
                    Bs[ch * VN + q][r] = vb[q];
                }
            }
            __syncthreads();
#pragma unroll 8
            for (int kk = 0; kk < kMergeTK; ++kk) {
                float a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) a[i] = As[kk][ty + 16 * i];
#pragma unroll
                for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx + 16 * j];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {                 // ascending slot within this thread
            const int col = tx + 16 * j;
            const int slot = n0 + col;
            if (slot < s1) {
                const float inv = s_inv[col];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float v = acc[i][j] * inv;
                    if (v > best_v[i]) { best_v[i] = v; best_s[i] = slot; }
                }
            }
        }
    }
    // combine the 16 column owners of each row: larger value, then lower slot
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xFFFFFFFFu, best_v[i], o);
            const int os = __shfl_xor_sync(0xFFFFFFFFu, best_s[i], o);
            if (ov > best_v[i] || (ov == best_v[i] && os < best_s[i])) { best_v[i] = ov; best_s[i] = os; }
        }
        const int row = row0 + ty + 16 * i;
        if (tx == 0 && row < row_end && !is_key[row]) assign[row] = best_s[i];
    }
}


// --------------------------------------------------------------------------- //
// Merge-assign on the tensor cores (bf16).
//
// Work unit = up to 256 consecutive token rows of one event x one chunk of the event's
// key tokens (up to 256 columns; an event's keys are cut into equal chunks).  The two
// 128-row halves of a unit are two accumulators in TMEM (2 x 256 columns) that share
// every key tile brought into shared memory: the main loop is fed at a fixed rate per
// SM, so what counts is the work done per byte loaded -- a 256 x 256 unit needs a third
// fewer bytes per flop than a 128 x 256 one.  The units of all events form one list; a
// persistent CTA takes every gridDim-th unit.
//   warp 0   : TMA producer -- per 64-wide K step one 256x64 (or, for an event's last
//              rows, 128x64) tile of V (rows are contiguous in V), 3-stage ring that
//              runs on across units;
//   warps 10-13: key producers -- the chunk's key rows are rows of V scattered over the
//              event, so their 128-byte slices come by 16-byte asynchronous copies
//              straight from V into the ring, written in the 128-byte swizzle the MMA
//              expects (eight threads per row, sixteen rows per thread and K step); the
//              copies of a stage report to the stage's barrier when they have landed;
//   warp 1   : allocates TMEM, issues tcgen05.mma (M=128, N=16..256, K=16), two per K
//              slice (one per row half), and commits to the ring / accumulator barriers;
//   warps 2-9: epilogue, four warps per row half -- read the accumulator with
//              tcgen05.ld, scale each column by 1/|key|, take the (value, slot) argmax of
//              the thread's row over the chunk.
// Chunks of one row tile may be handled by different CTAs: a row's result is combined
// with a 64-bit atomicMax on (order-preserving key of the value) << 32 | ~slot, which
// does not depend on the order of arrival (larger value first, then the lower slot).
// Every wait is bounded; on a timeout the CTA unwinds and writes METOK_ERR_TIMEOUT.
// --------------------------------------------------------------------------- //
constexpr int kMmaBM = 256, kMmaBK = 64, kMmaBN = 256, kMmaStages = 3;
constexpr int kMmaThreads = 448;
constexpr int kMmaKeyThreads = 128;                        // warps 10-13
constexpr uint32_t kMmaABytes = kMmaBM * kMmaBK * 2;       // 32 KiB
constexpr uint32_t kMmaBBytes = kMmaBN * kMmaBK * 2;       // 32 KiB
constexpr size_t kMmaSmemBytes = (size_t)kMmaStages * (kMmaABytes + kMmaBBytes) + 1024;

struct MergeUnit { int row0, row_end, col0, nvalid; };     // rows of V; first key slot and number of keys

__device__ __forceinline__ MergeUnit merge_unit(int u, const int32_t* __restrict__ ev_unit_off,
                                                const int32_t* __restrict__ ev_lo,
                                                const int32_t* __restrict__ ev_out_off, int k, int N) {
    const int e = find_event(ev_unit_off, k, u);
    const int s0 = ev_out_off[e], nk = ev_out_off[e + 1] - s0;
    const int nchunks = (nk + kMmaBN - 1) / kMmaBN;
    const int cols = (((nk + nchunks - 1) / nchunks) + 15) & ~15;       // equal chunks, whole MMA columns
    const int local = u - ev_unit_off[e];
    const int tile = local / nchunks, c = local - tile * nchunks;
    MergeUnit m;
    m.row0 = ev_lo[e] * N + tile * kMmaBM;
    m.row_end = ev_lo[e + 1] * N;
    m.col0 = s0 + c * cols;
    m.nvalid = min(cols, nk - c * cols);
    return m;
}

__global__ void __launch_bounds__(kMmaThreads, 1)
merge_assign_mma_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA_half,
                        const __nv_bfloat16* __restrict__ feats, int d, int N,
                        const int32_t* __restrict__ ev_lo, int k, const int32_t* __restrict__ ev_out_off,
                        const int32_t* __restrict__ ev_unit_off, const int32_t* __restrict__ out_src,
                        const float* __restrict__ inv_norm, const uint8_t* __restrict__ is_key,
                        unsigned long long* __restrict__ best64, int32_t* __restrict__ status) {
    grid_dep_wait();
    using namespace sm100;
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t full_bar[kMmaStages], empty_bar[kMmaStages], tfull_bar, tempty_bar, drain_bar;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ float s_keyinv[2][kMmaBN];

    const int total_units = ev_unit_off[k];
    if ((int)blockIdx.x >= total_units) return;
    const int ksteps = (d + kMmaBK - 1) / kMmaBK;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        // a stage is full when the tile of V has landed (one arrival with its byte count) and every
        // key-producer thread's copies have (one arrival each)
        for (int s = 0; s < kMmaStages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1 + kMmaKeyThreads); mbar_init(smem_u32(&empty_bar[s]), 1); }
        mbar_init(smem_u32(&tfull_bar), 1);
        mbar_init(smem_u32(&tempty_bar), 8);
        mbar_init(smem_u32(&drain_bar), 1);
        s_abort = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;

    // The two single-thread loops below run once per K step with nothing to hide their latency:
    // stage and phase are counted (no division), addresses and descriptor words only move by adds.
    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmA_half);
            int s = 0, issued = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
                const MergeUnit mu = merge_unit(u, ev_unit_off, ev_lo, ev_out_off, k, N);
                const bool two = mu.row_end - mu.row0 > 128;           // both row halves hold rows of the event
                const CUtensorMap* a0 = two ? &tmA : &tmA_half;
                const uint32_t tx = two ? kMmaABytes : kMmaABytes / 2;
                for (int ks = 0; ks < ksteps; ++ks) {
                    if (!mbar_wait(smem_u32(&empty_bar[0]) + 8u * s, ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = smem_u32(&full_bar[0]) + 8u * s;
                    mbar_arrive_expect_tx(fb, tx);
                    if (!(dbg_withhold(status, kDbgMergeAssign) && blockIdx.x == 0 && issued == 0))   // debug builds: one copy never sent
                        tma_load_2d(smem_base + (uint32_t)s * (kMmaABytes + kMmaBBytes), a0, ks * kMmaBK, mu.row0, fb);
                    ++issued;
                    if (++s == kMmaStages) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA's shared memory goes away
                for (int back = 1; back <= kMmaStages && back <= issued; ++back) {
                    const int j = issued - back;
                    mbar_wait(smem_u32(&full_bar[j % kMmaStages]), (uint32_t)(j / kMmaStages) & 1u, abort_flag);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int s = 0, n = 0;
            uint32_t ph = 0;
            bool ok = true;
            const uint32_t a_lo0 = desc_k128_lo(smem_base);
            constexpr uint32_t kStageWords = (kMmaABytes + kMmaBBytes) >> 4, kBWords = kMmaABytes >> 4,
                               kHalfWords = (kMmaABytes / 2) >> 4;
            for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++n) {
                const MergeUnit mu = merge_unit(u, ev_unit_off, ev_lo, ev_out_off, k, N);
                const bool two = mu.row_end - mu.row0 > 128;
                if (!mbar_wait(smem_u32(&tempty_bar), ((uint32_t)n & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = make_idesc_bf16(128, (mu.nvalid + 15) & ~15);
                for (int ks = 0; ks < ksteps; ++ks) {
                    if (!mbar_wait(smem_u32(&full_bar[0]) + 8u * s, ph, abort_flag)) { ok = false; break; }
                    fence_proxy_async();                             // the key rows were written by ordinary (non-bulk) copies
                    tc_fence_after();
                    const uint32_t a_lo = a_lo0 + (uint32_t)s * kStageWords, b_lo = a_lo + kBWords;
                    const uint32_t acc0 = ks != 0 ? 1u : 0u;
                    if (two) {                                       // rows 128..255 of the tile: 16 KiB further on
#pragma unroll
                        for (int kk = 0; kk < kMmaBK / 16; ++kk) {
                            umma_bf16_words(tmem_base, a_lo + 2 * kk, b_lo + 2 * kk, idesc, kk ? 1u : acc0);
                            umma_bf16_words(tmem_base + kMmaBN, a_lo + kHalfWords + 2 * kk, b_lo + 2 * kk, idesc, kk ? 1u : acc0);
                        }
                    } else {
#pragma unroll
                        for (int kk = 0; kk < kMmaBK / 16; ++kk)
                            umma_bf16_words(tmem_base, a_lo + 2 * kk, b_lo + 2 * kk, idesc, kk ? 1u : acc0);
                    }
                    umma_commit(smem_u32(&empty_bar[0]) + 8u * s);   // frees the stage when these MMAs retire
                    if (++s == kMmaStages) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&tfull_bar));         // both accumulators of this unit complete
            }
            if (!ok) {                                             // wait until whatever was issued has retired
                umma_commit(smem_u32(&drain_bar));
                mbar_wait(smem_u32(&drain_bar), 0u, abort_flag);
            }
        }
    } else if (warp >= 10) {
        // Key producers.  Thread pt copies 16-byte chunk c = pt % 8 of the rows r = pt / 8 + 16 i,
        // i = 0..15, of the chunk's keys: eight consecutive threads read the 128 contiguous bytes of
        // one row's K slice.  In the swizzled tile row r lies at r * 128 bytes and its chunk c at
        // position c ^ (r % 8).  Rows past the chunk's keys up to the next multiple of 16 (the MMA's
        // column count) are written as zeros; rows beyond are not touched.
        const int pt = (int)threadIdx.x - 320, c = pt & 7, rsub = pt >> 3;
        const uint32_t dst0 = smem_base + kMmaABytes + (uint32_t)rsub * 128u + (uint32_t)((c ^ (rsub & 7)) << 4);   // (r % 8) == (rsub % 8)
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
            const MergeUnit mu = merge_unit(u, ev_unit_off, ev_lo, ev_out_off, k, N);
            const int npad = (mu.nvalid + 15) & ~15;
            const __nv_bfloat16* src[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = rsub + 16 * i;
                const int row = r < mu.nvalid ? (int)dbg_bound(out_src[mu.col0 + r], (long long)ev_lo[k] * N, status) : 0;
                src[i] = feats + (size_t)row * d + c * 8;
            }
            for (int ks = 0; ks < ksteps; ++ks) {
                if (!mbar_wait(smem_u32(&empty_bar[0]) + 8u * s, ph ^ 1u, abort_flag)) { ok = false; break; }
                const uint32_t dst = dst0 + (uint32_t)s * (kMmaABytes + kMmaBBytes);
                // a K slice that reaches past d (d is a multiple of 8, not of 64) reads zeros there
                const bool in_k = ks * kMmaBK + c * 8 < d;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int r = rsub + 16 * i;
                    if (r < npad)
                        cp_async16_zfill(dst + (uint32_t)i * 2048u, src[i] + (in_k ? ks * kMmaBK : 0),
                                         (r < mu.nvalid && in_k) ? 16u : 0u);
                }
                cp_async_arrive_noinc(smem_u32(&full_bar[0]) + 8u * s);   // arrives when this thread's copies have landed
                if (++s == kMmaStages) { s = 0; ph ^= 1u; }
            }
        }
        cp_async_wait_all();                                       // nothing may land after the CTA's shared memory is gone
    } else {
        const int grp = warp & 3;                                   // TMEM lanes 32*grp .. 32*grp+31
        const int half = (warp - 2) >> 2;                           // row half = accumulator
        const int et = (warp - 2) * 32 + lane;                      // 0..255 among the epilogue threads
        bool ok = true;
        int n = 0;
        for (int u = blockIdx.x; u < total_units; u += gridDim.x, ++n) {
            const MergeUnit mu = merge_unit(u, ev_unit_off, ev_lo, ev_out_off, k, N);
            const int b = n & 1;                                    // s_keyinv alternates: a slow warp may still read the last one
            s_keyinv[b][et] = (et < mu.nvalid) ? inv_norm[out_src[mu.col0 + et]] : 0.f;
            named_bar_sync(1, 256);
            if (ok && !mbar_wait(smem_u32(&tfull_bar), (uint32_t)n & 1u, abort_flag)) ok = false;
            ok = __all_sync(0xFFFFFFFFu, ok);                      // tcgen05.ld below is warp-collective
            if (!ok) continue;                                     // keep meeting the others at the named barrier
            tc_fence_after();
            const int row = mu.row0 + half * 128 + grp * 32 + lane;
            float best_v = -3.4e38f;
            int best_c = 0;
            if (half == 0 || mu.row_end - mu.row0 > 128) {          // the second accumulator of a short unit holds nothing
                const uint32_t t_row = tmem_base + ((uint32_t)(grp * 32) << 16) + (uint32_t)half * kMmaBN;
                for (int c0 = 0; c0 < mu.nvalid; c0 += 32) {
                    float v[32];
                    tmem_ld32(t_row + (uint32_t)c0, v);
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int col = c0 + j;
                        const float val = v[j] * s_keyinv[b][col];
                        if (col < mu.nvalid && val > best_v) { best_v = val; best_c = col; }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tempty_bar));
            if (row < mu.row_end && !is_key[row]) {
                const unsigned long long packed =
                    ((unsigned long long)float_key(best_v) << 32) | (unsigned long long)(~(uint32_t)(mu.col0 + best_c));
                atomicMax(&best64[row], packed);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0 && s_abort) *status = METOK_ERR_TIMEOUT;
}

// An event's tokens are cut into at most 64 blocks of this many tokens; per output token one
// bit per block says whether the block holds a member.
__host__ __device__ __forceinline__ int avg_block_tokens(int m) {
    const int g = (((m + 63) / 64) + 3) & ~3;
    return g < 256 ? 256 : g;
}

// assign[row] of every non-key token from the packed argmax (tensor-core path; best64 is null when
// the CUDA-core kernel has written assign itself), and the member-block bits of every output token.
__global__ void __launch_bounds__(256)
merge_decode_kernel(const unsigned long long* __restrict__ best64, const uint8_t* __restrict__ is_key, int Nv,
                    int N, const int32_t* __restrict__ ev_lo, int k, int32_t* __restrict__ assign,
                    unsigned long long* __restrict__ slot_blocks, int32_t* __restrict__ slot_cnt,
                    int32_t* __restrict__ long_index, int32_t* __restrict__ long_slot,
                    int32_t* __restrict__ long_counter, int long_threshold, int long_cap,
                    int32_t* __restrict__ few_members, int few_cap, int32_t* __restrict__ heavy_index,
                    int32_t* __restrict__ heavy_slot, int32_t* __restrict__ heavy_counter, int heavy_threshold,
                    int heavy_cap,
                    const int32_t* __restrict__ n_out) {
    grid_dep_wait();
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= Nv) return;
    int slot;
    if (best64 && !is_key[row]) {
        slot = (int32_t)(~(uint32_t)(best64[row] & 0xFFFFFFFFull));
        assign[row] = slot;
    } else {
        slot = assign[row];
    }
    // a token whose unit gave up on a wait has no maximum: it stays out of every member list (the
    // call's status word already says that the results are not valid)
    if (slot < 0 || slot >= *n_out) return;
    const int e = find_event(ev_lo, k, row / N);
    const int lo = ev_lo[e] * N, m = ev_lo[e + 1] * N - lo;
    atomicOr(&slot_blocks[slot], 1ull << ((row - lo) / avg_block_tokens(m)));
    // member count; the token that takes an output past the threshold books scratch for it (which
    // scratch an output gets depends on arrival order, what is computed in it does not)
    const int pos = atomicAdd(&slot_cnt[slot], 1);
    if (pos < few_cap) few_members[(size_t)slot * few_cap + pos] = row;   // the first few_cap arrivals are listed
    if (pos == heavy_threshold) {                             // many members: an output to be started early
        const int hh = atomicAdd(heavy_counter, 1);
        heavy_index[slot] = hh;
        if (hh < heavy_cap) heavy_slot[hh] = slot;
    }
    if (pos == long_threshold) {
        const int l = atomicAdd(long_counter, 1);
        long_index[slot] = l;
        if (l < long_cap) long_slot[l] = slot;
    }
}

// --------------------------------------------------------------------------- //
// Averaging: one CTA per output token.  Only the blocks of the event that hold a member
// (one bit each, set by merge_decode) are searched: their `assign` entries are read in
// passes in which every thread takes a contiguous run (16-byte loads, all issued before
// the first is looked at), the matches are packed in token order by one block-wide
// scan, and the member rows are then added in that order (so the
// summation order is fixed).  The rows come in by bulk copies into shared memory, up to
// kAvgStages rows at once (usually all members of an output), so that the bytes in
// flight do not depend on registers.  fp32 sum, one division, one rounding.
// --------------------------------------------------------------------------- //
constexpr int kAvgThreads = 128;
constexpr int kAvgChunks = 4;      // 16-byte chunks per thread per pass over d
constexpr int kAvgQuads = 5;       // 16-byte groups of `assign` per thread and pass
constexpr int kAvgStages = 3;      // member rows in flight when a pass over a row fills a stage (more than 4 KiB); the same
                                   // bytes hold 6 or 12 shorter rows (template parameter NST of the kernel)
constexpr int kAvgList = 512;      // members listed at a time
constexpr int kAvgStageBytes = kAvgThreads * kAvgChunks * 16;
constexpr size_t kAvgSmemBytes = (size_t)kAvgStages * kAvgStageBytes + 128;
constexpr int kAvgFew = 32;        // outputs with at most this many members get them listed by merge_decode (a warp ranks them)
constexpr int kAvgHeavy = 16;      // outputs with more members than this are listed to be started first
constexpr int kAvgLong = 32;       // outputs with more members than this (= kAvgFew: the others need no search) are split ...
constexpr int kAvgParts = 8;       // ... over up to this many CTAs (fp32 partial sums, added in part order)
constexpr int kAvgLongCapMax = 1024;   // most long outputs that get scratch for their partial sums ...
constexpr size_t kAvgLongBytes = (size_t)32 << 20;   // ... within this much scratch
constexpr int kAvgHeavyCap = 2048;  // outputs with more than kAvgHeavy members that are listed to be started first
constexpr int kAvgFrontCtas = 8 * kNumSMs;   // CTAs at the front of the grid that take the listed outputs and parts
// long outputs that get scratch: as many as kAvgLongBytes hold (kAvgParts rows of d floats each)
__host__ __device__ inline int avg_long_cap(int d) {
    const long long c = (long long)(kAvgLongBytes / ((size_t)kAvgParts * (size_t)d * sizeof(float)));
    return (int)(c < 64 ? 64 : c > kAvgLongCapMax ? kAvgLongCapMax : c);
}
// parts of an output with `count` > kAvgLong members: about eight members each if they lie evenly
__host__ __device__ inline int avg_parts(int count) {
    const int p = (count + 7) / 8;
    return p < kAvgParts ? p : kAvgParts;
}

// One (output, part): the members of output c in this part's share of the search, added in token order.
// What a CTA needs to know about its output before it can fetch a row; the loads are independent of
// one another, so a caller issues them together with whatever else it has to look up about the output.
struct AvgMeta {
    int count, few_tok, li, e;
    unsigned long long blocks;
};
__device__ __forceinline__ AvgMeta avg_meta(int c, const int32_t* __restrict__ slot_cnt,
                                            const int32_t* __restrict__ few_members,
                                            const int32_t* __restrict__ long_index,
                                            const int32_t* __restrict__ out_event,
                                            const unsigned long long* __restrict__ slot_blocks) {
    AvgMeta m;
    const int lane = threadIdx.x & 31;
    m.few_tok = lane < kAvgFew ? few_members[(size_t)c * kAvgFew + lane] : 0;
    m.count = slot_cnt[c];
    m.li = long_index[c];
    m.e = out_event[c];
    m.blocks = slot_blocks[c];
    return m;
}

template <typename T, int NST>
__device__ __forceinline__ void
merge_avg_item(int c, int part, const AvgMeta& meta, uint32_t& phase, uint8_t* avg_dyn, uint64_t* s_bar, int* s_list, int* s_wtot,
               int* s_blocks, int* s_abort_p, int* s_last_p,
               const T* __restrict__ feats, int d, int N, int Nv, const int32_t* __restrict__ ev_lo,
               const int32_t* __restrict__ out_event, const int32_t* __restrict__ assign,
               const unsigned long long* __restrict__ slot_blocks, const int32_t* __restrict__ slot_cnt,
               const int32_t* __restrict__ long_index, const int32_t* __restrict__ few_members,
               float* __restrict__ long_sums, int32_t* __restrict__ long_done, T* __restrict__ out_feats, int32_t* __restrict__ out_members,
               int32_t* __restrict__ status) {
    using namespace sm100;
    constexpr int VN = Vec16<T>::N;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int& s_abort = *s_abort_p;
    int& s_last = *s_last_p;
    // an output with at most kAvgFew members has them listed by merge_decode (in arrival order):
    // fetched together with the output's other data, no search of `assign`
    const int few_tok = meta.few_tok;
    const int count = meta.count;
    const bool few = count <= kAvgFew;
    int li = meta.li;
    if (li >= avg_long_cap(d)) li = -1;                        // no scratch left: one CTA does it all
    const int nparts = li >= 0 ? avg_parts(count) : 1;
    const int e = meta.e;
    const int lo = ev_lo[e] * N, hi = ev_lo[e + 1] * N;
    const int nchunk = d / VN;
    const int4* assign4 = reinterpret_cast<const int4*>(assign);
    const uint32_t stage0 = (smem_u32(avg_dyn) + 127u) & ~127u;
    constexpr int nst = NST;
    constexpr uint32_t stage_stride = (uint32_t)(kAvgStages * kAvgStageBytes) / NST;   // a pass over a row moves no more
    // the blocks to search, in order; a block is searched as bt/4 + 1 groups of four tokens (its
    // first token need not start a group)
    const unsigned long long blocks = meta.blocks;
    const int nblk = __popcll(blocks);
    const int bt = avg_block_tokens(hi - lo), qpb = bt / 4 + 1;
    const int total_q = nblk * qpb;
    // a part takes an equal share of the groups to search (not of the members): what it finds there
    // it adds up, so an output's search is done once however many parts it has
    const int q_per = (total_q + nparts - 1) / nparts;
    const int q_begin = min(total_q, part * q_per), q_end = min(total_q, q_begin + q_per);
    if (few) {
        if (warp == 0) {                                       // into token order: rank = members before it
            const int mine = lane < count ? few_tok : 0x7FFFFFFF;
            int rank = 0;
            for (int j = 0; j < count; ++j) rank += __shfl_sync(0xFFFFFFFFu, mine, j) < mine;
            if (lane < count) s_list[rank] = mine;
        }
    } else if (tid == 0) {
        unsigned long long mm = blocks;
        for (int i = 0; mm; ++i, mm &= mm - 1) s_blocks[i] = __ffsll((long long)mm) - 1;
    }
    __syncthreads();
    volatile int* abort_flag = &s_abort;
    for (int cb = 0; cb < nchunk; cb += kAvgThreads * kAvgChunks) {
        const uint32_t seg_bytes = (uint32_t)min(kAvgThreads * kAvgChunks, nchunk - cb) * 16u;
        float acc[kAvgChunks][VN];
#pragma unroll
        for (int u = 0; u < kAvgChunks; ++u) Vec16<T>::zero(acc[u]);
        // the listed members' rows, nst in flight, added in list order
        auto consume = [&](int nlist) {
        // a ring: row m goes to stage m % nst; the stage is refilled with row m + nst as
        // soon as every thread has added row m, so nst rows stay in flight until the list ends
        auto issue = [&](int m) {
            const int j = m % nst;                             // nst is a constant: no division
            const uint32_t bar = smem_u32(&s_bar[j]);
            mbar_arrive_expect_tx(bar, seg_bytes);
            const long long src_row = dbg_bound(s_list[m], Nv, status);
            if (!(dbg_withhold(status, kDbgMergeAvg) && blockIdx.x == (unsigned)kAvgFrontCtas && m == 0 && cb == 0))   // debug builds: one copy never sent
                bulk_load(stage0 + (uint32_t)j * stage_stride, feats + (size_t)src_row * d + (size_t)cb * VN, seg_bytes, bar);
        };
        if (tid == 0)
            for (int m = 0; m < nlist && m < nst; ++m) issue(m);
        for (int m = 0; m < nlist; ++m) {
            const int j = m % nst;
            const bool ok = mbar_wait(smem_u32(&s_bar[j]), (phase >> j) & 1u, abort_flag);
            phase ^= 1u << j;
            if (ok) {
                const uint8_t* row = avg_dyn + (stage0 - smem_u32(avg_dyn)) + (size_t)j * stage_stride;
#pragma unroll
                for (int u = 0; u < kAvgChunks; ++u) {
                    const int ch = cb + u * kAvgThreads + tid;
                    if (ch < nchunk) {
                        const uint4 raw = *reinterpret_cast<const uint4*>(row + (size_t)(u * kAvgThreads + tid) * 16);
                        float v[VN];
                        if constexpr (sizeof(T) == 4) {
                            v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y);
                            v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
                        } else {
                            const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                v[2 * i]     = __uint_as_float(w4[i] << 16);
                                v[2 * i + 1] = __uint_as_float(w4[i] & 0xFFFF0000u);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < VN; ++q) acc[u][q] += v[q];
                    }
                }
            }
            __syncthreads();                                   // every thread is done with stage j
            if (tid == 0 && m + nst < nlist && !*abort_flag) issue(m + nst);
        }
        };
        if (few) {
            consume(count);                                    // s_list holds them already
        } else {
        // a thread's run is qpt consecutive groups: as few as cover the search in one pass
        const int qpt = max(1, min(kAvgQuads, (q_end - q_begin + kAvgThreads - 1) / kAvgThreads));
        for (int qs = q_begin; qs < q_end; qs += kAvgThreads * qpt) {
            int4 a[kAvgQuads];
            int qidx[kAvgQuads], j_lo[kAvgQuads], j_hi[kAvgQuads];   // group index; the block's token range
#pragma unroll
            for (int u = 0; u < kAvgQuads; ++u) {
                const int qf = qs + tid * qpt + u;
                a[u] = make_int4(-1, -1, -1, -1);
                qidx[u] = 0; j_lo[u] = 0; j_hi[u] = 0;
                if (u < qpt && qf < q_end) {
                    const int bi = qf / qpb, wq = qf - bi * qpb;
                    const int st = lo + s_blocks[bi] * bt;
                    const int q = (st >> 2) + wq;
                    qidx[u] = q; j_lo[u] = st; j_hi[u] = min(st + bt, hi);
                    if (q * 4 + 3 < Nv) {
                        a[u] = assign4[q];
                    } else {                                   // the array ends inside this group
                        if (q * 4 + 0 < Nv) a[u].x = assign[q * 4 + 0];
                        if (q * 4 + 1 < Nv) a[u].y = assign[q * 4 + 1];
                        if (q * 4 + 2 < Nv) a[u].z = assign[q * 4 + 2];
                    }
                }
            }
            unsigned match = 0;                                // bit 4u+i: token 4*qidx[u]+i belongs to output c
#pragma unroll
            for (int u = 0; u < kAvgQuads; ++u) {
                if (u >= qpt) break;
                const int j = qidx[u] * 4;
                match |= (unsigned)(a[u].x == c && j + 0 >= j_lo[u] && j + 0 < j_hi[u]) << (4 * u + 0);
                match |= (unsigned)(a[u].y == c && j + 1 >= j_lo[u] && j + 1 < j_hi[u]) << (4 * u + 1);
                match |= (unsigned)(a[u].z == c && j + 2 >= j_lo[u] && j + 2 < j_hi[u]) << (4 * u + 2);
                match |= (unsigned)(a[u].w == c && j + 3 >= j_lo[u] && j + 3 < j_hi[u]) << (4 * u + 3);
            }
            const int mine = __popc(match);
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31) s_wtot[warp] = incl;
            __syncthreads();
            int before = incl - mine, total = 0;               // rank of this thread's first member in the pass
#pragma unroll
            for (int w = 0; w < kAvgThreads / 32; ++w) {
                const int v = s_wtot[w];
                if (w < warp) before += v;
                total += v;
            }
            // the members of the pass, listed kAvgList at a time
            for (int b0 = 0; b0 < total; b0 += kAvgList) {
                const int nlist = min(kAvgList, total - b0);
                {
                    unsigned mm = match;
                    int r = before;
                    while (mm) {
                        const int b = __ffs(mm) - 1;
                        mm &= mm - 1;
                        if (r >= b0 && r < b0 + nlist) s_list[r - b0] = qidx[b >> 2] * 4 + (b & 3);
                        ++r;
                    }
                }
                __syncthreads();
                consume(nlist);
            }
            __syncthreads();                                   // s_wtot and s_list are reused by the next pass
        }
        }
        if (nparts == 1) {
            const float inv = 1.0f / (float)count;
#pragma unroll
            for (int u = 0; u < kAvgChunks; ++u) {
                const int ch = cb + u * kAvgThreads + tid;
                if (ch < nchunk) {
                    T* o = out_feats + (size_t)c * d + (size_t)ch * VN;
                    alignas(16) T tmp[VN];
#pragma unroll
                    for (int q = 0; q < VN; ++q) from_float(tmp[q], acc[u][q] * inv);
                    *reinterpret_cast<uint4*>(o) = *reinterpret_cast<const uint4*>(tmp);
                }
            }
        } else {
            float* ps = long_sums + ((size_t)li * kAvgParts + part) * d;
#pragma unroll
            for (int u = 0; u < kAvgChunks; ++u) {
                const int ch = cb + u * kAvgThreads + tid;
                if (ch < nchunk) {
#pragma unroll
                    for (int q = 0; q < VN; ++q) ps[(size_t)ch * VN + q] = acc[u][q];
                }
            }
        }
    }
    if (part == 0 && tid == 0) out_members[c] = count;
    if (tid == 0 && s_abort) *status = METOK_ERR_TIMEOUT;
    if (nparts > 1) {
        // the last part to finish adds the partial sums in part order
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = atomicAdd(&long_done[li], 1) == nparts - 1;
        __syncthreads();
        if (s_last) {
            __threadfence();
            const float inv = 1.0f / (float)count;
            const float* ps = long_sums + (size_t)li * kAvgParts * d;
            // four elements per thread and trip, the parts' loads all in flight, added in part order
            // (d is a multiple of 4: rows are whole 16-byte chunks)
            for (int i = tid * 4; i < d; i += kAvgThreads * 4) {
                float4 v[kAvgParts];
#pragma unroll
                for (int q = 0; q < kAvgParts; ++q)
                    v[q] = q < nparts ? __ldcg(reinterpret_cast<const float4*>(ps + (size_t)q * d + i))
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int q = 0; q < kAvgParts; ++q) {
                    if (q < nparts) { a.x += v[q].x; a.y += v[q].y; a.z += v[q].z; a.w += v[q].w; }
                }
                T* o = out_feats + (size_t)c * d + i;
                from_float(o[0], a.x * inv); from_float(o[1], a.y * inv);
                from_float(o[2], a.z * inv); from_float(o[3], a.w * inv);
            }
        }
    }
}

template <typename T, int NST>
__global__ void __launch_bounds__(kAvgThreads, 8)
merge_avg_kernel(const T* __restrict__ feats, int d, int N, int Nv, const int32_t* __restrict__ ev_lo,
                 const int32_t* __restrict__ out_event, const int32_t* __restrict__ assign,
                 const unsigned long long* __restrict__ slot_blocks, const int32_t* __restrict__ slot_cnt,
                 const int32_t* __restrict__ long_index, const int32_t* __restrict__ long_slot,
                 const int32_t* __restrict__ long_counter, const int32_t* __restrict__ few_members,
                 const int32_t* __restrict__ heavy_index, const int32_t* __restrict__ heavy_slot,
                 const int32_t* __restrict__ heavy_counter,
                 float* __restrict__ long_sums, int32_t* __restrict__ long_done, int front_ctas, const int32_t* __restrict__ n_out,
                 T* __restrict__ out_feats, int32_t* __restrict__ out_members, int32_t* __restrict__ status) {
    grid_dep_wait();
    using namespace sm100;
    extern __shared__ uint8_t avg_dyn[];
    __shared__ __align__(8) uint64_t s_bar[NST];
    __shared__ int s_list[kAvgList];
    __shared__ int s_wtot[kAvgThreads / 32];
    __shared__ int s_blocks[64];
    __shared__ int s_abort, s_last;
    // A CTA adds the rows of its output about three at a time, one memory latency per three rows:
    // an output with many members lasts many times longer than the usual one, and would set the
    // kernel's time if it started late.  So merge_decode lists every output with more than kAvgHeavy
    // members, and the first front_ctas CTAs of the grid take the listed work round-robin, before the
    // other outputs' CTAs start: the outputs with more than kAvgLong members part by part (up to
    // kAvgParts parts, each an equal share of the blocks to search, partial sums combined in part
    // order by the last part to finish), the others whole (their members are listed: no search).
    // A listed output's own CTA leaves at once.  The other CTAs start
    // in index order and take the outputs from the last one down, so that this pass begins with the
    // rows of V that the preceding (ascending) pass left in L2.
    const int tid = threadIdx.x;
    const int long_cap = avg_long_cap(d);
    if (tid == 32) {                                           // not thread 0: it is busy with the block list below
        for (int j = 0; j < NST; ++j) mbar_init(smem_u32(&s_bar[j]), 1);
        s_abort = 0;
        mbar_fence_init();
    }
    uint32_t phase = 0;                                        // bit j: parity of the next completion of barrier j
#define METOK_AVG_ITEM(C, PART, META)                                                                                     \
    merge_avg_item<T, NST>(C, PART, META, phase, avg_dyn, s_bar, s_list, s_wtot, s_blocks, &s_abort, &s_last, feats, d, N, Nv,  \
                      ev_lo, out_event, assign, slot_blocks, slot_cnt, long_index, few_members, long_sums, long_done,  \
                      out_feats, out_members, status)
    if ((int)blockIdx.x >= front_ctas) {
        const int c = *n_out - 1 - ((int)blockIdx.x - front_ctas);
        if (c < 0) return;
        // everything about output c in one round trip: whether it is listed, and what its own CTA needs if not
        const int hh = heavy_index[c];
        const AvgMeta meta = avg_meta(c, slot_cnt, few_members, long_index, out_event, slot_blocks);
        if ((hh >= 0 && hh < kAvgHeavyCap) || (meta.li >= 0 && meta.li < long_cap)) return;   // listed: the front CTAs have it
        METOK_AVG_ITEM(c, 0, meta);
        return;
    }
    const int n_long = min(*long_counter, long_cap), n_heavy = min(*heavy_counter, kAvgHeavyCap);
    const int n_items = n_long * kAvgParts + n_heavy;
    for (int it = (int)blockIdx.x; it < n_items; it += front_ctas) {
        int c, part;
        if (it < n_long * kAvgParts) {
            c = long_slot[it / kAvgParts];
            part = it % kAvgParts;
            if (part >= avg_parts(slot_cnt[c])) continue;
        } else {
            c = heavy_slot[it - n_long * kAvgParts];
            part = 0;
            const int li = long_index[c];
            if (li >= 0 && li < long_cap) continue;            // split into parts: taken above
        }
        const AvgMeta meta = avg_meta(c, slot_cnt, few_members, long_index, out_event, slot_blocks);
        METOK_AVG_ITEM(c, part, meta);
        __syncthreads();                                       // the shared lists are reused by the next item
    }
#undef METOK_AVG_ITEM
}

// --------------------------------------------------------------------------- //
// host side
// --------------------------------------------------------------------------- //
struct VisionWs {
    int32_t* status;          // device status word, first in the workspace
    float* inv_norm;
    uint8_t* is_key;
    int32_t *ev_lo, *ev_budget, *ev_out_off, *ev_tile_off, *ev_unit_off;
    int32_t *frame_ev, *frame_stride, *frame_off;   // POOL mode
    unsigned long long* best64;   // packed argmax per token (tensor-core path)
    unsigned long long* slot_blocks;   // per output token: which blocks of its event hold a member
    int32_t* slot_cnt;                 // per output token: members
    int32_t* long_counter;             // outputs with more than kAvgLong members ...
    int32_t* long_done;                // ... parts of each that have finished
    int32_t* long_index;               // output -> index among the long ones, -1 otherwise
    int32_t* long_slot;                // and back
    int32_t* heavy_counter;            // outputs with more than kAvgHeavy members ...
    int32_t* heavy_index;              // ... output -> index among them, -1 otherwise (directly after long_index)
    int32_t* heavy_slot;               // ... and back
    int32_t* few_members;              // per output token: its first kAvgFew members, in arrival order
    float* long_sums;                  // partial sums of their parts
    size_t zero_bytes;                 // slot_blocks .. long_done are cleared together
};

static VisionWs carve_vision(Carver& cv, int Tn, int N, int k, int d, int cap, bool mma) {
    VisionWs w;
    w.status = cv.take<int32_t>(64);
    w.inv_norm = cv.take<float>((size_t)Tn * N);
    w.is_key = cv.take<uint8_t>((size_t)Tn * N);
    w.ev_lo = cv.take<int32_t>((size_t)k + 1);
    w.ev_budget = cv.take<int32_t>((size_t)k + 1);
    w.ev_out_off = cv.take<int32_t>((size_t)k + 1);
    w.ev_tile_off = cv.take<int32_t>((size_t)k + 1);
    w.ev_unit_off = cv.take<int32_t>((size_t)k + 1);
    w.frame_ev = cv.take<int32_t>((size_t)Tn);
    w.frame_stride = cv.take<int32_t>((size_t)Tn);
    w.frame_off = cv.take<int32_t>((size_t)Tn + 1);
    w.best64 = mma ? cv.take<unsigned long long>((size_t)Tn * N) : nullptr;
    {
        const size_t n = (size_t)cap + 64;
        w.zero_bytes = n * 8 + n * 4 + (size_t)(64 + kAvgLongCapMax + 64) * 4;
        unsigned char* z = cv.take<unsigned char>(w.zero_bytes);
        w.slot_blocks = reinterpret_cast<unsigned long long*>(z);
        w.slot_cnt = reinterpret_cast<int32_t*>(z + n * 8);
        w.long_counter = w.slot_cnt + n;
        w.long_done = w.long_counter + 64;
        w.heavy_counter = w.long_done + kAvgLongCapMax;
        w.long_index = cv.take<int32_t>(2 * n);         // long_index, then heavy_index: filled with -1 together
        w.heavy_index = w.long_index + n;
        w.heavy_slot = cv.take<int32_t>(kAvgHeavyCap);
        w.long_slot = cv.take<int32_t>(kAvgLongCapMax);
        w.few_members = cv.take<int32_t>(n * kAvgFew);
        w.long_sums = cv.take<float>((size_t)avg_long_cap(d) * kAvgParts * d);
    }
    return w;
}

// The tensor-core merge path needs bf16 rows that TMA can address (16-byte row pitch);
// METOK_DEBUG_FORCE_SIMT=1 in the environment selects the CUDA-core kernels (debugging aid).
static bool use_mma_path(int d) {
    static const bool force_simt = [] { const char* e = getenv("METOK_DEBUG_FORCE_SIMT"); return e && e[0] == '1'; }();
    return !force_simt && d % 8 == 0;
}

static bool ratio_ok(double r) { return r > 0.0 && r <= 1.0; }

template <typename T>
static int launch_vision(const void* feats_, int Tn, int N, int d, const int32_t* event_offsets, int k,
                         const void* text_, const metok_vision_params* p, void* out_feats_, int32_t* out_src,
                         int32_t* out_event, int32_t* out_members, int32_t* assign, float* token_score,
                         float* frame_score, float* event_score, uint8_t* event_is_key, int32_t* n_out, int cap,
                         void* ws, cudaStream_t st) {
    const T* feats = reinterpret_cast<const T*>(feats_);
    const T* text = reinterpret_cast<const T*>(text_);
    T* out_feats = reinterpret_cast<T*>(out_feats_);
    const int Nv = Tn * N;
    constexpr bool kBf16 = sizeof(T) == 2;
    const bool mma = kBf16 && use_mma_path(d) && p->mode == METOK_MODE_TOPK_MERGE;
    Carver cv(ws);
    VisionWs w = carve_vision(cv, Tn, N, k, d, cap, mma);
    // (the status word and the scratch that must start cleared are written by event_plan_kernel)
    if (const int rc = debug_arm(w.status, st)) return rc;

    // Eq. 5 per token, unless the caller brings the scores and norms from metok_segment_score_events
    const float* inv_norm = p->token_inv_norm ? p->token_inv_norm : w.inv_norm;
    if (!p->token_inv_norm) {
        const int grid = min(ceil_div(Nv, 8), kNumSMs * 8);
        const size_t smem = (size_t)d * sizeof(float);
        if (smem > 48 * 1024)
            METOK_CUDA_TRY(cudaFuncSetAttribute(tok_score_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)smem));
        {
            METOK_TIMED("tok_score_kernel", st);
            tok_score_kernel<T><<<grid, 256, smem, st>>>(feats, text, Nv, d, token_score, w.inv_norm);
        }
        METOK_LAUNCH_CHECK();
    }
    PlanParams pp;
    pp.Tn = Tn; pp.N = N; pp.k = k;
    pp.n_key_events = min(k, ceilq(p->alpha * (double)k));
    pp.event_agg = p->event_agg; pp.mode = p->mode; pp.tile_rows = mma ? kMmaBM : kMergeTM;
    pp.chunk_cols = kMmaBN;
    pp.keep_key = p->keep_key; pp.keep_nonkey = p->keep_nonkey; pp.beta = p->beta;
    pp.key_given = p->key_events_given;
    pp.key_frames_given = p->key_frames_given;
    pp.grid = 1;
    while (pp.grid * pp.grid < N) ++pp.grid;
    pp.s1 = p->s1; pp.s2 = p->s2; pp.s1_nonkey = p->s1_nonkey; pp.s2_nonkey = p->s2_nonkey;
    const size_t plan_smem = (size_t)(k + Tn) * sizeof(float) + (size_t)k * (3 * sizeof(int) + 1);
    if (plan_smem > 40 * 1024)
        METOK_CUDA_TRY(cudaFuncSetAttribute(event_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)plan_smem));
    PlanClears clr;
    const bool merging = p->mode == METOK_MODE_TOPK_MERGE;
    clr.zero_a = mma ? w.best64 : nullptr;
    clr.zero_a_bytes = (size_t)Nv * sizeof(unsigned long long);
    clr.zero_b = merging ? w.slot_blocks : nullptr;
    clr.zero_b_bytes = w.zero_bytes;
    clr.ones = merging ? w.long_index : nullptr;
    clr.ones_bytes = 2 * ((size_t)cap + 64) * sizeof(int32_t);
    clr.status = w.status;
    {
        METOK_TIMED("event_plan_kernel", st);
        launch_chained(event_plan_kernel, dim3(1 + kPlanFillCtas), dim3(1024), plan_smem, st, token_score, frame_score, event_offsets, pp, event_score,
                                                                  event_is_key, w.ev_lo, w.ev_budget, w.ev_out_off,
                                                                  w.ev_tile_off, w.ev_unit_off, w.frame_ev,
                                                                  w.frame_stride, w.frame_off, n_out, clr);
    }
    METOK_LAUNCH_CHECK();

    if (p->mode == METOK_MODE_POOL) {
        {
            METOK_TIMED("pool_kernel", st);
            pool_kernel<T><<<cap, kPoolThreads, 0, st>>>(feats, d, N, pp.grid, Tn, w.frame_off, w.frame_stride,
                                                     w.frame_ev, n_out, out_feats, out_src, out_event, out_members,
                                                     assign);
        }
        METOK_LAUNCH_CHECK();
        return METOK_OK;
    }

    {
        // the cache is sized for the longest event there can be, the thread count for twice the mean
        // an event has at most Tn - (k - 1) frames
        const BlockSelLayout bl = block_sel_layout(1, (long long)(Tn - (k - 1)) * N, 0);
        if (bl.fits) {
            if (bl.bytes > 32 * 1024)
                METOK_CUDA_TRY(cudaFuncSetAttribute(event_block_topk_kernel,
                                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bl.bytes));
            METOK_TIMED("event_topk_kernel", st);
            launch_chained(event_block_topk_kernel, dim3(k), dim3(kBsThreads), bl.bytes, st, token_score, w.ev_lo, N, w.ev_budget, w.ev_out_off,
                                                                     bl, w.is_key, out_src, out_event, assign);
        } else {
            const SelectLayout lay = select_layout(1, select_items_per_cta((long long)(Tn - (k - 1)) * N));
            const int nthreads = select_threads(select_items_per_cta(2LL * Nv / k));
            if (lay.bytes > 32 * 1024)                    // static + dynamic beyond 48 KiB needs the opt-in
                METOK_CUDA_TRY(cudaFuncSetAttribute(event_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)lay.bytes));
            METOK_TIMED("event_topk_kernel", st);
            event_topk_kernel<<<k * kSelCluster, nthreads, lay.bytes, st>>>(
                token_score, w.ev_lo, N, w.ev_budget, w.ev_out_off, lay, w.is_key, out_src, out_event, assign);
        }
        METOK_LAUNCH_CHECK();
    }

    if (mma) {
        CUtensorMap tmA, tmA_half;
        int r2 = make_tmap_bf16_2d(&tmA, feats, (uint64_t)Nv, (uint64_t)d, kMmaBM);
        if (r2 != METOK_OK) return r2;
        r2 = make_tmap_bf16_2d(&tmA_half, feats, (uint64_t)Nv, (uint64_t)d, kMmaBM / 2);
        if (r2 != METOK_OK) return r2;
        METOK_CUDA_TRY(cudaFuncSetAttribute(merge_assign_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kMmaSmemBytes));
        {
            METOK_TIMED("merge_assign_mma_kernel", st);
            launch_chained(merge_assign_mma_kernel, dim3(kNumSMs), dim3(kMmaThreads), kMmaSmemBytes, st, 
                tmA, tmA_half, reinterpret_cast<const __nv_bfloat16*>(feats), d, N, w.ev_lo, k, w.ev_out_off, w.ev_unit_off, out_src, inv_norm, w.is_key, w.best64,
                w.status);
        }
        METOK_LAUNCH_CHECK();
    } else {
        const int max_tiles = Nv / kMergeTM + k;
        {
            METOK_TIMED("merge_assign_simt_kernel", st);
            merge_assign_simt_kernel<T><<<max_tiles, 256, 0, st>>>(feats, d, N, w.ev_lo, k, w.ev_out_off,
                                                                   w.ev_tile_off, out_src, inv_norm, w.is_key,
                                                                   assign);
        }
        METOK_LAUNCH_CHECK();
    }

    {
        METOK_TIMED("merge_decode_kernel", st);
        launch_chained(merge_decode_kernel, dim3(ceil_div(Nv, 256)), dim3(256), 0, st, mma ? w.best64 : nullptr, w.is_key, Nv, N, w.ev_lo, k,
                                                               assign, w.slot_blocks, w.slot_cnt, w.long_index,
                                                               w.long_slot, w.long_counter, kAvgLong, avg_long_cap(d),
                                                               w.few_members, kAvgFew, w.heavy_index, w.heavy_slot,
                                                               w.heavy_counter, kAvgHeavy, kAvgHeavyCap, n_out);
    }
    METOK_LAUNCH_CHECK();
    // rows in flight per CTA: a pass over a row moves at most seg0 bytes, the ring holds 24 KiB
    const uint32_t seg0 = (uint32_t)std::min<long long>(kAvgThreads * kAvgChunks, (long long)d * sizeof(T) / 16) * 16u;
    auto launch = [&](auto kernel) -> int {
        METOK_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAvgSmemBytes));
        {
            METOK_TIMED("merge_avg_kernel", st);
            launch_chained(kernel, dim3(kAvgFrontCtas + cap), dim3(kAvgThreads), kAvgSmemBytes, st,
                feats, d, N, Nv, w.ev_lo, out_event, assign, w.slot_blocks, w.slot_cnt, w.long_index, w.long_slot,
                w.long_counter, w.few_members, w.heavy_index, w.heavy_slot, w.heavy_counter, w.long_sums, w.long_done,
                kAvgFrontCtas, n_out, out_feats, out_members,
                w.status);
        }
        METOK_LAUNCH_CHECK();
        return METOK_OK;
    };
    if (seg0 > (uint32_t)kAvgStageBytes / 2) return launch(merge_avg_kernel<T, kAvgStages>);
    if (seg0 > (uint32_t)kAvgStageBytes / 4) return launch(merge_avg_kernel<T, 2 * kAvgStages>);
    return launch(merge_avg_kernel<T, 4 * kAvgStages>);
}

}  // namespace metok

using namespace metok;

static int vision_params_ok(const metok_vision_params* p, int N) {
    if (!p) return 0;
    if (!ratio_ok(p->alpha)) return 0;
    if (p->event_agg != METOK_AGG_MEAN && p->event_agg != METOK_AGG_MAX) return 0;
    if (p->mode == METOK_MODE_TOPK_MERGE) return ratio_ok(p->keep_key) && ratio_ok(p->keep_nonkey);
    if (p->mode == METOK_MODE_POOL) {
        if (!ratio_ok(p->beta)) return 0;
        if (p->s1 < 1 || p->s2 < 1 || p->s1_nonkey < 1 || p->s2_nonkey < 1) return 0;
        int g = 1;
        while (g * g < N) ++g;
        return g * g == N;
    }
    return 0;
}

extern "C" int metok_compress_vision_bound(int T, int N, int k, const metok_vision_params* p) {
    if (T < 1 || N < 1 || k < 1 || k > T || !vision_params_ok(p, N)) return METOK_ERR_INVALID_ARG;
    const long long Nv = (long long)T * N;
    if (p->mode == METOK_MODE_TOPK_MERGE) {
        const double r = p->keep_key > p->keep_nonkey ? p->keep_key : p->keep_nonkey;
        long long b = (long long)ceilq(r * (double)Nv) + k;     // sum of per-event ceilings
        if (b > Nv) b = Nv;
        return (int)b;
    }
    int smin = p->s1;
    if (p->s2 < smin) smin = p->s2;
    if (p->s1_nonkey < smin) smin = p->s1_nonkey;
    if (p->s2_nonkey < smin) smin = p->s2_nonkey;
    int g = 1;
    while (g * g < N) ++g;
    const int go = (g + smin - 1) / smin;
    return T * go * go;
}

extern "C" size_t metok_compress_vision_workspace_bytes(int dtype, int T, int N, int d, int k, int cap,
                                                        const metok_vision_params* p) {
    if (T < 1 || N < 1 || k < 1 || d < 1 || cap < 0) return 0;
    Carver cv(nullptr);
    carve_vision(cv, T, N, k, d, cap, dtype == METOK_BF16 && !(p && p->mode == METOK_MODE_POOL));
    return cv.total();
}

extern "C" int metok_compress_vision(const void* feats, int dtype, int T, int N, int d,
                                     const int32_t* event_offsets, int k, const void* text_emb,
                                     const metok_vision_params* p, void* out_feats, int32_t* out_src,
                                     int32_t* out_event, int32_t* out_members, int32_t* assign,
                                     float* token_score, float* frame_score, float* event_score,
                                     uint8_t* event_is_key, int32_t* n_out, int cap, void* ws, size_t ws_bytes,
                                     void* stream) {
    if (!feats || !event_offsets || !text_emb || !p || !out_feats || !out_src || !out_event || !out_members ||
        !assign || !token_score || !frame_score || !event_score || !event_is_key || !n_out)
        return METOK_ERR_INVALID_ARG;
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (T < 1 || N < 1 || d < 1 || k < 1 || k > T) return METOK_ERR_INVALID_ARG;
    if ((long long)T * N > 0x7FFFFFFFLL / 2) return METOK_ERR_INVALID_ARG;
    if (!vision_params_ok(p, N)) return METOK_ERR_INVALID_ARG;
    if (!aligned16(feats) || !aligned16(text_emb) || !aligned16(out_feats)) return METOK_ERR_INVALID_ARG;
    const int bound = metok_compress_vision_bound(T, N, k, p);
    if (bound < 0 || cap < bound) return METOK_ERR_INVALID_ARG;
    const int eb = dtype == METOK_F32 ? 4 : 2;
    if (((long long)d * eb) % 16 != 0 || T > 8192) return METOK_ERR_UNSUPPORTED;
    const size_t need = metok_compress_vision_workspace_bytes(dtype, T, N, d, k, cap, p);
    if (!ws || ws_bytes < need || !aligned16(ws)) return METOK_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (dtype == METOK_F32)
        return launch_vision<float>(feats, T, N, d, event_offsets, k, text_emb, p, out_feats, out_src, out_event,
                                    out_members, assign, token_score, frame_score, event_score, event_is_key,
                                    n_out, cap, ws, st);
    return launch_vision<__nv_bfloat16>(feats, T, N, d, event_offsets, k, text_emb, p, out_feats, out_src,
                                        out_event, out_members, assign, token_score, frame_score, event_score,
                                        event_is_key, n_out, cap, ws, st);
}
