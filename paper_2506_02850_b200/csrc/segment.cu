// metok_segment_events: adjacent-frame cosine similarity (Eq. 4) and the split at
// the k-1 lowest similarities.
//
// FLATTEN mode is one streaming pass over V.  The flattened frame vector (N*d
// elements) is cut into slabs of 256 threads x 4 x 16 bytes; a CTA walks a run of
// consecutive frames of one slab, keeps the previous frame's chunks in registers
// and accumulates <v_f, v_f> and <v_f, v_{f+1}> in fp32.  Per-(slab, frame)
// partial sums go to the workspace and are added in a fixed order by the finishing
// kernel, so the result does not depend on scheduling.
#include "common.cuh"

namespace metok {

constexpr int kSegThreads = 256;
constexpr int kSegUnroll = 4;     // 16-byte chunks per thread per frame
constexpr int kMaxFrames = 8192;

// Raw 16-byte chunk of either dtype, widened on use.
template <typename T>
__device__ __forceinline__ void widen16(const uint4& r, float (&v)[16 / sizeof(T)]) {
    if constexpr (sizeof(T) == 4) {
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y);
        v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    } else {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i]     = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
}

constexpr int kSegMaxRun = 16;    // frames per CTA at most

template <typename T>
__global__ void __launch_bounds__(kSegThreads)
seg_partial_kernel(const T* __restrict__ feats, int Tn, long long chunks_per_frame, int frames_per_cta,
                   float* __restrict__ part_dot, float* __restrict__ part_nrm) {
    constexpr int VN = Vec16<T>::N;
    constexpr int NW = kSegThreads / 32;
    __shared__ float s_nn[kSegMaxRun + 1][NW], s_dp[kSegMaxRun + 1][NW];
    const int slab = blockIdx.x;
    const int f0 = blockIdx.y * frames_per_cta;
    const int f1 = min(Tn, f0 + frames_per_cta);          // own frames [f0, f1)
    const int f_last = min(Tn - 1, f1);                   // halo frame for the last dot
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    long long chunk[kSegUnroll];
    bool ok[kSegUnroll];
#pragma unroll
    for (int u = 0; u < kSegUnroll; ++u) {
        chunk[u] = (long long)slab * (kSegThreads * kSegUnroll) + u * kSegThreads + tid;
        ok[u] = chunk[u] < chunks_per_frame;
    }
    const uint4* base = reinterpret_cast<const uint4*>(feats);
    auto fetch = [&](int f, uint4 (&r)[kSegUnroll]) {
        const uint4* frame = base + (size_t)f * (size_t)chunks_per_frame;
#pragma unroll
        for (int u = 0; u < kSegUnroll; ++u) r[u] = ok[u] ? __ldg(frame + chunk[u]) : make_uint4(0u, 0u, 0u, 0u);
    };
    uint4 prev[kSegUnroll], cur[kSegUnroll], nxt[kSegUnroll];   // raw chunks: widened when used
#pragma unroll
    for (int u = 0; u < kSegUnroll; ++u) prev[u] = make_uint4(0u, 0u, 0u, 0u);
    fetch(f0, cur);
    // the next frame's loads are in flight while this frame is reduced; nothing inside the
    // loop waits for another warp
    for (int f = f0; f <= f_last; ++f) {
        if (f < f_last) fetch(f + 1, nxt);
        float nn = 0.f, dp = 0.f;
#pragma unroll
        for (int u = 0; u < kSegUnroll; ++u) {
            float c[VN], p[VN];
            widen16<T>(cur[u], c);
            widen16<T>(prev[u], p);
#pragma unroll
            for (int e = 0; e < VN; ++e) {
                nn = fmaf(c[e], c[e], nn);
                dp = fmaf(c[e], p[e], dp);
            }
        }
        nn = warp_sum(nn);
        dp = warp_sum(dp);
        if (lane == 0) { s_nn[f - f0][warp] = nn; s_dp[f - f0][warp] = dp; }
#pragma unroll
        for (int u = 0; u < kSegUnroll; ++u) { prev[u] = cur[u]; cur[u] = nxt[u]; }
    }
    __syncthreads();
    // the warps' sums in warp order: <v_f, v_f> for own frames, <v_{f-1}, v_f> for every frame after the first
    const int nf = f_last - f0 + 1;
    if (tid < nf) {
        const int f = f0 + tid;
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) { a += s_nn[tid][w]; b += s_dp[tid][w]; }
        if (f < f1) part_nrm[(size_t)slab * Tn + f] = a;
        if (f > f0) part_dot[(size_t)slab * Tn + (f - 1)] = b;
    }
}

// MEANPOOL: mean over the N tokens of each frame, per 16-byte column chunk.
template <typename T>
__global__ void __launch_bounds__(128)
seg_mean_kernel(const T* __restrict__ feats, int N, int d, float* __restrict__ mean) {
    constexpr int VN = Vec16<T>::N;
    const int f = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c * VN >= d) return;
    const T* base = feats + ((size_t)f * N) * d + (size_t)c * VN;
    float acc[VN];
    Vec16<T>::zero(acc);
    for (int p = 0; p < N; ++p) {
        float v[VN];
        Vec16<T>::load(base + (size_t)p * d, v);
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[e] += v[e];
    }
    const float inv = 1.0f / (float)N;
#pragma unroll
    for (int e = 0; e < VN; ++e) mean[(size_t)f * d + c * VN + e] = acc[e] * inv;
}

// dot / norm of consecutive mean vectors: one CTA per frame, written as a single "slab".
__global__ void __launch_bounds__(256)
seg_meandot_kernel(const float* __restrict__ mean, int Tn, int d, float* __restrict__ part_dot,
                   float* __restrict__ part_nrm) {
    __shared__ float red[2][8];
    const int f = blockIdx.x;
    const float* a = mean + (size_t)f * d;
    const float* b = mean + (size_t)(f + 1 < Tn ? f + 1 : f) * d;
    float nn = 0.f, dp = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        nn = fmaf(a[i], a[i], nn);
        dp = fmaf(a[i], b[i], dp);
    }
    nn = warp_sum(nn);
    dp = warp_sum(dp);
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = nn; red[1][threadIdx.x >> 5] = dp; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float x = 0.f, y = 0.f;
        for (int w = 0; w < 8; ++w) { x += red[0][w]; y += red[1][w]; }
        part_nrm[f] = x;
        if (f + 1 < Tn) part_dot[f] = y;
    }
}

// Order-preserving key of a similarity; NaN (a non-finite frame) ranks above everything.
__device__ __forceinline__ uint32_t sim_key(float f) { return f != f ? 0xFFFFFFFFu : float_key(f); }

// Adds the slab partials in slab order, forms the cosines, picks the k-1 smallest
// (rank by counting; ties to the lower index) and writes boundaries, CSR offsets
// and per-frame event ids.  One CTA of 1024 threads; T <= kMaxFrames.
__global__ void __launch_bounds__(1024)
seg_finish_kernel(const float* __restrict__ part_dot, const float* __restrict__ part_nrm, int nslab,
                  int Tn, int k, float* __restrict__ sims, int32_t* __restrict__ boundaries,
                  int32_t* __restrict__ event_offsets, int32_t* __restrict__ frame_event) {
    grid_dep_wait();
    extern __shared__ float sm_f[];
    float* s_sim = sm_f;                                   // [Tn]   (Tn-1 used)
    float* s_nrm = sm_f + Tn;                              // [Tn]
    int* s_flag = reinterpret_cast<int*>(sm_f + 2 * Tn);   // [Tn]  boundary after frame i
    __shared__ int s_scan[32];
    const int tid = threadIdx.x, nthr = blockDim.x;

    // The partial sums: 128 consecutive frames per sweep, eight groups of 128 threads; a group takes the
    // slabs 8 apart, so a warp's load is 128 contiguous bytes of one slab (one CTA's L1 handles a sector
    // per cycle: whole sectors matter), six loads in flight; the eight groups' sums are then added in
    // group order.
    __shared__ float s_pn[8][128], s_pd[8][128];
    for (int f0 = 0; f0 < Tn; f0 += 128) {
        const int fl = tid & 127, part = tid >> 7;            // nthr == 1024
        const int f = f0 + fl;
        float a = 0.f, b = 0.f;
        if (f < Tn) {
            const bool has_dot = f < Tn - 1;
            constexpr int kB = 6;                           // loads in flight; the additions keep their order
            for (int s0 = part; s0 < nslab; s0 += 8 * kB) {
                float x[kB], y[kB];
#pragma unroll
                for (int u = 0; u < kB; ++u) {
                    const int s = s0 + 8 * u;
                    x[u] = s < nslab ? part_nrm[(size_t)s * Tn + f] : 0.f;
                    y[u] = s < nslab && has_dot ? part_dot[(size_t)s * Tn + f] : 0.f;
                }
#pragma unroll
                for (int u = 0; u < kB; ++u) {
                    if (s0 + 8 * u < nslab) { a += x[u]; b += y[u]; }
                }
            }
        }
        s_pn[part][fl] = a;
        s_pd[part][fl] = b;
        __syncthreads();
        if (tid < 128 && f < Tn) {
            float an = 0.f, ad = 0.f;
#pragma unroll
            for (int g = 0; g < 8; ++g) { an += s_pn[g][tid]; ad += s_pd[g][tid]; }
            s_nrm[f] = fmaxf(sqrtf(an), kEps);
            s_sim[f] = ad;                                  // dot product for now
        }
        __syncthreads();
    }
    __syncthreads();
    for (int i = tid; i < Tn - 1; i += nthr) {
        const float c = s_sim[i] / (s_nrm[i] * s_nrm[i + 1]);
        s_sim[i] = c;
        sims[i] = c;
    }
    __syncthreads();
    const int nb = k - 1;
    for (int i = tid; i < Tn; i += nthr) {
        int flag = 0;
        if (i < Tn - 1 && nb > 0) {
            // integer keys give a total order even with non-finite similarities (a NaN ranks as the
            // largest value), so exactly k-1 boundaries are flagged whatever the input holds
            const uint32_t v = sim_key(s_sim[i]);
            int rank = 0;
            for (int j = 0; j < Tn - 1; ++j) {
                const uint32_t w = sim_key(s_sim[j]);
                rank += (w < v) || (w == v && j < i);
            }
            flag = rank < nb;
        }
        s_flag[i] = flag;
    }
    __syncthreads();
    // exclusive scan of the flags: contiguous ranges per thread, a shuffle scan inside each warp,
    // then the warps' totals
    const int per = (Tn + nthr - 1) / nthr;
    const int lo = min(Tn, tid * per), hi = min(Tn, lo + per);
    int local = 0;
    for (int i = lo; i < hi; ++i) local += s_flag[i];
    const int lane = tid & 31, warp = tid >> 5;
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += s_scan[w];
    int run = before + incl - local;                       // boundaries before frame lo
    for (int i = lo; i < hi; ++i) {
        frame_event[i] = run;                              // event id = boundaries strictly before i
        if (s_flag[i] && run < nb) {
            boundaries[run] = i;
            event_offsets[run + 1] = i + 1;
            ++run;
        }
    }
    if (tid == 0) {
        event_offsets[0] = 0;
        event_offsets[k] = Tn;
    }
}

template <typename T>
static int launch_segment(const void* feats, int Tn, int N, int d, int k, int sim_mode, float* sims,
                          int32_t* boundaries, int32_t* event_offsets, int32_t* frame_event, void* ws,
                          cudaStream_t st) {
    constexpr int VN = 16 / sizeof(T);
    Carver cv(ws);
    int nslab;
    float *part_dot, *part_nrm;
    if (sim_mode == METOK_SIM_FLATTEN) {
        const long long chunks = (long long)N * d / VN;
        nslab = (int)((chunks + kSegThreads * kSegUnroll - 1) / (kSegThreads * kSegUnroll));
        int fpc = kSegMaxRun;
        while (fpc > 1 && (long long)nslab * ceil_div(Tn, fpc) < 4 * kNumSMs) fpc >>= 1;
        part_dot = cv.take<float>((size_t)nslab * Tn);
        part_nrm = cv.take<float>((size_t)nslab * Tn);
        dim3 grid(nslab, ceil_div(Tn, fpc));
        {
            METOK_TIMED("seg_partial_kernel", st);
            seg_partial_kernel<T><<<grid, kSegThreads, 0, st>>>(reinterpret_cast<const T*>(feats), Tn, chunks, fpc,
                                                            part_dot, part_nrm);
        }
        METOK_LAUNCH_CHECK();
    } else {
        nslab = 1;
        part_dot = cv.take<float>((size_t)Tn);
        part_nrm = cv.take<float>((size_t)Tn);
        float* mean = cv.take<float>((size_t)Tn * d);
        dim3 grid(ceil_div(d / VN, 128), Tn);
        {
            METOK_TIMED("seg_mean_kernel", st);
            seg_mean_kernel<T><<<grid, 128, 0, st>>>(reinterpret_cast<const T*>(feats), N, d, mean);
        }
        METOK_LAUNCH_CHECK();
        {
            METOK_TIMED("seg_meandot_kernel", st);
            seg_meandot_kernel<<<Tn, 256, 0, st>>>(mean, Tn, d, part_dot, part_nrm);
        }
        METOK_LAUNCH_CHECK();
    }
    const size_t smem = (size_t)Tn * 3 * sizeof(float);
    if (smem > 48 * 1024) {
        METOK_CUDA_TRY(cudaFuncSetAttribute(seg_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)smem));
    }
    {
        METOK_TIMED("seg_finish_kernel", st);
        launch_chained(seg_finish_kernel, dim3(1), dim3(1024), smem, st, part_dot, part_nrm, nslab, Tn, k, sims, boundaries, event_offsets,
                                             frame_event);
    }
    METOK_LAUNCH_CHECK();
    return METOK_OK;
}

}  // namespace metok

using namespace metok;

extern "C" size_t metok_segment_events_workspace_bytes(int dtype, int T, int N, int d, int sim_mode) {
    if (T < 1 || N < 1 || d < 1) return 0;
    const int VN = dtype == METOK_F32 ? 4 : 8;
    Carver cv(nullptr);
    if (sim_mode == METOK_SIM_FLATTEN) {
        const long long chunks = ((long long)N * d + VN - 1) / VN;
        const size_t nslab = (size_t)((chunks + kSegThreads * kSegUnroll - 1) / (kSegThreads * kSegUnroll));
        cv.take<float>(nslab * T);
        cv.take<float>(nslab * T);
    } else {
        cv.take<float>((size_t)T);
        cv.take<float>((size_t)T);
        cv.take<float>((size_t)T * d);
    }
    return cv.total();
}

extern "C" int metok_segment_events(const void* feats, int dtype, int T, int N, int d, int k, int sim_mode,
                                    float* sims, int32_t* boundaries, int32_t* event_offsets,
                                    int32_t* frame_event, void* ws, size_t ws_bytes, void* stream) {
    if (!feats || !sims || !boundaries || !event_offsets || !frame_event) return METOK_ERR_INVALID_ARG;
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (sim_mode != METOK_SIM_FLATTEN && sim_mode != METOK_SIM_MEANPOOL) return METOK_ERR_INVALID_ARG;
    if (T < 1 || N < 1 || d < 1 || k < 1 || k > T) return METOK_ERR_INVALID_ARG;
    if (!aligned16(feats) || (reinterpret_cast<uintptr_t>(sims) & 3) || (reinterpret_cast<uintptr_t>(boundaries) & 3) ||
        (reinterpret_cast<uintptr_t>(event_offsets) & 3) || (reinterpret_cast<uintptr_t>(frame_event) & 3))
        return METOK_ERR_INVALID_ARG;
    const int eb = dtype == METOK_F32 ? 4 : 2;
    if (((long long)d * eb) % 16 != 0 || T > kMaxFrames) return METOK_ERR_UNSUPPORTED;
    const size_t need = metok_segment_events_workspace_bytes(dtype, T, N, d, sim_mode);
    if (!ws || ws_bytes < need || !aligned16(ws)) return METOK_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (dtype == METOK_F32)
        return launch_segment<float>(feats, T, N, d, k, sim_mode, sims, boundaries, event_offsets, frame_event, ws, st);
    return launch_segment<__nv_bfloat16>(feats, T, N, d, k, sim_mode, sims, boundaries, event_offsets, frame_event,
                                         ws, st);
}

// --------------------------------------------------------------------------- //
// metok_segment_score_events: segmentation and the per-token text relevance of Eq. 5
// in ONE pass over V: per token row its squared norm, its dot product with the text
// embedding and its dot product with the same position's row of the previous frame.
// Token score and 1/norm are final in the kernel; the per-(position, frame) norms and
// dots are added over the positions by seg_finish in a fixed order.
//
// fp32 rows (seg_score_kernel): a warp owns one token position and a run of frames, holds
// the row in registers (the next row's loads in flight meanwhile) and the previous row in
// shared memory, and takes the three sums with multiply-adds.
//
// bf16 rows (seg_score_mma_kernel).  The multiply-add form costs 40 instructions per 16
// bytes (widening, three fma per element) and needs the whole row in registers, which
// leaves an SM with 12 warps.  Here the rows land in shared memory by 16-byte
// asynchronous copies (a ring of kFsDepth stages per warp, no registers held while in
// flight) and the sums run on the tensor cores.  A warp owns one position and
// EIGHT consecutive frames; a stage holds 512 contiguous bytes of those eight rows and
// of the frame before them (one copy instruction per row, 16 bytes per lane: the memory
// system sees long pieces of a row).  A stage is consumed as eight 64-byte slices.  Lane
// (g, q) = (lane / 4, lane % 4) reads chunk q of frame g's
// slice: the 16 bytes, as they lie in memory (dwords m0..m3), are the A operand of
// m16n8k16 mma, which gives row g of A the k-slots (m0, m2) and row 8 + g the slots
// (m1, m3).  The other vector is the B operand, whose two registers pair with (m0, m2)
// in the upper half of C and with (m1, m3) in the lower half: with B = (y0, y2) the
// diagonal element C[g][g] adds the products of the even dwords of frame g's slice, with
// B = (y1, y3) C[8 + g][g] those of the odd dwords -- the order of k inside a dot product
// is free as long as both operands use the same one.  Two mma per slice and vector pair,
// accumulated over the slices of the row: at the end the lane that holds C[g][g] has the
// complete sum of frame g, with no shuffle and no widening.  The previous frame's slice
// is the same slice of the row before it in the stage.  Products of bf16 are exact in fp32 and
// the sums are fp32; the off-diagonal entries are never read.
// --------------------------------------------------------------------------- //
namespace metok {

constexpr int kFsThreads = 128;

template <typename T, int kCH>
__global__ void __launch_bounds__(kFsThreads, 3)
seg_score_kernel(const T* __restrict__ feats, const T* __restrict__ text, int Tn, int N, int d, int frames_per_warp,
                 float* __restrict__ part_dot, float* __restrict__ part_nrm, float* __restrict__ token_score,
                 float* __restrict__ inv_norm) {
    constexpr int VN = Vec16<T>::N;
    extern __shared__ float s_t[];                 // [d], in planes of 4 floats per chunk (conflict-free 16-byte reads)
                                                   // then [warps][nchunk] raw 16-byte chunks: the previous frame's row
    __shared__ float s_red[kFsThreads / 32];
    __shared__ float s_tn;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nchunk = d / VN;
    for (int i = tid; i < d; i += kFsThreads) {
        const int c = i / VN, q = i % VN;
        s_t[(q >> 2) * (nchunk * 4) + c * 4 + (q & 3)] = to_float(text[i]);
    }
    __syncthreads();
    float a = 0.f;
    for (int i = tid; i < d; i += kFsThreads) a = fmaf(s_t[i], s_t[i], a);
    a = warp_sum(a);
    if (lane == 0) s_red[warp] = a;
    __syncthreads();
    if (tid == 0) {
        float sum = 0.f;
        for (int w = 0; w < kFsThreads / 32; ++w) sum += s_red[w];
        s_tn = fmaxf(sqrtf(sum), kEps);
    }
    __syncthreads();
    const float tn = s_tn;
    const int nruns = (Tn + frames_per_warp - 1) / frames_per_warp;
    const int gw = blockIdx.x * (kFsThreads / 32) + warp;
    if (gw >= N * nruns) return;
    const int p = gw % N, run = gw / N;
    const int f0 = run * frames_per_warp;
    const int f1 = min(Tn, f0 + frames_per_warp);           // own frames [f0, f1)
    const int f_last = min(Tn - 1, f1);                     // halo frame for the last dot
    const uint4* base = reinterpret_cast<const uint4*>(feats);
    uint4* prev = reinterpret_cast<uint4*>(s_t + d) + (size_t)warp * nchunk;   // d floats = a multiple of 16 bytes
    uint4 cur[kCH], nxt[kCH];
#pragma unroll
    for (int u = 0; u < kCH; ++u) {
        const int c = u * 32 + lane;
        if (c < nchunk) prev[c] = make_uint4(0u, 0u, 0u, 0u);
    }
    auto fetch = [&](int f, uint4 (&r)[kCH]) {
        const uint4* x = base + ((size_t)f * N + p) * (size_t)nchunk;
#pragma unroll
        for (int u = 0; u < kCH; ++u) {
            const int c = u * 32 + lane;
            r[u] = c < nchunk ? __ldg(x + c) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    fetch(f0, cur);
    // the next row's loads are in flight while this row is reduced
    for (int f = f0; f <= f_last; ++f) {
        const size_t row = (size_t)f * N + p;
        if (f < f_last) fetch(f + 1, nxt);
        float nn = 0.f, dt = 0.f, dp = 0.f;
#pragma unroll
        for (int u = 0; u < kCH; ++u) {
            const int c = u * 32 + lane;
            if (c < nchunk) {
                float v[VN], pv[VN];
                widen16<T>(cur[u], v);
                widen16<T>(prev[c], pv);
                prev[c] = cur[u];                           // a lane only ever touches its own chunks
#pragma unroll
                for (int h = 0; h < VN / 4; ++h) {
                    const float4 tt = reinterpret_cast<const float4*>(s_t + h * (nchunk * 4))[c];
                    nn = fmaf(v[4 * h + 0], v[4 * h + 0], nn); dt = fmaf(v[4 * h + 0], tt.x, dt); dp = fmaf(v[4 * h + 0], pv[4 * h + 0], dp);
                    nn = fmaf(v[4 * h + 1], v[4 * h + 1], nn); dt = fmaf(v[4 * h + 1], tt.y, dt); dp = fmaf(v[4 * h + 1], pv[4 * h + 1], dp);
                    nn = fmaf(v[4 * h + 2], v[4 * h + 2], nn); dt = fmaf(v[4 * h + 2], tt.z, dt); dp = fmaf(v[4 * h + 2], pv[4 * h + 2], dp);
                    nn = fmaf(v[4 * h + 3], v[4 * h + 3], nn); dt = fmaf(v[4 * h + 3], tt.w, dt); dp = fmaf(v[4 * h + 3], pv[4 * h + 3], dp);
                }
            }
        }
        nn = warp_sum(nn);
        dt = warp_sum(dt);
        dp = warp_sum(dp);
        if (lane == 0) {
            if (f < f1) {
                const float n = fmaxf(sqrtf(nn), kEps);
                part_nrm[(size_t)p * Tn + f] = nn;
                token_score[row] = dt / (n * tn);
                inv_norm[row] = 1.0f / n;
            }
            if (f > f0) part_dot[(size_t)p * Tn + (f - 1)] = dp;   // dot of frames f-1 and f at position p
        }
#pragma unroll
        for (int u = 0; u < kCH; ++u) cur[u] = nxt[u];
    }
}

// D += A * B for one m16n8k16 bf16 tile, fp32 accumulators; A is a 16-byte chunk as loaded.
__device__ __forceinline__ void mma_bf16_m16n8k16(float (&c)[4], const uint4& a, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

// 16-byte asynchronous copy global -> shared that bypasses L1; src_bytes = 0 writes zeros.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int kFsDepth = 4;                        // stages of a warp's ring
constexpr int kFsFrames = 8;                       // frames per warp = row groups of the mma tile
constexpr int kFsSlices = 8;                       // 64-byte slices of a row per stage: 512 contiguous bytes
constexpr int kFsRowPitch = kFsSlices * 64 + 64;   // bytes between a stage's rows (see the bank note in the kernel)
constexpr int kFsStageBytes = (kFsFrames + 1) * kFsRowPitch;

// Shared memory: the text embedding as 16-byte chunks with the dwords in the order
// (0, 2, 1, 3), zero-padded to whole slices; then per warp kFsDepth stages of nine rows
// (512 bytes of frame f0 - 1, then of frames f0 .. f0 + 7).
template <bool kFull>                               // kFull: the row is a whole number of 512-byte pieces
__global__ void __launch_bounds__(kFsThreads)
seg_score_mma_kernel(const __nv_bfloat16* __restrict__ feats, const __nv_bfloat16* __restrict__ text, int Tn, int N,
                     int d, float* __restrict__ part_dot, float* __restrict__ part_nrm,
                     float* __restrict__ token_score, float* __restrict__ inv_norm) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char s_dyn[];
    __shared__ float s_red[kFsThreads / 32];
    __shared__ float s_tn;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nchunk = d / 8;
    const int nslice = (nchunk + 3) >> 2;
    uint4* s_text = reinterpret_cast<uint4*>(s_dyn);
    float a = 0.f;
    for (int c = tid; c < nslice * 4; c += kFsThreads) {
        const uint4 r = c < nchunk ? __ldg(reinterpret_cast<const uint4*>(text) + c) : make_uint4(0u, 0u, 0u, 0u);
        s_text[c] = make_uint4(r.x, r.z, r.y, r.w);
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
            a = fmaf(lo, lo, a);
            a = fmaf(hi, hi, a);
        }
    }
    a = warp_sum(a);
    if (lane == 0) s_red[warp] = a;
    __syncthreads();
    if (tid == 0) {
        float sum = 0.f;
        for (int w = 0; w < kFsThreads / 32; ++w) sum += s_red[w];
        s_tn = fmaxf(sqrtf(sum), kEps);
    }
    __syncthreads();
    const float tn = s_tn;
    // the CTA owns eight frames and four consecutive positions, one per warp: their norms and dots are
    // added here (in warp order), so that seg_finish has a quarter of the partial sums to read
    constexpr int kFsWarps = kFsThreads / 32;
    const int pgroups = (N + kFsWarps - 1) / kFsWarps;
    const int run = blockIdx.x / pgroups, pg = blockIdx.x - run * pgroups;
    const int p_raw = pg * kFsWarps + warp;
    const bool has_p = p_raw < N;
    const int p = has_p ? p_raw : N - 1;                    // an idle warp repeats the last position and writes nothing
    const int f0 = run * kFsFrames;
    const int g = lane >> 2, q = lane & 3;
    const int f = f0 + g;                                   // this lane's frame
    const bool has_f = f < Tn;
    // Copies: a stage holds 512 contiguous bytes (eight 64-byte slices) of each of the nine rows -- the
    // frame before the run, then the run's eight frames.  One copy instruction moves a row's 512 bytes
    // (16 per lane), so what reaches the memory system is long contiguous pieces of a row.  Rows of a
    // stage lie kFsRowPitch bytes apart: with 16 words more than a multiple of 32 the 16-byte reads of
    // the eight lanes of a quarter warp (two frames, four chunks each) fall into different banks.
    const uint4* row0 = reinterpret_cast<const uint4*>(feats) + ((size_t)max(f0 - 1, 0) * N + p) * (size_t)nchunk;
    const size_t frame_pitch = (size_t)N * nchunk;          // 16-byte chunks from a frame's row to the next frame's
    const int nsuper = (nslice + kFsSlices - 1) / kFsSlices;
    unsigned char* ring = s_dyn + (size_t)nslice * 4 * sizeof(uint4) + (size_t)warp * kFsDepth * kFsStageBytes;
    const unsigned char* mine = ring + (g + 1) * kFsRowPitch + q * 16;
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + (uint32_t)lane * 16u;
    const uint4* tq = s_text + q;
    // 512-byte piece `sup` of the nine rows into stage `stage` (a constant where the caller is unrolled); one group per call
    auto issue = [&](int sup, int stage) {
        if (sup < nsuper) {
            const int c = sup * 32 + lane;                  // this lane's chunk of every row
            const bool in = c < nchunk;
#pragma unroll
            for (int r = 0; r <= kFsFrames; ++r) {
                const int fr = f0 - 1 + r;                  // r = 0: the frame before the run
                const bool ok = in && fr >= 0 && fr < Tn;
                const uint4* src = ok ? row0 + (size_t)(fr - max(f0 - 1, 0)) * frame_pitch + c : row0;
                cp_async16(dst + stage * kFsStageBytes + r * kFsRowPitch, src, ok ? 16u : 0u);   // 0 bytes read = zeros written
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int j = 0; j < kFsDepth - 1; ++j) issue(j, j);
    // accumulators: [0] pairs the even dwords (diagonal of the upper half), [1] the odd ones (lower half)
    float cn[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    float cp[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    float ct[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll 1
    for (int base = 0; base < nsuper; base += kFsDepth) {
#pragma unroll
        for (int j = 0; j < kFsDepth; ++j) {
            const int sup = base + j;
            if (sup < nsuper) {                             // the same for the whole warp
                cp_async_wait<kFsDepth - 2>();              // this lane's copies of the piece have landed
                __syncwarp();                               // ... and every lane's; the piece before it has been read by all
                issue(sup + kFsDepth - 1, (j + kFsDepth - 1) % kFsDepth);     // into the stage that held the piece before
#pragma unroll
                for (int i = 0; i < kFsSlices; ++i) {
                    const int sl = sup * kFsSlices + i;
                    if (kFull || sl < nslice) {
                        const uint4 x = *reinterpret_cast<const uint4*>(mine + j * kFsStageBytes + i * 64);
                        const uint4 pv = *reinterpret_cast<const uint4*>(mine + j * kFsStageBytes + i * 64 - kFsRowPitch);
                        const uint4 tt = tq[sl * 4];
                        const uint4 xs = make_uint4(x.x, x.z, x.y, x.w);
                        mma_bf16_m16n8k16(cn[0], x, xs.x, xs.y);
                        mma_bf16_m16n8k16(cn[1], x, xs.z, xs.w);
                        mma_bf16_m16n8k16(cp[0], pv, xs.x, xs.y);
                        mma_bf16_m16n8k16(cp[1], pv, xs.z, xs.w);
                        mma_bf16_m16n8k16(ct[0], x, tt.x, tt.y);
                        mma_bf16_m16n8k16(ct[1], x, tt.z, tt.w);
                    }
                }
            }
        }
    }
    cp_async_wait<0>();
    // the diagonal element of group g sits in the lane with q == g / 2, at column g % 2
    __shared__ float s_nn[kFsWarps][kFsFrames], s_dp[kFsWarps][kFsFrames];
    if (q == (g >> 1)) {
        const bool odd = g & 1;
        const float nn = odd ? cn[0][1] + cn[1][3] : cn[0][0] + cn[1][2];
        const float dp = odd ? cp[0][1] + cp[1][3] : cp[0][0] + cp[1][2];
        const float dt = odd ? ct[0][1] + ct[1][3] : ct[0][0] + ct[1][2];
        s_nn[warp][g] = has_p && has_f ? nn : 0.f;
        s_dp[warp][g] = has_p && has_f ? dp : 0.f;
        if (has_p && has_f) {
            const size_t r = (size_t)f * N + p;
            const float n = fmaxf(sqrtf(nn), kEps);
            token_score[r] = dt / (n * tn);
            inv_norm[r] = 1.0f / n;
        }
    }
    __syncthreads();
    if (tid < kFsFrames && f0 + tid < Tn) {
        float nn = 0.f, dp = 0.f;
#pragma unroll
        for (int w = 0; w < kFsWarps; ++w) { nn += s_nn[w][tid]; dp += s_dp[w][tid]; }
        const int ff = f0 + tid;
        part_nrm[(size_t)pg * Tn + ff] = nn;
        if (ff > 0) part_dot[(size_t)pg * Tn + (ff - 1)] = dp;    // dots of frames ff-1 and ff, four positions
    }
}

// Frame runs sized so that all warps are resident at once: a second, partly filled wave of
// CTAs would cost as much time as the first.
template <typename KernelT>
static int seg_score_runs(KernelT kernel, size_t smem, int Tn, int N, int* frames_per_warp) {
    if (smem > 40 * 1024)
        METOK_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    METOK_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kFsThreads, smem));
    const long long slots = (long long)kNumSMs * (per_sm > 0 ? per_sm : 1) * (kFsThreads / 32);
    long long nruns = slots / N;
    nruns = nruns < 1 ? 1 : nruns > Tn ? Tn : nruns;
    *frames_per_warp = ceil_div(Tn, (int)nruns);
    return METOK_OK;
}

template <typename T, int kCH>
static int launch_seg_score(const void* feats, const void* text, int Tn, int N, int d, int k, float* sims,
                            int32_t* boundaries, int32_t* event_offsets, int32_t* frame_event,
                            float* token_score, float* inv_norm, void* ws, cudaStream_t st) {
    Carver cv(ws);
    float* part_dot = cv.take<float>((size_t)N * Tn);
    float* part_nrm = cv.take<float>((size_t)N * Tn);
    int fpw = 1;
    int nslab = N;                                         // partial sums per frame that seg_finish adds up
    if constexpr (sizeof(T) == 2) {
        const int nslice = (d / 8 + 3) / 4;
        const size_t smem_t = (size_t)nslice * 4 * sizeof(uint4) + (size_t)(kFsThreads / 32) * kFsDepth * kFsStageBytes;
        auto kernel = (d / 8) % (4 * kFsSlices) == 0 ? seg_score_mma_kernel<true> : seg_score_mma_kernel<false>;
        if (smem_t > 40 * 1024)
            METOK_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_t));
        nslab = ceil_div(N, kFsThreads / 32);              // the kernel adds the four positions of a CTA
        METOK_TIMED("seg_score_kernel", st);
        launch_chained(kernel, dim3(nslab * ceil_div(Tn, kFsFrames)), dim3(kFsThreads), smem_t, st, 
            reinterpret_cast<const __nv_bfloat16*>(feats), reinterpret_cast<const __nv_bfloat16*>(text), Tn, N, d,
            part_dot, part_nrm, token_score, inv_norm);
    } else {
        const size_t smem_t = (size_t)d * sizeof(float) + (size_t)(kFsThreads / 32) * d * sizeof(T);
        const int rc = seg_score_runs(seg_score_kernel<T, kCH>, smem_t, Tn, N, &fpw);
        if (rc != METOK_OK) return rc;
        const int warps = N * ceil_div(Tn, fpw);
        METOK_TIMED("seg_score_kernel", st);
        seg_score_kernel<T, kCH><<<ceil_div(warps, kFsThreads / 32), kFsThreads, smem_t, st>>>(
            reinterpret_cast<const T*>(feats), reinterpret_cast<const T*>(text), Tn, N, d, fpw, part_dot, part_nrm,
            token_score, inv_norm);
    }
    METOK_LAUNCH_CHECK();
    const size_t smem = (size_t)Tn * 3 * sizeof(float);
    if (smem > 48 * 1024)
        METOK_CUDA_TRY(cudaFuncSetAttribute(seg_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    {
        METOK_TIMED("seg_finish_kernel", st);
        launch_chained(seg_finish_kernel, dim3(1), dim3(1024), smem, st, part_dot, part_nrm, nslab, Tn, k, sims, boundaries, event_offsets,
                                             frame_event);
    }
    METOK_LAUNCH_CHECK();
    return METOK_OK;
}

}  // namespace metok

extern "C" size_t metok_segment_score_events_workspace_bytes(int dtype, int T, int N, int d) {
    (void)dtype; (void)d;
    if (T < 1 || N < 1) return 0;
    Carver cv(nullptr);
    cv.take<float>((size_t)N * T);
    cv.take<float>((size_t)N * T);
    return cv.total();
}

extern "C" int metok_segment_score_events(const void* feats, int dtype, int T, int N, int d, int k,
                                          const void* text_emb, float* sims, int32_t* boundaries,
                                          int32_t* event_offsets, int32_t* frame_event, float* token_score,
                                          float* token_inv_norm, void* ws, size_t ws_bytes, void* stream) {
    if (!feats || !text_emb || !sims || !boundaries || !event_offsets || !frame_event || !token_score || !token_inv_norm)
        return METOK_ERR_INVALID_ARG;
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (T < 1 || N < 1 || d < 1 || k < 1 || k > T) return METOK_ERR_INVALID_ARG;
    if (!aligned16(feats) || !aligned16(text_emb)) return METOK_ERR_INVALID_ARG;
    const int eb = dtype == METOK_F32 ? 4 : 2;
    if (((long long)d * eb) % 16 != 0 || T > kMaxFrames) return METOK_ERR_UNSUPPORTED;
    const long long nchunk = (long long)d * eb / 16;
    if (nchunk > 32 * 16) return METOK_ERR_UNSUPPORTED;          // rows of more than 8 KiB: use the two separate calls
    const size_t need = metok_segment_score_events_workspace_bytes(dtype, T, N, d);
    if (!ws || ws_bytes < need || !aligned16(ws)) return METOK_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
#define METOK_FS(TYPE, CH)                                                                                        \
    return launch_seg_score<TYPE, CH>(feats, text_emb, T, N, d, k, sims, boundaries, event_offsets, frame_event, \
                                      token_score, token_inv_norm, ws, st)
    if (dtype == METOK_F32) {
        if (nchunk <= 32 * 4) METOK_FS(float, 4);
        if (nchunk <= 32 * 8) METOK_FS(float, 8);
        METOK_FS(float, 16);
    }
    METOK_FS(__nv_bfloat16, 4);                                  // the bf16 kernel has no per-width variants
#undef METOK_FS
}

// --------------------------------------------------------------------------- //
// metok_segment_events_static: the same computation with the scratch in a fixed
// array that lives inside the library image instead of a caller workspace.
// --------------------------------------------------------------------------- //
namespace metok {
constexpr size_t kStaticScratchBytes = (size_t)1 << 20;      // 1 MiB per GPU that loads the library
static __device__ __align__(256) unsigned char g_seg_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_seg_scratch_addr[kMaxDevices] = {nullptr};    // device address of the array, per device

// `g_seg_scratch` in host code is only a handle; the address kernels can use has to be
// asked for, once per device, with that device current.
static int static_scratch_address(void** out, cudaStream_t st) {
    int dev = -1;
    METOK_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return METOK_ERR_UNSUPPORTED;
    if (!g_seg_scratch_addr[dev]) {
        // the look-up is not a stream operation: made while `st` is being captured it could end the
        // caller's capture, so the first call on a device has to come before any capture
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        METOK_CUDA_TRY(cudaStreamIsCapturing(st, &cs));
        if (cs != cudaStreamCaptureStatusNone) return METOK_ERR_UNSUPPORTED;
        void* p = nullptr;
        METOK_CUDA_TRY(cudaGetSymbolAddress(&p, g_seg_scratch));
        g_seg_scratch_addr[dev] = p;
    }
    *out = g_seg_scratch_addr[dev];
    return METOK_OK;
}
}  // namespace metok

extern "C" size_t metok_segment_events_static_capacity(void) { return metok::kStaticScratchBytes; }

extern "C" int metok_segment_events_static(const void* feats, int dtype, int T, int N, int d, int k, int sim_mode,
                                           float* sims, int32_t* boundaries, int32_t* event_offsets,
                                           int32_t* frame_event, void* stream) {
    if (dtype != METOK_F32 && dtype != METOK_BF16) return METOK_ERR_INVALID_ARG;
    if (T < 1 || N < 1 || d < 1) return METOK_ERR_INVALID_ARG;
    const size_t need = metok_segment_events_workspace_bytes(dtype, T, N, d, sim_mode);
    if (need > metok::kStaticScratchBytes) return METOK_ERR_TOO_LARGE;
    void* scratch = nullptr;
    const int rc = metok::static_scratch_address(&scratch, reinterpret_cast<cudaStream_t>(stream));
    if (rc != METOK_OK) return rc;
    return metok_segment_events(feats, dtype, T, N, d, k, sim_mode, sims, boundaries, event_offsets, frame_event,
                                scratch, metok::kStaticScratchBytes, stream);
}
