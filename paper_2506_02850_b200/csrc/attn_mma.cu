// Text->visual attention scores on the tensor cores (bf16, head dim 64 or 128).
//
// Per KV head g the rep = Hq/Hkv query heads of the group give R = rep*Lt query rows
// (row r = local head * Lt + q) that all multiply the same K[g].  The R x S matrix of
// probabilities is never stored.  Two kernels, both TMA -> shared memory ->
// tcgen05.mma -> TMEM -> registers:
//
//   stats  : D = Q_tile (128 query rows = TMEM lanes) x K_tile^T (256 keys = columns).
//            A thread owns one query row, so the running (max, sum) of the softmax is
//            thread-local.  The keys are split over CTAs; each CTA leaves one (max,
//            sum) pair per row (the column quarters are merged in the CTA).
//   colsum : D = K_tile (128 keys = TMEM lanes) x Q_chunk^T (up to 256 query rows =
//            columns).  The row normalisers are known now (log-sum-exp per query row,
//            kept in shared memory), a thread owns one key and adds up
//            exp2(logit - lse) over its columns: the sum over queries is thread-local
//            too.  Only key tiles that touch the visual span are visited.
//
// Warp roles in both: warp 0 = TMA producer, warp 1 = MMA issuer (one elected lane),
// the others = epilogue: four (stats) or two (colsum) warps per TMEM lane quadrant, each
// taking a quarter or half of the columns.  Two accumulators in TMEM (2 x 256 columns) so
// that the epilogue of tile i overlaps the MMA of tile i+1.  Every wait is bounded.
#include "common.cuh"
#include "launchers.h"
#include "sm100.cuh"

namespace metok {

namespace {

constexpr int kAmThreads = 320;
constexpr int kAmEpiWarps = 8;
constexpr int kStEpiWarps = 16;           // stats: four warps per TMEM lane quadrant, 64 columns of a tile each
constexpr int kStThreads = 64 + kStEpiWarps * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegInf = -3.0e38f;       // finite stand-in: keeps (m_old - m_new) free of inf - inf

constexpr int kStBM = 128;                // stats: query rows per CTA
constexpr int kStBN = 256;                // stats: keys per tile
constexpr int kStStages = 2;
constexpr int kCsBM = 128;                // colsum: keys per tile
constexpr int kCsMaxNQ = 256;             // colsum: query rows per chunk (multiple of 16)
constexpr int kCsStages = 4;
constexpr int kStMinTiles = 2;            // fewest key tiles a stats CTA is started for
constexpr int kCsMinTiles = 3;            // the same for colsum

struct AttnMmaDims {
    int Hq, Hkv, Lt, S, vis_start, n_vis, R;
    int st_nrt, st_tiles, st_per, st_nsplit;          // stats: row tiles, key tiles, tiles per split, splits
    int cs_nq, cs_nchunk, cs_t0, cs_tiles, cs_per, cs_nsplit;   // colsum
    float scale_log2;
};

__host__ AttnMmaDims make_mma_dims(int Hq, int Hkv, int Lt, int S, int vis_start, int n_vis, float scale) {
    AttnMmaDims dm;
    dm.Hq = Hq; dm.Hkv = Hkv; dm.Lt = Lt; dm.S = S; dm.vis_start = vis_start; dm.n_vis = n_vis;
    dm.R = (Hq / Hkv) * Lt;
    dm.scale_log2 = scale * kLog2e;
    // one CTA per SM: as many key splits as keep the grid within one wave
    dm.st_nrt = ceil_div(dm.R, kStBM);
    dm.st_tiles = ceil_div(S, kStBN);
    // ... but a CTA gets at least kStMinTiles tiles: a launch that is mostly prologue on every SM
    // keeps other streams' kernels off the GPU for nothing
    int ns = kNumSMs / (Hkv * dm.st_nrt);
    if (ns > ceil_div(dm.st_tiles, kStMinTiles)) ns = ceil_div(dm.st_tiles, kStMinTiles);
    if (ns < 1) ns = 1;
    if (ns > dm.st_tiles) ns = dm.st_tiles;
    dm.st_per = ceil_div(dm.st_tiles, ns);
    dm.st_nsplit = ceil_div(dm.st_tiles, dm.st_per);   // every split owns at least one tile
    dm.cs_nchunk = ceil_div(dm.R, kCsMaxNQ);
    dm.cs_nq = ceil_div(ceil_div(dm.R, dm.cs_nchunk), 16) * 16;
    dm.cs_t0 = vis_start / kCsBM;
    dm.cs_tiles = (vis_start + n_vis - 1) / kCsBM - dm.cs_t0 + 1;
    ns = kNumSMs / (Hkv * dm.cs_nchunk);
    if (ns > ceil_div(dm.cs_tiles, kCsMinTiles)) ns = ceil_div(dm.cs_tiles, kCsMinTiles);
    if (ns < 1) ns = 1;
    if (ns > dm.cs_tiles) ns = dm.cs_tiles;
    dm.cs_per = ceil_div(dm.cs_tiles, ns);
    dm.cs_nsplit = ceil_div(dm.cs_tiles, dm.cs_per);
    return dm;
}

// --------------------------------------------------------------------------- //
// stats
// --------------------------------------------------------------------------- //
template <int DH>
__global__ void __launch_bounds__(kStThreads, 1)
attn_stats_mma_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      AttnMmaDims dm, float* __restrict__ part_m, float* __restrict__ part_l,
                      int32_t* __restrict__ status) {
    grid_dep_wait();
    using namespace sm100;
    constexpr int KB = DH / 64;                               // 64-element (128-byte) K blocks
    constexpr uint32_t kQBlk = kStBM * 128, kKBlk = kStBN * 128;
    constexpr uint32_t kQBytes = KB * kQBlk, kKBytes = KB * kKBlk;
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t q_bar, drain_bar, full_bar[kStStages], empty_bar[kStStages], tfull_bar[2],
        tempty_bar[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ float s_pm[4][kStBM], s_pl[4][kStBM];          // the column quarters' (max, sum) per query row

    const int split = blockIdx.x, rt = blockIdx.y, g = blockIdx.z;
    // The call's status word starts cleared: written by the first CTA of the call's first kernel
    // instead of by a memset node.  A CTA that gives up writes it only after its waits have run
    // out, seconds later.
    if (split == 0 && rt == 0 && g == 0 && threadIdx.x == 0) *status = 0;
    const int t_lo = split * dm.st_per;
    const int nt = min(dm.st_tiles, t_lo + dm.st_per) - t_lo;          // >= 1 by construction
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int text_start = dm.S - dm.Lt;

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t q_addr = smem_base;
    auto k_addr = [&](int s) { return smem_base + kQBytes + (uint32_t)s * kKBytes; };

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&q_bar), 1);
        mbar_init(smem_u32(&drain_bar), 1);
        for (int s = 0; s < kStStages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&tfull_bar[b]), 1); mbar_init(smem_u32(&tempty_bar[b]), kStEpiWarps); }
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

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmQ);
            prefetch_tmap(&tmK);
            mbar_arrive_expect_tx(smem_u32(&q_bar), kQBytes);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
                tma_load_2d(q_addr + kb * kQBlk, &tmQ, kb * 64, g * dm.R + rt * kStBM, smem_u32(&q_bar));
            int it = 0;
            bool ok = true;
            for (; it < nt; ++it) {
                const int s = it % kStStages;
                const uint32_t ph = (uint32_t)(it / kStStages) & 1u;
                if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
                const uint32_t fb = smem_u32(&full_bar[s]);
                mbar_arrive_expect_tx(fb, kKBytes);
                if (dbg_withhold(status, kDbgAttnStats) && split == 0 && rt == 0 && g == 0 && it == 0) continue;   // debug builds: one copy never sent
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_2d(k_addr(s) + kb * kKBlk, &tmK, kb * 64, g * dm.S + (t_lo + it) * kStBN, fb);
            }
            // every copy issued has landed before the CTA's shared memory goes away, whichever way the
            // other warps leave (in a normal run these waits are over already)
            mbar_wait(smem_u32(&q_bar), 0u, abort_flag);
            for (int back = 1; back <= kStStages && back <= it; ++back) {
                const int j = it - back;
                mbar_wait(smem_u32(&full_bar[j % kStStages]), (uint32_t)(j / kStStages) & 1u, abort_flag);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(kStBM, kStBN);
            bool ok = mbar_wait(smem_u32(&q_bar), 0u, abort_flag);
            for (int it = 0; it < nt && ok; ++it) {
                const int b = it & 1, s = it % kStStages;
                if (!mbar_wait(smem_u32(&tempty_bar[b]), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                if (!mbar_wait(smem_u32(&full_bar[s]), (uint32_t)(it / kStStages) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)b * kStBN;
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    const uint64_t ad = make_desc_k128(q_addr + (kk >> 2) * kQBlk + (kk & 3) * 32);
                    const uint64_t bd = make_desc_k128(k_addr(s) + (kk >> 2) * kKBlk + (kk & 3) * 32);
                    umma_bf16(d_tmem, ad, bd, idesc, kk != 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&empty_bar[s]));
                umma_commit(smem_u32(&tfull_bar[b]));
            }
            if (!ok) {                                         // wait until whatever was issued has retired
                umma_commit(smem_u32(&drain_bar));
                mbar_wait(smem_u32(&drain_bar), 0u, abort_flag);
            }
        }
    } else {
        const int quad = warp & 3;                             // TMEM lanes 32*quad .. 32*quad+31
        const int part = (warp - 2) >> 2;                      // column quarter of every tile
        const int r = rt * kStBM + quad * 32 + lane;
        const bool valid = r < dm.R;
        const int limit = valid ? text_start + (r % dm.Lt) : -1;     // last key this query may see
        const float sc = dm.scale_log2;
        float m_run = kNegInf, l_run = 0.f;
        bool ok = true;
        for (int it = 0; it < nt; ++it) {
            const int b = it & 1;
            if (!mbar_wait(smem_u32(&tfull_bar[b]), (uint32_t)(it >> 1) & 1u, abort_flag)) ok = false;
            ok = __all_sync(0xFFFFFFFFu, ok);                  // tcgen05.ld below is warp-collective
            if (!ok) break;
            tc_fence_after();
            const int u_tile = (t_lo + it) * kStBN;
            const int u0 = u_tile + part * (kStBN / 4);
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(b * kStBN + part * (kStBN / 4));
            const bool masked = u_tile + kStBN - 1 > text_start;       // some query cannot see some key of the tile
            uint32_t raw[2][32];
            tmem_ld32_issue(taddr, raw[0]);
#pragma unroll
            for (int ci = 0; ci < kStBN / 128; ++ci) {
                // the next 32 columns are fetched while these are reduced
                const int c0 = ci * 32;
                tmem_ld32_wait(raw[ci & 1]);
                if (ci + 1 < kStBN / 128) tmem_ld32_issue(taddr + (uint32_t)(c0 + 32), raw[(ci + 1) & 1]);
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(raw[ci & 1][j]);
                float a0 = 0.f, a1 = 0.f;
                float m_new;
                if (masked) {                                  // hidden keys add exactly nothing
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = (u0 + c0 + j <= limit) ? v[j] * sc : kNegInf;
                    float cm = v[0];
#pragma unroll
                    for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
                    m_new = fmaxf(m_run, cm);
#pragma unroll
                    for (int j = 0; j < 32; ++j) a0 += (v[j] > kNegInf) ? fast_exp2(v[j] - m_new) : 0.f;
                } else {
                    // the scale is positive: the maximum of the raw logits, scaled, is the maximum of the
                    // scaled ones, and scaling folds into the exponent's multiply-add
                    float t16[16];                             // a tree: the maximum is five steps deep, not 31
#pragma unroll
                    for (int j = 0; j < 16; ++j) t16[j] = fmaxf(v[2 * j], v[2 * j + 1]);
#pragma unroll
                    for (int w = 8; w >= 1; w >>= 1) {
#pragma unroll
                        for (int j = 0; j < w; ++j) t16[j] = fmaxf(t16[j], t16[j + w]);
                    }
                    const float cm = t16[0];
                    m_new = fmaxf(m_run, cm * sc);
                    const float neg_m = -m_new;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {           // every fourth exponential on the FMA pipe
                        a0 += fast_exp2(fmaf(v[j], sc, neg_m));
                        a1 += fast_exp2(fmaf(v[j + 1], sc, neg_m));
                        a0 += fast_exp2(fmaf(v[j + 2], sc, neg_m));
                        a1 += exp2_fma(fmaf(v[j + 3], sc, neg_m));
                    }
                }
                l_run = l_run * fast_exp2(m_run - m_new) + (a0 + a1);
                m_run = m_new;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tempty_bar[b]));
        }
        // the four column quarters of a row are merged here, in quarter order: one pair per row and split
        const int rl = quad * 32 + lane;
        s_pm[part][rl] = m_run;
        s_pl[part][rl] = l_run;
        asm volatile("bar.sync 1, %0;" ::"n"(kStEpiWarps * 32) : "memory");
        if (part == 0 && ok && valid) {
            float M = s_pm[0][rl];
#pragma unroll
            for (int p2 = 1; p2 < 4; ++p2) M = fmaxf(M, s_pm[p2][rl]);
            float Z = 0.f;
#pragma unroll
            for (int p2 = 0; p2 < 4; ++p2) Z += s_pl[p2][rl] * fast_exp2(s_pm[p2][rl] - M);
            const size_t o = ((size_t)g * dm.st_nsplit + (size_t)split) * dm.R + r;
            part_m[o] = M;
            part_l[o] = Z;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0 && s_abort) *status = METOK_ERR_TIMEOUT;
}

// --------------------------------------------------------------------------- //
// colsum
// --------------------------------------------------------------------------- //
template <int DH>
__global__ void __launch_bounds__(kAmThreads, 1)
attn_colsum_mma_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       AttnMmaDims dm, const float* __restrict__ part_m, const float* __restrict__ part_l,
                       float* __restrict__ part_col, int32_t* __restrict__ status) {
    grid_dep_wait();
    using namespace sm100;
    constexpr int KB = DH / 64;
    constexpr uint32_t kKBlk = kCsBM * 128;
    constexpr uint32_t kKBytes = KB * kKBlk;
    extern __shared__ uint8_t smem_dyn[];
    __shared__ __align__(8) uint64_t q_bar, drain_bar, full_bar[kCsStages], empty_bar[kCsStages], tfull_bar[2],
        tempty_bar[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ __align__(16) float s_nlse[kCsMaxNQ];           // -(log-sum-exp) per query row of the chunk, log2 units

    const int split = blockIdx.x, chunk = blockIdx.y, g = blockIdx.z;
    const int NQ = dm.cs_nq;
    const uint32_t kQBlk = (uint32_t)NQ * 128;
    const uint32_t kQBytes = KB * kQBlk;
    const int t_lo = dm.cs_t0 + split * dm.cs_per;
    const int nt = min(dm.cs_t0 + dm.cs_tiles, t_lo + dm.cs_per) - t_lo;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t q_addr = smem_base;
    auto k_addr = [&](int s) { return smem_base + kQBytes + (uint32_t)s * kKBytes; };

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&q_bar), 1);
        mbar_init(smem_u32(&drain_bar), 1);
        for (int s = 0; s < kCsStages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&tfull_bar[b]), 1); mbar_init(smem_u32(&tempty_bar[b]), kAmEpiWarps); }
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

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmQ);
            prefetch_tmap(&tmK);
            mbar_arrive_expect_tx(smem_u32(&q_bar), kQBytes);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
                tma_load_2d(q_addr + kb * kQBlk, &tmQ, kb * 64, g * dm.R + chunk * NQ, smem_u32(&q_bar));
            int it = 0;
            bool ok = true;
            for (; it < nt; ++it) {
                const int s = it % kCsStages;
                const uint32_t ph = (uint32_t)(it / kCsStages) & 1u;
                if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
                const uint32_t fb = smem_u32(&full_bar[s]);
                mbar_arrive_expect_tx(fb, kKBytes);
                if (dbg_withhold(status, kDbgAttnColsum) && split == 0 && chunk == 0 && g == 0 && it == 0) continue;   // debug builds: one copy never sent
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_2d(k_addr(s) + kb * kKBlk, &tmK, kb * 64, g * dm.S + (t_lo + it) * kCsBM, fb);
            }
            mbar_wait(smem_u32(&q_bar), 0u, abort_flag);         // as in the stats kernel
            for (int back = 1; back <= kCsStages && back <= it; ++back) {
                const int j = it - back;
                mbar_wait(smem_u32(&full_bar[j % kCsStages]), (uint32_t)(j / kCsStages) & 1u, abort_flag);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(kCsBM, NQ);
            bool ok = mbar_wait(smem_u32(&q_bar), 0u, abort_flag);
            for (int it = 0; it < nt && ok; ++it) {
                const int b = it & 1, s = it % kCsStages;
                if (!mbar_wait(smem_u32(&tempty_bar[b]), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                if (!mbar_wait(smem_u32(&full_bar[s]), (uint32_t)(it / kCsStages) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)b * kCsMaxNQ;
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    const uint64_t ad = make_desc_k128(k_addr(s) + (kk >> 2) * kKBlk + (kk & 3) * 32);
                    const uint64_t bd = make_desc_k128(q_addr + (kk >> 2) * kQBlk + (kk & 3) * 32);
                    umma_bf16(d_tmem, ad, bd, idesc, kk != 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&empty_bar[s]));
                umma_commit(smem_u32(&tfull_bar[b]));
            }
            if (!ok) {
                umma_commit(smem_u32(&drain_bar));
                mbar_wait(smem_u32(&drain_bar), 0u, abort_flag);
            }
        }
    } else {
        // The epilogue warps first turn the key-split partials into the log-sum-exp of the chunk's
        // query rows, one row per thread, while the producer's first copies and the first MMA are
        // already under way; nobody else reads s_nlse, so a barrier among these 256 threads is enough.
        {
            const int c = threadIdx.x - 64;                    // 0 .. kCsMaxNQ - 1
            const int r = chunk * NQ + c;
            float nl = kNegInf;                                // rows past R contribute exp2(x - 3e38) = 0
            if (c < NQ && r < dm.R) {
                const int ns2 = dm.st_nsplit;                  // one (max, sum) pair per key split
                const float* pm = part_m + (size_t)g * ns2 * dm.R + r;
                const float* pl = part_l + (size_t)g * ns2 * dm.R + r;
                float M = kNegInf, Z = 0.f;                    // running maximum and sum, partials in order
                for (int s0 = 0; s0 < ns2; s0 += 8) {
                    float m8[8], l8[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const bool in = s0 + u < ns2;
                        m8[u] = in ? pm[(size_t)(s0 + u) * dm.R] : kNegInf;
                        l8[u] = in ? pl[(size_t)(s0 + u) * dm.R] : 0.f;
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const float Mn = fmaxf(M, m8[u]);
                        Z = Z * exp2f(M - Mn) + l8[u] * exp2f(m8[u] - Mn);
                        M = Mn;
                    }
                }
                nl = -(M + log2f(Z));
            }
            s_nlse[c] = nl;
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;
        const int h0 = ((NQ / 16 + 1) / 2) * 16;               // first column of the second half
        const int c_lo = half ? h0 : 0, c_hi = half ? NQ : h0;
        const float sc = dm.scale_log2;
        const int vis_end = dm.vis_start + dm.n_vis;
        float* plane = part_col + ((size_t)(g * dm.cs_nchunk + chunk) * 2 + half) * dm.n_vis;
        bool ok = true;
        for (int it = 0; it < nt; ++it) {
            const int b = it & 1;
            if (!mbar_wait(smem_u32(&tfull_bar[b]), (uint32_t)(it >> 1) & 1u, abort_flag)) ok = false;
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(b * kCsMaxNQ);
            float a0 = 0.f, a1 = 0.f;
            int c = c_lo;
#pragma unroll 1
            for (; c + 32 <= c_hi; c += 32) {
                float v[32];
                tmem_ld32(taddr + (uint32_t)c, v);
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float4 nl = *reinterpret_cast<const float4*>(&s_nlse[c + j]);
                    a0 += fast_exp2(fmaf(v[j], sc, nl.x));
                    a1 += fast_exp2(fmaf(v[j + 1], sc, nl.y));
                    a0 += fast_exp2(fmaf(v[j + 2], sc, nl.z));
                    a1 += exp2_fma(fmaf(v[j + 3], sc, nl.w));     // every fourth exponential on the FMA pipe
                }
            }
            if (c < c_hi) {                                    // halves are multiples of 16 columns
                float v[16];
                tmem_ld16(taddr + (uint32_t)c, v);
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    const float4 nl = *reinterpret_cast<const float4*>(&s_nlse[c + j]);
                    a0 += fast_exp2(fmaf(v[j], sc, nl.x));
                    a1 += fast_exp2(fmaf(v[j + 1], sc, nl.y));
                    a0 += fast_exp2(fmaf(v[j + 2], sc, nl.z));
                    a1 += exp2_fma(fmaf(v[j + 3], sc, nl.w));     // every fourth exponential on the FMA pipe
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tempty_bar[b]));
            const int u = (t_lo + it) * kCsBM + quad * 32 + lane;
            if (u >= dm.vis_start && u < vis_end) plane[u - dm.vis_start] = a0 + a1;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0 && s_abort) *status = METOK_ERR_TIMEOUT;
}

template <int DH>
int launch_dh(const void* q_text, const void* k_all, const AttnMmaDims& dm, float* part_m, float* part_l,
              float* part_col, int32_t* status, cudaStream_t st) {
    CUtensorMap tmQs, tmKs, tmQc, tmKc;
    const uint64_t qrows = (uint64_t)dm.Hq * dm.Lt, krows = (uint64_t)dm.Hkv * dm.S;
    int rc;
    if ((rc = make_tmap_bf16_2d(&tmQs, q_text, qrows, DH, kStBM)) != METOK_OK) return rc;
    if ((rc = make_tmap_bf16_2d(&tmKs, k_all, krows, DH, kStBN)) != METOK_OK) return rc;
    if ((rc = make_tmap_bf16_2d(&tmQc, q_text, qrows, DH, (uint32_t)dm.cs_nq)) != METOK_OK) return rc;
    if ((rc = make_tmap_bf16_2d(&tmKc, k_all, krows, DH, kCsBM)) != METOK_OK) return rc;
    constexpr int KB = DH / 64;
    const size_t smem_st = (size_t)KB * (kStBM + kStStages * kStBN) * 128 + 1024;
    const size_t smem_cs = (size_t)KB * (dm.cs_nq + kCsStages * kCsBM) * 128 + 1024;
    METOK_CUDA_TRY(cudaFuncSetAttribute(attn_stats_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)smem_st));
    METOK_CUDA_TRY(cudaFuncSetAttribute(attn_colsum_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)((size_t)KB * (kCsMaxNQ + kCsStages * kCsBM) * 128 + 1024)));
    {
        METOK_TIMED("attn_stats_mma_kernel", st);
        launch_chained(attn_stats_mma_kernel<DH>, dim3(dim3(dm.st_nsplit, dm.st_nrt, dm.Hkv)), dim3(kStThreads), smem_st, st, 
            tmQs, tmKs, dm, part_m, part_l, status);
    }
    METOK_LAUNCH_CHECK();
    {
        METOK_TIMED("attn_colsum_mma_kernel", st);
        launch_chained(attn_colsum_mma_kernel<DH>, dim3(dim3(dm.cs_nsplit, dm.cs_nchunk, dm.Hkv)), dim3(kAmThreads), smem_cs, st, 
            tmQc, tmKc, dm, part_m, part_l, part_col, status);
    }
    METOK_LAUNCH_CHECK();
    return METOK_OK;
}

}  // namespace

void attn_mma_workspace(int Hq, int Hkv, int Lt, int S, int n_vis, size_t* n_part_ml, size_t* n_part_col,
                        int* n_planes) {
    const AttnMmaDims dm = make_mma_dims(Hq, Hkv, Lt, S, 0, n_vis, 1.f);
    *n_part_ml = (size_t)Hkv * dm.st_nsplit * 2 * dm.R;
    *n_planes = Hkv * dm.cs_nchunk * 2;
    *n_part_col = (size_t)(*n_planes) * n_vis;
}

int launch_attn_scores_mma(const void* q_text, const void* k_all, int Hq, int Hkv, int Lt, int S, int dh,
                           int vis_start, int n_vis, float scale, float* part_m, float* part_l, float* part_col,
                           int32_t* status, cudaStream_t st) {
    const AttnMmaDims dm = make_mma_dims(Hq, Hkv, Lt, S, vis_start, n_vis, scale);
    if (dh == 128) return launch_dh<128>(q_text, k_all, dm, part_m, part_l, part_col, status, st);
    if (dh == 64) return launch_dh<64>(q_text, k_all, dm, part_m, part_l, part_col, status, st);
    return METOK_ERR_UNSUPPORTED;
}

}  // namespace metok
