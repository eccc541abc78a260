// Shared device/host helpers of the METok CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/metok.h"

namespace metok {

constexpr float kEps = 1e-8f;            // lower clamp of every norm
constexpr int kNumSMs = 148;             // B200

// ---- host-side error plumbing ------------------------------------------------
void set_last_cuda_error(int e);
#define METOK_CUDA_TRY(expr)                                   \
    do {                                                       \
        cudaError_t _e = (expr);                               \
        if (_e != cudaSuccess) {                               \
            ::metok::set_last_cuda_error((int)_e);             \
            return METOK_ERR_CUDA;                             \
        }                                                      \
    } while (0)
#define METOK_LAUNCH_CHECK() METOK_CUDA_TRY(cudaGetLastError())

// Brackets one kernel launch with CUDA events while profiling is on (see
// metok_profile_begin); costs one predictable branch otherwise.
extern bool g_profiling;
struct KernelTimer {
    const char* name;
    cudaStream_t st;
    cudaEvent_t a, b;
    bool active;
    KernelTimer(const char* n, cudaStream_t s);
    ~KernelTimer();
    void record(cudaEvent_t e);
};
#define METOK_TIMED(name, st) ::metok::KernelTimer _metok_kt(name, st)

// Launch with programmatic stream serialisation: the grid may be scheduled while the kernel before it
// on the stream is still draining, and every one of its CTAs calls grid_dep_wait() before it touches
// memory, which returns once that kernel has completed and its writes are visible.  Because every CTA
// of every kernel launched this way waits first, completion of a kernel implies completion of all
// kernels before it on the stream.  The launch error is picked up by METOK_LAUNCH_CHECK().
template <typename... P, typename... A>
inline void launch_chained(void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    (void)cudaLaunchKernelEx(&cfg, kern, static_cast<P>(args)...);
}

#ifdef __CUDACC__
// First statements of a kernel launched by launch_chained(): wait for the kernel before it, then let
// the kernel after it be scheduled as soon as all CTAs of this one have started.
__device__ __forceinline__ void grid_dep_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

// ---- debug builds ------------------------------------------------------------------
// Two compile-time switches give a second library (lib/libmetok_debug.so) that exercises what a
// normal run never reaches:
//   METOK_DEBUG_SHORT_WAIT  bounded waits give up after a few thousand polls, and metok_debug_set
//                           can make a producer skip ONE copy, so that the consumer's wait runs out,
//                           the CTA unwinds and the call's status word reads METOK_ERR_TIMEOUT;
//   METOK_DEBUG_BOUNDS      every data-dependent row or slot index is checked against its range; a bad
//                           one is counted in word 2 of the call's status area and replaced by 0
//                           (no trap, no fault).
// Words 1 and 2 of the status area (the 64 int32 at the start of a workspace) belong to these builds:
// word 1 = the copies to withhold (bit mask, written by the host when the call is made), word 2 = the
// number of out-of-range indices met.
enum { kDbgMergeAssign = 1, kDbgAttnStats = 2, kDbgAttnColsum = 4, kDbgMergeAvg = 8, kDbgGatherRows = 16 };
int debug_arm(int32_t* status, cudaStream_t st);          // debug builds: writes words 1 and 2; else does nothing
#ifdef __CUDACC__
__device__ __forceinline__ bool dbg_withhold(const int32_t* status, int bit) {
#ifdef METOK_DEBUG_SHORT_WAIT
    return (status[1] & bit) != 0;
#else
    (void)status; (void)bit;
    return false;
#endif
}
__device__ __forceinline__ long long dbg_bound(long long idx, long long limit, int32_t* status) {
#ifdef METOK_DEBUG_BOUNDS
    if (idx < 0 || idx >= limit) {
        atomicAdd(status + 2, 1);
        return 0;
    }
#else
    (void)limit; (void)status;
#endif
    return idx;
}
#endif

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int ceilq(double x) {
    double c = x - 1e-9;
    long long f = (long long)c;
    if ((double)f < c) f += 1;
    return (int)f;
}

// Carves 256-byte aligned pieces out of the caller's workspace; with base == nullptr
// it only adds up sizes.
struct Carver {
    char* base;
    size_t off;
    explicit Carver(void* b) : base(reinterpret_cast<char*>(b)), off(0) {}
    template <typename T>
    T* take(size_t count) {
        off = align_up(off, 256);
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += count * sizeof(T);
        return p;
    }
    size_t total() const { return align_up(off, 256); }
};

// ---- element access: 16-byte vectors of either dtype, widened to fp32 ---------
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const float* p, float (&v)[4]) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    __device__ static __forceinline__ void zero(float (&v)[4]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = 0.f;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i]     = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static __forceinline__ void zero(float (&v)[8]) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
    }
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_float(float& o, float x) { o = x; }
__device__ __forceinline__ void from_float(__nv_bfloat16& o, float x) { o = __float2bfloat16_rn(x); }

// ---- warp / block reductions ---------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Order-preserving map float -> uint32 (larger float <=> larger key); -0 and +0 differ
// by one step, which no selection here can observe as a tie on equal values... so
// fold -0 onto +0 first.
__device__ __forceinline__ uint32_t float_key(float f) {
    uint32_t b = __float_as_uint(f + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

}  // namespace metok
