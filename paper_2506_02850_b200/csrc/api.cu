// Host-only helpers of the C ABI: status strings, last CUDA error, version.
#include <deque>
#include <mutex>
#include <string>
#include <vector>
#include <cstdio>
#include <cstring>

#include "common.cuh"
#include "sm100.cuh"

namespace metok {
static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

bool g_profiling = false;
namespace {
struct Rec { const char* scope; const char* name; cudaEvent_t a, b; };
std::vector<Rec> g_recs;
std::deque<std::string> g_scopes;            // interned scope labels: pointers into it stay valid
const char* g_scope = "";                    // label of the brackets recorded from now on
std::mutex g_mu;
}  // namespace

KernelTimer::KernelTimer(const char* n, cudaStream_t s) : name(n), st(s), a(nullptr), b(nullptr), active(g_profiling) {
    if (!active) return;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { active = false; return; }
    record(a);
}
// On a stream that is being captured the bracket becomes an event-record node of the graph, so that a
// replay of the graph times its kernels without the host's launch gaps between them.
void KernelTimer::record(cudaEvent_t e) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusActive)
        cudaEventRecordWithFlags(e, st, cudaEventRecordExternal);
    else
        cudaEventRecord(e, st);
}
KernelTimer::~KernelTimer() {
    if (!active) return;
    record(b);
    std::lock_guard<std::mutex> lk(g_mu);
    g_recs.push_back({g_scope, name, a, b});
}
}  // namespace metok

namespace metok {
int make_tmap_bf16_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        METOK_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (!fn || q != cudaDriverEntryPointSuccess) return METOK_ERR_UNSUPPORTED;
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};                 // bytes between rows
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error((int)r);
        return METOK_ERR_CUDA;
    }
    return METOK_OK;
}
}  // namespace metok

extern "C" int metok_profile_begin(void) {
    std::lock_guard<std::mutex> lk(metok::g_mu);
    for (auto& r : metok::g_recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    metok::g_recs.clear();
    metok::g_scope = "";
    metok::g_profiling = true;
    return METOK_OK;
}

extern "C" int metok_profile_scope(const char* label) {
    std::lock_guard<std::mutex> lk(metok::g_mu);
    if (!label || !*label) { metok::g_scope = ""; return METOK_OK; }
    for (const char* c = label; *c; ++c)
        if (*c == ' ' || *c == '\n' || *c == '/') return METOK_ERR_INVALID_ARG;
    for (auto& sc : metok::g_scopes)
        if (sc == label) { metok::g_scope = sc.c_str(); return METOK_OK; }
    metok::g_scopes.emplace_back(label);
    metok::g_scope = metok::g_scopes.back().c_str();
    return METOK_OK;
}

// Elapsed times of all recorded brackets, one line per kernel name; `release` destroys the events.
static int profile_collect(char* out, size_t cap, bool release) {
    metok::g_profiling = false;
    std::lock_guard<std::mutex> lk(metok::g_mu);
    struct Agg { std::string name; int n; double ms; };
    std::vector<Agg> agg;
    int launches = 0;
    for (auto& r : metok::g_recs) {
        float ms = 0.f;
        if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) {
            metok::set_last_cuda_error((int)cudaGetLastError());
            return METOK_ERR_CUDA;
        }
        ++launches;
        bool found = false;
        const std::string full = *r.scope ? std::string(r.scope) + "/" + r.name : std::string(r.name);
        for (auto& g : agg)
            if (g.name == full) { g.n += 1; g.ms += ms; found = true; break; }
        if (!found) agg.push_back({full, 1, (double)ms});
        if (release) {
            cudaEventDestroy(r.a);
            cudaEventDestroy(r.b);
        }
    }
    if (release) metok::g_recs.clear();
    if (out && cap > 0) {
        std::string text;
        char line[256];
        for (auto& g : agg) {
            std::snprintf(line, sizeof line, "%s %d %.6f\n", g.name.c_str(), g.n, g.ms);
            text += line;
        }
        const size_t n = text.size() < cap - 1 ? text.size() : cap - 1;
        std::memcpy(out, text.data(), n);
        out[n] = 0;
    }
    return launches;
}

extern "C" int metok_profile_read(char* out, size_t cap) { return profile_collect(out, cap, false); }
extern "C" int metok_profile_end(char* out, size_t cap) { return profile_collect(out, cap, true); }

namespace metok {
#if defined(METOK_DEBUG_SHORT_WAIT) || defined(METOK_DEBUG_BOUNDS)
static int g_dbg_withhold = 0;
#endif
int debug_arm(int32_t* status, cudaStream_t st) {
#if defined(METOK_DEBUG_SHORT_WAIT) || defined(METOK_DEBUG_BOUNDS)
    const int32_t words[2] = {g_dbg_withhold, 0};
    METOK_CUDA_TRY(cudaMemcpyAsync(status + 1, words, sizeof words, cudaMemcpyHostToDevice, st));
#else
    (void)status; (void)st;
#endif
    return METOK_OK;
}
}  // namespace metok

extern "C" int metok_debug_set(int what, int value) {
#if defined(METOK_DEBUG_SHORT_WAIT) || defined(METOK_DEBUG_BOUNDS)
    if (what == METOK_DEBUG_WITHHOLD_COPY) { metok::g_dbg_withhold = value; return METOK_OK; }
    return METOK_ERR_INVALID_ARG;
#else
    (void)what; (void)value;
    return METOK_ERR_UNSUPPORTED;
#endif
}

extern "C" int metok_debug_build(void) {
    int flags = 0;
#ifdef METOK_DEBUG_SHORT_WAIT
    flags |= 1;
#endif
#ifdef METOK_DEBUG_BOUNDS
    flags |= 2;
#endif
    return flags;
}

extern "C" const char* metok_status_string(int status) {
    switch (status) {
        case METOK_OK: return "ok";
        case METOK_ERR_INVALID_ARG: return "invalid argument";
        case METOK_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case METOK_ERR_WORKSPACE: return "workspace missing or too small";
        case METOK_ERR_CUDA: return "CUDA error";
        case METOK_ERR_TIMEOUT: return "device-side wait timed out";
        case METOK_ERR_TOO_LARGE: return "problem exceeds the built-in scratch capacity";
        default: return "unknown status";
    }
}

extern "C" int metok_last_cuda_error(void) { return metok::g_last_cuda_error; }

extern "C" int metok_version(void) { return 100; }
