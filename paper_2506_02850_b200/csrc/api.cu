// Host-only helpers of the C ABI: status strings, last CUDA error, version.
#include "common.cuh"

namespace metok {
static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }
}  // namespace metok

extern "C" const char* metok_status_string(int status) {
    switch (status) {
        case METOK_OK: return "ok";
        case METOK_ERR_INVALID_ARG: return "invalid argument";
        case METOK_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case METOK_ERR_WORKSPACE: return "workspace missing or too small";
        case METOK_ERR_CUDA: return "CUDA error";
        case METOK_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

extern "C" int metok_last_cuda_error(void) { return metok::g_last_cuda_error; }

extern "C" int metok_version(void) { return 100; }
