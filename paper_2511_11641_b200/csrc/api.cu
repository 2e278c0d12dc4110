// Status strings and per-thread CUDA error record of libecospa.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace ecospa {

static thread_local char g_cuda_error[256] = "";
static std::atomic<uint64_t> g_launches{0};

void set_cuda_error(cudaError_t e, const char* where) {
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
}

ecospa_status_t check_launch(const char* where) {
    const cudaError_t e = cudaGetLastError();
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e == cudaSuccess) return ECOSPA_OK;
    set_cuda_error(e, where);
    return ECOSPA_ERR_CUDA;
}

}  // namespace ecospa

extern "C" const char* ecospa_status_string(ecospa_status_t s) {
    switch (s) {
        case ECOSPA_OK: return "ok";
        case ECOSPA_ERR_INVALID: return "invalid argument";
        case ECOSPA_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
        case ECOSPA_ERR_UNSUPPORTED: return "unsupported configuration";
        case ECOSPA_ERR_CUDA: return "CUDA error";
        case ECOSPA_ERR_TIMEOUT: return "device-side wait timed out";
        case ECOSPA_ERR_WORKSPACE: return "workspace missing or too small";
    }
    return "unknown status";
}

extern "C" const char* ecospa_last_cuda_error(void) { return ecospa::g_cuda_error; }

extern "C" uint64_t ecospa_launch_count(void) { return ecospa::g_launches.load(std::memory_order_relaxed); }
