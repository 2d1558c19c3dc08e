// Status plumbing of libchai: error text, status strings, the blocking status-word read.
#include <stdarg.h>
#include <string.h>

#include "chai_common.cuh"

namespace chai {

static thread_local char g_last_error[512] = "";

void set_last_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char* what) {
    set_last_error("%s: %s", what, cudaGetErrorString(e));
    return CHAI_ERR_CUDA;
}

}  // namespace chai

extern "C" {

const char* chai_status_string(int status) {
    switch (status) {
        case CHAI_OK: return "ok";
        case CHAI_ERR_INVALID_ARG: return "invalid argument";
        case CHAI_ERR_UNSUPPORTED: return "unsupported configuration";
        case CHAI_ERR_WORKSPACE: return "workspace too small";
        case CHAI_ERR_BAD_MEMBERSHIP: return "inconsistent membership / representatives";
        case CHAI_ERR_TIMEOUT: return "device-side wait expired";
        case CHAI_ERR_CUDA: return "CUDA error";
        case CHAI_ERR_CACHE_FULL: return "cache position outside [0, T_cap)";
        default: return "unknown status";
    }
}

const char* chai_last_error(void) { return chai::g_last_error; }

int chai_version(void) { return 100; }

int chai_device_status(const void* workspace, int* status_out, void* stream) {
    CHAI_REQUIRE(workspace && status_out, CHAI_ERR_INVALID_ARG, "chai_device_status: null argument");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int st = 0;
    cudaError_t e = cudaMemcpyAsync(&st, workspace, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return chai::cuda_fail(e, "chai_device_status copy");
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return chai::cuda_fail(e, "chai_device_status sync");
    *status_out = st;
    return CHAI_OK;
}

}  // extern "C"
