// Status plumbing of libchai: error text, status strings, the blocking status-word read.
#include <stdarg.h>
#include <stdlib.h>
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

// Cycle limit of the decode kernel's device-side waits (see chai_set_decode_wait_limit_cycles).
static std::atomic<long long> g_decode_wait_limit{kDefaultWaitLimitCycles};
long long decode_wait_limit_cycles() { return g_decode_wait_limit.load(std::memory_order_relaxed); }

// CHAI_LOG=1 in the environment: one line per call on stderr (entry point, shapes, what was launched).
bool log_enabled() {
    static const bool on = [] {
        const char* e = getenv("CHAI_LOG");
        return e != nullptr && e[0] != '\0' && e[0] != '0';
    }();
    return on;
}
void log_line(const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    fprintf(stderr, "[chai] %s\n", buf);
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

void chai_set_decode_wait_limit_cycles(long long cycles) {
    chai::g_decode_wait_limit.store(cycles > 0 ? cycles : chai::kDefaultWaitLimitCycles, std::memory_order_relaxed);
}

int chai_device_status(const void* workspace, int* status_out, void* stream) {
    CHAI_REQUIRE(workspace && status_out, CHAI_ERR_INVALID_ARG, "chai_device_status: null argument");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    chai::WsHeader h;
    cudaError_t e = cudaMemcpyAsync(&h, workspace, sizeof(h), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return chai::cuda_fail(e, "chai_device_status copy");
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return chai::cuda_fail(e, "chai_device_status sync");
    // A decode launch in which a wait ran out says so with its own token (see WsHeader): that cannot be lost to
    // the status word's reset by the CTA that owns the launch's first tile, whichever of the two comes first.
    unsigned long long gave_up, latest;
    memcpy(&gave_up, &h.pad[chai::kHdrGaveUpToken], 8);
    memcpy(&latest, &h.pad[chai::kHdrLaunchToken], 8);
    *status_out = (gave_up != 0 && gave_up == latest) ? (int)CHAI_ERR_TIMEOUT : h.status;
    return CHAI_OK;
}

}  // extern "C"
