// Shared host/device helpers of libchai: status plumbing, argument checks, dtype loads.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <atomic>
#include <mutex>
#include <utility>

#include "chai.h"

namespace chai {

// The first 256 bytes of every workspace.  `status` is a chai_status_t; the other words say where
// the first inconsistency was seen (debugging aid only).
struct WsHeader {
    int status;
    int bad_b;
    int bad_h;
    int pad[61];
};
static_assert(sizeof(WsHeader) == 256, "workspace header is 256 bytes");
// Words of pad[] with a fixed meaning.  Decode: pad[0] work counter, pad[8] launch count of the workspace, and two
// 64-bit launch tokens (8-byte aligned): the token of the latest launch that started or gave up, and the token of
// the latest launch in which a bounded wait ran out.  Equal and non-zero = the latest launch timed out.  Prefill:
// pad[0..59] are per-launch work counters, cleared by the planner (both tokens then read 0).
constexpr int kHdrGaveUpToken = 11, kHdrLaunchToken = 13;
static_assert((12 + 4 * kHdrGaveUpToken) % 8 == 0 && (12 + 4 * kHdrLaunchToken) % 8 == 0, "token words are 8-byte aligned");

// Every device-side wait is bounded by a cycle count; this is the default (about a second).
constexpr long long kDefaultWaitLimitCycles = 2000000000ll;
long long decode_wait_limit_cycles();  // current limit of the decode kernel's waits (api.cu)

void set_last_error(const char* fmt, ...);
bool log_enabled();                      // CHAI_LOG set in the environment (read once)
void log_line(const char* fmt, ...);     // one line on stderr
#define CHAI_LOG_CALL(...)                                   \
    do {                                                     \
        if (::chai::log_enabled()) ::chai::log_line(__VA_ARGS__); \
    } while (0)
int cuda_fail(cudaError_t e, const char* what);  // records the text, returns CHAI_ERR_CUDA

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t elem_size(int dtype) { return dtype == CHAI_BF16 ? 2 : (dtype == CHAI_FP8_E4M3 ? 1 : 4); }

// Per-device set-up that the first call on a device performs (attribute queries, a kernel's opt-in to its
// shared-memory size), safe when several host threads make their first call at once: the flag is read with
// acquire order, the set-up runs under a mutex, and the flag is set only when it succeeded (a failed set-up is
// tried again by the next call).  What the set-up stored is visible to every thread that sees the flag.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    std::atomic<bool> done[kMaxDevices];
    std::mutex lock;
    PerDeviceOnce() {
        for (auto& d : done) d.store(false, std::memory_order_relaxed);
    }
    template <typename F>
    int run(int dev, F&& setup) {  // setup() returns a chai status
        std::atomic<bool>& flag = done[dev & (kMaxDevices - 1)];
        if (flag.load(std::memory_order_acquire)) return CHAI_OK;
        std::lock_guard<std::mutex> guard(lock);
        if (flag.load(std::memory_order_relaxed)) return CHAI_OK;
        const int rc = setup();
        if (rc == CHAI_OK) flag.store(true, std::memory_order_release);
        return rc;
    }
};

#define CHAI_REQUIRE(cond, code, ...)            \
    do {                                         \
        if (!(cond)) {                           \
            ::chai::set_last_error(__VA_ARGS__); \
            return (code);                       \
        }                                        \
    } while (0)

#define CHAI_LAUNCH_CHECK(what)                                   \
    do {                                                          \
        cudaError_t e__ = cudaGetLastError();                     \
        if (e__ != cudaSuccess) return ::chai::cuda_fail(e__, what); \
    } while (0)

// Launches `kernel` as a programmatic dependent of whatever precedes it on the stream: if that kernel lets its
// dependents go early (ours do, first thing), this one is scheduled while the predecessor drains and blocks in
// dependent_grid_sync() until the predecessor has completed and its writes are visible, which hides the launch
// latency in chains of short kernels.  After any other kernel, a copy or a memset the attribute changes nothing.
// Every kernel launched this way calls dependent_grid_sync() before its first access to global memory.
// Not a default: measured on the prefill flow (features, clustering, compaction, planner, attention; 144 us),
// the clustering kernel and the planner gain a little from it, while the feature kernel (128 small CTAs
// behind the attention kernel of the previous call) made the flow 17 us slower, so that one and the copy
// kernels with grids of hundreds of CTAs are launched the ordinary way.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args&&... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

#define CHAI_LAUNCH_DEPENDENT(what, ...)                               \
    do {                                                               \
        cudaError_t e__ = ::chai::launch_dependent(__VA_ARGS__);        \
        if (e__ != cudaSuccess) return ::chai::cuda_fail(e__, what);    \
    } while (0)

// ---- device helpers ---------------------------------------------------------------------------

// First statement of a kernel launched with launch_dependent(): release our own dependents, then wait for
// the grid before us.  Both instructions do nothing in a kernel launched the ordinary way.
__device__ __forceinline__ void dependent_grid_sync() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// 16-byte vector of T unpacked to floats: 8 bf16 or 4 fp32.
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
    static constexpr int N = 4;
    __device__ __forceinline__ static void unpack(const uint4& r, float* f) {
        f[0] = __uint_as_float(r.x);
        f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z);
        f[3] = __uint_as_float(r.w);
    }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    // bf16 -> fp32 is a 16-bit shift
    __device__ __forceinline__ static void unpack(const uint4& r, float* f) {
        f[0] = __uint_as_float(r.x << 16);
        f[1] = __uint_as_float(r.x & 0xffff0000u);
        f[2] = __uint_as_float(r.y << 16);
        f[3] = __uint_as_float(r.y & 0xffff0000u);
        f[4] = __uint_as_float(r.z << 16);
        f[5] = __uint_as_float(r.z & 0xffff0000u);
        f[6] = __uint_as_float(r.w << 16);
        f[7] = __uint_as_float(r.w & 0xffff0000u);
    }
};

// One byte per element: fp8 e4m3 (4 exponent bits, bias 7, 3 mantissa bits, no infinities) as stored by
// chai_quantize_cache_fp8; the value it stands for is the decoded number times the plane's scale.
struct Fp8E4M3 {
    unsigned char bits;
};
template <>
struct Vec16<Fp8E4M3> {
    static constexpr int N = 16;
    __device__ __forceinline__ static void unpack(const uint4& r, float* f) {
        const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(w[i] & 0xffffu), __NV_E4M3);
            const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(w[i] >> 16), __NV_E4M3);
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&lo));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&hi));
            f[4 * i + 0] = a.x;
            f[4 * i + 1] = a.y;
            f[4 * i + 2] = b.x;
            f[4 * i + 3] = b.y;
        }
    }
    // the same 16 values as eight fp16 pairs (every e4m3 value is an fp16 value): h[j] = elements 2j, 2j + 1
    __device__ __forceinline__ static void unpack_h2(const uint4& r, __half2* h) {
        const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(w[i] & 0xffffu), __NV_E4M3);
            const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(w[i] >> 16), __NV_E4M3);
            h[2 * i] = *reinterpret_cast<const __half2*>(&lo);
            h[2 * i + 1] = *reinterpret_cast<const __half2*>(&hi);
        }
    }
};

// Streaming 16-byte load that does not pollute L1 (cache data are read exactly once).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// Start of a call that reports through the status word: no error yet, and no launch token that says "gave up"
// (a fresh workspace may hold anything there, two equal words included).
__device__ __forceinline__ void reset_status(WsHeader* hdr) {
    hdr->status = CHAI_OK;
    hdr->bad_b = -1;
    hdr->bad_h = -1;
    *reinterpret_cast<unsigned long long*>(&hdr->pad[kHdrGaveUpToken]) = 0ull;
}

// Records the first data inconsistency a kernel meets; never traps.
__device__ __forceinline__ void flag_bad_membership(WsHeader* hdr, int b, int h) {
    if (atomicCAS(&hdr->status, CHAI_OK, CHAI_ERR_BAD_MEMBERSHIP) == CHAI_OK) {
        hdr->bad_b = b;
        hdr->bad_h = h;
    }
}

// Resolves head h of request b to (cluster, representative); returns false (and flags) when the
// membership data are inconsistent.  No address outside the arrays is formed.
__device__ __forceinline__ bool resolve_head(const int32_t* membership, const int32_t* reps, int b, int h,
                                             int H, int k, int* c_out, int* r_out) {
    int c = membership[(size_t)b * H + h];
    if (c < 0 || c >= k) return false;
    int r = reps[(size_t)b * k + c];
    if (r < 0 || r >= H) return false;
    if (membership[(size_t)b * H + r] != c) return false;
    *c_out = c;
    *r_out = r;
    return true;
}

}  // namespace chai
