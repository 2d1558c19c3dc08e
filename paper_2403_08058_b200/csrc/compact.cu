// K-cache compaction: gather the representative heads' key planes (Section 3.5; Section 4.3).
// Pure HBM copy: 2*k*B*T*D*es algorithmic bytes.  Each thread moves 8 independent 16-byte
// vectors (all loads issued before the first store) so that a CTA keeps 32 KB in flight.
#include "chai_common.cuh"

namespace chai {

constexpr int kCompactThreads = 256;
constexpr int kCompactUnroll = 8;

__global__ void __launch_bounds__(kCompactThreads) compact_k_kernel(const uint4* __restrict__ k_full,
                                                                    uint4* __restrict__ k_rep,
                                                                    const int32_t* __restrict__ reps, int H, int k,
                                                                    size_t plane_cap_vec, size_t copy_vec) {
    const int c = blockIdx.y, b = blockIdx.z;
    const int r = reps[(size_t)b * k + c];
    const bool valid = r >= 0 && r < H;
    const uint4* src = k_full + ((size_t)b * H + (valid ? r : 0)) * plane_cap_vec;
    uint4* dst = k_rep + ((size_t)b * k + c) * plane_cap_vec;
    const size_t base = (size_t)blockIdx.x * (kCompactThreads * kCompactUnroll) + threadIdx.x;
    uint4 buf[kCompactUnroll];
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
        size_t i = base + (size_t)u * kCompactThreads;
        buf[u] = make_uint4(0, 0, 0, 0);
        if (valid && i < copy_vec) buf[u] = ld_stream16(src + i);
    }
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
        size_t i = base + (size_t)u * kCompactThreads;
        if (i < copy_vec) __stcs(dst + i, buf[u]);
    }
}

}  // namespace chai

extern "C" int chai_compact_k_cache(const void* k_full, void* k_rep, const int32_t* reps, int B, int H, int k,
                                    int T, int T_cap, int D, int dtype, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(k_full && k_rep && reps, CHAI_ERR_INVALID_ARG, "chai_compact_k_cache: null pointer");
    CHAI_REQUIRE(aligned16(k_full) && aligned16(k_rep), CHAI_ERR_INVALID_ARG,
                 "chai_compact_k_cache: pointers must be 16-byte aligned");
    CHAI_REQUIRE(B > 0 && H > 0 && T > 0 && D > 0, CHAI_ERR_INVALID_ARG, "chai_compact_k_cache: sizes must be positive");
    CHAI_REQUIRE(k >= 1 && k <= H && T <= T_cap, CHAI_ERR_INVALID_ARG,
                 "chai_compact_k_cache: need 1 <= k <= H and T <= T_cap");
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED, "chai_compact_k_cache: dtype");
    const size_t es = elem_size(dtype);
    CHAI_REQUIRE(((size_t)D * es) % 16 == 0, CHAI_ERR_UNSUPPORTED, "chai_compact_k_cache: D*elem_size must be a multiple of 16");
    CHAI_REQUIRE(k <= 65535 && B <= 65535, CHAI_ERR_UNSUPPORTED, "chai_compact_k_cache: k and B must be <= 65535");
    const char* a = static_cast<const char*>(k_full);
    const char* o = static_cast<const char*>(k_rep);
    const size_t in_bytes = (size_t)B * H * T_cap * D * es, out_bytes = (size_t)B * k * T_cap * D * es;
    CHAI_REQUIRE(a + in_bytes <= o || o + out_bytes <= a, CHAI_ERR_INVALID_ARG,
                 "chai_compact_k_cache: k_full and k_rep overlap");
    const size_t plane_cap_vec = (size_t)T_cap * D * es / 16, copy_vec = (size_t)T * D * es / 16;
    const size_t per_cta = (size_t)kCompactThreads * kCompactUnroll;
    dim3 grid((unsigned)((copy_vec + per_cta - 1) / per_cta), k, B);
    // an ordinary launch: as a programmatic dependent of the clustering kernel this grid of hundreds of CTAs made
    // the prefill flow 4 us slower (measured)
    CHAI_LOG_CALL("chai_compact_k_cache: B=%d H=%d k=%d T=%d T_cap=%d D=%d dtype=%d, %zu bytes gathered", B, H, k, T, T_cap, D, dtype,
                  (size_t)B * k * T * D * elem_size(dtype));
    compact_k_kernel<<<grid, kCompactThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(k_full), static_cast<uint4*>(k_rep), reps, H, k, plane_cap_vec, copy_vec);
    CHAI_LAUNCH_CHECK("compact_k_kernel launch");
    return CHAI_OK;
}
