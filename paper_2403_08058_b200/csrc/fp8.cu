// fp8 (e4m3) caches for the clustered decode step.  The paper presents head clustering as orthogonal to
// quantisation (Section 2, related work on quantised KV caches): storing the representative keys and the
// values in one byte per element halves the bytes the decode step has to stream once more.
//
//   chai_quantize_cache_fp8     bf16 cache planes -> e4m3 bytes + one fp32 scale per plane
//   chai_decode_attention_fp8   the decode step on such caches (bf16 queries and output, fp32 accumulation)
#include "decode_layout.cuh"

namespace chai {

constexpr float kE4M3Max = 448.f;  // largest finite e4m3 value

// absmax per plane over rows [0,T): positive floats order like their bit patterns, so an integer atomicMax does it.
// VEC: 16-byte loads of 8 elements (the host checks alignment and that the row count allows it).
template <bool VEC>
__global__ void __launch_bounds__(256)
fp8_absmax_kernel(const __nv_bfloat16* __restrict__ src, int* __restrict__ absmax_bits, int T, int T_cap, int D) {
    const int plane = blockIdx.y;
    const size_t n = (size_t)T * D;
    const __nv_bfloat16* p = src + (size_t)plane * T_cap * D;
    const size_t first = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
    float m = 0.f;
    if constexpr (VEC) {
        const uint4* p4 = reinterpret_cast<const uint4*>(p);
        const size_t n4 = n / 8;
        for (size_t i = first; i < n4; i += 4 * stride) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i + u * stride < n4) v[u] = __ldg(p4 + i + u * stride); else v[u] = make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    m = fmaxf(m, fabsf(__uint_as_float(w[e] << 16)));
                    m = fmaxf(m, fabsf(__uint_as_float(w[e] & 0xffff0000u)));
                }
            }
        }
    } else {
        for (size_t i = first; i < n; i += stride) m = fmaxf(m, fabsf(__bfloat162float(p[i])));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(absmax_bits + plane, __float_as_int(m));
}

__device__ __forceinline__ unsigned quant1(float x, float scale) {
    return (unsigned)__nv_cvt_float_to_fp8(__fdiv_rn(x, scale), __NV_SATFINITE, __NV_E4M3);
}

// q = round-to-nearest-even e4m3 of (x / scale), scale = absmax / 448 in fp32 (1 for an all-zero plane)
template <bool VEC>
__global__ void __launch_bounds__(256)
fp8_quantize_kernel(const __nv_bfloat16* __restrict__ src, unsigned char* __restrict__ dst,
                    const int* __restrict__ absmax_bits, int T, int T_cap, int D) {
    const int plane = blockIdx.y;
    const float amax = __int_as_float(absmax_bits[plane]);
    const float scale = amax > 0.f ? __fdiv_rn(amax, kE4M3Max) : 1.f;
    const size_t n = (size_t)T * D;
    const __nv_bfloat16* p = src + (size_t)plane * T_cap * D;
    unsigned char* q = dst + (size_t)plane * T_cap * D;
    const size_t first = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
    if constexpr (VEC) {
        const uint4* p4 = reinterpret_cast<const uint4*>(p);
        uint2* q2 = reinterpret_cast<uint2*>(q);
        const size_t n4 = n / 8;
        for (size_t i = first; i < n4; i += 4 * stride) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i + u * stride < n4) v[u] = __ldg(p4 + i + u * stride);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (i + u * stride >= n4) break;
                const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                unsigned b[8];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    b[2 * e] = quant1(__uint_as_float(w[e] << 16), scale);
                    b[2 * e + 1] = quant1(__uint_as_float(w[e] & 0xffff0000u), scale);
                }
                uint2 o;
                o.x = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
                o.y = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
                q2[i + u * stride] = o;
            }
        }
    } else {
        for (size_t i = first; i < n; i += stride) q[i] = (unsigned char)quant1(__bfloat162float(p[i]), scale);
    }
}

__global__ void fp8_scales_kernel(int* __restrict__ absmax_bits_to_scale, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float amax = __int_as_float(absmax_bits_to_scale[i]);
    absmax_bits_to_scale[i] = __float_as_int(amax > 0.f ? __fdiv_rn(amax, kE4M3Max) : 1.f);
}

}  // namespace chai

extern "C" {

int chai_quantize_cache_fp8(const void* src, void* dst, float* scales, int n_planes, int T, int T_cap, int D,
                            void* stream) {
    using namespace chai;
    CHAI_REQUIRE(src && dst && scales, CHAI_ERR_INVALID_ARG, "chai_quantize_cache_fp8: null pointer");
    CHAI_REQUIRE(n_planes > 0 && T > 0 && T <= T_cap && D > 0, CHAI_ERR_INVALID_ARG,
                 "chai_quantize_cache_fp8: need n_planes, D > 0 and 0 < T <= T_cap");
    CHAI_REQUIRE(n_planes <= 65535, CHAI_ERR_UNSUPPORTED, "chai_quantize_cache_fp8: at most 65535 planes per call");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(scales, 0, sizeof(float) * (size_t)n_planes, s);
    if (e != cudaSuccess) return cuda_fail(e, "chai_quantize_cache_fp8: clearing the scales");
    // 16-byte loads need every plane to start on a 16-byte boundary and hold a multiple of 8 elements
    const bool vec = ((size_t)T * D) % 8 == 0 && ((size_t)T_cap * D) % 16 == 0 && aligned16(src) && aligned16(dst);
    const size_t n = (size_t)T * D;
    const size_t per_cta = vec ? 256 * 8 * 4 : 256 * 16;
    unsigned chunks = (unsigned)((n + per_cta - 1) / per_cta);
    chunks = chunks < 1 ? 1 : (chunks > 64 ? 64 : chunks);
    int* bits = reinterpret_cast<int*>(scales);
    const dim3 grid(chunks, n_planes);
    const __nv_bfloat16* sp = static_cast<const __nv_bfloat16*>(src);
    unsigned char* dp = static_cast<unsigned char*>(dst);
    if (vec) fp8_absmax_kernel<true><<<grid, 256, 0, s>>>(sp, bits, T, T_cap, D);
    else fp8_absmax_kernel<false><<<grid, 256, 0, s>>>(sp, bits, T, T_cap, D);
    CHAI_LAUNCH_CHECK("fp8_absmax_kernel launch");
    if (vec) fp8_quantize_kernel<true><<<grid, 256, 0, s>>>(sp, dp, bits, T, T_cap, D);
    else fp8_quantize_kernel<false><<<grid, 256, 0, s>>>(sp, dp, bits, T, T_cap, D);
    CHAI_LAUNCH_CHECK("fp8_quantize_kernel launch");
    fp8_scales_kernel<<<(n_planes + 255) / 256, 256, 0, s>>>(bits, n_planes);
    CHAI_LAUNCH_CHECK("fp8_scales_kernel launch");
    return CHAI_OK;
}

size_t chai_decode_fp8_workspace_bytes(int B, int H, int k, int T, int D) {
    chai::DecodeLayout L;
    if (B <= 0 || H <= 0 || k <= 0 || T <= 0) return 0;
    if (!chai::decode_layout(B, H, k, T, D, CHAI_FP8_E4M3, &L)) return 0;
    return L.total;
}

int chai_decode_attention_fp8(const void* q, const void* k_rep, const void* v, const float* k_scale, const float* v_scale,
                              const int32_t* membership, const int32_t* reps, const int32_t* seq_lens, void* out, int B,
                              int H, int k, int T, int T_cap, int D, size_t k_batch_stride, float scale, void* workspace,
                              size_t workspace_bytes, void* stream) {
    using namespace chai;
    const char* fn = "chai_decode_attention_fp8";
    CHAI_REQUIRE(q && k_rep && v && k_scale && v_scale && membership && reps && out && workspace, CHAI_ERR_INVALID_ARG,
                 "%s: null pointer", fn);
    CHAI_REQUIRE(aligned16(q) && aligned16(k_rep) && aligned16(v) && aligned16(out) && aligned16(workspace),
                 CHAI_ERR_INVALID_ARG, "%s: pointers must be 16-byte aligned", fn);
    CHAI_REQUIRE(B > 0 && H > 0 && T > 0 && k >= 1 && k <= H && T <= T_cap, CHAI_ERR_INVALID_ARG,
                 "%s: need B, H, T > 0, 1 <= k <= H, T <= T_cap", fn);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED, "%s: head_dim %d (64 or 128 supported)", fn, D);
    CHAI_REQUIRE(H <= 65535 && B <= 65535, CHAI_ERR_UNSUPPORTED, "%s: H and B must be <= 65535", fn);
    const size_t dense = (size_t)k * T_cap * D;
    if (k_batch_stride == 0) k_batch_stride = dense;
    CHAI_REQUIRE(k_batch_stride >= dense && k_batch_stride % 16 == 0, CHAI_ERR_INVALID_ARG,
                 "%s: k_batch_stride=%zu must be at least k*T_cap*D=%zu elements and a multiple of 16", fn, k_batch_stride,
                 dense);
    DecodeLayout L;
    decode_layout(B, H, k, T, D, CHAI_FP8_E4M3, &L);
    CHAI_REQUIRE(workspace_bytes >= L.total, CHAI_ERR_WORKSPACE, "%s: workspace has %zu bytes, %zu needed", fn,
                 workspace_bytes, L.total);
    CHAI_LOG_CALL("chai_decode_attention_fp8: B=%d H=%d k=%d T=%d T_cap=%d D=%d %se4m3 caches, persistent kernel, one CTA per SM", B, H, k,
                  T, T_cap, D, seq_lens ? "ragged " : "");
    const int rc = launch_decode_persistent(q, k_rep, v, membership, reps, seq_lens, out, B, H, k, T, T_cap, D,
                                            k_batch_stride, scale, CHAI_FP8_E4M3, static_cast<char*>(workspace), L,
                                            static_cast<cudaStream_t>(stream), k_scale, v_scale);
    CHAI_REQUIRE(rc != kDecodeNotLaunched, CHAI_ERR_UNSUPPORTED,
                 "%s: this device cannot run the persistent decode kernel (no cooperative launch)", fn);
    return rc;
}

}  // extern "C"
