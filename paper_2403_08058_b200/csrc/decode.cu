// Clustered decode attention (Fig. 3(b), Section 3.4): one query row per head against the caches.
//
// HBM-bound: (k + H) cache planes are read once per layer and nothing else of size moves.  The work
// is cut into two streaming kernels whose items are all the same size whatever the cluster sizes:
//
//   decode_scores_kernel   item (b, cluster, key chunk): streams a K_rep chunk once, writes the
//                          scaled scores s_t (fp32, B*k*T floats, L2 resident) and the chunk maximum.
//   decode_pv_kernel       item (b, head, value chunk): reads its cluster's global maximum and the
//                          chunk's scores, forms p_t = exp(s_t - max), streams the head's V chunk and
//                          writes the partial sums (sum_t p_t V_t, sum_t p_t).  The CTA that finishes
//                          last for a head (atomic ticket, no waiting) adds the partials in chunk order
//                          and writes out = sum / l.  The result does not depend on scheduling.
//
// Because the softmax reference maximum is global (two-pass), partials need no rescaling.
#include <stdlib.h>
#include <string.h>

#include "decode_layout.cuh"

namespace chai {

template <typename T, int D>
struct DecodeGeom {
    static constexpr int EPV = 16 / (int)sizeof(T);  // elements per 16-byte vector
    static constexpr int LPR = D / EPV;              // lanes that cover one row
    static constexpr int RPW = 32 / LPR;             // rows covered by one warp-wide load
    static constexpr int RPS = kDecWarps * RPW;      // rows covered by one CTA-wide load
    static constexpr int CK = RPS * kStepsK;         // rows per key chunk
    static constexpr int CV = RPS * kStepsV;         // rows per value chunk
    static_assert(LPR >= 1 && LPR <= 32 && (32 % LPR) == 0, "row must split evenly over a warp");
};

__device__ __forceinline__ float block_max(float v, float* s_w) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = s_w[0];
#pragma unroll
    for (int w = 1; w < kDecWarps; ++w) r = fmaxf(r, s_w[w]);
    __syncthreads();
    return r;
}

__device__ __forceinline__ float block_sum(float v, float* s_w) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = s_w[0];
#pragma unroll
    for (int w = 1; w < kDecWarps; ++w) r += s_w[w];
    __syncthreads();
    return r;
}

template <typename T, int D>
__global__ void __launch_bounds__(kDecThreads)
decode_scores_kernel(const T* __restrict__ q, const T* __restrict__ k_rep, const int32_t* __restrict__ reps,
                     const int32_t* __restrict__ seq_lens, WsHeader* __restrict__ hdr, int* __restrict__ counters,
                     float* __restrict__ scores, float* __restrict__ cmax, int H, int k, int T_len, int T_cap,
                     size_t k_batch_stride, float scale, int nK) {
    using G = DecodeGeom<T, D>;
    __shared__ float s_w[kDecWarps];
    const int chunk = blockIdx.x, c = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // housekeeping for the value kernel that follows on the stream: tickets and status word
    if (chunk == 0 && c == 0) {
        for (int h = tid; h < H; h += kDecThreads) counters[(size_t)b * H + h] = 0;
        if (b == 0 && tid == 0) reset_status(hdr);
    }
    const int r = reps[(size_t)b * k + c];
    if (r < 0 || r >= H) return;  // unused cluster slot: nothing reads its scores
    const int len = seq_lens ? min(max(seq_lens[b], 0), T_len) : T_len;  // this request's context length

    const int sub = lane / G::LPR, part = lane % G::LPR;
    float qf[G::EPV];
    {
        const uint4 qv = *reinterpret_cast<const uint4*>(q + ((size_t)b * H + r) * D + part * G::EPV);
        Vec16<T>::unpack(qv, qf);
    }
    const T* kbase = k_rep + (size_t)b * k_batch_stride + (size_t)c * T_cap * D + part * G::EPV;
    const int row0 = chunk * G::CK + warp * G::RPW + sub;

    uint4 buf[kStepsK];
#pragma unroll
    for (int u = 0; u < kStepsK; ++u) {
        const int row = row0 + u * G::RPS;
        buf[u] = make_uint4(0, 0, 0, 0);
        if (row < len) buf[u] = ld_stream16(kbase + (size_t)row * D);
    }
    float lmax = -INFINITY;
    float* srow = scores + ((size_t)b * k + c) * (size_t)T_len;
#pragma unroll
    for (int u = 0; u < kStepsK; ++u) {
        const int row = row0 + u * G::RPS;
        float kf[G::EPV];
        Vec16<T>::unpack(buf[u], kf);
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < G::EPV; ++e) s = fmaf(qf[e], kf[e], s);
#pragma unroll
        for (int o = G::LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= scale;
        if (row < len) {
            if (part == 0) srow[row] = s;
            lmax = fmaxf(lmax, s);
        }
    }
    const float m = block_max(lmax, s_w);
    if (tid == 0) cmax[((size_t)b * k + c) * nK + chunk] = m;
}

template <typename T, int D>
__global__ void __launch_bounds__(kDecThreads)
decode_pv_kernel(const T* __restrict__ v, const int32_t* __restrict__ membership, const int32_t* __restrict__ reps,
                 const int32_t* __restrict__ seq_lens, WsHeader* __restrict__ hdr, int* __restrict__ counters, const float* __restrict__ scores,
                 const float* __restrict__ cmax, float* __restrict__ lpart, float* __restrict__ opart,
                 T* __restrict__ out, int H, int k, int T_len, int T_cap, int nK, int nV) {
    using G = DecodeGeom<T, D>;
    __shared__ float s_p[G::CV];
    __shared__ float s_red[kDecWarps][D];
    __shared__ float s_w[kDecWarps];
    __shared__ int s_ticket;
    const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    int c, r;
    if (!resolve_head(membership, reps, b, h, H, k, &c, &r)) {  // uniform over the CTA
        if (chunk == 0) {
            if (tid == 0) flag_bad_membership(hdr, b, h);
            for (int d = tid; d < D; d += kDecThreads) out[((size_t)b * H + h) * D + d] = from_float<T>(0.f);
        }
        return;
    }

    const int len = seq_lens ? min(max(seq_lens[b], 0), T_len) : T_len;  // this request's context length
    // reference maximum of the whole row of scores (exact two-pass softmax)
    float m = -INFINITY;
    for (int i = tid; i < nK; i += kDecThreads) m = fmaxf(m, cmax[((size_t)b * k + c) * nK + i]);
    m = block_max(m, s_w);

    const int row_base = chunk * G::CV;
    const float* srow = scores + ((size_t)b * k + c) * (size_t)T_len;
    float lsum = 0.f;
    for (int t = tid; t < G::CV; t += kDecThreads) {
        const int row = row_base + t;
        const float p = row < len ? expf(srow[row] - m) : 0.f;
        s_p[t] = p;
        lsum += p;
    }
    const float l = block_sum(lsum, s_w);  // also orders s_p before the reads below

    const int sub = lane / G::LPR, part = lane % G::LPR;
    const T* vbase = v + ((size_t)b * H + h) * (size_t)T_cap * D + part * G::EPV;
    float acc[G::EPV];
#pragma unroll
    for (int e = 0; e < G::EPV; ++e) acc[e] = 0.f;
#pragma unroll
    for (int half = 0; half < kStepsV / 8; ++half) {
        uint4 buf[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int lrow = (half * 8 + u) * G::RPS + warp * G::RPW + sub;
            buf[u] = make_uint4(0, 0, 0, 0);
            if (row_base + lrow < len) buf[u] = ld_stream16(vbase + (size_t)(row_base + lrow) * D);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int lrow = (half * 8 + u) * G::RPS + warp * G::RPW + sub;
            const float p = s_p[lrow];
            float vf[G::EPV];
            Vec16<T>::unpack(buf[u], vf);
#pragma unroll
            for (int e = 0; e < G::EPV; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
        }
    }
    // fold the RPW row slots of the warp, then the warps
#pragma unroll
    for (int o = G::LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int e = 0; e < G::EPV; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    }
    if (lane < G::LPR) {
#pragma unroll
        for (int e = 0; e < G::EPV; ++e) s_red[warp][part * G::EPV + e] = acc[e];
    }
    __syncthreads();
    const size_t head = (size_t)b * H + h;
    if (tid < D) {
        float o = s_red[0][tid];
#pragma unroll
        for (int w = 1; w < kDecWarps; ++w) o += s_red[w][tid];
        opart[(head * nV + chunk) * D + tid] = o;
    }
    if (tid == 0) lpart[head * nV + chunk] = l;

    // last CTA of this head combines the partials in chunk order
    __threadfence();
    __syncthreads();
    if (tid == 0) s_ticket = atomicAdd(&counters[head], 1);
    __syncthreads();
    if (s_ticket != nV - 1) return;
    __threadfence();
    if (tid < D) {
        float o = 0.f, ll = 0.f;
        for (int i = 0; i < nV; ++i) {
            o += __ldcg(&opart[(head * nV + i) * D + tid]);
            ll += __ldcg(&lpart[head * nV + i]);
        }
        out[head * D + tid] = from_float<T>(ll > 0.f ? o / ll : 0.f);  // empty context: zero output
    }
    if (tid == 0) counters[head] = 0;
}

template <typename T, int D>
static int launch_decode(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                         const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k, int T_len,
                         int T_cap, size_t k_batch_stride, float scale, char* ws, const DecodeLayout& L, cudaStream_t s) {
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws);
    int* counters = reinterpret_cast<int*>(ws + L.off_counters);
    float* scores = reinterpret_cast<float*>(ws + L.off_scores);
    float* cmax = reinterpret_cast<float*>(ws + L.off_cmax);
    float* lpart = reinterpret_cast<float*>(ws + L.off_lpart);
    float* opart = reinterpret_cast<float*>(ws + L.off_opart);
    decode_scores_kernel<T, D><<<dim3(L.nK, k, B), kDecThreads, 0, s>>>(
        static_cast<const T*>(q), static_cast<const T*>(k_rep), reps, seq_lens, hdr, counters, scores, cmax, H, k, T_len,
        T_cap, k_batch_stride, scale, L.nK);
    CHAI_LAUNCH_CHECK("decode_scores_kernel launch");
    decode_pv_kernel<T, D><<<dim3(L.nV, H, B), kDecThreads, 0, s>>>(static_cast<const T*>(v), membership, reps, seq_lens,
                                                                   hdr, counters, scores, cmax, lpart, opart,
                                                                   static_cast<T*>(out), H, k, T_len, T_cap, L.nK, L.nV);
    CHAI_LAUNCH_CHECK("decode_pv_kernel launch");
    return CHAI_OK;
}

}  // namespace chai

extern "C" {

size_t chai_decode_workspace_bytes(int B, int H, int k, int T, int D, int dtype) {
    chai::DecodeLayout L;
    if (B <= 0 || H <= 0 || k <= 0 || T <= 0 || (dtype != CHAI_F32 && dtype != CHAI_BF16)) return 0;
    if (!chai::decode_layout(B, H, k, T, D, dtype, &L)) return 0;
    return L.total;
}

namespace {
// Common body of the decode entry points.  `fn` names the caller in messages.
int decode_impl(const char* fn, const void* q, const void* k_rep, const void* v, const int32_t* membership,
                const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k, int T, int T_cap, int D,
                size_t k_batch_stride, float scale, int dtype, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(q && k_rep && v && membership && reps && out && workspace, CHAI_ERR_INVALID_ARG, "%s: null pointer", fn);
    CHAI_REQUIRE(aligned16(q) && aligned16(k_rep) && aligned16(v) && aligned16(out) && aligned16(workspace),
                 CHAI_ERR_INVALID_ARG, "%s: pointers must be 16-byte aligned", fn);
    CHAI_REQUIRE(B > 0 && H > 0 && T > 0 && D > 0, CHAI_ERR_INVALID_ARG, "%s: sizes must be positive", fn);
    CHAI_REQUIRE(k >= 1 && k <= H, CHAI_ERR_INVALID_ARG, "%s: need 1 <= k <= H (k=%d, H=%d)", fn, k, H);
    CHAI_REQUIRE(T <= T_cap, CHAI_ERR_INVALID_ARG, "%s: T=%d exceeds T_cap=%d", fn, T, T_cap);
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED, "%s: unknown dtype %d", fn, dtype);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED, "%s: head_dim %d (64 or 128 supported)", fn, D);
    CHAI_REQUIRE(H <= 65535 && B <= 65535, CHAI_ERR_UNSUPPORTED, "%s: H and B must be <= 65535", fn);
    const size_t dense = (size_t)k * T_cap * D;
    if (k_batch_stride == 0) k_batch_stride = dense;
    CHAI_REQUIRE(k_batch_stride >= dense && (k_batch_stride * elem_size(dtype)) % 16 == 0, CHAI_ERR_INVALID_ARG,
                 "%s: k_batch_stride=%zu must be at least k*T_cap*D=%zu elements and a multiple of 16 bytes", fn,
                 k_batch_stride, dense);
    DecodeLayout L;
    decode_layout(B, H, k, T, D, dtype, &L);
    CHAI_REQUIRE(workspace_bytes >= L.total, CHAI_ERR_WORKSPACE, "%s: workspace has %zu bytes, %zu needed", fn,
                 workspace_bytes, L.total);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    // The persistent streaming kernel is the product path; the split kernels remain for devices
    // without cooperative launch and for A/B measurements (CHAI_DECODE_IMPL=split).
    static const bool force_split = [] {
        const char* e = getenv("CHAI_DECODE_IMPL");
        return e != nullptr && strcmp(e, "split") == 0;
    }();
    CHAI_LOG_CALL("%s: B=%d H=%d k=%d T=%d T_cap=%d D=%d dtype=%d %s%s workspace=%zu of %zu bytes, kernel=%s", fn, B, H, k, T, T_cap,
                  D, dtype, seq_lens ? "ragged " : "", k_batch_stride != dense ? "strided-K " : "", L.total, workspace_bytes,
                  force_split ? "split (CHAI_DECODE_IMPL)" : "persistent, one CTA per SM");
    if (!force_split) {
        const int rc = launch_decode_persistent(q, k_rep, v, membership, reps, seq_lens, out, B, H, k, T, T_cap, D,
                                                k_batch_stride, scale, dtype, ws, L, s);
        if (rc != kDecodeNotLaunched) return rc;
    }
    if (dtype == CHAI_BF16) {
        if (D == 128)
            return launch_decode<__nv_bfloat16, 128>(q, k_rep, v, membership, reps, seq_lens, out, B, H, k, T, T_cap,
                                                     k_batch_stride, scale, ws, L, s);
        return launch_decode<__nv_bfloat16, 64>(q, k_rep, v, membership, reps, seq_lens, out, B, H, k, T, T_cap,
                                                k_batch_stride, scale, ws, L, s);
    }
    if (D == 128)
        return launch_decode<float, 128>(q, k_rep, v, membership, reps, seq_lens, out, B, H, k, T, T_cap, k_batch_stride,
                                         scale, ws, L, s);
    return launch_decode<float, 64>(q, k_rep, v, membership, reps, seq_lens, out, B, H, k, T, T_cap, k_batch_stride, scale,
                                    ws, L, s);
}
}  // namespace

int chai_decode_attention(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                          const int32_t* reps, void* out, int B, int H, int k, int T, int T_cap, int D, float scale,
                          int dtype, void* workspace, size_t workspace_bytes, void* stream) {
    return decode_impl("chai_decode_attention", q, k_rep, v, membership, reps, nullptr, out, B, H, k, T, T_cap, D, 0,
                       scale, dtype, workspace, workspace_bytes, stream);
}

int chai_decode_attention_ragged(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                 const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k,
                                 int T_max, int T_cap, int D, size_t k_batch_stride, float scale, int dtype,
                                 void* workspace, size_t workspace_bytes, void* stream) {
    CHAI_REQUIRE(seq_lens != nullptr, CHAI_ERR_INVALID_ARG, "chai_decode_attention_ragged: seq_lens is null");
    return decode_impl("chai_decode_attention_ragged", q, k_rep, v, membership, reps, seq_lens, out, B, H, k, T_max,
                       T_cap, D, k_batch_stride, scale, dtype, workspace, workspace_bytes, stream);
}

int chai_decode_attention_host_async(const void* q_host, void* out_host, void* q_stage, void* out_stage,
                                     const void* k_rep, const void* v, const int32_t* membership, const int32_t* reps,
                                     int B, int H, int k, int T, int T_cap, int D, float scale, int dtype,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    using namespace chai;
    const char* fn = "chai_decode_attention_host_async";
    CHAI_REQUIRE(q_host && out_host && q_stage && out_stage, CHAI_ERR_INVALID_ARG, "%s: null pointer", fn);
    CHAI_REQUIRE(B > 0 && H > 0 && D > 0 && (dtype == CHAI_F32 || dtype == CHAI_BF16), CHAI_ERR_INVALID_ARG,
                 "%s: bad sizes or dtype", fn);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)B * H * D * elem_size(dtype);
    cudaError_t e = cudaMemcpyAsync(q_stage, q_host, bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(e, "chai_decode_attention_host_async: query upload");
    int rc = chai_decode_attention(q_stage, k_rep, v, membership, reps, out_stage, B, H, k, T, T_cap, D, scale, dtype,
                                   workspace, workspace_bytes, stream);
    if (rc != CHAI_OK) return rc;
    e = cudaMemcpyAsync(out_host, out_stage, bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(e, "chai_decode_attention_host_async: output download");
    return CHAI_OK;
}

int chai_decode_attention_host_streams(const void* q_host, void* out_host, void* q_stage, void* out_stage,
                                       const void* k_rep, const void* v, const int32_t* membership, const int32_t* reps,
                                       int B, int H, int k, int T, int T_cap, int D, float scale, int dtype,
                                       void* workspace, size_t workspace_bytes, void* stream, void* upload_stream,
                                       void* download_stream, void* uploaded_event, void* computed_event) {
    using namespace chai;
    const char* fn = "chai_decode_attention_host_streams";
    CHAI_REQUIRE(q_host && out_host && q_stage && out_stage, CHAI_ERR_INVALID_ARG, "%s: null pointer", fn);
    CHAI_REQUIRE(uploaded_event && computed_event, CHAI_ERR_INVALID_ARG, "%s: both events are required", fn);
    CHAI_REQUIRE(B > 0 && H > 0 && D > 0 && (dtype == CHAI_F32 || dtype == CHAI_BF16), CHAI_ERR_INVALID_ARG,
                 "%s: bad sizes or dtype", fn);
    cudaStream_t s = static_cast<cudaStream_t>(stream), up = static_cast<cudaStream_t>(upload_stream),
                 down = static_cast<cudaStream_t>(download_stream);
    cudaEvent_t e_up = static_cast<cudaEvent_t>(uploaded_event), e_k = static_cast<cudaEvent_t>(computed_event);
    const size_t bytes = (size_t)B * H * D * elem_size(dtype);
    cudaError_t e = cudaMemcpyAsync(q_stage, q_host, bytes, cudaMemcpyHostToDevice, up);
    if (e == cudaSuccess) e = cudaEventRecord(e_up, up);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, e_up, 0);
    if (e != cudaSuccess) return cuda_fail(e, "chai_decode_attention_host_streams: query upload");
    int rc = chai_decode_attention(q_stage, k_rep, v, membership, reps, out_stage, B, H, k, T, T_cap, D, scale, dtype,
                                   workspace, workspace_bytes, stream);
    if (rc != CHAI_OK) return rc;
    e = cudaEventRecord(e_k, s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(down, e_k, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, out_stage, bytes, cudaMemcpyDeviceToHost, down);
    if (e != cudaSuccess) return cuda_fail(e, "chai_decode_attention_host_streams: output download");
    return CHAI_OK;
}

int chai_decode_attention_host(const void* q_host, void* out_host, void* q_stage, void* out_stage, const void* k_rep,
                               const void* v, const int32_t* membership, const int32_t* reps, int B, int H, int k,
                               int T, int T_cap, int D, float scale, int dtype, void* workspace,
                               size_t workspace_bytes, void* stream) {
    const int rc = chai_decode_attention_host_async(q_host, out_host, q_stage, out_stage, k_rep, v, membership, reps, B,
                                                    H, k, T, T_cap, D, scale, dtype, workspace, workspace_bytes, stream);
    if (rc != CHAI_OK) return rc;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return chai::cuda_fail(e, "chai_decode_attention_host: synchronize");
    return CHAI_OK;
}


// ---- decode without any caller-provided or allocated scratch -------------------------------------------
//
// Some callers cannot hand the library a workspace and cannot let it allocate one either: a serving
// engine that reserved all of HBM for its KV-cache pool at start-up has nothing left for cudaMalloc
// to return, and a caller that is inside a latency-critical loop (or between two captured regions)
// must not trigger the device-wide synchronisation an allocation implies.  For them the scratch of the
// decode kernels lives in this fixed array, which is part of the loaded library image: every GPU
// that loads libchai.so carries these 8 MiB until the process exits.
constexpr size_t kStaticScratchBytes = CHAI_DECODE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

int chai_decode_attention_static(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                 const int32_t* reps, void* out, int B, int H, int k, int T, int T_cap, int D,
                                 float scale, int dtype, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(B > 0 && H > 0 && k > 0 && T > 0, CHAI_ERR_INVALID_ARG,
                 "chai_decode_attention_static: sizes must be positive");
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED,
                 "chai_decode_attention_static: unknown dtype %d", dtype);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED,
                 "chai_decode_attention_static: head_dim %d (64 or 128 supported)", D);
    DecodeLayout L;
    CHAI_REQUIRE(decode_layout(B, H, k, T, D, dtype, &L), CHAI_ERR_UNSUPPORTED,
                 "chai_decode_attention_static: no scratch layout for head_dim %d, dtype %d", D, dtype);
    CHAI_REQUIRE(L.total <= kStaticScratchBytes, CHAI_ERR_WORKSPACE,
                 "chai_decode_attention_static: this problem needs %zu bytes of scratch but the built-in array holds "
                 "%zu; use chai_decode_attention with a caller-owned workspace",
                 L.total, kStaticScratchBytes);
    // The array's name is only a host-side handle here; kernels need the address it has on the current
    // device.  It is looked up on every call (a table lookup in the runtime once this device has the
    // library's module loaded) rather than remembered: an address kept across a cudaDeviceReset would dangle.
    // The first call on a device is the one that loads the module: make it before any stream capture.
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return cuda_fail(e, "chai_decode_attention_static: cudaGetSymbolAddress");
    // The decode kernels reset the tickets and the status word themselves at the start of every
    // call, so whatever the previous call left in the array does not matter.
    return chai_decode_attention(q, k_rep, v, membership, reps, out, B, H, k, T, T_cap, D, scale, dtype, ptr,
                                 kStaticScratchBytes, stream);
}

}  // extern "C"
