// Clustered prefill attention on CUDA cores: the fp32 path and the general-shape kernel.
//
// One CTA = (request, cluster member group of <= 2 heads, tile of 32 query rows).  It walks the
// key tiles of the cluster's representative with an online softmax and applies each probability
// tile to every member head's value tile.  fp32 accumulation throughout; inputs are widened to
// fp32 in shared memory.  The bf16 / head_dim-128 tensor-core kernel lives in prefill_tc.cu.
#include <stdlib.h>

#include "prefill_plan.cuh"

namespace chai {

constexpr int kSimtBQ = 32, kSimtBK = 32, kSimtThreads = 128, kSimtG = 2;

template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
prefill_simt_kernel(const T* __restrict__ q, const T* __restrict__ k_rep, const T* __restrict__ v,
                    const int* __restrict__ n_groups, const GroupEntry* __restrict__ groups, T* __restrict__ out,
                    WsHeader* __restrict__ hdr, const int* __restrict__ bad, int H, int k, int T_len, int q_start,
                    float scale, int causal, int n_qtiles) {
    constexpr int DP = D + 1;         // padded row: conflict-free column walks
    constexpr int DPT = D / 4;        // output columns per thread
    extern __shared__ float smem_f[];
    float* Qs = smem_f;               // [32][DP]
    float* Ks = Qs + kSimtBQ * DP;    // [32][DP]
    float* Vs = Ks + kSimtBK * DP;    // [32][D]
    float* Ps = Vs + kSimtBK * D;     // [32][33]

    const int b = blockIdx.z, slot = blockIdx.y;
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) publish_plan_status(hdr, bad, gridDim.z);
    if (slot >= n_groups[b]) return;
    const int qt = n_qtiles - 1 - (int)blockIdx.x;  // longest (latest) query tiles first
    const GroupEntry e = groups[(size_t)b * H + slot];
    const int q0 = qt * kSimtBQ;
    const int tid = threadIdx.x, i = tid >> 2, jq = tid & 3;
    const int i_abs = q0 + i;

    if (e.cluster < 0) {  // heads that could not be resolved: zero rows
        for (int g = 0; g < e.n; ++g)
            for (int idx = tid; idx < kSimtBQ * D; idx += kSimtThreads) {
                const int row = q0 + idx / D;
                if (row >= q_start && row < T_len)
                    out[(((size_t)b * H + e.heads[g]) * T_len + row) * D + idx % D] = from_float<T>(0.f);
            }
        return;
    }

    const T* qh = q + ((size_t)b * H + e.rep) * (size_t)T_len * D;
    const T* kc = k_rep + ((size_t)b * k + e.cluster) * (size_t)T_len * D;
    for (int idx = tid; idx < kSimtBQ * D; idx += kSimtThreads) {
        const int r = idx / D, d = idx % D;
        Qs[r * DP + d] = (q0 + r < T_len) ? to_float(qh[(size_t)(q0 + r) * D + d]) : 0.f;
    }

    float acc[kSimtG][DPT];
#pragma unroll
    for (int g = 0; g < kSimtG; ++g)
#pragma unroll
        for (int dd = 0; dd < DPT; ++dd) acc[g][dd] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;

    const int kv_end = causal ? min(T_len, q0 + kSimtBQ) : T_len;
    for (int j0 = 0; j0 < kv_end; j0 += kSimtBK) {
        __syncthreads();  // previous tile's Ks / Vs / Ps fully consumed
        for (int idx = tid; idx < kSimtBK * D; idx += kSimtThreads) {
            const int r = idx / D, d = idx % D;
            Ks[r * DP + d] = (j0 + r < T_len) ? to_float(kc[(size_t)(j0 + r) * D + d]) : 0.f;
        }
        __syncthreads();
        float s[8];
        float tmax = -INFINITY;
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int j = jq + 4 * jj, j_abs = j0 + j;
            float dot = 0.f;
            for (int d = 0; d < D; ++d) dot = fmaf(Qs[i * DP + d], Ks[j * DP + d], dot);
            const bool visible = j_abs < T_len && (!causal || j_abs <= i_abs);
            s[jj] = visible ? dot * scale : -INFINITY;
            tmax = fmaxf(tmax, s[jj]);
        }
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        const float m_new = fmaxf(m_run, tmax);
        // a row with nothing visible so far keeps m = -inf; use 0 as a harmless reference then
        const float m_ref = m_new == -INFINITY ? 0.f : m_new;
        const float corr = expf(m_run - m_ref);
        float psum = 0.f;
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const float p = expf(s[jj] - m_ref);
            Ps[i * 33 + jq + 4 * jj] = p;
            psum += p;
        }
        psum += __shfl_xor_sync(0xffffffffu, psum, 1);
        psum += __shfl_xor_sync(0xffffffffu, psum, 2);
        l_run = l_run * corr + psum;
        m_run = m_new;
#pragma unroll
        for (int g = 0; g < kSimtG; ++g)
#pragma unroll
            for (int dd = 0; dd < DPT; ++dd) acc[g][dd] *= corr;

        for (int g = 0; g < e.n; ++g) {
            const T* vh = v + ((size_t)b * H + e.heads[g]) * (size_t)T_len * D;
            __syncthreads();  // Ps written (first pass) / previous member's Vs consumed
            for (int idx = tid; idx < kSimtBK * D; idx += kSimtThreads) {
                const int r = idx / D, d = idx % D;
                Vs[idx] = (j0 + r < T_len) ? to_float(vh[(size_t)(j0 + r) * D + d]) : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int gg = 0; gg < kSimtG; ++gg) {
                if (gg != g) continue;
                for (int j = 0; j < kSimtBK; ++j) {
                    const float p = Ps[i * 33 + j];
#pragma unroll
                    for (int dd = 0; dd < DPT; ++dd) acc[gg][dd] = fmaf(p, Vs[j * D + jq + 4 * dd], acc[gg][dd]);
                }
            }
        }
    }
    if (i_abs >= q_start && i_abs < T_len) {  // rows before q_start belong to the caller (prefix computed earlier)
        const float inv = 1.f / l_run;
#pragma unroll
        for (int gg = 0; gg < kSimtG; ++gg) {
            if (gg >= e.n) continue;
            T* o = out + (((size_t)b * H + e.heads[gg]) * T_len + i_abs) * D;
#pragma unroll
            for (int dd = 0; dd < DPT; ++dd) o[jq + 4 * dd] = from_float<T>(acc[gg][dd] * inv);
        }
    }
}

template <typename T, int D>
static int launch_prefill_simt(const void* q, const void* k_rep, const void* v, const int* n_groups,
                               const GroupEntry* groups, void* out, WsHeader* hdr, const int* bad, int B, int H, int k,
                               int T_len, int q_start, float scale, int causal, cudaStream_t s) {
    const int n_qtiles = (T_len + kSimtBQ - 1) / kSimtBQ;
    const int qt0 = q_start / kSimtBQ;  // query tiles below this one hold no row to compute
    const size_t smem = sizeof(float) * ((size_t)kSimtBQ * (D + 1) + (size_t)kSimtBK * (D + 1) + (size_t)kSimtBK * D + 32 * 33);
    cudaError_t e = cudaFuncSetAttribute(prefill_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "prefill_simt_kernel shared-memory opt-in");
    prefill_simt_kernel<T, D><<<dim3(n_qtiles - qt0, H, B), kSimtThreads, smem, s>>>(
        static_cast<const T*>(q), static_cast<const T*>(k_rep), static_cast<const T*>(v), n_groups, groups,
        static_cast<T*>(out), hdr, bad, H, k, T_len, q_start, scale, causal, n_qtiles);
    CHAI_LAUNCH_CHECK("prefill_simt_kernel launch");
    return CHAI_OK;
}

int prefill_check_args(const char* fn, const void* q, const void* k_rep, const void* v, const int32_t* membership,
                       const int32_t* reps, void* out, int B, int H, int k, int T, int D, int dtype, void* workspace,
                       size_t workspace_bytes) {
    CHAI_REQUIRE(q && k_rep && v && membership && reps && out && workspace, CHAI_ERR_INVALID_ARG, "%s: null pointer", fn);
    CHAI_REQUIRE(aligned16(q) && aligned16(k_rep) && aligned16(v) && aligned16(out) && aligned16(workspace),
                 CHAI_ERR_INVALID_ARG, "%s: pointers must be 16-byte aligned", fn);
    CHAI_REQUIRE(B > 0 && H > 0 && T > 0 && D > 0, CHAI_ERR_INVALID_ARG, "%s: sizes must be positive", fn);
    CHAI_REQUIRE(k >= 1 && k <= H, CHAI_ERR_INVALID_ARG, "%s: need 1 <= k <= H (k=%d, H=%d)", fn, k, H);
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED, "%s: unknown dtype %d", fn, dtype);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED, "%s: head_dim %d (64 or 128 supported)", fn, D);
    CHAI_REQUIRE(H <= 65535 && B <= 65535, CHAI_ERR_UNSUPPORTED, "%s: H and B must be <= 65535", fn);
    CHAI_REQUIRE(prefill_plan_smem(H, k) <= 48 * 1024, CHAI_ERR_UNSUPPORTED,
                 "%s: too many heads and clusters for the planner (H=%d, k=%d need %zu bytes of shared memory, limit 49152)",
                 fn, H, k, prefill_plan_smem(H, k));
    const PrefillLayout L = prefill_layout(B, H);
    CHAI_REQUIRE(workspace_bytes >= L.total, CHAI_ERR_WORKSPACE, "%s: workspace has %zu bytes, %zu needed", fn,
                 workspace_bytes, L.total);
    return CHAI_OK;
}

int prefill_run_plan(const int32_t* membership, const int32_t* reps, int B, int H, int k, int gmax, char* ws,
                     cudaStream_t s) {
    const PrefillLayout L = prefill_layout(B, H);
    const size_t smem = prefill_plan_smem(H, k);
    // Launched as a programmatic dependent: when the kernel before it on the stream lets its dependents go
    // early (the tensor-core prefill kernel does), the planner's CTAs are placed while that kernel drains and
    // wait inside griddepcontrol.wait for it to complete, which hides the launch latency between
    // back-to-back prefill calls (+1.3 % measured).  After any other kernel the attribute changes nothing.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill_plan_kernel, membership, reps, reinterpret_cast<WsHeader*>(ws),
                                       reinterpret_cast<int*>(ws + L.off_ngroups), reinterpret_cast<int*>(ws + L.off_bad),
                                       reinterpret_cast<GroupEntry*>(ws + L.off_groups), H, k, gmax);
    if (e != cudaSuccess) return cuda_fail(e, "prefill_plan_kernel launch");
    return CHAI_OK;
}

}  // namespace chai

extern "C" {

size_t chai_prefill_workspace_bytes(int B, int H, int k, int T, int D, int dtype) {
    (void)k;
    (void)T;
    (void)D;
    (void)dtype;
    if (B <= 0 || H <= 0) return 0;
    return chai::prefill_layout(B, H).total;
}

int chai_prefill_attention_simt_from(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                     const int32_t* reps, void* out, int B, int H, int k, int T, int q_start, int D,
                                     float scale, int causal, int dtype, void* workspace, size_t workspace_bytes,
                                     void* stream) {
    using namespace chai;
    const char* fn = "chai_prefill_attention_simt";
    int rc = prefill_check_args(fn, q, k_rep, v, membership, reps, out, B, H, k, T, D, dtype, workspace, workspace_bytes);
    if (rc != CHAI_OK) return rc;
    CHAI_REQUIRE(q_start >= 0 && q_start < T, CHAI_ERR_INVALID_ARG, "%s: need 0 <= q_start < T (q_start=%d, T=%d)", fn,
                 q_start, T);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    CHAI_LOG_CALL("%s: B=%d H=%d k=%d T=%d q_start=%d D=%d causal=%d dtype=%d CUDA-core kernel, grid (%d, %d, %d)", fn, B, H, k, T,
                  q_start, D, causal, dtype, (T + kSimtBQ - 1) / kSimtBQ - q_start / kSimtBQ, H, B);
    rc = prefill_run_plan(membership, reps, B, H, k, kSimtG, ws, s);
    if (rc != CHAI_OK) return rc;
    const PrefillLayout L = prefill_layout(B, H);
    const int* ng = reinterpret_cast<const int*>(ws + L.off_ngroups);
    const GroupEntry* gr = reinterpret_cast<const GroupEntry*>(ws + L.off_groups);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws);
    const int* bad = reinterpret_cast<const int*>(ws + L.off_bad);
    if (dtype == CHAI_BF16) {
        if (D == 128)
            return launch_prefill_simt<__nv_bfloat16, 128>(q, k_rep, v, ng, gr, out, hdr, bad, B, H, k, T, q_start, scale, causal, s);
        return launch_prefill_simt<__nv_bfloat16, 64>(q, k_rep, v, ng, gr, out, hdr, bad, B, H, k, T, q_start, scale, causal, s);
    }
    if (D == 128) return launch_prefill_simt<float, 128>(q, k_rep, v, ng, gr, out, hdr, bad, B, H, k, T, q_start, scale, causal, s);
    return launch_prefill_simt<float, 64>(q, k_rep, v, ng, gr, out, hdr, bad, B, H, k, T, q_start, scale, causal, s);
}

int chai_prefill_attention_simt(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                const int32_t* reps, void* out, int B, int H, int k, int T, int D, float scale,
                                int causal, int dtype, void* workspace, size_t workspace_bytes, void* stream) {
    return chai_prefill_attention_simt_from(q, k_rep, v, membership, reps, out, B, H, k, T, 0, D, scale, causal, dtype,
                                            workspace, workspace_bytes, stream);
}

}  // extern "C"
