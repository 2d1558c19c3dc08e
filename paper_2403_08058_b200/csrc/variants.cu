// Variants of the method that the paper evaluates next to the main one.
//
//   CHAI-QKV (Table 4): besides the queries and keys, the VALUES of non-representative heads are dropped
//       too, so a member head's output IS its representative's output.  Per cluster this is one plain
//       attention head (the representative's Q, K, V).  The streaming decode kernel and the tensor-core prefill
//       kernel take the clusters as their heads / work items, read each representative's query rows where they lie
//       among the H heads and write a cluster's rows to all of its members (one launch each); where those
//       kernels do not apply (fp32 prefill, devices without cooperative launch) the entry points gather the
//       query rows, run the k-head problem with identity maps, and copy each cluster's output to its members.
//   CHAI-static (Section 3.5): one membership, found offline, is used for every request: the per-request
//       arrays the other entry points expect are then B copies of it (chai_broadcast_membership).
#include "decode_layout.cuh"
#include "prefill_plan.cuh"

namespace chai {

// CHAI-QKV prefill on the tensor-core kernel (prefill_tc.cu); -1 when the call is outside its range.
int prefill_qkv_tc(const void* q, const void* k_rep, const void* v_rep, const int32_t* membership, const int32_t* reps,
                   void* out, int B, int H, int k, int T, int q_start, int D, float scale, int causal, int dtype, void* workspace,
                   size_t workspace_bytes, cudaStream_t s);

// rows of `rows_per_head` * vec_per_row 16-byte vectors per head.
// gather:  dst[b][c] = src[b][reps[b][c]]   (zero for an unused slot); also writes the identity maps of the
// inner k-head problem: membership[b][c] = c, reps[b][c] = c
__global__ void __launch_bounds__(256)
gather_rep_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, const int32_t* __restrict__ reps,
                       int32_t* __restrict__ ident, int H, int k, size_t vecs_per_head) {
    dependent_grid_sync();
    const int c = blockIdx.y, b = blockIdx.z;
    if (blockIdx.x == 0 && threadIdx.x == 0) ident[(size_t)b * k + c] = c;
    const int r = reps[(size_t)b * k + c];
    const bool live = r >= 0 && r < H;
    const uint4* s = src + ((size_t)b * H + (live ? r : 0)) * vecs_per_head;
    uint4* d = dst + ((size_t)b * k + c) * vecs_per_head;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < vecs_per_head; i += (size_t)gridDim.x * blockDim.x)
        d[i] = live ? s[i] : make_uint4(0, 0, 0, 0);
}

// scatter: out[b][h] = inner[b][membership[b][h]]; rows [row0, rows) of each head only (prefill from q_start);
// a head whose membership cannot be resolved gets zeros and is reported.
__global__ void __launch_bounds__(256)
scatter_members_kernel(const uint4* __restrict__ inner, uint4* __restrict__ out, const int32_t* __restrict__ membership,
                       const int32_t* __restrict__ reps, WsHeader* __restrict__ hdr, int H, int k, size_t vecs_per_head,
                       size_t vec0) {
    const int h = blockIdx.y, b = blockIdx.z;
    int c, r;
    const bool live = resolve_head(membership, reps, b, h, H, k, &c, &r);
    if (!live && blockIdx.x == 0 && threadIdx.x == 0) flag_bad_membership(hdr, b, h);
    const uint4* s = inner + ((size_t)b * k + (live ? c : 0)) * vecs_per_head;
    uint4* d = out + ((size_t)b * H + h) * vecs_per_head;
    for (size_t i = vec0 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < vecs_per_head; i += (size_t)gridDim.x * blockDim.x)
        d[i] = live ? s[i] : make_uint4(0, 0, 0, 0);
}

__global__ void broadcast_membership_kernel(const int32_t* __restrict__ m_static, const int32_t* __restrict__ r_static,
                                            int32_t* __restrict__ membership, int32_t* __restrict__ reps, int B, int H,
                                            int k) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < B * H) membership[i] = m_static[i % H];
    if (i < B * k) reps[i] = r_static[i % k];
}

struct QkvLayout {
    size_t off_q, off_out, off_ident, total;  // after the inner call's own workspace (which starts at 0)
};

static QkvLayout qkv_layout(size_t inner_bytes, int B, int k, size_t elems_per_head, int dtype) {
    QkvLayout L;
    size_t off = round_up(inner_bytes, 256);
    L.off_q = off;
    off = round_up(off + (size_t)B * k * elems_per_head * elem_size(dtype), 256);
    L.off_out = off;
    off = round_up(off + (size_t)B * k * elems_per_head * elem_size(dtype), 256);
    L.off_ident = off;
    off = round_up(off + sizeof(int32_t) * (size_t)B * k, 256);
    L.total = off;
    return L;
}

static unsigned blocks_for(size_t vecs) {
    const size_t b = (vecs + 255) / 256;
    return (unsigned)(b < 1 ? 1 : (b > 64 ? 64 : b));
}

}  // namespace chai

extern "C" {

int chai_broadcast_membership(const int32_t* membership_static, const int32_t* reps_static, int32_t* membership,
                              int32_t* reps, int B, int H, int k, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(membership_static && reps_static && membership && reps, CHAI_ERR_INVALID_ARG,
                 "chai_broadcast_membership: null pointer");
    CHAI_REQUIRE(B > 0 && H > 0 && k >= 1 && k <= H, CHAI_ERR_INVALID_ARG,
                 "chai_broadcast_membership: need B, H > 0 and 1 <= k <= H");
    const int n = B * H;
    broadcast_membership_kernel<<<(n + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        membership_static, reps_static, membership, reps, B, H, k);
    CHAI_LAUNCH_CHECK("broadcast_membership_kernel launch");
    return CHAI_OK;
}

size_t chai_decode_qkv_workspace_bytes(int B, int H, int k, int T, int D, int dtype) {
    (void)H;
    const size_t inner = chai_decode_workspace_bytes(B, k, k, T, D, dtype);
    if (inner == 0) return 0;
    return chai::qkv_layout(inner, B, k, (size_t)D, dtype).total;
}

int chai_decode_attention_qkv(const void* q, const void* k_rep, const void* v_rep, const int32_t* membership,
                              const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k, int T,
                              int T_cap, int D, float scale, int dtype, void* workspace, size_t workspace_bytes,
                              void* stream) {
    using namespace chai;
    const char* fn = "chai_decode_attention_qkv";
    CHAI_REQUIRE(q && k_rep && v_rep && membership && reps && out && workspace, CHAI_ERR_INVALID_ARG, "%s: null pointer", fn);
    CHAI_REQUIRE(aligned16(q) && aligned16(out) && aligned16(workspace), CHAI_ERR_INVALID_ARG,
                 "%s: pointers must be 16-byte aligned", fn);
    CHAI_REQUIRE(B > 0 && H > 0 && k >= 1 && k <= H && T > 0, CHAI_ERR_INVALID_ARG, "%s: bad sizes", fn);
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED, "%s: unknown dtype %d", fn, dtype);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED, "%s: head_dim %d (64 or 128 supported)", fn, D);
    CHAI_REQUIRE(H <= 65535 && B <= 65535, CHAI_ERR_UNSUPPORTED, "%s: H and B must be <= 65535", fn);
    const size_t inner = chai_decode_workspace_bytes(B, k, k, T, D, dtype);
    const QkvLayout L = qkv_layout(inner, B, k, (size_t)D, dtype);
    CHAI_REQUIRE(workspace_bytes >= L.total, CHAI_ERR_WORKSPACE, "%s: workspace has %zu bytes, %zu needed", fn,
                 workspace_bytes, L.total);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    // One launch of the streaming decode kernel with the k clusters as its heads: it reads each representative's
    // query row where it lies among the H heads and writes a cluster's row to all of its member heads itself.
    CHAI_REQUIRE(T <= T_cap, CHAI_ERR_INVALID_ARG, "%s: T=%d exceeds T_cap=%d", fn, T, T_cap);
    CHAI_REQUIRE(aligned16(k_rep) && aligned16(v_rep), CHAI_ERR_INVALID_ARG, "%s: pointers must be 16-byte aligned", fn);
    DecodeLayout DL;
    if (decode_layout(B, k, k, T, D, dtype, &DL) && DL.total <= inner) {
        const int rc = launch_decode_persistent(q, k_rep, v_rep, membership, reps, seq_lens, out, B, k, k, T, T_cap, D,
                                                (size_t)k * T_cap * D, scale, dtype, ws, DL, s, nullptr, nullptr, membership, H);
        if (rc != kDecodeNotLaunched) return rc;
    }
    // (devices without cooperative launch: gather the query rows, run the k-head problem, copy to the members)
    int32_t* ident = reinterpret_cast<int32_t*>(ws + L.off_ident);
    const size_t vecs = (size_t)D * elem_size(dtype) / 16;
    CHAI_LAUNCH_DEPENDENT("gather_rep_rows_kernel launch", gather_rep_rows_kernel, dim3(1, k, B), dim3(32), 0, s,
                          static_cast<const uint4*>(q), reinterpret_cast<uint4*>(ws + L.off_q), reps, ident, H, k, vecs);
    int rc;
    if (seq_lens != nullptr)
        rc = chai_decode_attention_ragged(ws + L.off_q, k_rep, v_rep, ident, ident, seq_lens, ws + L.off_out, B, k, k, T,
                                          T_cap, D, 0, scale, dtype, ws, inner, stream);
    else
        rc = chai_decode_attention(ws + L.off_q, k_rep, v_rep, ident, ident, ws + L.off_out, B, k, k, T, T_cap, D, scale,
                                   dtype, ws, inner, stream);
    if (rc != CHAI_OK) return rc;
    scatter_members_kernel<<<dim3(1, H, B), 32, 0, s>>>(reinterpret_cast<const uint4*>(ws + L.off_out),
                                                       static_cast<uint4*>(out), membership, reps,
                                                       reinterpret_cast<WsHeader*>(ws), H, k, vecs, 0);
    CHAI_LAUNCH_CHECK("scatter_members_kernel launch");
    return CHAI_OK;
}

size_t chai_prefill_qkv_workspace_bytes(int B, int H, int k, int T, int D, int dtype) {
    (void)H;
    const size_t inner = chai_prefill_workspace_bytes(B, k, k, T, D, dtype);
    if (inner == 0 || T <= 0 || D <= 0) return 0;
    const size_t general = chai::qkv_layout(inner, B, k, (size_t)T * D, dtype).total;  // copies of Q rows and outputs
    const size_t fused = chai::prefill_layout(B, H + k).total;                           // the plan alone
    return general > fused ? general : fused;
}

int chai_prefill_attention_qkv(const void* q, const void* k_rep, const void* v_rep, const int32_t* membership,
                               const int32_t* reps, void* out, int B, int H, int k, int T, int q_start, int D,
                               float scale, int causal, int dtype, void* workspace, size_t workspace_bytes,
                               void* stream) {
    using namespace chai;
    const char* fn = "chai_prefill_attention_qkv";
    CHAI_REQUIRE(q && k_rep && v_rep && membership && reps && out && workspace, CHAI_ERR_INVALID_ARG, "%s: null pointer", fn);
    CHAI_REQUIRE(aligned16(q) && aligned16(out) && aligned16(workspace), CHAI_ERR_INVALID_ARG,
                 "%s: pointers must be 16-byte aligned", fn);
    CHAI_REQUIRE(B > 0 && H > 0 && k >= 1 && k <= H && T > 0 && q_start >= 0 && q_start < T, CHAI_ERR_INVALID_ARG,
                 "%s: bad sizes", fn);
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED, "%s: unknown dtype %d", fn, dtype);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED, "%s: head_dim %d (64 or 128 supported)", fn, D);
    CHAI_REQUIRE(H <= 65535 && B <= 65535, CHAI_ERR_UNSUPPORTED, "%s: H and B must be <= 65535", fn);
    const size_t inner = chai_prefill_workspace_bytes(B, k, k, T, D, dtype);
    const QkvLayout L = qkv_layout(inner, B, k, (size_t)T * D, dtype);
    CHAI_REQUIRE(workspace_bytes >= L.total, CHAI_ERR_WORKSPACE, "%s: workspace has %zu bytes, %zu needed", fn,
                 workspace_bytes, L.total);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    int32_t* ident = reinterpret_cast<int32_t*>(ws + L.off_ident);
    // bf16: one launch of the tensor-core kernel with the clusters as its work items (it reads the representatives'
    // query tiles in place and writes every member's rows itself)
    CHAI_REQUIRE(aligned16(k_rep) && aligned16(v_rep), CHAI_ERR_INVALID_ARG, "%s: pointers must be 16-byte aligned", fn);
    {
        const int rc = prefill_qkv_tc(q, k_rep, v_rep, membership, reps, out, B, H, k, T, q_start, D, scale, causal, dtype,
                                      workspace, workspace_bytes, s);
        if (rc != -1) return rc;
    }
    // otherwise: gather the query rows, run the k-head problem, copy each cluster's rows to its members
    const size_t row_vecs = (size_t)D * elem_size(dtype) / 16;
    const size_t vecs = (size_t)T * row_vecs;
    gather_rep_rows_kernel<<<dim3(blocks_for(vecs), k, B), 256, 0, s>>>(
        static_cast<const uint4*>(q), reinterpret_cast<uint4*>(ws + L.off_q), reps, ident, H, k, vecs);
    CHAI_LAUNCH_CHECK("gather_rep_rows_kernel launch");
    const int rc = chai_prefill_attention_from(ws + L.off_q, k_rep, v_rep, ident, ident, ws + L.off_out, B, k, k, T, q_start,
                                               D, scale, causal, dtype, ws, inner, stream);
    if (rc != CHAI_OK) return rc;
    scatter_members_kernel<<<dim3(blocks_for(vecs), H, B), 256, 0, s>>>(
        reinterpret_cast<const uint4*>(ws + L.off_out), static_cast<uint4*>(out), membership, reps,
        reinterpret_cast<WsHeader*>(ws), H, k, vecs, (size_t)q_start * row_vecs);
    CHAI_LAUNCH_CHECK("scatter_members_kernel launch");
    return CHAI_OK;
}

}  // extern "C"
