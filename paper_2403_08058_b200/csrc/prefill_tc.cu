// Clustered prefill attention entry point.  (Tensor-core kernel: see below; dispatch by dtype.)
#include "prefill_plan.cuh"

extern "C" int chai_prefill_attention(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                      const int32_t* reps, void* out, int B, int H, int k, int T, int D, float scale,
                                      int causal, int dtype, void* workspace, size_t workspace_bytes, void* stream) {
    return chai_prefill_attention_simt(q, k_rep, v, membership, reps, out, B, H, k, T, D, scale, causal, dtype,
                                       workspace, workspace_bytes, stream);
}
