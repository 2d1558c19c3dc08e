/*
 * chai.h -- C ABI of the B200 clustered-head-attention library (libchai.so).
 *
 * The library implements the inference hot path of CHAI (Clustered Head
 * Attention, arXiv 2403.08058): per request, the heads of a layer are grouped by
 * k-means over attention-score features of a five-token prompt prefix; afterwards
 * only each cluster's representative head computes Q K^T and the softmax, against
 * a key cache that stores representative heads only, and every member head
 * applies those shared probabilities to its own value cache.
 *
 * Conventions common to every entry point
 *   - All tensor arguments are DEVICE pointers to contiguous row-major arrays
 *     unless the name ends in _host.  Pointers must be 16-byte aligned.
 *   - Ownership: the caller allocates and frees every buffer, including the
 *     workspace.  The library allocates no device memory.  State it keeps between
 *     calls, all of it host-side and safe to reach from several host threads at
 *     once: the text of the last error (per thread); per device, what the first
 *     call on that device found out or set up (SM count, cooperative-launch
 *     support, each kernel's opt-in to its shared-memory size); a process-wide
 *     counter from which decode launches draw their tokens; the wait limit set by
 *     chai_set_decode_wait_limit_cycles.  On the device it owns one thing, the
 *     8 MiB scratch array of chai_decode_attention_static.
 *   - Asynchrony: a call validates its scalar arguments on the host, enqueues its
 *     kernels on `stream` (a cudaStream_t passed as void*) and returns; it never
 *     synchronises, except chai_device_status and chai_decode_attention_host (the
 *     other host-buffer entry points, *_host_async and *_host_streams, leave the wait to the caller).
 *   - Errors: the return value is a chai_status_t.  Anything checkable on the host
 *     (null or misaligned pointer, non-positive size, k > H, unsupported head
 *     dimension, workspace too small) is refused before any launch.  Errors in
 *     device-resident data (membership[b][h] outside [0,k), reps[b][c] outside
 *     {-1} U [0,H), membership[b][reps[b][c]] != c) cannot be seen by the host:
 *     the kernels record CHAI_ERR_BAD_MEMBERSHIP in the status word at the head of
 *     the workspace, give the affected heads an all-zero output and never form an
 *     out-of-range address.  Read the word with chai_device_status.
 *   - Logging: with CHAI_LOG=1 in the environment (read once per process) the main entry points
 *     write one line per call to stderr: their name, the shapes, and what they launch.
 *   - dtype: CHAI_F32 or CHAI_BF16 for Q, K, V and the output; accumulation is
 *     always fp32.  Head dimension D must be 64 or 128.
 *   - T counts cached positions INCLUDING the current token; T_cap (>= T) is the
 *     row capacity of the caches, i.e. the stride between heads is T_cap*D.
 *   - membership [B,H] int32: cluster id of each head.  reps [B,k] int32: head
 *     index of each cluster's representative, or -1 for an unused cluster slot.
 *     Both are per request (Section 3.5: membership is decided for each request).
 */
#ifndef CHAI_H_
#define CHAI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CHAI_OK = 0,
    CHAI_ERR_INVALID_ARG = 1,    /* null/misaligned pointer, non-positive size, k > H, T > T_cap ... */
    CHAI_ERR_UNSUPPORTED = 2,    /* head_dim not 64/128, unknown dtype, problem too large for a kernel */
    CHAI_ERR_WORKSPACE = 3,      /* workspace_bytes smaller than the matching *_workspace_bytes() */
    CHAI_ERR_BAD_MEMBERSHIP = 4, /* device status word only: inconsistent membership / reps */
    CHAI_ERR_TIMEOUT = 5,        /* device status word only: a bounded device-side wait expired */
    CHAI_ERR_CUDA = 6,           /* a CUDA call failed; text in chai_last_error() */
    CHAI_ERR_CACHE_FULL = 7      /* device status word only: chai_append_kv found seq_lens[b] outside [0, T_cap) */
} chai_status_t;

typedef enum { CHAI_F32 = 0, CHAI_BF16 = 1, CHAI_FP8_E4M3 = 2 /* caches of chai_decode_attention_fp8 only */ } chai_dtype_t;

/* size of the built-in scratch array used by chai_decode_attention_static */
#define CHAI_DECODE_STATIC_SCRATCH_BYTES (8u << 20)

/*
 * Prefix score features (Section 3.3 and Fig. 6(b): the first five tokens of a
 * request run with plain multi-head attention and their attention scores are what
 * is clustered; Section 3.1 defines head similarity on softmax(Q K^T)).
 *   q_full, k_full  [B,H,T_cap,D]  every head's own queries / keys; rows 0..P-1 are read
 *   features        [B,H,P*P] fp32 out: entry i*P+j = causal softmax probability of
 *                   query i on key j (j <= i) of that head, 0 for j > i
 * 1 <= P <= 32, P <= T_cap.
 */
int chai_prefix_features(const void* q_full, const void* k_full, int B, int H, int T_cap, int D, int P,
                         float scale, int dtype, float* features, void* stream);

/*
 * Cluster membership by k-means (Section 3.5: K-Means once five tokens have been
 * processed; Section 3.2: error = sum of squared distances to the closest centre).
 * Deterministic: seeded farthest-first initial centres (first = seed mod H; ties
 * to the lowest index), Lloyd iterations in fp64 until the assignment repeats or
 * max_iter assignments were made, empty clusters keep their centre, clusters are
 * renumbered by their lowest member and the lowest member is the representative.
 *   features   [B,H,F] fp32         one request = one independent problem
 *   membership [B,H] int32 out      cluster id in [0,k_eff)
 *   reps       [B,k] int32 out      representative head; -1 for slots >= k_eff
 *   k_eff      [B] int32 out        number of non-empty clusters (< k only when fewer
 *                                   than k distinct feature vectors exist)
 *   inertia    [B] fp64 out or NULL sum of squared distances to the members' means
 * 1 <= k <= H <= 1024; (H+k)*F + H*k doubles must fit in 200 KB of shared memory.
 */
int chai_cluster_heads(const float* features, int B, int H, int F, int k, int max_iter, uint64_t seed,
                       int32_t* membership, int32_t* reps, int32_t* k_eff, double* inertia, void* stream);

/*
 * Offline choice of the number of clusters (Section 3.2, Fig. 8: the clustering error is plotted against the
 * number of clusters and the count is taken where the curve flattens; the paper reads the plot by eye).
 * Runs chai_cluster_heads' k-means for every k = 1..k_max on every request at once (one CTA per (request, k))
 * and returns the error curve; optionally picks the knee: with k scaled to x in [0,1] and the error to y in
 * [0,1], the k farthest below the line from (0,1) to (1,0), ties to the smaller k (a flat curve gives 1).
 *   features [B,H,F] fp32 -> inertia_curve [B,k_max] fp64 (entry k-1 = inertia with k clusters),
 *   k_pick [B] int32 or NULL.  Same seed / max_iter meaning and size limits as chai_cluster_heads.
 */
int chai_cluster_sweep(const float* features, int B, int H, int F, int k_max, int max_iter, uint64_t seed,
                       double* inertia_curve, int32_t* k_pick, void* stream);

/*
 * Alternative choice of representatives: for every cluster the member whose feature vector is nearest
 * (squared Euclidean distance, fp64) to the mean of the cluster's members; ties go to the lowest head index
 * (the paper does not say which member stands for a cluster; chai_cluster_heads takes the lowest member).
 *   features [B,H,F] fp32, membership [B,H] int32 (as written by chai_cluster_heads) -> reps [B,k] int32,
 *   -1 for a cluster without members.  Cluster numbering is not changed, so reps[b][c] >= c still holds, but
 *   the representatives are no longer ascending: chai_compact_k_cache_inplace refuses such reps (use the
 *   out-of-place compaction).  Same size limits as chai_cluster_heads.
 */
int chai_select_representatives(const float* features, const int32_t* membership, int B, int H, int F, int k,
                                int32_t* reps, void* stream);

/*
 * K-cache compaction (Section 3.5: once membership is fixed the keys of pruned
 * heads are removed; Section 4.3: all values are kept).
 *   k_full [B,H,T_cap,D] -> k_rep [B,k,T_cap,D]:  k_rep[b][c][0..T) = k_full[b][reps[b][c]][0..T)
 * Bit copy, out of place; the buffers must not overlap.  A slot with reps = -1 (or
 * an out-of-range head) is zero-filled.
 */
int chai_compact_k_cache(const void* k_full, void* k_rep, const int32_t* reps, int B, int H, int k, int T,
                         int T_cap, int D, int dtype, void* stream);

/*
 * Clustered decode attention, one new token per request (Fig. 3(b), Section 3.4,
 * Section 4.3; A = softmax(Q K^T / sqrt(d)) of Section 2 with `scale` given explicitly).
 *   q    [B,H,D]         all heads' queries; only q[b][reps[b][c]] is read
 *   k_rep[B,k,T_cap,D]   representative-only key cache
 *   v    [B,H,T_cap,D]   full value cache
 *   out  [B,H,D]         out[b][h] = sum_t softmax_t(scale * q[b][r] . k_rep[b][c][t]) * v[b][h][t],
 *                        c = membership[b][h], r = reps[b][c], over t in [0,T)
 * The workspace holds the scores, split-KV partials and the status word; calls
 * that share a workspace must be ordered on one stream.
 */
int chai_decode_attention(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                          const int32_t* reps, void* out, int B, int H, int k, int T, int T_cap, int D,
                          float scale, int dtype, void* workspace, size_t workspace_bytes, void* stream);
size_t chai_decode_workspace_bytes(int B, int H, int k, int T, int D, int dtype);

/*
 * The same decode step for a ragged batch, as a serving loop holds it (Section 3.5: membership, hence the
 * caches, are per request; requests of a batch are at different positions).
 *   seq_lens [B] int32, device   cached positions of each request, INCLUDING the current token; values are
 *                                clamped to [0, T_max]; a request with length 0 gets an all-zero output
 *   T_max                        upper bound of seq_lens known to the host: sizes the workspace
 *                                (chai_decode_workspace_bytes(B, H, k, T_max, D, dtype)) and the launch
 *   k_batch_stride               elements between the first representative planes of two consecutive requests
 *                                in k_rep: 0 or k*T_cap*D for a dense [B,k,T_cap,D] cache, H*T_cap*D for a
 *                                full cache compacted in place by chai_compact_k_cache_inplace
 * Everything else as chai_decode_attention.  Cache rows at or beyond a request's length are never read.
 */
int chai_decode_attention_ragged(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                 const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k,
                                 int T_max, int T_cap, int D, size_t k_batch_stride, float scale, int dtype,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * Cache append for one new token per request (Section 3.5 / 4.3: after clustering only the representative
 * heads' keys are cached, every head's values are).
 *   k_new, v_new [B,H,D]   the token's keys / values of all heads (the layer's projection output)
 *   k_rep                  representative key cache, request stride k_batch_stride (see above), plane stride T_cap*D
 *   v     [B,H,T_cap,D]    value cache
 *   seq_lens [B] int32     device; the row written is pos = seq_lens[b] (the number of positions cached so far):
 *                          k_rep[b][c][pos] = k_new[b][reps[b][c]],  v[b][h][pos] = v_new[b][h]
 *   advance                non-zero: seq_lens[b] becomes pos + 1 afterwards, so that the following decode call
 *                          sees the new token
 *   workspace              NULL, or >= 256 bytes: its status word is set to CHAI_OK, or to CHAI_ERR_CACHE_FULL
 *                          if some seq_lens[b] was outside [0, T_cap) (that request is skipped, nothing faults)
 */
int chai_append_kv(const void* k_new, const void* v_new, void* k_rep, void* v, const int32_t* reps, int32_t* seq_lens,
                   int B, int H, int k, int T_cap, int D, size_t k_batch_stride, int dtype, int advance,
                   void* workspace, void* stream);

/*
 * K-cache compaction in place (Section 3.5: "remove" the keys of the non-representative heads): afterwards
 * planes 0..k-1 of every request of k_cache [B,H,T_cap,D] hold the representatives' keys, rows [0,T); the
 * other planes are dead and may be reused by the caller; decode / append then address the buffer with
 * k_batch_stride = H*T_cap*D.  Requires what chai_cluster_heads guarantees: reps strictly ascending with
 * reps[b][c] >= c and unused slots (-1) only at the end.  A request whose reps break that rule is left
 * untouched and CHAI_ERR_BAD_MEMBERSHIP is recorded in the status word of `workspace` (NULL or >= 256 bytes).
 */
int chai_compact_k_cache_inplace(void* k_cache, const int32_t* reps, int B, int H, int k, int T, int T_cap, int D,
                                 int dtype, void* workspace, void* stream);

/*
 * The same decode step with the per-step tensors in HOST memory: q_host [B,H,D] is
 * copied to q_stage, the kernels run, out_stage is copied to out_host [B,H,D] and
 * the call returns after the stream has drained.  q_stage / out_stage are device
 * buffers of B*H*D elements owned by the caller; the caches stay device resident
 * (they are state, not per-step input).  Pinned host memory makes the copies
 * asynchronous; pageable memory works too.
 */
int chai_decode_attention_host(const void* q_host, void* out_host, void* q_stage, void* out_stage,
                               const void* k_rep, const void* v, const int32_t* membership,
                               const int32_t* reps, int B, int H, int k, int T, int T_cap, int D, float scale,
                               int dtype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * As chai_decode_attention_host, but the call only enqueues upload, kernels and download on `stream` and
 * returns: out_host is valid once the caller has synchronised the stream (or an event recorded after the call).
 * q_host must stay unchanged and out_host untouched until then; with pageable instead of pinned host memory the
 * copies fall back to synchronous staging by the CUDA runtime.  Successive calls on one stream may share q_stage
 * and out_stage (stream order keeps them apart), so a whole decode step of layer calls needs one
 * synchronisation, not one per layer.
 */
int chai_decode_attention_host_async(const void* q_host, void* out_host, void* q_stage, void* out_stage,
                                     const void* k_rep, const void* v, const int32_t* membership,
                                     const int32_t* reps, int B, int H, int k, int T, int T_cap, int D, float scale,
                                     int dtype, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The host-buffer decode step spread over three streams, so that in a run of layer calls the upload of the next
 * call's queries and the download of the previous call's outputs overlap the kernels: q_host -> q_stage on
 * upload_stream, the kernels on `stream` (after uploaded_event), out_stage -> out_host on download_stream (after
 * computed_event).  Streams and events (cudaStream_t / cudaEvent_t passed as void*) belong to the caller; the
 * two events are recorded by this call and must not be reused before it has run.  Nothing is synchronised:
 * out_host is valid once download_stream has drained.  Calls that may be in flight together need staging
 * buffers of their own (q_stage is overwritten as soon as upload_stream gets there; out_stage is read until
 * download_stream is done), while the workspace may be shared, since the kernels of all calls run in order on
 * `stream`.  Pinned host memory is required for the copies to overlap anything.
 */
int chai_decode_attention_host_streams(const void* q_host, void* out_host, void* q_stage, void* out_stage,
                                       const void* k_rep, const void* v, const int32_t* membership,
                                       const int32_t* reps, int B, int H, int k, int T, int T_cap, int D, float scale,
                                       int dtype, void* workspace, size_t workspace_bytes, void* stream,
                                       void* upload_stream, void* download_stream, void* uploaded_event,
                                       void* computed_event);

/*
 * Decode step for callers that can neither pass a workspace nor let the library allocate one
 * (no counterpart in the paper: this is a deployment convenience).  Typical cases: a serving
 * engine that has already handed every free byte of HBM to its KV-cache pool, so a later
 * allocation would fail, and a latency-critical loop where the implicit device synchronisation
 * of an allocation is not acceptable.  Same arguments and result as chai_decode_attention, minus
 * the workspace: the scratch lives in an array of CHAI_DECODE_STATIC_SCRATCH_BYTES (8 MiB) that
 * is part of the library image, resident on every GPU that loads the library until the
 * process exits.  The call allocates nothing (no cudaMalloc / cudaFree, no allocating library
 * routine).
 *   - A problem whose scratch (chai_decode_workspace_bytes) exceeds the array is refused with
 *     CHAI_ERR_WORKSPACE and a message that states both sizes.
 *   - Every call looks up the array's address on the device that is current at the time of the
 *     call (nothing is remembered, so a cudaDeviceReset in between does no harm).  The first call
 *     on a device is the one that loads the library's module there: make it before any stream
 *     capture begins.
 *   - All calls on a device share the one array, which still holds whatever the previous call left;
 *     the kernels clear the parts that must start at zero.  Two calls that can overlap on the GPU
 *     (different streams without ordering) race on it: order them, or use chai_decode_attention
 *     with separate workspaces.  The status word of the last call is not readable through this
 *     entry point; inconsistent membership still yields zero rows and never faults.
 */
int chai_decode_attention_static(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                 const int32_t* reps, void* out, int B, int H, int k, int T, int T_cap, int D,
                                 float scale, int dtype, void* stream);

/*
 * Clustered prefill attention over a whole prompt (same operator as decode with T
 * query rows; decoder-only models attend causally, Section 2).
 *   q [B,H,T,D] (only representative heads' rows are read), k_rep [B,k,T,D],
 *   v [B,H,T,D], out [B,H,T,D];  causal != 0: row i sees keys j <= i.
 * bf16 (D = 128 or 64) with a positive, finite scale runs on the tcgen05 tensor-core
 * kernel; fp32 (and any other scale) on the CUDA-core kernel, a correct but far slower
 * path (milliseconds where the tensor-core kernel needs a tenth of one), which
 * chai_prefill_attention_simt selects for any dtype.
 * Errors: CHAI_ERR_INVALID_ARG / CHAI_ERR_WORKSPACE as for decode; CHAI_ERR_UNSUPPORTED for another head_dim or
 * dtype, for H or B above 65535, and when the work list of one request does not fit the planning kernel's
 * 48 KB of shared memory (4 * (H + 3 k + k * ceil(H / 32)) bytes: e.g. H = k = 512 still fits).  Inconsistent
 * membership data are reported through the status word of `workspace`; the heads concerned get zero rows.
 */
int chai_prefill_attention(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                           const int32_t* reps, void* out, int B, int H, int k, int T, int D, float scale,
                           int causal, int dtype, void* workspace, size_t workspace_bytes, void* stream);
int chai_prefill_attention_simt(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                const int32_t* reps, void* out, int B, int H, int k, int T, int D,
                                float scale, int causal, int dtype, void* workspace, size_t workspace_bytes,
                                void* stream);
size_t chai_prefill_workspace_bytes(int B, int H, int k, int T, int D, int dtype);

/*
 * Prefill that leaves the first q_start query rows alone (Section 3.3 / Fig. 6(b): the first five tokens
 * of a request run with plain multi-head attention, whose scores decide the clusters; clustered attention
 * takes over after them).  Rows [q_start, T) of `out` are computed exactly as by chai_prefill_attention --
 * they still attend to keys 0..i -- and rows [0, q_start) are neither computed nor written.
 * 0 <= q_start < T.  The plain-MHA rows themselves are a call with k = H and identity membership.
 */
int chai_prefill_attention_from(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                const int32_t* reps, void* out, int B, int H, int k, int T, int q_start, int D,
                                float scale, int causal, int dtype, void* workspace, size_t workspace_bytes,
                                void* stream);
int chai_prefill_attention_simt_from(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                     const int32_t* reps, void* out, int B, int H, int k, int T, int q_start, int D,
                                     float scale, int causal, int dtype, void* workspace, size_t workspace_bytes,
                                     void* stream);

/*
 * CHAI-QKV (Table 4 of the paper: besides Q and K, the V of non-representative heads is dropped as well, so a
 * member head's output equals its representative's).  Caches hold representatives only:
 *   k_rep, v_rep [B,k,T_cap,D] (decode) / [B,k,T,D] (prefill);  q and out keep all H heads:
 *   out[b][h] = attention(q[b][reps[b][c]], k_rep[b][c], v_rep[b][c]),  c = membership[b][h].
 * Decode: seq_lens may be NULL (every request has T positions) or a device array [B] as in
 * chai_decode_attention_ragged.  Prefill: rows [q_start, T) are computed and written.  The workspace
 * (chai_*_qkv_workspace_bytes) also holds the gathered query rows and the k per-cluster outputs.
 * v_rep is produced from a full value cache by chai_compact_k_cache (the same gather).
 * Heads whose membership cannot be resolved get zero rows and CHAI_ERR_BAD_MEMBERSHIP in the status word.
 */
size_t chai_decode_qkv_workspace_bytes(int B, int H, int k, int T, int D, int dtype);
int chai_decode_attention_qkv(const void* q, const void* k_rep, const void* v_rep, const int32_t* membership,
                              const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k, int T,
                              int T_cap, int D, float scale, int dtype, void* workspace, size_t workspace_bytes,
                              void* stream);
size_t chai_prefill_qkv_workspace_bytes(int B, int H, int k, int T, int D, int dtype);
int chai_prefill_attention_qkv(const void* q, const void* k_rep, const void* v_rep, const int32_t* membership,
                               const int32_t* reps, void* out, int B, int H, int k, int T, int q_start, int D,
                               float scale, int causal, int dtype, void* workspace, size_t workspace_bytes,
                               void* stream);

/*
 * CHAI-static (Section 3.5: a membership found offline is used for every request instead of clustering each
 * request's prefix): expands one membership [H] / representatives [k] into the per-request arrays [B,H] /
 * [B,k] that every other entry point takes.
 */
int chai_broadcast_membership(const int32_t* membership_static, const int32_t* reps_static, int32_t* membership,
                              int32_t* reps, int B, int H, int k, void* stream);

/*
 * fp8 caches (the paper treats head clustering as orthogonal to quantisation; one byte per cached element
 * halves the decode step's bytes once more).  Format: e4m3 (4 exponent bits, bias 7, 3 mantissa bits, no
 * infinities, largest finite value 448), one fp32 scale per cache plane; a stored byte stands for
 * decode(byte) * scale.
 *
 * chai_quantize_cache_fp8: src [n_planes,T_cap,D] bf16 -> dst [n_planes,T_cap,D] bytes + scales [n_planes].
 *   Per plane: scale = max|x| over rows [0,T) divided by 448 in fp32 (1 if the plane is all zero); each element
 *   is x / scale (fp32 division) rounded to the nearest e4m3 value, ties to even, saturating.  Rows >= T are not
 *   touched.  Works for K_rep (n_planes = B*k) and V (n_planes = B*H) alike.
 *
 * chai_decode_attention_fp8: the decode step of chai_decode_attention / _ragged on such caches.
 *   q, out [B,H,D] bf16; k_rep, v: e4m3 bytes; k_scale [B,k], v_scale [B,H] fp32 (device);
 *   seq_lens NULL or [B] device; k_batch_stride in elements (= bytes), 0 for dense.
 *   out[b][h] = v_scale[b][h] * sum_t softmax_t(scale * k_scale[b][c] * q[b][r] . k8[b][c][t]) * v8[b][h][t]
 *   with fp32 accumulation.  Workspace: chai_decode_fp8_workspace_bytes.  Runs on the persistent kernel only;
 *   CHAI_ERR_UNSUPPORTED on a device without cooperative launch.
 */
int chai_quantize_cache_fp8(const void* src, void* dst, float* scales, int n_planes, int T, int T_cap, int D,
                            void* stream);
size_t chai_decode_fp8_workspace_bytes(int B, int H, int k, int T, int D);
int chai_decode_attention_fp8(const void* q, const void* k_rep, const void* v, const float* k_scale, const float* v_scale,
                              const int32_t* membership, const int32_t* reps, const int32_t* seq_lens, void* out, int B,
                              int H, int k, int T, int T_cap, int D, size_t k_batch_stride, float scale, void* workspace,
                              size_t workspace_bytes, void* stream);

/* Blocking read of the status a decode/prefill call left in `workspace`
 * (synchronises `stream`).  *status_out receives a chai_status_t. */
int chai_device_status(const void* workspace, int* status_out, void* stream);

/*
 * Test hook (no counterpart in the paper).  Every wait inside the persistent decode kernel -- on a
 * ring slot, a copy, another CTA's flag -- gives up after a number of SM cycles, after which the
 * launch stops taking work, waits for the copies it has in flight, records CHAI_ERR_TIMEOUT for
 * chai_device_status and returns; the next launch on the same workspace starts clean.  The limit
 * is 2e9 cycles (about a second) unless this call changes it for the launches that follow, in
 * every thread of the process; cycles <= 0 restores the default.  Tests use a limit of a few
 * cycles to run the give-up path without any fault or hang; production code has no reason to call it.
 */
void chai_set_decode_wait_limit_cycles(long long cycles);

const char* chai_status_string(int status);
const char* chai_last_error(void); /* text of the last CHAI_ERR_CUDA / refusal on this thread */
int chai_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CHAI_H_ */
