// The steps either side of the attention calls in a serving loop (Section 3.5: once membership is known
// the keys of the non-representative heads are dropped, and from then on only representatives' keys are
// cached; Section 4.3: every head keeps its values).
//
//   chai_append_kv                 one new token per request: the representatives' key rows and every
//                                  head's value row go to position seq_lens[b] of the caches.
//   chai_compact_k_cache_inplace   K_full -> representatives in the first k planes of the same buffer.
#include "chai_common.cuh"

namespace chai {

// grid B, block 256.  Rows are D elements = D*es/16 vectors of 16 bytes.
__global__ void __launch_bounds__(256)
append_kv_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, uint4* __restrict__ k_rep,
                 uint4* __restrict__ v, const int32_t* __restrict__ reps, int32_t* __restrict__ seq_lens,
                 WsHeader* __restrict__ hdr, int H, int k, int T_cap, int vec_per_row, size_t k_batch_vecs, int advance) {
    dependent_grid_sync();
    const int b = blockIdx.x, tid = threadIdx.x;
    const int pos = seq_lens[b];
    __syncthreads();  // every thread holds the position before thread 0 may advance it
    if (pos < 0 || pos >= T_cap) {  // no room (or a corrupt length): nothing is written for this request
        if (tid == 0 && hdr != nullptr) {
            atomicCAS(&hdr->status, CHAI_OK, CHAI_ERR_CACHE_FULL);
            hdr->bad_b = b;
            hdr->bad_h = -1;
        }
        return;
    }
    const size_t plane_vecs = (size_t)T_cap * vec_per_row;
    // values: every head
    for (int i = tid; i < H * vec_per_row; i += blockDim.x) {
        const int h = i / vec_per_row, x = i - h * vec_per_row;
        v[((size_t)b * H + h) * plane_vecs + (size_t)pos * vec_per_row + x] = v_new[((size_t)b * H + h) * vec_per_row + x];
    }
    // keys: representatives only
    for (int i = tid; i < k * vec_per_row; i += blockDim.x) {
        const int c = i / vec_per_row, x = i - c * vec_per_row;
        const int r = reps[(size_t)b * k + c];
        if (r < 0 || r >= H) continue;  // unused cluster slot
        k_rep[(size_t)b * k_batch_vecs + (size_t)c * plane_vecs + (size_t)pos * vec_per_row + x] =
            k_new[((size_t)b * H + r) * vec_per_row + x];
    }
    if (advance && tid == 0) seq_lens[b] = pos + 1;
}

// In-place compaction.  Representatives are the lowest members of clusters that are numbered by their
// lowest member, so reps is strictly ascending and reps[c] >= c: moving plane reps[c] to plane c for
// c = 0, 1, ... never overwrites a plane that is still to be read -- as long as the moves of one cache
// ROW happen in that order, which they do here because one thread carries its rows through all clusters.
// Different rows are independent.  grid (row blocks, B), block 256; a thread owns one 16-byte column of
// kRowsPerThread rows.
constexpr int kRowsPerThread = 4;

__global__ void __launch_bounds__(256)
compact_inplace_kernel(uint4* __restrict__ k_cache, const int32_t* __restrict__ reps, WsHeader* __restrict__ hdr,
                       int H, int k, int T_len, int T_cap, int vec_per_row) {
    const int b = blockIdx.y, tid = threadIdx.x;
    // reps of this request must be ascending with reps[c] >= c, unused slots (-1) only at the end
    __shared__ int s_bad;
    if (tid == 0) {
        int bad = 0, prev = -1;
        bool tail = false;
        for (int c = 0; c < k; ++c) {
            const int r = reps[(size_t)b * k + c];
            if (r == -1) {
                tail = true;
                continue;
            }
            if (tail || r < c || r >= H || r <= prev) bad = 1;
            prev = r;
        }
        s_bad = bad;
        if (bad && blockIdx.x == 0 && hdr != nullptr) {
            atomicCAS(&hdr->status, CHAI_OK, CHAI_ERR_BAD_MEMBERSHIP);
            hdr->bad_b = b;
            hdr->bad_h = -1;
        }
    }
    __syncthreads();
    if (s_bad) return;  // the request's cache is left as it was
    const size_t plane_vecs = (size_t)T_cap * vec_per_row;
    uint4* base = k_cache + (size_t)b * H * plane_vecs;
    const size_t n_vecs = (size_t)T_len * vec_per_row;  // vectors of one plane that hold cached rows
    const size_t i0 = ((size_t)blockIdx.x * blockDim.x * kRowsPerThread) + tid;
    for (int c = 0; c < k; ++c) {
        const int r = reps[(size_t)b * k + c];
        if (r < 0) break;
        if (r == c) continue;  // already in place
        const uint4* src = base + (size_t)r * plane_vecs;
        uint4* dst = base + (size_t)c * plane_vecs;
        uint4 buf[kRowsPerThread];
#pragma unroll
        for (int u = 0; u < kRowsPerThread; ++u) {
            const size_t i = i0 + (size_t)u * blockDim.x;
            if (i < n_vecs) buf[u] = src[i];
        }
#pragma unroll
        for (int u = 0; u < kRowsPerThread; ++u) {
            const size_t i = i0 + (size_t)u * blockDim.x;
            if (i < n_vecs) dst[i] = buf[u];
        }
    }
}

__global__ void reset_status_kernel(WsHeader* hdr) {
    dependent_grid_sync();
    reset_status(hdr);
}

}  // namespace chai

extern "C" {

int chai_append_kv(const void* k_new, const void* v_new, void* k_rep, void* v, const int32_t* reps, int32_t* seq_lens,
                   int B, int H, int k, int T_cap, int D, size_t k_batch_stride, int dtype, int advance,
                   void* workspace, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(k_new && v_new && k_rep && v && reps && seq_lens, CHAI_ERR_INVALID_ARG, "chai_append_kv: null pointer");
    CHAI_REQUIRE(aligned16(k_new) && aligned16(v_new) && aligned16(k_rep) && aligned16(v), CHAI_ERR_INVALID_ARG,
                 "chai_append_kv: pointers must be 16-byte aligned");
    CHAI_REQUIRE(B > 0 && H > 0 && T_cap > 0 && k >= 1 && k <= H, CHAI_ERR_INVALID_ARG,
                 "chai_append_kv: need B, H, T_cap > 0 and 1 <= k <= H");
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED, "chai_append_kv: unknown dtype %d", dtype);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED, "chai_append_kv: head_dim %d (64 or 128 supported)", D);
    const size_t es = elem_size(dtype), dense = (size_t)k * T_cap * D;
    if (k_batch_stride == 0) k_batch_stride = dense;
    CHAI_REQUIRE(k_batch_stride >= dense && (k_batch_stride * es) % 16 == 0, CHAI_ERR_INVALID_ARG,
                 "chai_append_kv: k_batch_stride=%zu must be at least k*T_cap*D=%zu elements and a multiple of 16 bytes",
                 k_batch_stride, dense);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WsHeader* hdr = static_cast<WsHeader*>(workspace);
    if (hdr != nullptr) {
        CHAI_LAUNCH_DEPENDENT("chai_append_kv: status reset", reset_status_kernel, dim3(1), dim3(1), 0, s, hdr);
    }
    const int vec_per_row = (int)(D * es / 16);
    CHAI_LAUNCH_DEPENDENT("append_kv_kernel launch", append_kv_kernel, dim3(B), dim3(256), 0, s,
                          static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), static_cast<uint4*>(k_rep),
                          static_cast<uint4*>(v), reps, seq_lens, hdr, H, k, T_cap, vec_per_row,
                          (size_t)(k_batch_stride * es / 16), advance);
    return CHAI_OK;
}

int chai_compact_k_cache_inplace(void* k_cache, const int32_t* reps, int B, int H, int k, int T, int T_cap, int D,
                                 int dtype, void* workspace, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(k_cache && reps, CHAI_ERR_INVALID_ARG, "chai_compact_k_cache_inplace: null pointer");
    CHAI_REQUIRE(aligned16(k_cache), CHAI_ERR_INVALID_ARG, "chai_compact_k_cache_inplace: the cache must be 16-byte aligned");
    CHAI_REQUIRE(B > 0 && H > 0 && T > 0 && k >= 1 && k <= H && T <= T_cap, CHAI_ERR_INVALID_ARG,
                 "chai_compact_k_cache_inplace: need B, H, T > 0, 1 <= k <= H and T <= T_cap");
    CHAI_REQUIRE(B <= 65535, CHAI_ERR_UNSUPPORTED, "chai_compact_k_cache_inplace: B must be <= 65535");
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED,
                 "chai_compact_k_cache_inplace: unknown dtype %d", dtype);
    CHAI_REQUIRE(D == 64 || D == 128, CHAI_ERR_UNSUPPORTED,
                 "chai_compact_k_cache_inplace: head_dim %d (64 or 128 supported)", D);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WsHeader* hdr = static_cast<WsHeader*>(workspace);
    if (hdr != nullptr) {
        CHAI_LAUNCH_DEPENDENT("chai_compact_k_cache_inplace: status reset", reset_status_kernel, dim3(1), dim3(1), 0, s, hdr);
    }
    const int vec_per_row = (int)(D * elem_size(dtype) / 16);
    const size_t n_vecs = (size_t)T * vec_per_row;
    const size_t per_block = 256 * (size_t)kRowsPerThread;
    const unsigned blocks = (unsigned)((n_vecs + per_block - 1) / per_block);
    compact_inplace_kernel<<<dim3(blocks, B), 256, 0, s>>>(static_cast<uint4*>(k_cache), reps, hdr, H, k, T, T_cap,
                                                          vec_per_row);
    CHAI_LAUNCH_CHECK("compact_inplace_kernel launch");
    return CHAI_OK;
}

}  // extern "C"
