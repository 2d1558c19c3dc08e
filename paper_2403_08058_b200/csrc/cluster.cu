// Membership identification: prefix score features and k-means over heads.
//
// Both kernels are tiny and latency-bound (one CTA per (request, head) resp. per request); there is
// no roofline to chase.  The k-means kernel runs in fp64 with explicitly rounded operations in a
// fixed order, so its trajectory does not depend on the launch shape or on compiler contraction.
#include "chai_common.cuh"

namespace chai {

// ---- prefix score features (Section 3.3; similarity is defined on softmax(Q K^T), Section 3.1) ----
// grid (H, B), block P*P threads: thread (i,j) computes the scaled dot product of query i and key j
// of its own head, then thread (i,0) normalises row i causally.
template <typename T>
__global__ void prefix_features_kernel(const T* __restrict__ q_full, const T* __restrict__ k_full,
                                       float* __restrict__ features, int H, int T_cap, int D, int P,
                                       float scale) {
    extern __shared__ float s_scores[];  // [P*P]
    const int h = blockIdx.x, b = blockIdx.y;
    const int i = threadIdx.x / P, j = threadIdx.x % P;
    const size_t head = ((size_t)b * H + h) * (size_t)T_cap * D;
    if (j <= i) {
        const T* q = q_full + head + (size_t)i * D;
        const T* kk = k_full + head + (size_t)j * D;
        float s = 0.f;
        for (int d = 0; d < D; ++d) s = fmaf(to_float(q[d]), to_float(kk[d]), s);
        s_scores[i * P + j] = s * scale;
    }
    __syncthreads();
    if (j == 0) {
        float m = -INFINITY;
        for (int jj = 0; jj <= i; ++jj) m = fmaxf(m, s_scores[i * P + jj]);
        float z = 0.f;
        for (int jj = 0; jj <= i; ++jj) {
            float p = expf(s_scores[i * P + jj] - m);
            s_scores[i * P + jj] = p;
            z += p;
        }
        float* f = features + ((size_t)b * H + h) * (size_t)P * P + (size_t)i * P;
        for (int jj = 0; jj < P; ++jj) f[jj] = jj <= i ? s_scores[i * P + jj] / z : 0.f;
    }
}

// ---- k-means (Section 3.5; objective of Section 3.2) ------------------------------------------------
// Squared distance, summed in ascending f in one chain (the order the result is defined with).  Only the
// additions depend on one another: the loads, differences and squares of eight elements are issued ahead of
// the chain, which is what the time of the whole kernel hangs on.
__device__ __forceinline__ double sqdist(const double* x, const double* y, int F) {
    double s = 0.0;
    int f = 0;
    for (; f + 8 <= F; f += 8) {
        double q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const double d = __dsub_rn(x[f + u], y[f + u]);
            q[u] = __dmul_rn(d, d);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) s = __dadd_rn(s, q[u]);
    }
    for (; f < F; ++f) {
        const double d = __dsub_rn(x[f], y[f]);
        s = __dadd_rn(s, __dmul_rn(d, d));
    }
    return s;
}

// Sum over the members of cluster c of feature f, ascending h (the order the mean is defined with); the
// loads run ahead of the chain of additions.
__device__ __forceinline__ double member_sum(const double* X, const int* a, int c, int f, int H, int F) {
    double s = 0.0;
    int h = 0;
    for (; h + 8 <= H; h += 8) {
        double v[8];
        bool in[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            in[u] = a[h + u] == c;
            v[u] = X[(size_t)(h + u) * F + f];
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (in[u]) s = __dadd_rn(s, v[u]);
    }
    for (; h < H; ++h)
        if (a[h] == c) s = __dadd_rn(s, X[(size_t)h * F + f]);
    return s;
}

// One CTA per request.  Shared memory: X [H,F], C [k,F], dist [H,k] doubles; a, prev, count ints.
// Sweep mode (k_arg = 0, grid (B, k_max)): CTA (b, j) clusters request b with k = j + 1 and writes only the
// inertia, to inertia[b * k_max + j]; the other outputs are not written.
__global__ void __launch_bounds__(256) kmeans_kernel(const float* __restrict__ features, int H, int F, int k_arg,
                                                     int max_iter, unsigned long long seed,
                                                     int32_t* __restrict__ membership, int32_t* __restrict__ reps,
                                                     int32_t* __restrict__ k_eff, double* __restrict__ inertia) {
    dependent_grid_sync();
    const bool sweep = k_arg == 0;
    const int k = sweep ? (int)blockIdx.y + 1 : k_arg;
    if (sweep) inertia += (size_t)blockIdx.x * gridDim.y + blockIdx.y - blockIdx.x;  // so that inertia[b] below is the curve entry
    extern __shared__ double smem_d[];
    double* X = smem_d;
    double* C = X + (size_t)H * F;
    double* dist = C + (size_t)k * F;  // [H,k]; its first H entries double as dmin during initialisation
    int* a = reinterpret_cast<int*>(dist + (size_t)H * k);
    int* prev = a + H;
    int* count = prev + H;
    int* newid = count + k;
    __shared__ int s_ncentres, s_same;

    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    const float* xin = features + (size_t)b * H * F;
    for (int i = tid; i < H * F; i += nt) X[i] = (double)xin[i];
    __syncthreads();

    // farthest-first traversal: first centre = head (seed mod H)
    const int first = (int)(seed % (unsigned long long)H);
    for (int f = tid; f < F; f += nt) C[f] = X[(size_t)first * F + f];
    if (tid == 0) s_ncentres = 1;
    __syncthreads();
    double* dmin = dist;
    for (int h = tid; h < H; h += nt) dmin[h] = sqdist(X + (size_t)h * F, C, F);
    __syncthreads();
    // The traversal is a chain of k - 1 dependent steps (farthest head, then every head's distance to it).  Four
    // warps walk it, one per scheduler of the SM (the distances are bound by fp64 throughput, which is per
    // scheduler): warp w owns the heads h with h mod 4 = w and their dmin entries; per step the warps exchange
    // their candidates through shared memory and meet at one named barrier.
    if (tid < 128) {
        const int w = tid >> 5, lane = tid & 31;
        __shared__ double s_cd[2][4];
        __shared__ int s_ch[2][4];
        int ncent = 1;
        for (int n = 1; n < k; ++n) {
            double bd = -1.0;  // farthest head so far: largest dmin, lowest index on ties
            int bh = 0x7fffffff;
            for (int h = w + 4 * lane; h < H; h += 128) {
                const double d = dmin[h];
                if (d > bd) {
                    bd = d;
                    bh = h;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double od = __shfl_xor_sync(0xffffffffu, bd, o);
                const int oh = __shfl_xor_sync(0xffffffffu, bh, o);
                if (od > bd || (od == bd && oh < bh)) {
                    bd = od;
                    bh = oh;
                }
            }
            if (lane == 0) {
                s_cd[n & 1][w] = bd;
                s_ch[n & 1][w] = bh;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const double od = s_cd[n & 1][x];
                const int oh = s_ch[n & 1][x];
                if (od > bd || (od == bd && oh < bh)) {
                    bd = od;
                    bh = oh;
                }
            }
            if (bd == 0.0) break;  // fewer than k distinct points (the same decision in all four warps)
            const double* xf = X + (size_t)bh * F;
            if (w == 0)
                for (int f = lane; f < F; f += 32) C[(size_t)n * F + f] = xf[f];
            for (int h = w + 4 * lane; h < H; h += 128) {
                const double d = sqdist(X + (size_t)h * F, xf, F);
                if (d < dmin[h]) dmin[h] = d;
            }
            ncent = n + 1;
        }
        if (tid == 0) s_ncentres = ncent;
    }
    __syncthreads();
    const int nc = s_ncentres;

    // Lloyd iterations
    for (int it = 0; it < max_iter; ++it) {
        for (int p = tid; p < H * nc; p += nt) {
            int h = p / nc, c = p % nc;
            dist[(size_t)h * k + c] = sqdist(X + (size_t)h * F, C + (size_t)c * F, F);
        }
        if (tid == 0) s_same = 1;
        __syncthreads();
        for (int h = tid; h < H; h += nt) {
            int best = 0;
            double bd = dist[(size_t)h * k];
            for (int c = 1; c < nc; ++c) {
                double d = dist[(size_t)h * k + c];
                if (d < bd) {
                    bd = d;
                    best = c;
                }
            }
            a[h] = best;
            if (it == 0 || best != prev[h]) s_same = 0;  // benign race: every writer stores 0
        }
        __syncthreads();
        if (s_same) break;
        for (int h = tid; h < H; h += nt) prev[h] = a[h];
        for (int c = tid; c < nc; c += nt) {
            int n = 0;
            for (int h = 0; h < H; ++h) n += (a[h] == c);
            count[c] = n;
        }
        __syncthreads();
        for (int p = tid; p < nc * F; p += nt) {
            int c = p / F, f = p % F;
            if (count[c] == 0) continue;  // an empty cluster keeps its centre
            C[(size_t)c * F + f] = __ddiv_rn(member_sum(X, a, c, f, H, F), (double)count[c]);
        }
        __syncthreads();
    }
    __syncthreads();

    // canonical labels: clusters ordered by their lowest member; representative = lowest member
    if (tid == 0) {
        for (int c = 0; c < k; ++c) {
            newid[c] = -1;
            if (!sweep) reps[(size_t)b * k + c] = -1;
        }
        int next = 0;
        for (int h = 0; h < H; ++h) {
            if (newid[a[h]] < 0) {
                newid[a[h]] = next;
                if (!sweep) reps[(size_t)b * k + next] = h;
                ++next;
            }
        }
        if (!sweep) k_eff[b] = next;
        s_ncentres = next;
    }
    __syncthreads();
    for (int h = tid; h < H; h += nt) {
        a[h] = newid[a[h]];
        if (!sweep) membership[(size_t)b * H + h] = a[h];
    }
    if (inertia == nullptr) return;
    __syncthreads();

    // inertia against the final members' means, summed in (cluster, head) order
    const int ke = s_ncentres;
    for (int c = tid; c < ke; c += nt) {
        int n = 0;
        for (int h = 0; h < H; ++h) n += (a[h] == c);
        count[c] = n;
    }
    __syncthreads();
    for (int p = tid; p < ke * F; p += nt) {
        int c = p / F, f = p % F;
        C[(size_t)c * F + f] = __ddiv_rn(member_sum(X, a, c, f, H, F), (double)count[c]);
    }
    __syncthreads();
    // heads in (cluster, head) order: that is the order of the sum below
    for (int h = tid; h < H; h += nt) {
        dist[h] = sqdist(X + (size_t)h * F, C + (size_t)a[h] * F, F);
        int rank = 0;
        for (int h2 = 0; h2 < H; ++h2) rank += (a[h2] < a[h] || (a[h2] == a[h] && h2 < h)) ? 1 : 0;
        prev[rank] = h;
    }
    __syncthreads();
    if (tid == 0) {
        double total = 0.0;
        for (int i = 0; i < H; ++i) total = __dadd_rn(total, dist[prev[i]]);
        inertia[b] = total;
    }
}

// Representative of each cluster = the member nearest to the cluster's mean (an alternative to "lowest
// member"; ties go to the lowest head index).  One CTA per request; fp64 with the same explicitly rounded
// operations and summation orders as the clustering itself, so the choice is reproducible bit for bit.
// Shared memory: X [H,F], C [k,F], dist [H] doubles; a [H], count [k] ints.
__global__ void __launch_bounds__(256)
select_reps_kernel(const float* __restrict__ features, const int32_t* __restrict__ membership, int H, int F, int k,
                   int32_t* __restrict__ reps) {
    extern __shared__ double sh_sel[];
    double* X = sh_sel;
    double* C = X + (size_t)H * F;
    double* dist = C + (size_t)k * F;
    int* a = reinterpret_cast<int*>(dist + H);
    int* count = a + H;
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    for (int i = tid; i < H * F; i += nt) X[i] = (double)features[(size_t)b * H * F + i];
    for (int h = tid; h < H; h += nt) {
        const int c = membership[(size_t)b * H + h];
        a[h] = (c >= 0 && c < k) ? c : -1;  // heads with an invalid cluster id belong nowhere
    }
    __syncthreads();
    for (int c = tid; c < k; c += nt) {
        int n = 0;
        for (int h = 0; h < H; ++h) n += (a[h] == c);
        count[c] = n;
    }
    __syncthreads();
    for (int p = tid; p < k * F; p += nt) {
        const int c = p / F, f = p % F;
        if (count[c] == 0) continue;
        C[(size_t)c * F + f] = __ddiv_rn(member_sum(X, a, c, f, H, F), (double)count[c]);
    }
    __syncthreads();
    for (int h = tid; h < H; h += nt)
        if (a[h] >= 0) dist[h] = sqdist(X + (size_t)h * F, C + (size_t)a[h] * F, F);
    __syncthreads();
    for (int c = tid; c < k; c += nt) {
        int best = -1;
        for (int h = 0; h < H; ++h)
            if (a[h] == c && (best < 0 || dist[h] < dist[best])) best = h;
        reps[(size_t)b * k + c] = best;  // -1 for an empty cluster
    }
}

// Knee of a clustering-error curve e(1..n) (Section 3.2 / Fig. 8: the number of clusters is read off where
// the error stops falling quickly; the paper does it by eye).  Rule: scale k to x in [0,1] and the error to
// y in [0,1] (y = 1 at the largest error, 0 at the smallest); the knee is the k that lies farthest below the
// straight line from (0,1) to (1,0), i.e. maximises 1 - x - y; ties go to the smaller k.  One thread per request.
__global__ void knee_kernel(const double* __restrict__ curve, int B, int n, int32_t* __restrict__ k_pick) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const double* e = curve + (size_t)b * n;
    double lo = e[0], hi = e[0];
    for (int i = 1; i < n; ++i) {
        lo = e[i] < lo ? e[i] : lo;
        hi = e[i] > hi ? e[i] : hi;
    }
    int best = 1;
    if (n > 1 && hi > lo) {
        const double span = __dsub_rn(hi, lo);
        double best_v = 0.0;
        bool have = false;
        for (int i = 0; i < n; ++i) {
            const double x = __ddiv_rn((double)i, (double)(n - 1));
            const double y = __ddiv_rn(__dsub_rn(e[i], lo), span);
            const double v = __dsub_rn(__dsub_rn(1.0, x), y);
            if (!have || v > best_v) {
                best_v = v;
                best = i + 1;
                have = true;
            }
        }
    }
    k_pick[b] = best;
}

static size_t kmeans_smem_bytes(int H, int F, int k) {
    return sizeof(double) * ((size_t)H * F + (size_t)k * F + (size_t)H * k) + sizeof(int) * (2 * (size_t)H + 2 * (size_t)k);
}

}  // namespace chai

extern "C" {

int chai_prefix_features(const void* q_full, const void* k_full, int B, int H, int T_cap, int D, int P,
                         float scale, int dtype, float* features, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(q_full && k_full && features, CHAI_ERR_INVALID_ARG, "chai_prefix_features: null pointer");
    CHAI_REQUIRE(aligned16(q_full) && aligned16(k_full), CHAI_ERR_INVALID_ARG,
                 "chai_prefix_features: pointers must be 16-byte aligned");
    CHAI_REQUIRE(B > 0 && H > 0 && T_cap > 0 && D > 0 && P > 0, CHAI_ERR_INVALID_ARG,
                 "chai_prefix_features: sizes must be positive");
    CHAI_REQUIRE(P <= T_cap, CHAI_ERR_INVALID_ARG, "chai_prefix_features: P=%d exceeds T_cap=%d", P, T_cap);
    CHAI_REQUIRE(P <= 32 && B <= 65535, CHAI_ERR_UNSUPPORTED, "chai_prefix_features: P <= 32 and B <= 65535");
    CHAI_REQUIRE(dtype == CHAI_F32 || dtype == CHAI_BF16, CHAI_ERR_UNSUPPORTED, "chai_prefix_features: dtype");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    dim3 grid(H, B), block(P * P);
    size_t smem = sizeof(float) * P * P;
    if (dtype == CHAI_BF16)
        prefix_features_kernel<__nv_bfloat16><<<grid, block, smem, s>>>(
            static_cast<const __nv_bfloat16*>(q_full), static_cast<const __nv_bfloat16*>(k_full), features, H,
            T_cap, D, P, scale);
    else
        prefix_features_kernel<float><<<grid, block, smem, s>>>(static_cast<const float*>(q_full),
                                                               static_cast<const float*>(k_full), features, H,
                                                               T_cap, D, P, scale);
    CHAI_LAUNCH_CHECK("prefix_features_kernel launch");
    return CHAI_OK;
}

int chai_cluster_heads(const float* features, int B, int H, int F, int k, int max_iter, uint64_t seed,
                       int32_t* membership, int32_t* reps, int32_t* k_eff, double* inertia, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(features && membership && reps && k_eff, CHAI_ERR_INVALID_ARG,
                 "chai_cluster_heads: null pointer");
    CHAI_REQUIRE(B > 0 && H > 0 && F > 0 && max_iter > 0, CHAI_ERR_INVALID_ARG,
                 "chai_cluster_heads: sizes must be positive");
    CHAI_REQUIRE(k >= 1 && k <= H, CHAI_ERR_INVALID_ARG, "chai_cluster_heads: need 1 <= k <= H (k=%d, H=%d)", k, H);
    size_t smem = kmeans_smem_bytes(H, F, k);
    CHAI_REQUIRE(H <= 1024 && smem <= 200 * 1024, CHAI_ERR_UNSUPPORTED,
                 "chai_cluster_heads: problem needs %zu bytes of shared memory (limit 204800)", smem);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CHAI_LOG_CALL("chai_cluster_heads: B=%d H=%d F=%d k=%d max_iter=%d seed=%llu, %d CTAs x 256 threads, %zu bytes of shared memory",
                  B, H, F, k, max_iter, (unsigned long long)seed, B, smem);
    cudaError_t e = cudaFuncSetAttribute(kmeans_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "kmeans_kernel shared-memory opt-in");
    CHAI_LAUNCH_DEPENDENT("kmeans_kernel launch", kmeans_kernel, dim3(B), dim3(256), smem, s, features, H, F, k, max_iter,
                          (unsigned long long)seed, membership, reps, k_eff, inertia);
    return CHAI_OK;
}

int chai_select_representatives(const float* features, const int32_t* membership, int B, int H, int F, int k,
                                int32_t* reps, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(features && membership && reps, CHAI_ERR_INVALID_ARG, "chai_select_representatives: null pointer");
    CHAI_REQUIRE(B > 0 && H > 0 && F > 0 && k >= 1 && k <= H, CHAI_ERR_INVALID_ARG,
                 "chai_select_representatives: need B, H, F > 0 and 1 <= k <= H");
    const size_t smem = sizeof(double) * ((size_t)H * F + (size_t)k * F + (size_t)H) + sizeof(int) * ((size_t)H + k);
    CHAI_REQUIRE(H <= 1024 && smem <= 200 * 1024, CHAI_ERR_UNSUPPORTED,
                 "chai_select_representatives: problem needs %zu bytes of shared memory (limit 204800)", smem);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaFuncSetAttribute(select_reps_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "select_reps_kernel shared-memory opt-in");
    select_reps_kernel<<<B, 256, smem, s>>>(features, membership, H, F, k, reps);
    CHAI_LAUNCH_CHECK("select_reps_kernel launch");
    return CHAI_OK;
}

int chai_cluster_sweep(const float* features, int B, int H, int F, int k_max, int max_iter, uint64_t seed,
                       double* inertia_curve, int32_t* k_pick, void* stream) {
    using namespace chai;
    CHAI_REQUIRE(features && inertia_curve, CHAI_ERR_INVALID_ARG, "chai_cluster_sweep: null pointer");
    CHAI_REQUIRE(B > 0 && H > 0 && F > 0 && max_iter > 0, CHAI_ERR_INVALID_ARG, "chai_cluster_sweep: sizes must be positive");
    CHAI_REQUIRE(k_max >= 1 && k_max <= H, CHAI_ERR_INVALID_ARG, "chai_cluster_sweep: need 1 <= k_max <= H (k_max=%d, H=%d)",
                 k_max, H);
    const size_t smem = kmeans_smem_bytes(H, F, k_max);
    CHAI_REQUIRE(H <= 1024 && B <= 65535 && smem <= 200 * 1024, CHAI_ERR_UNSUPPORTED,
                 "chai_cluster_sweep: problem needs %zu bytes of shared memory (limit 204800)", smem);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaFuncSetAttribute(kmeans_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "kmeans_kernel shared-memory opt-in");
    kmeans_kernel<<<dim3(B, k_max), 256, smem, s>>>(features, H, F, 0, max_iter, (unsigned long long)seed, nullptr,
                                                    nullptr, nullptr, inertia_curve);
    CHAI_LAUNCH_CHECK("kmeans_kernel (sweep) launch");
    if (k_pick != nullptr) {
        knee_kernel<<<(B + 127) / 128, 128, 0, s>>>(inertia_curve, B, k_max, k_pick);
        CHAI_LAUNCH_CHECK("knee_kernel launch");
    }
    return CHAI_OK;
}

}  // extern "C"
