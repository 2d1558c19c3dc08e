/*
 * CPU oracle for clustered-head attention (CHAI) -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the CUDA library must compute.  It is
 * called by the tests, by the smoke check and by the timed CPU-baseline leg of
 * the benchmark; the product path never links, imports or executes it.  It
 * shares no source, header, table or helper with the CUDA library.
 *
 * Every routine is the definition written out (attention, features,
 * compaction) or the algorithm step by step (k-means); the only parallelism is
 * an OpenMP loop over independent (request, cluster, query row) triples.
 * Build with -ffp-contract=off so that the k-means arithmetic is a fixed
 * sequence of IEEE double operations.
 *
 * Pins (tests/test_oracle_*.py): k = H reduces to textbook multi-head
 * attention (checked against torch's scaled_dot_product_attention in fp64 and
 * a dense masked-matrix numpy restatement); identical Q,K inside a cluster
 * reduces to multi-head attention; closed forms (Q = 0, V = 1, V = I, one
 * dominant key); softmax-shift and relabelling invariances; decode equals the
 * last prefill row; k-means recovers planted partitions for every seed, agrees
 * with scikit-learn's Lloyd from the same initial centres, never increases the
 * inertia, and is bounded below by exhaustive search on tiny inputs.
 * The paper prints no numeric example of an attention or clustering output,
 * so agreement with the authors' own implementation is "parity unpinned"
 * beyond those checks.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * Clustered-head attention (Section 3.4 and Fig. 3(b) for the operator,
 * Section 2 for A_h = softmax(Q K^T / sqrt(d)) and y = concat_h A_h V_h,
 * Section 4.3: only keys are dropped, every head keeps its values).
 *
 *   Q     [B,H,Tq,D]   all heads' queries; only representatives' rows are read
 *   Krep  [B,k,T,D]    keys of the representative heads, slot c = cluster c
 *   V     [B,H,T,D]    every head's values
 *   membership [B,H]   cluster id of each head;  reps [B,k]  head index or -1
 *   O     [B,H,Tq,D]   output
 *
 * Query row i (0-based, of Tq) is the token at absolute position
 * i + (T - Tq); with causal != 0 it sees keys j <= i + (T - Tq), otherwise all
 * T keys.  Decode is Tq = 1.  A head whose cluster id is out of range or whose
 * cluster has no representative gets a zero output.
 */
int oracle_cha_attention(const double* Q, const double* Krep, const double* V,
                         const int32_t* membership, const int32_t* reps, double* O,
                         int B, int H, int k, int Tq, int T, int D, double scale, int causal) {
    if (B <= 0 || H <= 0 || k <= 0 || Tq <= 0 || T <= 0 || D <= 0 || Tq > T) return 1;
    memset(O, 0, sizeof(double) * (size_t)B * H * Tq * D);
    long long n_units = (long long)B * k * Tq;
#pragma omp parallel
    {
        double* a = (double*)malloc(sizeof(double) * (size_t)T);
#pragma omp for schedule(dynamic, 8)
        for (long long u = 0; u < n_units; ++u) {
            int i = (int)(u % Tq);
            int c = (int)((u / Tq) % k);
            int b = (int)(u / ((long long)Tq * k));
            int r = reps[(size_t)b * k + c];
            if (r < 0 || r >= H) continue;
            int jmax = causal ? i + (T - Tq) : T - 1;
            const double* q = Q + (((size_t)b * H + r) * Tq + i) * D;
            const double* Kc = Krep + ((size_t)b * k + c) * (size_t)T * D;
            /* scores of the representative head */
            double m = -INFINITY;
            for (int j = 0; j <= jmax; ++j) {
                double s = 0.0;
                for (int d = 0; d < D; ++d) s += q[d] * Kc[(size_t)j * D + d];
                s *= scale;
                a[j] = s;
                if (s > m) m = s;
            }
            /* softmax over the visible keys */
            double Z = 0.0;
            for (int j = 0; j <= jmax; ++j) {
                a[j] = exp(a[j] - m);
                Z += a[j];
            }
            for (int j = 0; j <= jmax; ++j) a[j] /= Z;
            /* every member head applies the shared probabilities to its own values */
            for (int h = 0; h < H; ++h) {
                if (membership[(size_t)b * H + h] != c) continue;
                const double* Vh = V + ((size_t)b * H + h) * (size_t)T * D;
                double* o = O + (((size_t)b * H + h) * Tq + i) * D;
                for (int j = 0; j <= jmax; ++j) {
                    double aj = a[j];
                    for (int d = 0; d < D; ++d) o[d] += aj * Vh[(size_t)j * D + d];
                }
            }
        }
        free(a);
    }
    return 0;
}

/*
 * Prefix score features (Section 3.3: membership is decided from what plain
 * multi-head attention produced on the first five tokens; the problem
 * statement of Section 3.1 defines similarity on softmax(Q K^T)).
 *
 *   Q, K  [B,H,T,D] (row stride between heads is T*D); the first P rows are read
 *   features [B,H,P*P]: entry i*P+j is the causal attention probability of
 *   head h's own query i on its own key j (j <= i), and 0 for j > i.
 */
int oracle_prefix_features(const double* Q, const double* K, double* features,
                           int B, int H, int T, int D, int P, double scale) {
    if (B <= 0 || H <= 0 || T <= 0 || D <= 0 || P <= 0 || P > T) return 1;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const double* q = Q + ((size_t)b * H + h) * (size_t)T * D;
            const double* kk = K + ((size_t)b * H + h) * (size_t)T * D;
            double* f = features + ((size_t)b * H + h) * (size_t)P * P;
            for (int i = 0; i < P; ++i) {
                double m = -INFINITY;
                for (int j = 0; j <= i; ++j) {
                    double s = 0.0;
                    for (int d = 0; d < D; ++d) s += q[(size_t)i * D + d] * kk[(size_t)j * D + d];
                    s *= scale;
                    f[i * P + j] = s;
                    if (s > m) m = s;
                }
                double Z = 0.0;
                for (int j = 0; j <= i; ++j) {
                    f[i * P + j] = exp(f[i * P + j] - m);
                    Z += f[i * P + j];
                }
                for (int j = 0; j <= i; ++j) f[i * P + j] /= Z;
                for (int j = i + 1; j < P; ++j) f[i * P + j] = 0.0;
            }
        }
    return 0;
}

static double sqdist(const double* x, const double* y, int F) {
    double s = 0.0;
    for (int f = 0; f < F; ++f) {
        double d = x[f] - y[f];
        s += d * d;
    }
    return s;
}

/*
 * K-means membership of the H heads of one request (Section 3.5: "K-Means
 * clustering" on the activations observed after five tokens; Section 3.2:
 * clustering error = sum of squared distance to the closest centre, hence
 * squared Euclidean distance and mean centroids).  The paper fixes nothing
 * below the name; this is the reading used throughout this repository:
 *
 *   init    seeded farthest-first traversal: first centre = point (seed mod H),
 *           each next centre = the point farthest from the centres so far
 *           (ties -> lowest index); stops early when every point coincides
 *           with a centre (fewer than k distinct points)
 *   Lloyd   assign each point to its nearest centre (ties -> lowest centre),
 *           stop when an assignment repeats, else move every non-empty centre
 *           to the mean of its members (summed in ascending head order); an
 *           empty cluster keeps its centre; at most max_iter assignments
 *   output  clusters renumbered by their lowest member head; reps[c] = lowest
 *           member head of cluster c, -1 for c >= k_eff; inertia = sum of
 *           squared distances to the final members' means
 *
 *   X [H,F]; membership [H]; reps [k]; k_eff [1]; inertia [1] (may be NULL);
 *   trace [max_iter] (may be NULL): clustering error right after each
 *   assignment step, against the centres used for that assignment; unused
 *   entries are set to -1.  init_idx [k] (may be NULL): the head chosen as each
 *   initial centre, -1 where the traversal stopped early.
 */
int oracle_kmeans(const double* X, int H, int F, int k, int max_iter, uint64_t seed,
                  int32_t* membership, int32_t* reps, int32_t* k_eff, double* inertia,
                  double* trace, int32_t* init_idx) {
    if (H <= 0 || F <= 0 || k <= 0 || k > H || max_iter <= 0) return 1;
    double* C = (double*)calloc((size_t)k * F, sizeof(double));
    double* dmin = (double*)malloc(sizeof(double) * (size_t)H);
    int* a = (int*)malloc(sizeof(int) * (size_t)H);
    int* prev = (int*)malloc(sizeof(int) * (size_t)H);
    int* count = (int*)malloc(sizeof(int) * (size_t)k);
    int* newid = (int*)malloc(sizeof(int) * (size_t)k);
    if (trace)
        for (int it = 0; it < max_iter; ++it) trace[it] = -1.0;

    /* farthest-first initial centres */
    int first = (int)(seed % (uint64_t)H);
    int n_centres = 1;
    if (init_idx) {
        for (int c = 0; c < k; ++c) init_idx[c] = -1;
        init_idx[0] = first;
    }
    memcpy(C, X + (size_t)first * F, sizeof(double) * (size_t)F);
    for (int h = 0; h < H; ++h) dmin[h] = sqdist(X + (size_t)h * F, C, F);
    while (n_centres < k) {
        int far = 0;
        for (int h = 1; h < H; ++h)
            if (dmin[h] > dmin[far]) far = h;
        if (dmin[far] == 0.0) break;
        double* cn = C + (size_t)n_centres * F;
        if (init_idx) init_idx[n_centres] = far;
        memcpy(cn, X + (size_t)far * F, sizeof(double) * (size_t)F);
        for (int h = 0; h < H; ++h) {
            double d = sqdist(X + (size_t)h * F, cn, F);
            if (d < dmin[h]) dmin[h] = d;
        }
        ++n_centres;
    }

    /* Lloyd iterations over the n_centres centres that exist */
    for (int it = 0; it < max_iter; ++it) {
        double err = 0.0;
        for (int h = 0; h < H; ++h) {
            int best = 0;
            double bd = sqdist(X + (size_t)h * F, C, F);
            for (int c = 1; c < n_centres; ++c) {
                double d = sqdist(X + (size_t)h * F, C + (size_t)c * F, F);
                if (d < bd) {
                    bd = d;
                    best = c;
                }
            }
            a[h] = best;
            err += bd;
        }
        if (trace) trace[it] = err;
        if (it > 0) {
            int same = 1;
            for (int h = 0; h < H; ++h)
                if (a[h] != prev[h]) same = 0;
            if (same) break;
        }
        memcpy(prev, a, sizeof(int) * (size_t)H);
        for (int c = 0; c < n_centres; ++c) count[c] = 0;
        for (int h = 0; h < H; ++h) count[a[h]]++;
        for (int c = 0; c < n_centres; ++c) {
            if (count[c] == 0) continue;
            double* cc = C + (size_t)c * F;
            for (int f = 0; f < F; ++f) {
                double s = 0.0;
                for (int h = 0; h < H; ++h)
                    if (a[h] == c) s += X[(size_t)h * F + f];
                cc[f] = s / (double)count[c];
            }
        }
    }

    /* canonical labels: clusters ordered by their lowest member head */
    for (int c = 0; c < k; ++c) {
        newid[c] = -1;
        reps[c] = -1;
    }
    int next = 0;
    for (int h = 0; h < H; ++h) {
        if (newid[a[h]] < 0) {
            newid[a[h]] = next;
            reps[next] = h;
            ++next;
        }
        membership[h] = newid[a[h]];
    }
    *k_eff = next;

    if (inertia) {
        /* distance of every head to the mean of the cluster it ended in */
        double total = 0.0;
        double* mean = (double*)malloc(sizeof(double) * (size_t)F);
        for (int c = 0; c < next; ++c) {
            int n = 0;
            for (int h = 0; h < H; ++h) n += (membership[h] == c);
            for (int f = 0; f < F; ++f) {
                double s = 0.0;
                for (int h = 0; h < H; ++h)
                    if (membership[h] == c) s += X[(size_t)h * F + f];
                mean[f] = s / (double)n;
            }
            for (int h = 0; h < H; ++h)
                if (membership[h] == c) total += sqdist(X + (size_t)h * F, mean, F);
        }
        free(mean);
        *inertia = total;
    }
    free(C);
    free(dmin);
    free(a);
    free(prev);
    free(count);
    free(newid);
    return 0;
}

/*
 * K-cache compaction (Section 3.5: once membership is fixed, the keys of the
 * pruned heads are removed; Section 4.3: values are all kept).
 *   Kfull [B,H,T,D] -> Krep [B,k,T,D], slot c = head reps[b][c]; a slot whose
 *   representative is -1 is zero-filled.  elem_bytes is the element size; the
 *   copy is bit-for-bit.  bytes[0] = K+V bytes before, bytes[1] = after.
 */
int oracle_compact_k_cache(const void* Kfull, void* Krep, const int32_t* reps,
                           int B, int H, int k, int T, int D, int elem_bytes, int64_t* bytes) {
    if (B <= 0 || H <= 0 || k <= 0 || k > H || T <= 0 || D <= 0 || elem_bytes <= 0) return 1;
    size_t plane = (size_t)T * D * elem_bytes;
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < k; ++c) {
            int r = reps[(size_t)b * k + c];
            char* dst = (char*)Krep + ((size_t)b * k + c) * plane;
            if (r < 0 || r >= H)
                memset(dst, 0, plane);
            else
                memcpy(dst, (const char*)Kfull + ((size_t)b * H + r) * plane, plane);
        }
    if (bytes) {
        bytes[0] = (int64_t)2 * B * H * (int64_t)plane;
        bytes[1] = (int64_t)B * (H + k) * (int64_t)plane;
    }
    return 0;
}
