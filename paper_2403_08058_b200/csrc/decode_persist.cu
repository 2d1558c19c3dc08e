// Clustered decode attention, persistent streaming kernel (Fig. 3(b), Section 3.4).
//
// One CTA per SM, launched cooperatively.  Warp 8 is the producer: it streams the cache rows of this
// CTA's work, 32 KB tile by tile, into a shared-memory ring with bulk async copies that complete on
// mbarriers, and runs ahead of the consumers by the depth of the ring, so HBM stays busy while a
// consumer does an item's serial prologue and epilogue.  Warps 0..7 consume, each on its own: ring
// position n belongs to one consumer warp, nothing is synchronised across warps.
//
//   phase K   unit = one key tile (TR rows of one cluster's K_rep): scaled scores s_t -> workspace
//             (fp32, stays in L2) and the tile's maximum.  Every K_rep row is read exactly once.
//   grid-wide barrier (cooperative groups).  The producer has already filled the ring with value
//             tiles by then.
//   phase V   unit = item (request, head, IV value tiles) owned by one warp: reference maximum of the
//             cluster's whole score row, p_t = exp(s_t - max), partial sums (sum p_t V_t, sum p_t)
//             -> workspace; the warp that completes a head's last item (atomic ticket, nobody waits)
//             adds the partials in chunk order and writes out = sum / l.
//
// Units have the same size whatever the cluster sizes and are dealt round-robin over CTAs and warps, so
// the schedule is static and balanced for skewed memberships too.  The softmax is the exact two-pass
// form; results do not depend on timing.  Every wait is bounded; on expiry the CTA records
// CHAI_ERR_TIMEOUT, stops consuming, still joins the grid barrier and returns.
#include <cooperative_groups.h>
#include <stdlib.h>

#include "decode_layout.cuh"

namespace cg = cooperative_groups;

namespace chai {
namespace pd {

// per-CTA phase timestamps (ns) of the most recent launch: debugging aid read by chai_debug_decode_stats
__device__ unsigned long long g_cta_stats[1024][4];

constexpr int CONSUMER_WARPS = 8;
constexpr int CONSUMERS = CONSUMER_WARPS * 32;
constexpr int THREADS = CONSUMERS + 32;
constexpr int STAGES = 5;                  // 176 KB of cache rows in flight per SM
constexpr int TABLE_CAP = 2048;            // heads whose cluster id is cached in shared memory
constexpr long long TIMEOUT_CYCLES = 2000000000ll;

struct Smem {
    alignas(128) unsigned char ring[STAGES][kTileBytes];
    alignas(8) unsigned long long full[STAGES];
    unsigned long long empty[STAGES];
    int table[TABLE_CAP];
    int seq[STAGES];   // sequence number of the tile most recently issued into each slot
    int abort_flag;
};

struct Params {
    const void* q;
    const void* k_rep;
    const void* v;
    const int32_t* membership;
    const int32_t* reps;
    void* out;
    WsHeader* hdr;
    int* counters;
    float* scores;
    float* cmax;
    float* lpart;
    float* opart;
    int B, H, k, T, T_cap;
    int IK, IV;      // tiles per key / value item
    int nKi, nVi;    // items per plane
    float scale;
    int debug;       // bit 0: consumers only drain the ring (streaming-rate experiments; results are garbage)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long* stall_cycles = nullptr) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    bool done = false;
    while (true) {
        if (mbar_try_wait(bar, parity)) {
            done = true;
            break;
        }
        if (*abort_flag) break;
        if (clock64() - t0 > TIMEOUT_CYCLES) {
            *abort_flag = 1;
            break;
        }
    }
    if (stall_cycles) *stall_cycles += clock64() - t0;
    return done;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait until a ring slot carries the tile with sequence number n (see the producer's tagging).
__device__ __forceinline__ bool seq_wait(const int* seq_word, int n, volatile int* abort_flag, long long* stall_cycles) {
    const volatile int* w = seq_word;
    if (*w == n) return true;
    const long long t0 = clock64();
    bool done = false;
    while (true) {
        if (*w == n) {
            done = true;
            break;
        }
        if (*abort_flag) break;
        if (clock64() - t0 > TIMEOUT_CYCLES) {
            *abort_flag = 1;
            break;
        }
    }
    if (stall_cycles) *stall_cycles += clock64() - t0;
    return done;
}
// 1-D bulk async copy global -> shared, completion counted in bytes on an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
template <typename T, int D>
struct Geom {
    static constexpr int EPV = 16 / (int)sizeof(T);   // elements per 16-byte vector
    static constexpr int ROW_BYTES = D * (int)sizeof(T);
    static constexpr int TR = kTileBytes / ROW_BYTES;  // rows per tile (32, 64 or 128)
    static constexpr int LPR = ROW_BYTES / 16;         // lanes per row
    static constexpr int RPW = 32 / LPR;               // rows per warp-wide load
    static constexpr int PV = TR / 32;                 // probabilities per lane per tile
    static constexpr int IT = 32 / RPW;                // warp-wide loads per 32 rows
    static_assert(TR % 32 == 0 && PV >= 1, "a tile is a whole number of 32-row blocks");
};

struct Ring {
    uint32_t full0, empty0, data0;
    __device__ __forceinline__ uint32_t full(int slot) const { return full0 + 8 * slot; }
    __device__ __forceinline__ uint32_t empty(int slot) const { return empty0 + 8 * slot; }
    __device__ __forceinline__ uint32_t data(int slot) const { return data0 + kTileBytes * slot; }
};

// Work decomposition (identical arithmetic on the producer and consumer side).
//   tp   tiles per cache plane = ceil(T / TR)
//   phase K: this CTA's key tiles are the global tile ids g = cta, cta + ncta, ...  (g = plane * tp + tile);
//            its t-th tile has ring sequence number t and belongs to consumer warp t mod W.
//   phase V: value items (head, chunk of IV tiles), item id i = cta + jc * ncta for the CTA's jc-th item;
//            item jc belongs to warp jc mod W (its j = jc / W -th item).  The ring interleaves the warps'
//            tile streams: full rows of W warps first, then the last row of R = NI mod W warps.
struct Work {
    int tp, nkt, ni, full_rows, rem;  // tiles/plane, key tiles and value items of this CTA, NI / W, NI % W
    int IV;
    __device__ __forceinline__ int vseq(int w, int j, int t) const {  // ring sequence number of a value tile
        if (j < full_rows) return nkt + (j * IV + t) * CONSUMER_WARPS + w;
        return nkt + full_rows * IV * CONSUMER_WARPS + t * rem + w;
    }
};

template <typename T, int D>
__global__ void __launch_bounds__(THREADS, 1) decode_persistent_kernel(const Params P) {
    using G = Geom<T, D>;
    constexpr int W = CONSUMER_WARPS;
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, ncta = gridDim.x;
    volatile int* abort_flag = &sm.abort_flag;
    const Ring ring{smem_u32(&sm.full[0]), smem_u32(&sm.empty[0]), smem_u32(&sm.ring[0][0])};
    const int B = P.B, H = P.H, k = P.k, T_len = P.T;
    const bool use_table = B * H <= TABLE_CAP;
    Work wk;
    wk.tp = (T_len + G::TR - 1) / G::TR;
    wk.IV = P.IV;
    {
        const long long kt = (long long)B * k * wk.tp, vi = (long long)B * H * P.nVi;
        wk.nkt = (int)((kt - cta + ncta - 1) / ncta);
        wk.ni = (int)((vi - cta + ncta - 1) / ncta);
        if (wk.nkt < 0) wk.nkt = 0;
        if (wk.ni < 0) wk.ni = 0;
        wk.full_rows = wk.ni / W;
        wk.rem = wk.ni % W;
    }
    // timing breadcrumbs of CTA 0 (debugging aid): header words 16.. as 64-bit values
    unsigned long long* stats = reinterpret_cast<unsigned long long*>(&P.hdr->pad[1]);
    if (cta == 0 && tid == 0) stats[0] = global_ns();
    if (tid == 0 && cta < 1024) g_cta_stats[cta][0] = global_ns();

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(ring.full(s), 1);
            mbar_init(ring.empty(s), 1);
            sm.seq[s] = -1;
        }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // housekeeping for phase V (ordered by the grid barrier): tickets, status word, head table
    if (cta == 0 && tid == 0) {
        P.hdr->status = CHAI_OK;
        P.hdr->bad_b = -1;
        P.hdr->bad_h = -1;
    }
    for (int i = cta * THREADS + tid; i < B * H; i += ncta * THREADS) P.counters[i] = 0;
    if (use_table) {
        for (int i = tid; i < B * H; i += THREADS) {
            int c, r;
            sm.table[i] = resolve_head(P.membership, P.reps, i / H, i % H, H, k, &c, &r) ? c : -1;
        }
    }
    __syncthreads();

    const unsigned char* kc = static_cast<const unsigned char*>(P.k_rep);
    const unsigned char* vc = static_cast<const unsigned char*>(P.v);
    auto tile_rows = [&](int tile) { return max(0, min(G::TR, T_len - tile * G::TR)); };

    if (warp == W) {
        // ------------------------------ producer warp ------------------------------
        // Tiles are issued in strict ring order (ascending sequence number), which keeps the one-bit phase
        // parity of the slot barriers unambiguous on the producer side.  The loop control is uniform over
        // the warp; lane w (< W) keeps the addresses of consumer warp w's stream and is the one lane that
        // waits for the slot and issues when a tile of that stream is due, so the address arithmetic of
        // the W streams runs in parallel and a tile costs the warp a few dozen instructions.
        long long stall_k = 0, stall_v = 0;
        int n = 0, slot = 0;
        uint32_t parity = 1;  // parity to wait for on empty[slot]: ((n / STAGES) & 1) ^ 1
        auto next_slot = [&]() {
            ++n;
            if (++slot == STAGES) {
                slot = 0;
                parity ^= 1u;
            }
        };
        auto emit = [&](const unsigned char* base, int plane, int tile) {
            const int rows = tile_rows(tile);
            // Consumer warps run independently and bulk copies complete out of order, so a consumer may
            // reach this slot while the previous occupant's copy is still in flight; the one-bit phase
            // parity of the full barrier cannot tell those two fills apart.  The tag can: a consumer first
            // waits until the slot is tagged with its own sequence number (the previous occupant has then
            // been consumed, hence its phase completed) and only then waits on the barrier.
            *reinterpret_cast<volatile int*>(&sm.seq[slot]) = n;
            if (rows > 0) {
                const uint32_t bytes = (uint32_t)rows * G::ROW_BYTES;
                mbar_expect_tx(ring.full(slot), bytes);
                bulk_load(ring.data(slot), base + ((size_t)plane * P.T_cap + (size_t)tile * G::TR) * G::ROW_BYTES, bytes,
                          ring.full(slot));
            } else {
                mbar_arrive(ring.full(slot));  // padding tile past the end of the cache: nothing to copy
            }
        };
        // ---- key tiles: tile t of this CTA belongs to stream t mod W ----
        bool ok = true;
        {
            const long long g = (long long)cta + (long long)lane * ncta;  // meaningful for lanes < W
            int kplane = (int)(g / wk.tp), ktile = (int)(g % wk.tp);
            const int dplane = (int)(((long long)W * ncta) / wk.tp), dtile = (int)(((long long)W * ncta) % wk.tp);
            int w = 0;
            for (int t = 0; t < wk.nkt && ok; ++t) {
                int res = 1;
                if (lane == w) {
                    res = mbar_wait(ring.empty(slot), parity, abort_flag, &stall_k) ? 1 : 0;
                    if (res) {
                        emit(kc, kplane, ktile);
                        kplane += dplane;
                        ktile += dtile;
                        if (ktile >= wk.tp) {
                            ktile -= wk.tp;
                            ++kplane;
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, res, w) != 0;
                next_slot();
                if (++w == W) w = 0;
            }
        }
        // ---- value tiles: row j of items (one per stream), tile t of each, streams in order ----
        int j = 0, t = 0, w = 0, vplane = 0, vtile0 = 0;
        bool loaded = false;
        const int last_row = wk.rem > 0 ? wk.full_rows : wk.full_rows - 1;
        // returns 1 when every tile has been issued, 0 when a non-blocking probe found the slot busy, -1 on expiry
        auto pump_values = [&](bool blocking) -> int {
            while (j <= last_row) {
                const int nact = j < wk.full_rows ? W : wk.rem;
                if (!loaded) {  // every stream looks up its item of this row at once
                    if (lane < nact) {
                        const long long item = (long long)cta + (long long)(lane + j * W) * ncta;
                        vplane = (int)(item / P.nVi);
                        vtile0 = (int)(item % P.nVi) * wk.IV;
                    }
                    loaded = true;
                }
                int res = 1;
                if (lane == w) {
                    if (blocking)
                        res = mbar_wait(ring.empty(slot), parity, abort_flag, &stall_v) ? 1 : -1;
                    else
                        res = mbar_try_wait(ring.empty(slot), parity) ? 1 : 0;
                    if (res == 1) emit(vc, vplane, vtile0 + t);
                }
                res = __shfl_sync(0xffffffffu, res, w);
                if (res != 1) return res;
                next_slot();
                if (++w == nact) {
                    w = 0;
                    if (++t == wk.IV) {
                        t = 0;
                        ++j;
                        loaded = false;
                    }
                }
            }
            return 1;
        };
        // before the grid barrier value tiles only go into slots that are already free: the consumers
        // release value slots after the barrier, so a blocking wait here could never be satisfied
        const int r1 = ok ? pump_values(false) : -1;
        cg::this_grid().sync();
        if (r1 == 0) pump_values(true);
        if (cta == 0 && lane == 0) {
            stats[4] = (unsigned long long)stall_k;
            stats[5] = (unsigned long long)stall_v;
        }
    } else {
        // ------------------------------ consumers: every warp works alone ------------------------------
        const int sub = lane / G::LPR, part = lane % G::LPR;
        bool ok = true;
        long long stall_c = 0;
        // ---- phase K: one tile = TR scores and their maximum ----
        for (int t = warp; t < wk.nkt; t += W) {
            const long long g = (long long)cta + (long long)t * ncta;
            const int plane = (int)(g / wk.tp), tile = (int)(g % wk.tp);
            const int b = plane / k;
            const int rows = tile_rows(tile);
            const int rep = P.reps[plane];
            const bool live = rep >= 0 && rep < H;  // unused cluster slot: the tile is drained, nothing computed
            float qf[G::EPV];
#pragma unroll
            for (int e = 0; e < G::EPV; ++e) qf[e] = 0.f;
            if (live) {
                const uint4 qv = *reinterpret_cast<const uint4*>(static_cast<const T*>(P.q) + ((size_t)b * H + rep) * D + part * G::EPV);
                Vec16<T>::unpack(qv, qf);
            }
            const int slot = t % STAGES;
            if (ok) ok = __all_sync(0xffffffffu, seq_wait(&sm.seq[slot], t, abort_flag, &stall_c) &&
                                                     mbar_wait(ring.full(slot), (t / STAGES) & 1, abort_flag, &stall_c));
            if (ok && live && !(P.debug & 1)) {
                const unsigned char* data = sm.ring[slot];
                float* srow = P.scores + (size_t)plane * T_len + (size_t)tile * G::TR;
                float lmax = -INFINITY;
                // Each lane holds a 16-byte slice of a row; LPR lanes cover a row.  Partial dot products of
                // LPR rows are reduced together by a transposing butterfly (LPR - 1 shuffles per LPR rows),
                // after which lane `part` owns the score of row (batch * LPR + part) * RPW + sub: the 32
                // lanes of the warp then hold 32 consecutive rows and store them as one 128-byte line.
#pragma unroll
                for (int bt = 0; bt < G::TR / 32; ++bt) {
                    float v[G::LPR];
#pragma unroll
                    for (int ii = 0; ii < G::LPR; ++ii) {
                        const int row = (bt * G::LPR + ii) * G::RPW + sub;
                        const uint4 raw = *reinterpret_cast<const uint4*>(data + row * G::ROW_BYTES + part * 16);
                        float kf[G::EPV];
                        Vec16<T>::unpack(raw, kf);
                        float s0 = 0.f, s1 = 0.f;
#pragma unroll
                        for (int e = 0; e < G::EPV; e += 2) {
                            s0 = fmaf(qf[e], kf[e], s0);
                            s1 = fmaf(qf[e + 1], kf[e + 1], s1);
                        }
                        v[ii] = s0 + s1;
                    }
#pragma unroll
                    for (int o = G::LPR / 2; o >= 1; o >>= 1) {
                        const bool hi = (lane & o) != 0;
#pragma unroll
                        for (int x = 0; x < o; ++x) {
                            const float send = hi ? v[x] : v[x + o];
                            const float keep = hi ? v[x + o] : v[x];
                            v[x] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                        }
                    }
                    const float sc = v[0] * P.scale;
                    const int row = (bt * G::LPR + part) * G::RPW + sub;
                    if (row < rows) {  // rows past the end of a ragged last tile hold stale bytes
                        srow[row] = sc;
                        lmax = fmaxf(lmax, sc);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) lmax = fmaxf(lmax, __shfl_xor_sync(0xffffffffu, lmax, o));
                if (lane == 0) P.cmax[(size_t)plane * wk.tp + tile] = lmax;
            }
            __syncwarp();
            if (lane == 0 && ok) mbar_arrive(ring.empty(slot));
        }
        if (cta == 0 && tid == 0) {
            stats[1] = global_ns();
            stats[6] = (unsigned long long)stall_c;
        }
        if (tid == 0 && cta < 1024) g_cta_stats[cta][1] = global_ns();
        cg::this_grid().sync();
        if (cta == 0 && tid == 0) stats[2] = global_ns();
        if (tid == 0 && cta < 1024) g_cta_stats[cta][2] = global_ns();
        // ---- phase V: one item = IV tiles of one head; partial sums; combine by the last arriver ----
        T* outp = static_cast<T*>(P.out);
        for (int j = 0;; ++j) {
            const int jc = warp + j * W;
            if (jc >= wk.ni) break;
            const long long item = (long long)cta + (long long)jc * ncta;
            const int head = (int)(item / P.nVi), chunk = (int)(item % P.nVi);
            const int b = head / H, h = head % H;
            int c;
            if (use_table) {
                c = sm.table[head];
            } else {
                int rr;
                c = resolve_head(P.membership, P.reps, b, h, H, k, &c, &rr) ? c : -1;
            }
            const bool live = c >= 0;
            const size_t plane = (size_t)b * k + (live ? c : 0);
            float m = -INFINITY;
            if (live) {
                for (int x = lane; x < wk.tp; x += 32) m = fmaxf(m, __ldcg(&P.cmax[plane * wk.tp + x]));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            } else if (chunk == 0) {
                if (lane == 0) flag_bad_membership(P.hdr, b, h);
                for (int d = lane; d < D; d += 32) outp[(size_t)head * D + d] = from_float<T>(0.f);
            }
            float acc[G::EPV];
#pragma unroll
            for (int e = 0; e < G::EPV; ++e) acc[e] = 0.f;
            float lsum = 0.f;
            const float* srow = P.scores + plane * T_len;
            float sraw[G::PV];  // raw scores of the next tile, fetched one tile ahead
            auto fetch_scores = [&](int tile) {
                const int rows = tile_rows(tile);
#pragma unroll
                for (int u = 0; u < G::PV; ++u) {
                    const int r = u * 32 + lane;
                    sraw[u] = (live && r < rows) ? __ldcg(&srow[(size_t)tile * G::TR + r]) : -INFINITY;
                }
            };
            fetch_scores(chunk * wk.IV);
            for (int t = 0; t < wk.IV; ++t) {
                const int tile = chunk * wk.IV + t;
                const int rows = tile_rows(tile);
                float pv[G::PV];
#pragma unroll
                for (int u = 0; u < G::PV; ++u) {
                    pv[u] = sraw[u] == -INFINITY ? 0.f : expf(sraw[u] - m);
                    lsum += pv[u];
                }
                if (t + 1 < wk.IV) fetch_scores(tile + 1);
                const int n = wk.vseq(warp, j, t);
                const int slot = n % STAGES;
                if (ok) ok = __all_sync(0xffffffffu, seq_wait(&sm.seq[slot], n, abort_flag, &stall_c) &&
                                                         mbar_wait(ring.full(slot), (n / STAGES) & 1, abort_flag, &stall_c));
                if (ok && live && rows > 0 && !(P.debug & 1)) {
                    const unsigned char* data = sm.ring[slot];
                    if (rows == G::TR) {
#pragma unroll
                        for (int u = 0; u < G::PV; ++u) {
#pragma unroll
                            for (int i = 0; i < G::IT; ++i) {
                                const int r32 = i * G::RPW + sub;  // row within this block of 32
                                const float pr = __shfl_sync(0xffffffffu, pv[u], r32);
                                const uint4 raw = *reinterpret_cast<const uint4*>(data + (u * 32 + r32) * G::ROW_BYTES + part * 16);
                                float vf[G::EPV];
                                Vec16<T>::unpack(raw, vf);
#pragma unroll
                                for (int e = 0; e < G::EPV; ++e) acc[e] = fmaf(pr, vf[e], acc[e]);
                            }
                        }
                    } else {
#pragma unroll
                        for (int u = 0; u < G::PV; ++u) {
#pragma unroll 4
                            for (int i = 0; i < G::IT; ++i) {
                                const int r32 = i * G::RPW + sub;
                                const float pr = __shfl_sync(0xffffffffu, pv[u], r32);
                                const int row = u * 32 + r32;
                                if (row < rows) {  // never touch stale bytes of a ragged last tile
                                    const uint4 raw = *reinterpret_cast<const uint4*>(data + row * G::ROW_BYTES + part * 16);
                                    float vf[G::EPV];
                                    Vec16<T>::unpack(raw, vf);
#pragma unroll
                                    for (int e = 0; e < G::EPV; ++e) acc[e] = fmaf(pr, vf[e], acc[e]);
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0 && ok) mbar_arrive(ring.empty(slot));
            }
            if (!live || !ok) continue;  // warp-uniform
            // fold the RPW row slots of the warp; lanes 0..LPR-1 then hold the head's D partial sums
#pragma unroll
            for (int o = G::LPR; o < 32; o <<= 1) {
#pragma unroll
                for (int e = 0; e < G::EPV; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
            float* op = P.opart + ((size_t)head * P.nVi + chunk) * D;
            if (lane < G::LPR) {
#pragma unroll
                for (int e = 0; e < G::EPV; e += 4)
                    *reinterpret_cast<float4*>(op + part * G::EPV + e) = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
            }
            if (lane == 0) P.lpart[(size_t)head * P.nVi + chunk] = lsum;
            __threadfence();
            __syncwarp();
            int ticket = 0;
            if (lane == 0) ticket = atomicAdd(&P.counters[head], 1);
            ticket = __shfl_sync(0xffffffffu, ticket, 0);
            if (ticket == P.nVi - 1) {  // this warp completed the head: add the partials in chunk order
                __threadfence();
                constexpr int DPL = D / 32;  // output columns per lane
                float o[DPL];
#pragma unroll
                for (int e = 0; e < DPL; ++e) o[e] = 0.f;
                float ll = 0.f;
                for (int i = 0; i < P.nVi; ++i) {
                    const float* src = P.opart + ((size_t)head * P.nVi + i) * D + lane * DPL;
#pragma unroll
                    for (int e = 0; e < DPL; ++e) o[e] += __ldcg(src + e);
                    ll += __ldcg(&P.lpart[(size_t)head * P.nVi + i]);
                }
#pragma unroll
                for (int e = 0; e < DPL; ++e) outp[(size_t)head * D + lane * DPL + e] = from_float<T>(o[e] / ll);
            }
        }
        if (cta == 0 && tid == 0) stats[7] = (unsigned long long)stall_c;
    }
    if (cta == 0 && tid == 0) stats[3] = global_ns();
    __syncthreads();
    if (tid == 0 && cta < 1024) g_cta_stats[cta][3] = global_ns();
    if (tid == 0 && sm.abort_flag) atomicExch(&P.hdr->status, CHAI_ERR_TIMEOUT);
}

struct DeviceInfo {
    int sms = 0;
    int coop = 0;
    bool ready = false;
};

static DeviceInfo& device_info(int dev) {
    static DeviceInfo info[64];
    DeviceInfo& d = info[dev & 63];
    if (!d.ready) {
        cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&d.coop, cudaDevAttrCooperativeLaunch, dev);
        d.ready = true;
    }
    return d;
}

template <typename T, int D>
static int launch(const Params& P0, int ncta, int dev, cudaStream_t s) {
    Params P = P0;
    const size_t smem = sizeof(Smem) + 128;
    static bool configured_dev[64] = {};
    bool& configured = configured_dev[dev & 63];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(decode_persistent_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return cuda_fail(e, "decode_persistent_kernel shared-memory opt-in");
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_persistent_kernel<T, D>, THREADS, smem);
        if (e != cudaSuccess) return cuda_fail(e, "decode_persistent_kernel occupancy query");
        if (per_sm < 1) return kDecodeNotLaunched;
        configured = true;
    }
    void* args[] = {&P};
    cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(decode_persistent_kernel<T, D>), dim3(ncta),
                                                dim3(THREADS), args, smem, s);
    if (e != cudaSuccess) return cuda_fail(e, "decode_persistent_kernel launch");
    return CHAI_OK;
}

}  // namespace pd

int launch_decode_persistent(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                             const int32_t* reps, void* out, int B, int H, int k, int T, int T_cap, int D, float scale,
                             int dtype, char* ws, const DecodeLayout& L, cudaStream_t s) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return kDecodeNotLaunched;
    const pd::DeviceInfo& info = pd::device_info(dev);
    if (!info.coop || info.sms <= 0) return kDecodeNotLaunched;
    const int ncta = info.sms;
    const int tiles = (T + L.TR - 1) / L.TR;
    pd::Params P;
    P.q = q; P.k_rep = k_rep; P.v = v; P.membership = membership; P.reps = reps; P.out = out;
    P.hdr = reinterpret_cast<WsHeader*>(ws);
    P.counters = reinterpret_cast<int*>(ws + L.off_counters);
    P.scores = reinterpret_cast<float*>(ws + L.off_scores);
    P.cmax = reinterpret_cast<float*>(ws + L.off_cmax);
    P.lpart = reinterpret_cast<float*>(ws + L.off_lpart);
    P.opart = reinterpret_cast<float*>(ws + L.off_opart);
    P.B = B; P.H = H; P.k = k; P.T = T; P.T_cap = T_cap;
    // key work is dealt tile by tile; value items are runs of 4 tiles of one head (one consumer warp each)
    P.IK = 1;
    P.IV = tiles < 4 ? tiles : 4;
    P.nKi = tiles;
    P.nVi = (tiles + P.IV - 1) / P.IV;
    P.scale = scale;
    {
        static const int dbg = [] {
            const char* e = getenv("CHAI_DECODE_DEBUG");
            return e ? atoi(e) : 0;
        }();
        P.debug = dbg;
    }
    if (P.nKi > L.capK || P.nVi > L.capV) return kDecodeNotLaunched;
    if (dtype == CHAI_BF16) {
        if (D == 128) return pd::launch<__nv_bfloat16, 128>(P, ncta, dev, s);
        return pd::launch<__nv_bfloat16, 64>(P, ncta, dev, s);
    }
    if (D == 128) return pd::launch<float, 128>(P, ncta, dev, s);
    return pd::launch<float, 64>(P, ncta, dev, s);
}

}  // namespace chai

// Debugging aid (not part of the public interface): per-CTA phase timestamps of the last persistent launch.
extern "C" int chai_debug_decode_stats(unsigned long long* host_out, int n_ctas) {
    if (host_out == nullptr || n_ctas <= 0 || n_ctas > 1024) return CHAI_ERR_INVALID_ARG;
    cudaError_t e = cudaMemcpyFromSymbol(host_out, chai::pd::g_cta_stats, sizeof(unsigned long long) * 4 * n_ctas);
    return e == cudaSuccess ? CHAI_OK : chai::cuda_fail(e, "chai_debug_decode_stats");
}
