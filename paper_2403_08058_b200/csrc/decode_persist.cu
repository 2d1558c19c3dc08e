// Clustered decode attention, persistent streaming kernel (Fig. 3(b), Section 3.4).
//
// One CTA per SM (cooperative launch, for co-residency only).  The last warp is the producer: it streams
// cache rows, tile by tile, into a shared-memory ring with bulk async copies that complete on mbarriers, and
// runs ahead of the consumers by the depth of the ring, so HBM stays busy while a consumer does the serial
// part of a tile.  The other warps consume, each on its own: a free warp takes the next ring position (an
// atomic counter in shared memory), reads what the position holds from the slot's description and works on
// it; nothing else is synchronised across the warps of a CTA except item completion.
//
//   phase K   unit = one key tile (TR rows of one cluster's K_rep), dealt round-robin over CTAs: scaled
//             scores s_t -> workspace (fp32, stays in L2), the tile's maximum, then an arrival on the plane's
//             tile counter; the warp whose arrival completes a plane reduces the tile maxima to the plane's
//             largest score and sets the plane's flag word to this launch's token.  Every K_rep row is read
//             exactly once.
//   phase V   unit = item (request, head, run of IV value tiles), claimed by the producers from an atomic
//             counter, so fast SMs take more.  A tile waits (almost never in practice: planes complete in
//             request order) until the flag of its cluster's plane carries the token, takes the plane's
//             largest score, forms p_t = exp(s_t - max) and reduces its rows; the warp that finishes an
//             item's last tile adds the tile partials in tile order and publishes (sum p_t V_t, sum p_t);
//             the warp that completes a head's last item (atomic ticket, nobody waits) adds the item
//             partials in chunk order and writes out = sum / l.
//
// There is no grid-wide barrier and no state that must be cleared between launches: flags compare
// against a token that never repeats, and the few words that must start at zero (work counter, status,
// tickets) are reset by the warps that own the first key tile of the layer / of a plane, before their
// flags go up.  The softmax is the exact two-pass form; all sums are taken in a fixed order, so results
// are bitwise repeatable whatever the schedule.  Every wait is bounded; on expiry the CTA records
// CHAI_ERR_TIMEOUT, stops consuming and returns.
#include <type_traits>
#include <stdlib.h>

#include <atomic>
#include <chrono>

#include "decode_layout.cuh"

namespace chai {
namespace pd {

// Shape of the pipeline per cache element type: W consumer warps (+ 1 producer warp), a ring of STAGES slots
// of TILE bytes.  A slot is held while its tile is in flight AND while a warp works on it, so at most STAGES
// warps are busy at once.  For one-byte elements the per-element work (conversion, fused multiply-adds) is what
// limits the kernel, not the bytes: tiles keep the element count of the two-byte case (half the bytes), and more
// slots and more warps work side by side.
template <typename T>
struct Cfg {
    static constexpr int W = 12, STAGES = 6, TILE = kTileBytes;      // 192 KB of cache rows in flight per SM; 12 consumer warps
};
template <>
struct Cfg<Fp8E4M3> {
    static constexpr int W = 16, STAGES = 12, TILE = kTileBytesFp8;  // 192 KB in 12 slots, 16 consumer warps
};
constexpr int MAX_IV = 4;                  // tiles per value item
constexpr int ITEM_SLOTS = 8;              // value items whose tile partials may be open in one CTA
constexpr int TABLE_CAP = 2048;            // heads whose cluster id is cached in shared memory
constexpr int RAG_CAP = 1024;              // requests whose tile and item counts are kept in shared memory (ragged batches)
// groups a head's n items are first added in (1 = all at once)
__host__ __device__ inline int combine_groups(int n) { return n > 4 * kCombineGroup ? (n + kCombineGroup - 1) / kCombineGroup : 1; }
constexpr int LATE_ITEMS = 2;              // the last LATE_ITEMS items per CTA are claimed only when the producer is free
constexpr long long TIMEOUT_CYCLES = kDefaultWaitLimitCycles;  // bound of the final wait for copies in flight

// Shared by all waiting threads of a CTA: set when some wait ran out (everybody then stops), and the limit in
// cycles that the launch was given.  Waits receive a pointer to abort_flag and find the limit behind it.
struct alignas(8) WaitCtl {
    int abort_flag;
    int reserved;
    long long limit;
};
__device__ __forceinline__ long long wait_limit(const volatile int* abort_flag) {
    return reinterpret_cast<const volatile WaitCtl*>(abort_flag)->limit;
}

struct TileMeta {
    int item;      // value item id (phase V), -1: end of work for the warp that owns this ring position
    int t;         // tile index within the item
    int ntiles;    // real tiles of the item
    int islot;     // shared-memory slot of the item's tile partials
};

template <int STAGES, int TILE>
struct Smem {
    alignas(128) unsigned char ring[STAGES][TILE];
    alignas(16) float part[ITEM_SLOTS][MAX_IV][128];  // per-tile partial sums of open items
    float lpart[ITEM_SLOTS][MAX_IV];
    alignas(8) unsigned long long full[STAGES];
    unsigned long long empty[STAGES];
    TileMeta meta[STAGES];
    int seq[STAGES];            // sequence number of the tile most recently issued into each slot
    int item_cnt[ITEM_SLOTS];   // tiles of the open item finished so far
    int item_free[ITEM_SLOTS];  // 1 when the slot may be given to a new item
    int table[TABLE_CAP];
    unsigned ready[TABLE_CAP / 32];  // bit p: every key tile of plane p is known to carry this launch's token
    int tpre[RAG_CAP + 1];      // ragged batches: key tiles (per plane) of the requests before b, summed ...
    int ipre[RAG_CAP + 1];      // ... and value items (per head): work is dealt over what really exists
    WaitCtl wait;
    int next_pos;               // next ring position a consumer warp may take
    unsigned epoch;             // launch count of this workspace, read once at start
};

struct Params {
    const void* q;
    const void* k_rep;
    const void* v;
    const int32_t* membership;
    const int32_t* reps;
    const float* k_scale;        // fp8 caches: scale of each representative key plane [B,k] / value plane [B,H]
    const float* v_scale;
    const int32_t* seq_lens;     // per-request context length, or null (all T)
    size_t k_batch_bytes;        // bytes between two requests' representative planes in k_rep
    void* out;
    WsHeader* hdr;
    int* counters;               // tickets, one per head
    int* gcnt;                   // tickets of the groups of kCombineGroup items, capG per head
    int capG;
    unsigned long long* flags;   // [0]: the layer's first key tile is done
    unsigned long long* pflag;   // per key plane: all its tiles are done and pmax holds its largest score
    unsigned long long* pcnt;    // per key plane: finished tiles of this launch (launch tag in the upper bits)
    float* pmax;
    unsigned long long token;    // value unique to this launch (never seen in the flags before)
    float* scores;
    float* cmax;
    float* lpart;
    float* opart;
    int B, H, k, T, T_cap;
    int IV, nVi;                 // tiles per value item, items per head
    float scale;
    long long wait_limit;        // cycles after which a device-side wait gives up
    // CHAI-QKV (values of non-representative heads dropped too): the kernel's heads are the k clusters themselves
    // (H = k, v = the representatives' value planes), `reps` still names each cluster's representative among the
    // Hq heads that q and out have, and a cluster's output row is written to every head that out_membership [B,Hq]
    // assigns to it.  Null: the ordinary case, Hq = H and every head writes its own row.
    const int32_t* out_membership;
    int Hq;
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > wait_limit(abort_flag)) {
            *abort_flag = 1;
            return false;
        }
    }
}
// Bounded wait on a shared-memory word (slot tags, item-slot hand-back).
__device__ __forceinline__ bool word_wait(const int* word, int want, volatile int* abort_flag) {
    const volatile int* w = word;
    if (*w == want) return true;
    const long long t0 = clock64();
    while (true) {
        if (*w == want) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > wait_limit(abort_flag)) {
            *abort_flag = 1;
            return false;
        }
    }
}
// Flag words carry the token of the launch that wrote them.  Tokens come from a host-side counter that
// never repeats, so whatever earlier launches (or the allocator) left in a flag word cannot be mistaken
// for "ready".  Bounded wait by ONE thread for one flag ...
__device__ __forceinline__ bool flag_wait_one(const unsigned long long* flag, unsigned long long token,
                                              volatile int* abort_flag) {
    long long t0 = 0;
    bool first = true;
    while (true) {
        unsigned long long v;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(flag) : "memory");
        if (v == token) return true;
        if (first) {
            t0 = clock64();
            first = false;
        }
        if (*abort_flag) return false;
        if (clock64() - t0 > wait_limit(abort_flag)) {
            *abort_flag = 1;
            return false;
        }
        __nanosleep(100);
    }
}
// A key tile of a plane is done: returns how many of the plane's tiles are done now, this one included.  The
// counter word holds a tag of the launch (40 bits of its token) above a 24-bit count, so whatever an earlier
// launch or the allocator left there is recognised and replaced by the first arriver; after that every arrival
// is one atomic add.  The adds are acquire-release: the arriver that completes the plane has all the other
// tiles' scores and maxima visible.
__device__ __forceinline__ unsigned long long plane_peek(const unsigned long long* cnt) {
    unsigned long long cur;  // (issued early, while the tile's bytes are still on their way)
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(cur) : "l"(cnt) : "memory");
    return cur;
}
__device__ __forceinline__ unsigned plane_arrive(unsigned long long* cnt, unsigned long long token, unsigned long long cur) {
    const unsigned long long tag = (token ^ (token >> 24)) << 24;  // epoch and host counter both reach the upper 40 bits
    if ((cur >> 24) != (tag >> 24)) atomicCAS(cnt, cur, tag);  // stale word: one arriver installs this launch's tag
    unsigned long long prev;
    asm volatile("atom.acq_rel.gpu.global.add.u64 %0, [%1], 1;" : "=l"(prev) : "l"(cnt) : "memory");
    return (unsigned)(prev & 0xffffffull) + 1u;
}
// A ticket: an acquire-release increment by one lane.  Release: what the warp's lanes wrote before the __syncwarp()
// that precedes the call is visible to whoever draws a later ticket; acquire: what earlier ticket holders published
// is visible to this warp once the ticket has been passed round by a shuffle.  One instruction instead of a
// device-wide fence (a round trip of its own) before and after a plain atomic.
__device__ __forceinline__ unsigned ld_acquire_cta_shared(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"((unsigned)__cvta_generic_to_shared(p)) : "memory");
    return v;
}
__device__ __forceinline__ void or_release_cta_shared(unsigned* p, unsigned bits) {
    asm volatile("red.release.cta.shared.or.b32 [%0], %1;" ::"r"((unsigned)__cvta_generic_to_shared(p)), "r"(bits) : "memory");
}
__device__ __forceinline__ int ticket_acq_rel(int* counter) {
    int prev;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(prev) : "l"(counter) : "memory");
    return prev;
}
// ... and by a whole warp for `n` consecutive flags.
__device__ __forceinline__ bool flags_wait(const unsigned long long* flags, int n, unsigned long long token, int lane,
                                           volatile int* abort_flag) {
    long long t0 = 0;
    bool first = true;
    while (true) {
        bool all = true;
        for (int i = lane; i < n; i += 32) {
            unsigned long long v;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(flags + i) : "memory");
            all = all && (v == token);
        }
        if (__all_sync(0xffffffffu, all)) return true;
        if (first) {
            t0 = clock64();
            first = false;
        }
        const bool give_up = *abort_flag != 0 || clock64() - t0 > wait_limit(abort_flag);
        if (__any_sync(0xffffffffu, give_up)) {
            *abort_flag = 1;
            return false;
        }
        __nanosleep(100);
    }
}
// 1-D bulk async copy global -> shared, completion counted in bytes on an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

template <typename T, int D>
struct Geom {
    static constexpr int kTileBytes = Cfg<T>::TILE;
    static constexpr int EPV = 16 / (int)sizeof(T);   // elements per 16-byte vector
    static constexpr int ROW_BYTES = D * (int)sizeof(T);
    static constexpr int TR = kTileBytes / ROW_BYTES;  // rows per tile
    static constexpr int LPR = ROW_BYTES / 16;         // lanes per row
    static constexpr int RPW = 32 / LPR;               // rows per warp-wide load
    static constexpr int PV = TR / 32;                 // probabilities per lane per tile
    static constexpr int IT = 32 / RPW;                // warp-wide loads per 32 rows
    static_assert(TR % 32 == 0 && PV >= 1, "a tile is a whole number of 32-row blocks");
};

struct Ring {
    uint32_t full0, empty0, data0, tile_bytes;
    __device__ __forceinline__ uint32_t full(int slot) const { return full0 + 8 * slot; }
    __device__ __forceinline__ uint32_t empty(int slot) const { return empty0 + 8 * slot; }
    __device__ __forceinline__ uint32_t data(int slot) const { return data0 + tile_bytes * slot; }
};

// RAGGED = false is the equal-length, dense-cache case: per-request lengths, the K batch stride and the
// skipping of tiles beyond a request's end compile away (the streaming loops are sensitive to every
// instruction on the producer thread and in the per-tile consumer chain).
// T = element type of the caches, TQ = element type of the queries and the output (they differ for fp8 caches).
// Long contexts.  A head with hundreds of value items would have its item partials added by one warp in one go: a
// long chain of dependent L2 round trips (measured: 58 us of a 227 us call at T = 131072, H = 32).  Instead the
// items are added in groups of kCombineGroup by whichever warp completes a group (tickets, nobody waits; the
// group's sum replaces its first item's partial), and the warp that completes the head's last group adds the
// group sums: a fixed tree, so the result does not depend on who adds what.  Called by a whole warp that has
// just published item `chunk` of `head`; `done` is set in the warp that completed the head, with the head's
// sums (lane l holds columns l * DPL ..).  Kept out of line: the short-context path stays as it was.
template <int DPL>
struct GroupedSum {
    float o[DPL];
    float l;
    bool done;
};
template <int D>
__device__ __noinline__ GroupedSum<D / 32> combine_grouped(float* opart, float* lpart, int* gcnt, int* counters, int nVi,
                                                           int capG, int head, int chunk, int n_chunks, int lane) {
    constexpr int DPL = D / 32;
    GroupedSum<DPL> r;
    r.done = false;
    r.l = 0.f;
#pragma unroll
    for (int e = 0; e < DPL; ++e) r.o[e] = 0.f;
    const float* src = opart + (size_t)head * nVi * D + lane * DPL;
    const float* lsrc = lpart + (size_t)head * nVi;
    // adds `count` partials, `stride` slots apart, starting at slot `first`, in order, eight loads in flight
    auto add_partials = [&](int first, int count, int stride) {
#pragma unroll
        for (int e = 0; e < DPL; ++e) r.o[e] = 0.f;
        r.l = 0.f;
        int i = 0;
        for (; i + 8 <= count; i += 8) {
            float t8[8][DPL], l8[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const size_t slot = (size_t)first + (size_t)(i + u) * stride;
#pragma unroll
                for (int e = 0; e < DPL; ++e) t8[u][e] = __ldcg(src + slot * D + e);
                l8[u] = __ldcg(lsrc + slot);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
#pragma unroll
                for (int e = 0; e < DPL; ++e) r.o[e] += t8[u][e];
                r.l += l8[u];
            }
        }
        for (; i < count; ++i) {
            const size_t slot = (size_t)first + (size_t)i * stride;
#pragma unroll
            for (int e = 0; e < DPL; ++e) r.o[e] += __ldcg(src + slot * D + e);
            r.l += __ldcg(lsrc + slot);
        }
    };
    const int n_groups = combine_groups(n_chunks);
    const int grp = chunk / kCombineGroup;
    const int in_grp = min(kCombineGroup, n_chunks - grp * kCombineGroup);
    int ticket = 0;
    if (lane == 0) ticket = ticket_acq_rel(&gcnt[(size_t)head * capG + grp]);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    __syncwarp();  // what lane 0 acquired with the ticket is ordered before the other lanes' reads of the partials
    if (ticket != in_grp - 1) return r;
    add_partials(grp * kCombineGroup, in_grp, 1);
    float* gp = opart + ((size_t)head * nVi + (size_t)grp * kCombineGroup) * D;
#pragma unroll
    for (int e = 0; e < DPL; ++e) gp[lane * DPL + e] = r.o[e];
    if (lane == 0) lpart[(size_t)head * nVi + (size_t)grp * kCombineGroup] = r.l;
    __syncwarp();
    if (lane == 0) ticket = ticket_acq_rel(&counters[head]);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    __syncwarp();
    if (ticket != n_groups - 1) return r;
    add_partials(0, n_groups, kCombineGroup);
    r.done = true;
    return r;
}

template <typename T, typename TQ, int D, bool RAGGED>
__global__ void __launch_bounds__(Cfg<T>::W * 32 + 32, 1) decode_persistent_kernel(const Params P) {
    using G = Geom<T, D>;
    constexpr int W = Cfg<T>::W, STAGES = Cfg<T>::STAGES, THREADS = W * 32 + 32;
    using SmemT = Smem<STAGES, Cfg<T>::TILE>;
    extern __shared__ unsigned char smem_raw[];
    SmemT& sm = *reinterpret_cast<SmemT*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, ncta = gridDim.x;
    volatile int* abort_flag = &sm.wait.abort_flag;
    const Ring ring{smem_u32(&sm.full[0]), smem_u32(&sm.empty[0]), smem_u32(&sm.ring[0][0]), (uint32_t)Cfg<T>::TILE};
    const int B = P.B, H = P.H, k = P.k, T_len = P.T;
    const bool use_table = B * H <= TABLE_CAP;
    const int tp = (T_len + G::TR - 1) / G::TR;          // tiles per cache plane
    const long long n_ktiles = (long long)B * k * tp;    // key tiles of the layer
    const int nkt = n_ktiles > cta ? (int)((n_ktiles - cta + ncta - 1) / ncta) : 0;  // this CTA's share
    const int n_items_full = B * H * P.nVi;              // value items of the layer when every request has all T rows
    int* work_counter = &P.hdr->pad[0];
    int* launch_epoch = &P.hdr->pad[8];

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(ring.full(s), 1);
            mbar_init(ring.empty(s), 1);
            sm.seq[s] = -1;
        }
        for (int s = 0; s < ITEM_SLOTS; ++s) {
            sm.item_cnt[s] = 0;
            sm.item_free[s] = 1;
        }
        for (int i = 0; i < TABLE_CAP / 32; ++i) sm.ready[i] = 0;
        sm.wait.abort_flag = 0;
        sm.wait.limit = P.wait_limit;
        sm.next_pos = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // Launched as a programmatic dependent, the kernel gets here while its predecessor in the stream may still
    // be running: let our own dependents be scheduled, then wait for the predecessor to complete before the
    // first access to global memory (inputs, workspace, launch count).  Both are no-ops otherwise.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (tid == 0) sm.epoch = *reinterpret_cast<volatile unsigned*>(&P.hdr->pad[8]);
    const bool qkv = P.out_membership != nullptr;
    // head -> cluster, or -1.  CHAI-QKV: head c of request b is cluster c, usable when its representative is one
    // of the Hq heads and belongs to it.
    auto resolve_cluster = [&](int b, int h) -> int {
        if (qkv) {
            const int r = P.reps[(size_t)b * k + h];
            return (r >= 0 && r < P.Hq && P.out_membership[(size_t)b * P.Hq + r] == h) ? h : -1;
        }
        int c, r;
        return resolve_head(P.membership, P.reps, b, h, H, k, &c, &r) ? c : -1;
    };
    if (use_table) {
        for (int i = tid; i < B * H; i += THREADS) sm.table[i] = resolve_cluster(i / H, i % H);
    }
    // A ragged batch is dealt by what it really holds: with the running sums of every request's key tiles and value
    // items in shared memory, the producer walks (or claims) positions in the list of existing tiles and items, so
    // that neither a ring position nor a claim is spent on a tile beyond a request's end and every CTA gets the
    // same number of real key tiles.  (More than RAG_CAP requests: the positions are those of the full-length
    // batch and the missing ones are skipped.)
    const bool dealt_by_length = RAGGED && B <= RAG_CAP;
    if (dealt_by_length) {
        const int tr = G::TR;
        for (int b = tid; b < B; b += THREADS) {
            const int len = P.seq_lens ? min(max(__ldg(P.seq_lens + b), 0), T_len) : T_len;
            const int t = max(1, (len + tr - 1) / tr);
            sm.tpre[b + 1] = t;
            sm.ipre[b + 1] = (t + P.IV - 1) / P.IV;
        }
        __syncthreads();
        if (warp == 0) {  // inclusive scans, 32 requests at a time
            int tc = 0, ic = 0;
            for (int b0 = 0; b0 < B; b0 += 32) {
                const int b = b0 + lane;
                int tv = b < B ? sm.tpre[b + 1] : 0, iv = b < B ? sm.ipre[b + 1] : 0;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int tu = __shfl_up_sync(0xffffffffu, tv, o), iu = __shfl_up_sync(0xffffffffu, iv, o);
                    if (lane >= o) {
                        tv += tu;
                        iv += iu;
                    }
                }
                if (b < B) {
                    sm.tpre[b + 1] = tc + tv;
                    sm.ipre[b + 1] = ic + iv;
                }
                tc += __shfl_sync(0xffffffffu, tv, 31);
                ic += __shfl_sync(0xffffffffu, iv, 31);
            }
            if (lane == 0) sm.tpre[0] = sm.ipre[0] = 0;
        }
    }
    __syncthreads();
    // Token of this launch: the workspace's launch count (bumped once per launch, below) in the high word, a
    // host-side value in the low word.  It differs from the token of every earlier launch on this workspace --
    // also when the launch is a replay of a captured graph, whose kernel arguments never change -- so flag
    // words left by earlier launches cannot look ready.
    const unsigned long long token = ((unsigned long long)sm.epoch << 32) | (P.token & 0xffffffffull);
    auto cluster_of = [&](int b, int h) -> int {
        if (use_table) return sm.table[b * H + h];
        return resolve_cluster(b, h);
    };
    // A finished head's output row (lane l holds columns l * DPL ..).  CHAI-QKV: the row goes to every head of the
    // cluster, found by walking the request's membership.
    auto store_row = [&](int head, const float* vals) {
        constexpr int DPL = D / 32;
        TQ* outp = static_cast<TQ*>(P.out);
        if (!qkv) {
#pragma unroll
            for (int e = 0; e < DPL; ++e) outp[(size_t)head * D + lane * DPL + e] = from_float<TQ>(vals[e]);
            return;
        }
        const int b = head / H, c = head % H;
        const int32_t* mem = P.out_membership + (size_t)b * P.Hq;
        for (int h = 0; h < P.Hq; ++h)
            if (__ldg(mem + h) == c) {
#pragma unroll
                for (int e = 0; e < DPL; ++e) outp[((size_t)b * P.Hq + h) * D + lane * DPL + e] = from_float<TQ>(vals[e]);
            }
    };
    // rows of request b's tile: requests shorter than T leave whole tiles empty (they pass through the ring as
    // markers without data and contribute nothing)
    auto len_of = [&](int b) {
        if constexpr (RAGGED) return P.seq_lens ? min(max(__ldg(P.seq_lens + b), 0), T_len) : T_len;
        return T_len;
    };
    auto tile_rows = [&](int b, int tile) { return max(0, min(G::TR, len_of(b) - tile * G::TR)); };
    // Tiles that hold cached rows of request b (tile 0 always counts, so that an empty request still runs
    // through the bookkeeping once), and the value items (runs of IV tiles) they make.  Tiles and items
    // beyond these are skipped by the producer and the consumers alike: they never enter the ring.
    auto tiles_of = [&](int b) {
        if constexpr (RAGGED) return max(1, (len_of(b) + G::TR - 1) / G::TR);
        return tp;
    };
    auto items_of = [&](int b) {
        if constexpr (RAGGED) return (tiles_of(b) + P.IV - 1) / P.IV;
        return P.nVi;
    };
    const unsigned char* kc = static_cast<const unsigned char*>(P.k_rep);
    const unsigned char* vc = static_cast<const unsigned char*>(P.v);

    if (warp == W) {
        // ------------------------------ producer (one thread) ------------------------------
        // Tiles are issued in ring order (ascending sequence number): that keeps the one-bit phase parity
        // of the slot barriers unambiguous on this side.  Consumer warps run independently and bulk copies
        // complete out of order, so a consumer may reach a slot while the previous occupant's copy is
        // still in flight; the parity of the full barrier cannot tell those two fills apart, the slot's
        // sequence tag can: a consumer waits for its own sequence number in the tag (the previous occupant
        // has then been consumed, hence its phase completed) before it waits on the barrier.
        if (lane == 0) {
            int n = 0, slot = 0;
            uint32_t parity = 1;  // parity to wait for on empty[slot]: ((n / STAGES) & 1) ^ 1
            bool ok = true;
            auto issue = [&](const unsigned char* src, uint32_t bytes, const TileMeta& m) -> bool {
                if (!mbar_wait(ring.empty(slot), parity, abort_flag)) return false;
                sm.meta[slot] = m;
                __threadfence_block();
                *reinterpret_cast<volatile int*>(&sm.seq[slot]) = n;
                if (bytes > 0) {
                    mbar_expect_tx(ring.full(slot), bytes);
                    bulk_load(ring.data(slot), src, bytes, ring.full(slot));
                } else {
                    mbar_arrive(ring.full(slot));  // marker without data
                }
                ++n;
                if (++slot == STAGES) {
                    slot = 0;
                    parity ^= 1u;
                }
                return true;
            };
            // ---- key tiles: global tile ids cta, cta + ncta, ... ----
            if (dealt_by_length) {
                // positions cta, cta + ncta, ... in the list of the key tiles that exist, ordered by (request,
                // cluster, tile); positions only grow, so the request is found by walking forward
                const long long total = (long long)k * sm.tpre[B];
                int b = 0;
                for (long long r = cta; r < total && ok; r += ncta) {
                    while ((long long)k * sm.tpre[b + 1] <= r) ++b;
                    const int tb = sm.tpre[b + 1] - sm.tpre[b];
                    const int rem = (int)(r - (long long)k * sm.tpre[b]);
                    const int c = rem / tb, tile = rem - c * tb;
                    const TileMeta m{(int)(((long long)b * k + c) * tp + tile), -1, 0, 0};  // (the id consumers decode)
                    ok = issue(kc + (size_t)b * P.k_batch_bytes + ((size_t)c * P.T_cap + (size_t)tile * G::TR) * G::ROW_BYTES,
                               (uint32_t)tile_rows(b, tile) * G::ROW_BYTES, m);
                }
            } else {
                int plane = cta / tp, tile = cta % tp;
                const int dplane = ncta / tp, dtile = ncta % tp;
                constexpr bool plain = !RAGGED;
                for (int t = 0; t < nkt && ok; ++t) {
                    const TileMeta m{(int)(cta + (long long)t * ncta), -1, 0, 0};  // key tile: global tile id, t = -1
                    if constexpr (plain) {  // equal lengths, dense cache: no per-tile division on this (single) thread
                        ok = issue(kc + ((size_t)plane * P.T_cap + (size_t)tile * G::TR) * G::ROW_BYTES,
                                   (uint32_t)tile_rows(0, tile) * G::ROW_BYTES, m);
                    } else {
                        const int b = plane / k, c = plane - b * k;
                        if (tile < tiles_of(b))
                            ok = issue(kc + (size_t)b * P.k_batch_bytes + ((size_t)c * P.T_cap + (size_t)tile * G::TR) * G::ROW_BYTES,
                                       (uint32_t)tile_rows(b, tile) * G::ROW_BYTES, m);
                    }
                    plane += dplane;
                    tile += dtile;
                    if (tile >= tp) {
                        tile -= tp;
                        ++plane;
                    }
                }
            }
            // ---- value items, claimed one at a time; the next claim is in flight while this item streams ----
            // (the work counter is reset by the owner of the layer's first key tile before that tile's flag)
            if (ok) ok = flag_wait_one(P.flags, token, abort_flag);
            int n_open = 0;  // items this CTA has opened (item slots are handed out round-robin)
            // what is claimed: positions in the list of items -- of the items that exist, ordered by (request,
            // head, chunk), when the batch is dealt by length; of the full-length batch's items otherwise
            const int n_items = dealt_by_length ? H * sm.ipre[B] : n_items_full;
            int b_walk = 0;  // (claims only grow: the request of a position is found by walking forward)
            int next = ok ? atomicAdd(work_counter, 1) : n_items;
            while (ok && next < n_items) {
                const int pos = next;
                // The next claim is fetched while this item streams -- except near the end of the item list,
                // where a claimed but unstarted item on a slow SM is work a faster one could have taken.
                const bool ahead = pos < n_items - LATE_ITEMS * ncta;
                if (ahead) next = atomicAdd(work_counter, 1);
                int head, chunk;
                if (dealt_by_length) {
                    while (H * sm.ipre[b_walk + 1] <= pos) ++b_walk;
                    const int ib = sm.ipre[b_walk + 1] - sm.ipre[b_walk];
                    const int rem = pos - H * sm.ipre[b_walk];
                    const int h = rem / ib;
                    head = b_walk * H + h;
                    chunk = rem - h * ib;
                } else {
                    head = pos / P.nVi;
                    chunk = pos % P.nVi;
                }
                const int item = head * P.nVi + chunk;  // the id consumers decode
                const int tile0 = chunk * P.IV;
                const int b_item = RAGGED ? head / H : 0;
                const int ntiles = min(P.IV, tiles_of(b_item) - tile0);
                if (RAGGED && ntiles <= 0) {  // the request is shorter: this item does not exist
                    if (!ahead) next = atomicAdd(work_counter, 1);
                    continue;
                }
                const int islot = n_open % ITEM_SLOTS;
                ++n_open;
                ok = word_wait(&sm.item_free[islot], 1, abort_flag);  // the slot's previous item is fully reduced
                if (!ok) break;
                *reinterpret_cast<volatile int*>(&sm.item_free[islot]) = 0;
                for (int t = 0; t < ntiles && ok; ++t) {
                    const int tile = tile0 + t;
                    const TileMeta m{item, t, ntiles, islot};
                    ok = issue(vc + ((size_t)head * P.T_cap + (size_t)tile * G::TR) * G::ROW_BYTES,
                               (uint32_t)tile_rows(b_item, tile) * G::ROW_BYTES, m);
                }
                if (!ahead) next = atomicAdd(work_counter, 1);
            }
            // The claim that comes back with the largest id is the last one of the launch: every CTA has started
            // (and read the launch count) by then, so the count can move on for the next launch.
            if (ok && next == n_items + ncta - 1) atomicAdd(launch_epoch, 1);
            // ---- one end marker per consumer warp ----
            const TileMeta end{-1, 0, 0, 0};
            for (int w = 0; w < W && ok; ++w) ok = issue(nullptr, 0, end);
            // If the launch gave up, the copies already issued into the ring may still be in flight and nobody will
            // wait for them: this thread does, for the latest fill of every slot (with the default limit, whatever
            // limit the launch was given), so that the CTA does not leave while its shared memory is written.
            if (!ok || *abort_flag) {
                for (int i = n > STAGES ? n - STAGES : 0; i < n; ++i) {
                    const uint32_t bar = ring.full(i % STAGES), par = (uint32_t)(i / STAGES) & 1u;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(bar, par) && clock64() - t0 < TIMEOUT_CYCLES) {
                    }
                }
            }
        }
    } else {
        // ------------------------------ consumers: every warp works alone ------------------------------
        const int sub = lane / G::LPR, part = lane % G::LPR;
        bool ok = true;
        // Ring positions are taken in order by whichever warp is free (a warp that is held up -- an item or head
        // to combine, a ticket to fetch -- does not keep a filled slot waiting).  What a position holds is in
        // its description: a key tile (t < 0, item = global tile id), a value tile, or an end marker.
        TQ* outp = static_cast<TQ*>(P.out);
        for (;;) {
            int n = 0;
            if (lane == 0) n = atomicAdd(&sm.next_pos, 1);
            n = __shfl_sync(0xffffffffu, n, 0);
            const int slot = n % STAGES;
            // The description is in place as soon as the slot's tag says so, before the tile's bytes have
            // arrived: whatever does not need the bytes (the query row of a key tile; scores, maxima and the
            // probabilities of a value tile) is fetched and formed while the bulk copy is still in flight.
            if (ok) ok = __all_sync(0xffffffffu, word_wait(&sm.seq[slot], n, abort_flag));
            if (!ok) break;
            __threadfence_block();  // the description was written before the tag: read it after the tag
            const TileMeta m = sm.meta[slot];
            if (m.item < 0) {  // end marker
                ok = __all_sync(0xffffffffu, mbar_wait(ring.full(slot), (n / STAGES) & 1, abort_flag));
                __syncwarp();
                if (lane == 0) mbar_arrive(ring.empty(slot));
                break;
            }
          if (m.t < 0) {
            // ---- key tile: TR scores and their maximum ----
            const long long g = m.item;
            const int plane = (int)(g / tp), tile = (int)(g % tp);
            const int b = plane / k;
            const int rows = tile_rows(b, tile);
            const int rep = P.reps[plane];
            const bool live = rep >= 0 && rep < P.Hq;  // unused cluster slot: the tile is drained, nothing computed
            float qf[G::EPV];
#pragma unroll
            for (int e = 0; e < G::EPV; ++e) qf[e] = 0.f;
            if (live) {
                // the EPV query elements that face this lane's 16-byte slice of a key row
                const TQ* qsrc = static_cast<const TQ*>(P.q) + ((size_t)b * P.Hq + rep) * D + part * G::EPV;
#pragma unroll
                for (int x = 0; x < G::EPV / Vec16<TQ>::N; ++x)
                    Vec16<TQ>::unpack(*reinterpret_cast<const uint4*>(qsrc + x * Vec16<TQ>::N), qf + x * Vec16<TQ>::N);
            }
            float kscale = P.k_scale ? P.scale * __ldg(P.k_scale + plane) : P.scale;  // fp8 keys carry a scale per plane
            // fp8 keys: as on the value side, the conversions to fp32 bound the path, so a lane's 16 products are
            // formed and summed as fp16 pairs.  The query slice is brought below 16 in size by a power of two
            // (exact; undone in the score's scale), so that eight products with e4m3 values (at most 448) cannot
            // overflow fp16.
            __half2 qh[8];
            if constexpr (std::is_same<T, Fp8E4M3>::value) {
                static_assert(G::EPV == 16, "sixteen fp8 values per lane and row");
                float qmax = 0.f;
#pragma unroll
                for (int e = 0; e < G::EPV; ++e) qmax = fmaxf(qmax, fabsf(qf[e]));
#pragma unroll
                for (int o = G::LPR / 2; o >= 1; o >>= 1) qmax = fmaxf(qmax, __shfl_xor_sync(0xffffffffu, qmax, o));
                float fac = 1.f;
                if (qmax > 16.f && qmax < INFINITY) {
                    int ex;
                    frexpf(qmax, &ex);          // qmax = m * 2^ex with m in [0.5, 1)
                    fac = ldexpf(1.f, 4 - ex);  // qmax * fac in [8, 16)
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) qh[j] = __floats2half2_rn(qf[2 * j] * fac, qf[2 * j + 1] * fac);
                kscale /= fac;
            }
            unsigned long long cnt_seen = 0;
            if (lane == 0) cnt_seen = plane_peek(P.pcnt + plane);
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(ring.full(slot), (n / STAGES) & 1, abort_flag));
            if (ok && live && rows == 0) {  // tile beyond this request's length: no scores, neutral maximum
                if (lane == 0) P.cmax[(size_t)plane * tp + tile] = -INFINITY;
            } else if (ok && live) {
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
                        if constexpr (std::is_same<T, Fp8E4M3>::value) {
                            __half2 kh[8];
                            Vec16<T>::unpack_h2(raw, kh);
                            __half2 s2 = __hmul2(qh[0], kh[0]);
#pragma unroll
                            for (int j = 1; j < 8; ++j) s2 = __hfma2(qh[j], kh[j], s2);
                            const float2 f = __half22float2(s2);
                            v[ii] = f.x + f.y;
                        } else {
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
                    const float sc = v[0] * kscale;
                    const int row = (bt * G::LPR + part) * G::RPW + sub;
                    if (row < rows) {  // rows past the end of a ragged last tile hold stale bytes
                        srow[row] = sc;
                        lmax = fmaxf(lmax, sc);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) lmax = fmaxf(lmax, __shfl_xor_sync(0xffffffffu, lmax, o));
                if (lane == 0) P.cmax[(size_t)plane * tp + tile] = lmax;
            }
            __syncwarp();
            if (lane == 0 && ok) mbar_arrive(ring.empty(slot));
            if (ok) {
                if (g == 0 && lane == 0) {  // first key tile of the layer: reset status and work counter before its flag
                    P.hdr->status = CHAI_OK;
                    P.hdr->bad_b = -1;
                    P.hdr->bad_h = -1;
                    *reinterpret_cast<volatile unsigned long long*>(&P.hdr->pad[kHdrLaunchToken]) = token;
                    *work_counter = 0;
                }
                // the warp that owns tile 0 of a plane also clears the tickets of the plane's heads: every value
                // tile of those heads waits until all of the plane's tiles are done, this one included
                if (tile == 0 && live) {
                    const int c = plane % k;
                    for (int h = lane; h < H; h += 32)
                        if (cluster_of(b, h) == c) {
                            P.counters[(size_t)b * H + h] = 0;
                            const int n_groups = combine_groups(items_of(b));
                            if (n_groups > 1)
                                for (int gq = 0; gq < n_groups; ++gq) P.gcnt[((size_t)b * H + h) * P.capG + gq] = 0;
                        }
                }
                __syncwarp();
                unsigned done = 0;
                if (lane == 0) {
                    if (g == 0) asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(P.flags), "l"(token) : "memory");
                    done = plane_arrive(P.pcnt + plane, token, cnt_seen);
                }
                done = __shfl_sync(0xffffffffu, done, 0);
                if (done == (unsigned)tiles_of(b)) {
                    // the plane's last tile: every tile's scores and maximum are visible (acquire in the arrival);
                    // reduce the tile maxima to the plane's largest score and publish the plane
                    const float* cm = P.cmax + (size_t)plane * tp;
                    const int nx = tiles_of(b);
                    float mx = -INFINITY;
                    if (live) {
                        int x = lane;
                        for (; x + 7 * 32 < nx; x += 8 * 32) {
                            float t8[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) t8[u] = __ldcg(cm + x + u * 32);
#pragma unroll
                            for (int u = 0; u < 8; ++u) mx = fmaxf(mx, t8[u]);
                        }
                        for (; x < nx; x += 32) mx = fmaxf(mx, __ldcg(cm + x));
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    }
                    if (lane == 0) {
                        P.pmax[plane] = mx;
                        asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(P.pflag + plane), "l"(token) : "memory");
                    }
                }
            }
            if (!ok) break;
            continue;
          }
            // ---- value tile of a claimed item ----
            const int head = m.item / P.nVi, chunk = m.item % P.nVi;
            const int b = head / H, h = head % H;
            const int tile = chunk * P.IV + m.t;
            const int rows = tile_rows(b, tile);
            const int c = cluster_of(b, h);
            const bool live = c >= 0;
            float acc[G::EPV];
#pragma unroll
            for (int e = 0; e < G::EPV; ++e) acc[e] = 0.f;
            float lsum = 0.f;
            float pv[G::PV];
            bool have_p = false;
            if (live) {
                const size_t plane = (size_t)b * k + c;
                // all scores of the plane must exist; once seen, remembered per CTA (planes complete in order, so
                // after the first tiles of phase V this is a shared-memory bit test)
                // (the bit is set with release and read with acquire order within the CTA, so a warp that relies on
                // another warp's wait is ordered after the scores that wait made visible)
                const bool cached = plane < TABLE_CAP && ((ld_acquire_cta_shared(&sm.ready[plane >> 5]) >> (plane & 31)) & 1u);
                if (!cached) {
                    ok = flags_wait(P.pflag + plane, 1, token, lane, abort_flag);
                    if (ok && lane == 0 && plane < TABLE_CAP) or_release_cta_shared(&sm.ready[plane >> 5], 1u << (plane & 31));
                }
                if (ok && rows > 0) {  // (the only tile of an empty request has no rows: it just passes the ticket on,
                                       //  which the flag wait above has ordered after the ticket's reset)
                    const float mx = __ldcg(P.pmax + plane);  // the plane's largest score
                    const float* srow = P.scores + plane * T_len + (size_t)tile * G::TR;
#pragma unroll
                    for (int u = 0; u < G::PV; ++u) {
                        const int r = u * 32 + lane;
                        pv[u] = r < rows ? __ldcg(&srow[r]) : -INFINITY;
                    }
#pragma unroll
                    for (int u = 0; u < G::PV; ++u) {
                        pv[u] = pv[u] == -INFINITY ? 0.f : expf(pv[u] - mx);
                        lsum += pv[u];
                    }
                    have_p = true;
                }
            } else if (chunk == 0 && m.t == 0) {
                // unresolved head: zero output, flagged after the status reset (ordered by the layer's first flag)
                ok = flags_wait(P.flags, 1, token, lane, abort_flag);
                if (!qkv) {
                    if (ok && lane == 0) flag_bad_membership(P.hdr, b, h);
                    for (int d = lane; d < D; d += 32) outp[(size_t)head * D + d] = from_float<TQ>(0.f);
                }
            }
            if (qkv && ok && chunk == 0 && m.t == 0) {
                // CHAI-QKV, once per (request, cluster): the heads that name an unusable cluster get zero rows and
                // are reported; cluster 0's item also takes the heads whose cluster id is out of range.
                if (!live || h == 0) ok = flags_wait(P.flags, 1, token, lane, abort_flag);  // after the status reset
                const int32_t* mem = P.out_membership + (size_t)b * P.Hq;
                for (int hh = 0; hh < P.Hq && ok; ++hh) {
                    const int cc = __ldg(mem + hh);
                    const bool mine = (!live && cc == h) || (h == 0 && (cc < 0 || cc >= k));
                    if (!mine) continue;
                    if (lane == 0) flag_bad_membership(P.hdr, b, hh);
                    for (int d = lane; d < D; d += 32) outp[((size_t)b * P.Hq + hh) * D + d] = from_float<TQ>(0.f);
                }
            }
            // now the tile's bytes
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(ring.full(slot), (n / STAGES) & 1, abort_flag));
            if (ok && have_p) {
                {
                    unsigned char* data = sm.ring[slot];
                    if (rows < G::TR) {
                        // Ragged last tile: the copy brought `rows` rows, the rest of the slot holds whatever it held
                        // before.  Those rows' probabilities are 0, but 0 x (bytes that decode to NaN or infinity) is
                        // not, so the warp clears them in shared memory and then runs the one loop every tile runs
                        // (a separate loop with a test per row, visited once per plane, cost several full tiles each
                        // time: 61 us instead of 52 for lengths of 1407 instead of 1408).  The slot's next fill is
                        // by the copy engine: its writes are ordered after these by the proxy fence.
                        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                        uint4* v16 = reinterpret_cast<uint4*>(data);
                        for (int idx = rows * (G::ROW_BYTES / 16) + lane; idx < G::TR * (G::ROW_BYTES / 16); idx += 32) v16[idx] = zero;
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                    if constexpr (std::is_same<T, Fp8E4M3>::value) {
                        // fp8 values: the per-element conversions to fp32 are what bounds this path, so the
                        // products are formed and summed as fp16 pairs (every e4m3 value is an fp16 value; a
                        // probability is at most 1 and an e4m3 value at most 448, so FLUSH of them cannot
                        // overflow) and join the fp32 sums every FLUSH rows.
                        constexpr int FLUSH = 8;
                        static_assert(G::EPV == 16, "sixteen fp8 values per lane and row");
                        __half2 hacc[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) hacc[j] = __float2half2_rn(0.f);
                        auto flush = [&]() {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float2 f = __half22float2(hacc[j]);
                                acc[2 * j] += f.x;
                                acc[2 * j + 1] += f.y;
                                hacc[j] = __float2half2_rn(0.f);
                            }
                        };
#pragma unroll
                        for (int u = 0; u < G::PV; ++u) {
#pragma unroll
                            for (int i = 0; i < G::IT; ++i) {
                                const int r32 = i * G::RPW + sub;
                                const float pr = __shfl_sync(0xffffffffu, pv[u], r32);
                                const int row = u * 32 + r32;
                                const uint4 raw = *reinterpret_cast<const uint4*>(data + row * G::ROW_BYTES + part * 16);
                                __half2 vh[8];
                                Vec16<T>::unpack_h2(raw, vh);
                                const __half2 ph = __float2half2_rn(pr);
#pragma unroll
                                for (int j = 0; j < 8; ++j) hacc[j] = __hfma2(ph, vh[j], hacc[j]);
                                if ((u * G::IT + i) % FLUSH == FLUSH - 1) flush();
                            }
                        }
                        if ((G::PV * G::IT) % FLUSH != 0) flush();
                    } else {
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
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(ring.empty(slot));  // the tile's bytes are no longer needed
            if (!ok) break;
            // fold the RPW row slots of the warp; lanes 0..LPR-1 then hold the tile's D partial sums
#pragma unroll
            for (int o = G::LPR; o < 32; o <<= 1) {
#pragma unroll
                for (int e = 0; e < G::EPV; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
            if (lane < G::LPR) {
#pragma unroll
                for (int e = 0; e < G::EPV; ++e) sm.part[m.islot][m.t][part * G::EPV + e] = acc[e];
            }
            if (lane == 0) sm.lpart[m.islot][m.t] = lsum;
            __threadfence_block();
            __syncwarp();
            int done = 0;
            if (lane == 0) done = atomicAdd(&sm.item_cnt[m.islot], 1);
            done = __shfl_sync(0xffffffffu, done, 0);
            if (done != m.ntiles - 1) continue;
            // this warp finished the item's last open tile: add the tile partials in tile order
            __threadfence_block();
            constexpr int DPL = D / 32;  // output columns per lane
            float o[DPL];
#pragma unroll
            for (int e = 0; e < DPL; ++e) o[e] = 0.f;
            float l = 0.f;
            for (int t = 0; t < m.ntiles; ++t) {
#pragma unroll
                for (int e = 0; e < DPL; ++e) o[e] += *reinterpret_cast<volatile float*>(&sm.part[m.islot][t][lane * DPL + e]);
                l += *reinterpret_cast<volatile float*>(&sm.lpart[m.islot][t]);
            }
            __syncwarp();
            if (lane == 0) {
                sm.item_cnt[m.islot] = 0;
                __threadfence_block();
                *reinterpret_cast<volatile int*>(&sm.item_free[m.islot]) = 1;  // hand the slot back to the producer
            }
            if (!live) continue;
            float* op = P.opart + ((size_t)head * P.nVi + chunk) * D;
#pragma unroll
            for (int e = 0; e < DPL; ++e) op[lane * DPL + e] = o[e];
            if (lane == 0) P.lpart[(size_t)head * P.nVi + chunk] = l;
            __syncwarp();  // (the ticket below is the release of these stores)
            const int n_chunks = items_of(b);  // items this head really has
            if (combine_groups(n_chunks) > 1) {  // long context: the items are added group by group (see combine_grouped)
                const GroupedSum<D / 32> gs = combine_grouped<D>(P.opart, P.lpart, P.gcnt, P.counters, P.nVi, P.capG, head, chunk, n_chunks, lane);
                if (gs.done) {
                    const float vscale = P.v_scale ? __ldg(P.v_scale + head) : 1.f;
                    float fin[D / 32];
#pragma unroll
                    for (int e = 0; e < D / 32; ++e) fin[e] = gs.l > 0.f ? gs.o[e] / gs.l * vscale : 0.f;
                    store_row(head, fin);
                }
                continue;
            }
            int ticket = 0;
            if (lane == 0) ticket = ticket_acq_rel(&P.counters[head]);
            ticket = __shfl_sync(0xffffffffu, ticket, 0);
            __syncwarp();  // (as above: lane 0's acquire comes before every lane's reads of the partials)
            if (ticket == n_chunks - 1) {  // this warp completed the head: add the item partials in chunk order
#pragma unroll
                for (int e = 0; e < DPL; ++e) o[e] = 0.f;
                float ll = 0.f;
                const float* src = P.opart + (size_t)head * P.nVi * D + lane * DPL;
                const float* lsrc = P.lpart + (size_t)head * P.nVi;
                int i = 0;
                for (; i + 8 <= n_chunks; i += 8) {  // long contexts: eight chunks' loads in flight, added in chunk order
                    float t8[8][DPL], l8[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
#pragma unroll
                        for (int e = 0; e < DPL; ++e) t8[u][e] = __ldcg(src + (size_t)(i + u) * D + e);
                        l8[u] = __ldcg(lsrc + i + u);
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
#pragma unroll
                        for (int e = 0; e < DPL; ++e) o[e] += t8[u][e];
                        ll += l8[u];
                    }
                }
                for (; i < n_chunks; ++i) {
#pragma unroll
                    for (int e = 0; e < DPL; ++e) o[e] += __ldcg(src + (size_t)i * D + e);
                    ll += __ldcg(lsrc + i);
                }
                const float vscale = P.v_scale ? __ldg(P.v_scale + head) : 1.f;  // fp8 values carry a scale per plane
#pragma unroll
                for (int e = 0; e < DPL; ++e) o[e] = ll > 0.f ? o[e] / ll * vscale : 0.f;  // (an empty context has no probabilities: the output is zero)
                store_row(head, o);
            }
        }
    }
    __syncthreads();
    if (tid == 0 && sm.wait.abort_flag) {
        // (the status word alone could be reset afterwards by the CTA that owns the launch's first tile)
        *reinterpret_cast<volatile unsigned long long*>(&P.hdr->pad[kHdrGaveUpToken]) = token;
        *reinterpret_cast<volatile unsigned long long*>(&P.hdr->pad[kHdrLaunchToken]) = token;
        atomicExch(&P.hdr->status, CHAI_ERR_TIMEOUT);
        // A launch that gave up leaves flag words and counters of its token behind.  The launch count moves on
        // here too (the producer that sees the last claim may never have got there), so that a replay of a
        // captured graph, whose host token is the same every time, starts from a token nobody has used.
        atomicAdd(launch_epoch, 1);
    }
}

struct DeviceInfo {
    int sms = 0;
    int coop = 0;
};

// SM count and cooperative-launch support of a device, queried by the first call on it.
static int device_info(int dev, DeviceInfo* out) {
    static PerDeviceOnce once;
    static DeviceInfo info[kMaxDevices];
    if (dev < 0 || dev >= kMaxDevices) return CHAI_ERR_UNSUPPORTED;
    const int rc = once.run(dev, [&]() -> int {
        DeviceInfo d;
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess)
            return CHAI_ERR_CUDA;
        info[dev] = d;
        return CHAI_OK;
    });
    if (rc == CHAI_OK) *out = info[dev];
    return rc;
}

template <typename T, typename TQ, int D, bool RAGGED>
static int launch(const Params& P0, int ncta, int dev, cudaStream_t s) {
    Params P = P0;
    constexpr int THREADS = Cfg<T>::W * 32 + 32;
    const size_t smem = sizeof(Smem<Cfg<T>::STAGES, Cfg<T>::TILE>) + 128;
    static PerDeviceOnce once;  // (one per instantiation)
    const int rc = once.run(dev, [&]() -> int {
        cudaError_t e = cudaFuncSetAttribute(decode_persistent_kernel<T, TQ, D, RAGGED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return cuda_fail(e, "decode_persistent_kernel shared-memory opt-in");
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_persistent_kernel<T, TQ, D, RAGGED>, THREADS, smem);
        if (e != cudaSuccess) return cuda_fail(e, "decode_persistent_kernel occupancy query");
        return per_sm < 1 ? kDecodeNotLaunched : CHAI_OK;
    });
    if (rc != CHAI_OK) return rc;
    // Cooperative: value tiles wait for flags set by other CTAs, so all CTAs must be resident at once (a plain
    // launch would let two such kernels on different streams starve each other).  Programmatic stream
    // serialisation: the kernel may be scheduled while its predecessor in the stream drains and blocks in
    // griddepcontrol.wait until that predecessor has completed; worth 0.4 % on a replayed graph of layer calls.
    cudaLaunchAttribute attr[2];
    const unsigned n_attr = 2;
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ncta);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_persistent_kernel<T, TQ, D, RAGGED>, P);
    if (e != cudaSuccess) return cuda_fail(e, "decode_persistent_kernel launch");
    return CHAI_OK;
}

}  // namespace pd

int launch_decode_persistent(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                             const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k, int T,
                             int T_cap, int D, size_t k_batch_stride, float scale, int dtype, char* ws,
                             const DecodeLayout& L, cudaStream_t s, const float* k_scale, const float* v_scale,
                             const int32_t* out_membership, int Hq) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return kDecodeNotLaunched;
    pd::DeviceInfo info;
    if (pd::device_info(dev, &info) != CHAI_OK || !info.coop || info.sms <= 0) return kDecodeNotLaunched;
    const int ncta = info.sms;
    const int tiles = (T + L.TR - 1) / L.TR;
    pd::Params P;
    P.q = q; P.k_rep = k_rep; P.v = v; P.membership = membership; P.reps = reps; P.out = out;
    P.seq_lens = seq_lens;
    P.k_scale = k_scale;
    P.v_scale = v_scale;
    P.k_batch_bytes = k_batch_stride * elem_size(dtype);
    P.hdr = reinterpret_cast<WsHeader*>(ws);
    P.counters = reinterpret_cast<int*>(ws + L.off_counters);
    P.gcnt = reinterpret_cast<int*>(ws + L.off_gcnt);
    P.capG = L.capG;
    P.flags = reinterpret_cast<unsigned long long*>(ws + L.off_flags);
    P.pflag = P.flags + 2;
    P.pcnt = P.flags + 2 + (size_t)B * k;
    P.pmax = reinterpret_cast<float*>(ws + L.off_pmax);
    P.scores = reinterpret_cast<float*>(ws + L.off_scores);
    P.cmax = reinterpret_cast<float*>(ws + L.off_cmax);
    P.lpart = reinterpret_cast<float*>(ws + L.off_lpart);
    P.opart = reinterpret_cast<float*>(ws + L.off_opart);
    {
        // launch tokens never repeat within a process and start from a time-dependent value, so stale flag
        // words (earlier launches, other processes, fresh allocations) cannot look like "ready"
        static std::atomic<unsigned long long> counter{
            (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count() * 2654435761ull + 0x9E3779B97F4A7C15ull};
        P.token = counter.fetch_add(1) + 1;
    }
    P.B = B; P.H = H; P.k = k; P.T = T; P.T_cap = T_cap;
    // key work is dealt tile by tile; value items are runs of up to 4 tiles of one head
    P.IV = tiles < pd::MAX_IV ? tiles : pd::MAX_IV;
    P.nVi = (tiles + P.IV - 1) / P.IV;
    P.scale = scale;
    P.wait_limit = decode_wait_limit_cycles();
    P.out_membership = out_membership;
    P.Hq = out_membership != nullptr ? Hq : H;
    if (tiles > L.capK || P.nVi > L.capV || (long long)B * H * P.nVi > 0x7fffffffll ||
        (long long)B * k * tiles > 0x7fffffffll)  // item and key-tile ids travel as ints
        return kDecodeNotLaunched;
    const bool ragged = seq_lens != nullptr || k_batch_stride != (size_t)k * T_cap * D;
    using bf16 = __nv_bfloat16;
    if (dtype == CHAI_FP8_E4M3) {  // fp8 caches, bf16 queries and output
        if (D == 128) return ragged ? pd::launch<Fp8E4M3, bf16, 128, true>(P, ncta, dev, s) : pd::launch<Fp8E4M3, bf16, 128, false>(P, ncta, dev, s);
        return ragged ? pd::launch<Fp8E4M3, bf16, 64, true>(P, ncta, dev, s) : pd::launch<Fp8E4M3, bf16, 64, false>(P, ncta, dev, s);
    }
    if (dtype == CHAI_BF16) {
        if (D == 128) return ragged ? pd::launch<bf16, bf16, 128, true>(P, ncta, dev, s) : pd::launch<bf16, bf16, 128, false>(P, ncta, dev, s);
        return ragged ? pd::launch<bf16, bf16, 64, true>(P, ncta, dev, s) : pd::launch<bf16, bf16, 64, false>(P, ncta, dev, s);
    }
    if (D == 128) return ragged ? pd::launch<float, float, 128, true>(P, ncta, dev, s) : pd::launch<float, float, 128, false>(P, ncta, dev, s);
    return ragged ? pd::launch<float, float, 64, true>(P, ncta, dev, s) : pd::launch<float, float, 64, false>(P, ncta, dev, s);
}

}  // namespace chai
