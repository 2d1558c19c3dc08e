// Clustered causal prefill attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// A persistent kernel, one CTA per SM.  A unit of work = (request, member group of <= 2 heads of one
// cluster, tile of 128 query rows); units are handed out by an atomic counter, heaviest first.  The
// representative's Q tile and K tiles and the members' V tiles arrive by TMA (128-byte swizzle);
// S = Q K^T and O_g += P V_g are tcgen05.mma instructions with fp32 accumulators in tensor memory
// (one S buffer of 128 columns, two P buffers of 64 columns, one O accumulator of 128 columns per
// member: 512 columns).  The softmax threads read S from tensor memory, keep the running reference
// and sum of the softmax (the reference starts at 0 and moves, with a rescaling of O, only when a row maximum
// leaves a window of 2^32 around it, which leaves the result exact because p and l use the same reference) and write P as bf16 back into tensor memory,
// from where it is the A operand of the P V product; the probabilities of a cluster are therefore
// computed once and applied to every member's values (Fig. 3(b)).
//
// Warp roles: warp 0 = work distribution and TMA producer; warp 1 = issuer of the S = Q K^T batches
// (also owns the TMEM allocation); warps 2..9 = softmax / correction, two threads per query row
// (TMEM lane quadrant = warp index mod 4; warps 2..5 take columns 0..63 of a tile, warps 6..9
// columns 64..127); warps 10..13 = epilogue (O / l -> bf16 -> global) of the previous unit while
// the next one computes; warp 14 = issuer of the P V batches.
// head_dim 64 is a second instantiation: a tile is one 64-column block (two members' V tiles share a 32 KB
// slot), the accumulators have 64 columns, a work item carries up to four members, and one P V instruction of
// N = 64 x members serves them all.
// Every mbarrier wait is bounded: on expiry the CTA records CHAI_ERR_TIMEOUT in the workspace
// status word, skips the rest of its work, frees its tensor memory and returns.
// CHAI-QKV (Table 4: the values of non-representative heads are dropped too) is a third instantiation: the work
// items are the clusters themselves (one accumulator: the representative's Q, K and V), the representative's
// query tile is read where it lies among the H heads, and the epilogue writes a finished row to every head that
// the membership assigns to the cluster.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>
#include <type_traits>

#include "prefill_plan.cuh"
#include "tc_ptx.cuh"

namespace chai {

int prefill_check_args(const char* fn, const void* q, const void* k_rep, const void* v, const int32_t* membership,
                       const int32_t* reps, void* out, int B, int H, int k, int T, int D, int dtype, void* workspace,
                       size_t workspace_bytes);
int prefill_run_plan(const int32_t* membership, const int32_t* reps, int B, int H, int k, int gmax, char* ws,
                     cudaStream_t s);

namespace tc {

constexpr int BM = 128;            // query rows per CTA
constexpr int BN = 128;            // keys per tile
constexpr int G = 2;               // V tile slots per key tile: two 128-wide tiles, or four 64-wide ones (two per slot)
constexpr int GMAX = 4;            // member heads per work item at most (head_dim 64; two with head_dim 128)
constexpr int KST = 2;             // K tile stages (tile kt uses stage kt & 1)
constexpr int VST = 2 * G;         // V tile slots: tile kt uses slots (kt & 1) * G + g
constexpr int TILE_BYTES = BN * 128 * 2;       // 32 KB: a tile slot; a 128 x 128 bf16 tile fills it with two 64-column boxes,
                                               // a 128 x 64 tile (head_dim 64) uses its first half
constexpr int HALF_BYTES = TILE_BYTES / 2;     // 16 KB: one 128-row x 64-column swizzled box
constexpr int SOFTMAX_WARPS = 8;    // two per TMEM lane quadrant: each thread owns half a row (64 columns)
constexpr int EPILOGUE_WARPS = 4;   // one thread per query row: O / l -> bf16 -> global while the next item computes
constexpr int PV_WARP = 2 + SOFTMAX_WARPS + EPILOGUE_WARPS;  // the warp that issues the P V batches
constexpr int THREADS = 96 + (SOFTMAX_WARPS + EPILOGUE_WARPS) * 32;
constexpr float REF_WINDOW = 32.f;   // log2 of how far a row's maximum may be from the softmax reference
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t S_COL0 = 0, P_COL0 = 128, O_COL0 = 256;  // S at 0..127, P buffers at 128 + 64 i, O_g at 256 + 128 g

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + TILE_BYTES;
constexpr int OFF_V = OFF_K + KST * TILE_BYTES;
constexpr int OFF_BAR = OFF_V + VST * TILE_BYTES;
constexpr int NUM_BARS = 23;
constexpr int OFF_XCH = OFF_BAR + 8 * NUM_BARS + 16;               // after the barriers and the tmem slot / abort word
constexpr int XCH_BYTES = 2 * BM * 4;                              // row maxima exchanged between the two halves
constexpr int OFF_LSUM = OFF_XCH + XCH_BYTES;                      // row sums handed to the epilogue warps
constexpr int OFF_ITEM = OFF_LSUM + 2 * BM * 4;                    // two work-item descriptors + one for the epilogue
constexpr int ITEM_BYTES = 3 * 48;
constexpr int OFF_PREFIX = OFF_ITEM + ITEM_BYTES;                  // running sum of groups per request
constexpr int MAX_B = 64;                                          // requests per launch on this path
// No alignment slack: the dynamic shared memory of a kernel without static shared memory starts right
// after the 1 KB the system reserves per CTA, i.e. 1024-byte aligned; the kernel checks and refuses otherwise.
constexpr int SMEM_BYTES = OFF_PREFIX + 4 * (MAX_B + 1) + 12;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");

using namespace tcx;

// mbarrier addresses, computed rather than stored so that stage indices stay in registers.
// Tile-indexed barriers come in pairs: key tile number kt (counted over the CTA's whole life) uses
// entry kt & 1 in phase (kt >> 1) & 1.  qk_done[i] tells the softmax warps that S is ready AND the
// producer that the K stage is free; pv_done[i] tells the softmax warps that O may be touched AND
// the producer that the tile's V slots are free: one tcgen05.commit serves both waiters.
struct Bars {
    uint32_t base;
    __device__ __forceinline__ uint32_t q_full() const { return base; }
    __device__ __forceinline__ uint32_t q_empty() const { return base + 8; }
    __device__ __forceinline__ uint32_t o_free(int g) const { return g == 0 ? base + 16 : base + 8 * (18 + g); }  // per member
    // One arrival per softmax warp and tile; tiles alternate between two barriers.  With a single one, a warp of
    // one quadrant could arrive for tile kt + 1 while a warp of another quadrant (whose reference moved: it computes
    // its tile twice and rescales) has not arrived for tile kt -- the scores of tile kt + 1 only need everybody to
    // have LOADED tile kt -- and complete the wrong phase.  Two tiles ahead is impossible: P(kt + 2) overwrites
    // P(kt), which waits for the P V of tile kt, which waits for this barrier.
    __device__ __forceinline__ uint32_t p_full(int i) const { return i == 0 ? base + 24 : base + 8 * 22; }
    __device__ __forceinline__ uint32_t item_full(int i) const { return base + 8 * (4 + i); }
    __device__ __forceinline__ uint32_t item_empty(int i) const { return base + 8 * (6 + i); }
    __device__ __forceinline__ uint32_t k_full(int i) const { return base + 8 * (8 + i); }
    __device__ __forceinline__ uint32_t v_full(int i) const { return base + 8 * (10 + i); }
    __device__ __forceinline__ uint32_t qk_done(int i) const { return base + 8 * (12 + i); }
    __device__ __forceinline__ uint32_t pv_done(int i) const { return base + 8 * (14 + i); }
    __device__ __forceinline__ uint32_t epi_full() const { return base + 8 * 16; }
    __device__ __forceinline__ uint32_t epi_empty() const { return base + 8 * 17; }
    __device__ __forceinline__ uint32_t s_free() const { return base + 8 * 18; }
};
static_assert(NUM_BARS == 23, "barrier count");

// One unit of work, published by the producer to the other roles through shared memory.
template <int GM>
struct ItemT {
    int n_kv;        // key tiles to walk; 0 = zero-fill item (unresolved heads); -1 = no more work
    int n_members;   // heads in this group (1..GM)
    int q0;          // first query row of the tile
    int q_plane;     // b * H + representative head
    int k_plane;     // b * k + cluster
    int o_plane[GM]; // b * H + member head
    int pad[GM == 2 ? 1 : 3];
};
static_assert(sizeof(ItemT<2>) == 32 && sizeof(ItemT<4>) == 48, "item descriptors");

// Persistent kernel: one CTA per SM walks work items (request, member group, query tile) handed out
// by an atomic counter in descending order of cost.  While the softmax warps finish one item, the
// producer is already fetching the next item's Q, K and V tiles and the tensor core computes its
// first scores, so the pipeline fill of an item hides behind the drain of the previous one.
template <int HD, bool QKV>
__global__ void __launch_bounds__(THREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const int* __restrict__ n_groups,
                  const GroupEntry* __restrict__ groups, __nv_bfloat16* __restrict__ out, WsHeader* __restrict__ hdr,
                  const int* __restrict__ bad, int B_total, int b_begin, int B, int H, int k, int T_len, int q_start,
                  float scale_log2, int causal, int n_qtiles, int counter_slot, const int32_t* __restrict__ qkv_membership,
                  int Hq, int group_stride) {
    // QKV: H is the number of clusters (the heads of K_rep and V_rep), Hq the number of heads of q and out, and
    // qkv_membership [B_total, Hq] says which of those heads receive a cluster's rows.
    static_assert(HD == 128 || HD == 64, "head_dim 128 or 64");
    constexpr int LOAD_BYTES = BN * HD * 2;  // bytes one tile copy brings
    // stride between the 64-column blocks an MN-major V operand walks: the two halves of a 128-wide tile, or
    // (head_dim 64, two members in one instruction) the single blocks of two neighbouring slots
    constexpr int V_LBO = HALF_BYTES;        // (with head_dim 64 the members' single blocks lie 16 KB apart, two per slot)
    constexpr int GM = HD == 128 ? 2 : 4;    // member heads per work item
    using Item = ItemT<GM>;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    const uint32_t sbase = smem_u32(smem);
    if ((sbase & 1023u) != 0) {  // swizzled tiles need 1024-byte alignment; never observed, but refuse rather than corrupt
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the planner resets the header
        if (tid == 0) atomicExch(&hdr->status, CHAI_ERR_TIMEOUT);
        return;
    }
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 8 * NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    Item* items = reinterpret_cast<Item*>(smem + OFF_ITEM);          // [2] producer -> MMA / softmax; [2] = softmax -> epilogue
    int* prefix = reinterpret_cast<int*>(smem + OFF_PREFIX);         // [B + 1] running sum of n_groups
    const Bars bar{sbase + OFF_BAR};

    if (tid == 0) {
        mbar_init(bar.q_full(), 1);
        mbar_init(bar.q_empty(), 1);
        // Barriers that a whole role signals count warps, not threads: the lanes of a warp meet first and one
        // lane arrives (hundreds of arrivals on one barrier word serialise and cost more than the work between them).
        for (int g = 0; g < GMAX; ++g) mbar_init(bar.o_free(g), EPILOGUE_WARPS);
        mbar_init(bar.epi_full(), SOFTMAX_WARPS);
        mbar_init(bar.epi_empty(), EPILOGUE_WARPS);
        mbar_init(bar.s_free(), SOFTMAX_WARPS);
        mbar_init(bar.p_full(0), SOFTMAX_WARPS);
        mbar_init(bar.p_full(1), SOFTMAX_WARPS);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar.item_full(i), 1);
            mbar_init(bar.item_empty(i), 2 + SOFTMAX_WARPS);
            mbar_init(bar.k_full(i), 1);
            mbar_init(bar.v_full(i), 1);
            mbar_init(bar.qk_done(i), 1);
            mbar_init(bar.pv_done(i), 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_proxy();
    }
    if (warp == 1) {  // whole warp: allocate all 512 TMEM columns (one CTA per SM by shared-memory size)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Everything above is independent of the planning kernel, which may still be running (the launch is
    // programmatically dependent); its results are read only after this point.  Our own dependents (the
    // planner of a following prefill call) may be placed as soon as SMs free up; they wait for this grid's end.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (tid == 0) {
        if (blockIdx.x == 0 && counter_slot == 0) publish_plan_status(hdr, bad, B_total);
        prefix[0] = 0;
        for (int bb = 0; bb < B; ++bb) prefix[bb + 1] = prefix[bb] + n_groups[b_begin + bb];
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- producer: work distribution and TMA loads ----------------
        if (lane == 0) {
            const int n_pairs = prefix[B];                 // (request, group) pairs that exist
            const int n_items = n_pairs * (n_qtiles - q_start / BM);  // heaviest query tiles first; tiles below q_start hold no row to compute
            bool ok = true;
            int it = 0, qi = 0, kt = 0;                    // items published, items with loads, key tiles issued
            // Work items are fetched one ahead: the atomic that claims the next item is issued before the
            // current item's tiles are streamed and its group entry is read while they stream, so the two
            // dependent round trips to global memory never stall the pipeline between items.
            struct Claim {
                int id, qt, b;
                GroupEntry e;
            };
            auto resolve = [&](Claim& c) {                 // c.id -> query tile, request, group entry
                if (c.id >= n_items) return;
                const int pair = c.id % n_pairs;
                c.qt = n_qtiles - 1 - c.id / n_pairs;
                int lo = 0, hi = B;                        // largest b with prefix[b] <= pair
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (prefix[mid] <= pair) lo = mid; else hi = mid;
                }
                c.b = b_begin + lo;
                c.e = groups[(size_t)c.b * group_stride + (pair - prefix[lo])];
            };
            Claim cur, nxt;
            cur.id = atomicAdd(&hdr->pad[counter_slot], 1);  // (the counter was cleared by the planning kernel)
            resolve(cur);
            while (ok) {
                nxt.id = atomicAdd(&hdr->pad[counter_slot], 1);
                const int is = it & 1;
                ok = mbar_wait(bar.item_empty(is), ((it >> 1) & 1) ^ 1, abort_flag);
                if (!ok) break;
                Item& item = items[is];
                if (cur.id >= n_items) {
                    item.n_kv = -1;
                    mbar_arrive(bar.item_full(is));
                    break;
                }
                const int qt = cur.qt, b = cur.b;
                const GroupEntry e = cur.e;
                const int n_members = min(e.n, GM);
                item.q0 = qt * BM;
                item.n_members = n_members;
                // (CHAI-QKV: a zero-fill item names heads of the output, a computing item its cluster)
                for (int g = 0; g < GM; ++g) item.o_plane[g] = b * ((QKV && e.cluster < 0) ? Hq : H) + e.heads[g < n_members ? g : 0];
                if (e.cluster < 0) {                       // unresolved heads: zero rows, nothing to load
                    item.n_kv = 0;
                    item.q_plane = item.k_plane = 0;
                    mbar_arrive(bar.item_full(is));
                    ++it;
                    resolve(nxt);
                    cur = nxt;
                    continue;
                }
                const int n_kv = causal ? min(qt + 1, (T_len + BN - 1) / BN) : (T_len + BN - 1) / BN;
                item.n_kv = n_kv;
                item.q_plane = b * (QKV ? Hq : H) + e.rep;
                item.k_plane = b * k + e.cluster;
                mbar_arrive(bar.item_full(is));
                const int q_plane = item.q_plane, k_plane = item.k_plane, q0 = item.q0;
                int v_plane[GM];
                for (int g = 0; g < GM; ++g) v_plane[g] = item.o_plane[g];
                // Q: wait until the previous item's last S = Q K^T has been computed
                ok = mbar_wait(bar.q_empty(), (qi & 1) ^ 1, abort_flag);
                if (!ok) break;
                mbar_expect_tx(bar.q_full(), LOAD_BYTES);
                tma_load_4d(sbase + OFF_Q, &map_q, q0, q_plane, bar.q_full());
                // key tile number kt + j of this CTA's life: K stage and V slots (kt + j) & 1
                auto load_k = [&](int j) -> bool {
                    const int n = kt + j, ts = n & 1;
                    if (!mbar_wait(bar.qk_done(ts), ((n >> 1) & 1) ^ 1, abort_flag)) return false;  // stage free
                    mbar_expect_tx(bar.k_full(ts), LOAD_BYTES);
                    tma_load_4d(sbase + OFF_K + ts * TILE_BYTES, &map_k, j * BN, k_plane, bar.k_full(ts));
                    return true;
                };
                // order of need: K(0), K(1), V(0,*), K(2), V(1,*), ...  (S of tile j+1 is computed before P V of tile j)
                ok = load_k(0);
                for (int j = 0; j < n_kv && ok; ++j) {
                    if (j + 1 < n_kv) ok = load_k(j + 1);
                    if (!ok) break;
                    const int n = kt + j, ts = n & 1;
                    ok = mbar_wait(bar.pv_done(ts), ((n >> 1) & 1) ^ 1, abort_flag);  // the tile's V slots are free
                    if (!ok) break;
                    mbar_expect_tx(bar.v_full(ts), n_members * LOAD_BYTES);
#pragma unroll
                    for (int g = 0; g < GM; ++g)  // (member arrays are indexed statically: they stay in registers)
                        if (g < n_members) tma_load_4d(sbase + OFF_V + ts * G * TILE_BYTES + g * LOAD_BYTES, &map_v, j * BN, v_plane[g], bar.v_full(ts));
                    if (j == 0) resolve(nxt);  // two tiles are on their way: time to look at the claim's answer
                }
                kt += n_kv;
                ++it;
                ++qi;
                cur = nxt;
            }
        }
    } else if (warp == 1 || warp == PV_WARP) {
        // ---------------- MMA issuers ----------------
        // Two warps issue the tensor-core work, one the S = Q K^T batches and one the O += P V batches, so
        // that the barrier polling of either overlaps the other's instruction issue (issuing an MMA blocks
        // the thread for about as long as the tensor pipe needs to run it).  Every ordering between the two
        // streams goes through an mbarrier, and tcgen05.commit tracks the issuing thread's own MMAs, so the
        // streams need no program order between them.  Each warp walks its loop as a whole, which keeps the
        // control flow and the descriptor arithmetic warp-uniform; one elected lane issues.
        constexpr uint32_t IDESC_QK = make_idesc(false);
        auto desc = [](uint32_t hi, uint32_t lo) { return ((uint64_t)hi << 32) | lo; };
        auto wait_all = [&](uint32_t b, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait_polling(b, parity, abort_flag)); };
        const bool qk_role = warp == 1;
        // Descriptors are built once; inside the loops only the 14-bit start-address field (low word)
        // moves, by compile-time offsets, so issuing an MMA costs an add and the instruction.
        const uint64_t dq = make_desc(sbase + OFF_Q, 16, 1024);
        const uint64_t dk = make_desc(sbase + OFF_K, 16, 1024);
        const uint64_t dv = make_desc(sbase + OFF_V, V_LBO, 1024);
        const uint32_t hi_k = (uint32_t)(dq >> 32), hi_v = (uint32_t)(dv >> 32);
        const uint32_t q_lo = (uint32_t)dq, k_lo = (uint32_t)dk, v_lo = (uint32_t)dv;
        bool ok = true;
        int it = 0, qi = 0, kt = 0;  // items seen, items computed, key tiles issued so far
        while (ok) {
            const int is = it & 1;
            ok = wait_all(bar.item_full(is), (it >> 1) & 1);
            if (!ok) break;
            const int n_kv = items[is].n_kv, n_members = items[is].n_members;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.item_empty(is));  // the two fields are in registers
            if (n_kv < 0) break;
            if (n_kv == 0) {
                ++it;
                continue;
            }
            if (qk_role) {
                ok = wait_all(bar.q_full(), qi & 1);
                for (int j = 0; j < n_kv && ok; ++j, ++kt) {
                    // S(tile kt) = Q K^T into the S buffer, once the softmax warps hold the previous tile's scores
                    const int ts = kt & 1;
                    ok = wait_all(bar.k_full(ts), (kt >> 1) & 1) && (kt == 0 || wait_all(bar.s_free(), (kt - 1) & 1));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d = tmem_base + S_COL0;
                    const uint32_t kb = k_lo + ts * (TILE_BYTES >> 4);
                    if (elect_one()) {
#pragma unroll
                        for (int s = 0; s < HD / 16; ++s) {
                            const uint32_t off = ((s >> 2) * HALF_BYTES + (s & 3) * 32) >> 4;
                            tc_mma(d, desc(hi_k, q_lo + off), desc(hi_k, kb + off), IDESC_QK, s > 0);
                        }
                        tc_commit(bar.qk_done(ts));
                        if (j + 1 == n_kv) tc_commit(bar.q_empty());  // Q may be overwritten by the next item's tile
                    }
                    __syncwarp();
                }
            } else {
                for (int j = 0; j < n_kv && ok; ++j, ++kt) {
                    const int ts = kt & 1;
                    ok = wait_all(bar.p_full(ts), (kt >> 1) & 1) && wait_all(bar.v_full(ts), (kt >> 1) & 1);
                    if (!ok) break;
                    const uint32_t p_addr = tmem_base + P_COL0 + ts * 64;  // P buffer of this tile
                    const bool reuse = j == 0 && qi > 0;  // the accumulators still hold the previous item's output
                    // An item's first tile overwrites the accumulators, which still hold the previous item's output
                    // until the epilogue warps have drained them (each member's is released on its own).
                    if (reuse)
                        for (int g = 0; g < n_members && ok; ++g) ok = wait_all(bar.o_free(g), (qi - 1) & 1);
                    if (!ok) break;
                    // All members at once: their V tiles lie side by side in shared memory (64-column blocks at
                    // one stride) and so do their accumulators in tensor memory, so one instruction of
                    // N = head_dim x members per 16 keys serves them all and reads P once.
                    tc_fence_after();
                    if (elect_one()) {
                        const uint32_t d = tmem_base + O_COL0;
                        const uint32_t vb = v_lo + (ts * G) * (TILE_BYTES >> 4);
                        const uint32_t idesc_all = make_idesc_n(true, (unsigned)(HD * n_members));
#pragma unroll
                        for (int s = 0; s < BN / 16; ++s)  // 16 keys per step: 8 TMEM columns of P, 2048 bytes of each V block
                            tc_mma_ts(d, p_addr + s * 8, desc(hi_v, vb + s * (2048 >> 4)), idesc_all, (j > 0 || s > 0) ? 1u : 0u);
                        tc_commit(bar.pv_done(ts));
                    }
                    __syncwarp();
                }
            }
            ++it;
            ++qi;
        }
    } else if (warp < 2 + SOFTMAX_WARPS) {
        // ---------------- softmax / correction: two threads per query row ----------------
        // Warps 2..5 own columns 0..63 of their rows, warps 6..9 columns 64..127; the two threads of a row
        // sit in different warps of the same TMEM lane quadrant and meet once per tile at a 64-thread
        // named barrier, where they exchange their half-row maxima.
        const int quad = warp & 3;               // TMEM lanes this warp may touch
        const int half = (warp - 2) >> 2;        // which 64 columns of the tile
        const int row = quad * 32 + lane;        // row of the tile
        const int cbase = half * 64;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        __nv_bfloat16* xch = reinterpret_cast<__nv_bfloat16*>(smem + OFF_XCH);  // [tile parity][half][row]
        float* lsum = reinterpret_cast<float*>(smem + OFF_LSUM);  // [half][row]
        bool ok = true;
        int it = 0, ei = 0, kt = 0;  // items seen, items handed to the epilogue, key tiles processed so far
        uint32_t r[64];
        while (true) {
            const int is = it & 1;
            ok = ok && mbar_wait(bar.item_full(is), (it >> 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const Item item = items[is];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.item_empty(is));  // the item is in registers (all lanes: __syncwarp above)
            if (item.n_kv < 0) break;
            const int n_kv = item.n_kv, n_members = item.n_members, q0 = item.q0;
            const int row_abs = q0 + row;
            if (n_kv == 0) {  // unresolved heads: zero rows
                if (row_abs >= q_start && row_abs < T_len)
#pragma unroll
                    for (int g = 0; g < GM; ++g) {
                        if (g >= n_members) break;
                        uint4* o = reinterpret_cast<uint4*>(out + ((size_t)item.o_plane[g] * T_len + row_abs) * HD + half * (HD / 2));
#pragma unroll
                        for (int u = 0; u < HD / 16; ++u) o[u] = make_uint4(0, 0, 0, 0);
                    }
                ++it;
                continue;
            }
            // The reference the exponentials are taken against starts at 0 for every row and moves only when a
            // tile's row maximum leaves a window of 2^+-32 around it (first tile) or outgrows it by 2^32 (later
            // tiles): a common factor 2^-m cancels in P V / l, bf16 and fp32 keep their relative precision at
            // any magnitude, and 2^32 times the row's largest term is far from fp32's range for any number of
            // keys.  For scores of ordinary size the reference therefore never moves, no tile waits for its
            // maxima before its exponentials, and no accumulator is ever rescaled; the reference is a function
            // of the row's own scores alone, so results do not depend on how work was scheduled.
            float m_used = 0.f, l_run = 0.f;
            for (int j = 0; j < n_kv && ok; ++j, ++kt) {
                const int sb = kt & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(bar.qk_done(sb), (kt >> 1) & 1, abort_flag));
                if (!ok) break;  // warp-uniform: the tcgen05 loads below are warp-collective
                tc_fence_after();
                const uint32_t s_addr = lane_addr + S_COL0;
                const uint32_t p_st = lane_addr + P_COL0 + sb * 64 + half * 32;  // this thread's 32 columns of P(kt)
                const int col0 = j * BN;
                // columns of this thread's half that the row may see: col_abs < T and (causal: col_abs <= row_abs)
                int vis = T_len - col0;
                if (causal) vis = min(vis, row_abs - col0 + 1);
                vis = max(0, min(vis - cbase, 64));
                // the whole tile is visible to every row unless it is the diagonal tile or runs past T
                const bool full_tile = col0 + BN <= T_len && (!causal || col0 + BN - 1 <= q0);
                tc_ld64_wait(s_addr + cbase, r);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar.s_free());  // the scores are in registers: the next S = Q K^T may overwrite the buffer
                // Columns the row may not see (beyond the diagonal, beyond T) become -inf here, in registers:
                // they then lose every maximum and give probability 0, and the arithmetic below is the same
                // for every tile.
                if (!full_tile) {
#pragma unroll
                    for (int i = 0; i < 64; ++i)
                        if (i >= vis) r[i] = 0xff800000u;
                }
                // Own half-row maximum, eight independent chains, taken along with the exponentials (which run
                // against the current reference at once, see below) in the issue slots the special-function unit
                // leaves free.
                float mxa[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) mxa[c] = -INFINITY;
                // The two threads of a row must agree on one reference.  Each rounds its half-row maximum up to
                // bf16 and publishes it (slots alternate with the tile's parity); both take the larger of the two
                // rounded values, a reference slightly above the true maximum being as good.
                __nv_bfloat16 mx_up;
                __nv_bfloat16* xs = xch + (kt & 1) * 2 * BM;
                auto publish = [&]() {
                    mx_up = __float2bfloat16_ru(max3(max3(mxa[0], mxa[1], mxa[2]), max3(mxa[3], mxa[4], mxa[5]), fmaxf(mxa[6], mxa[7])));
                    xs[half * BM + row] = mx_up;
                };
                float m_new = m_used, corr = 1.f;
                // Meet the partner: reference of this tile, by the lazy-rescale rule above.
                auto meet = [&]() -> bool {
                    // The two warps of a quadrant meet at a named barrier (hardware barrier 1 + quad, 64 threads):
                    // a fraction of the latency of an mbarrier round trip, once per tile on the path that bounds
                    // the kernel.  It has no time limit of its own, so a warp that gives up (a bounded wait
                    // elsewhere ran out: the abort flag is set) arrives here once on its way out, and everyone
                    // looks at the flag right after the barrier: nobody can be left waiting for a warp that is gone.
                    asm volatile("bar.sync %0, 64;" ::"r"(quad + 1) : "memory");
                    if (*abort_flag) return false;
                    const float mx = fmaxf(__bfloat162float(mx_up), __bfloat162float(xs[(half ^ 1) * BM + row]));
                    const float m_tile = mx * scale_log2;
                    if (m_tile > m_used + REF_WINDOW || (j == 0 && m_tile < m_used - REF_WINDOW)) {
                        m_new = m_tile;
                        corr = j == 0 ? 1.f : fast_exp2(m_used - m_new);  // (nothing has been accumulated before the first tile)
                    }
                    return true;
                };
                // probabilities against reference m, rounded to bf16, two per 32-bit column: the layout of an A
                // operand in tensor memory (score columns 64 h + c map to column 32 h + c / 2 of the tile's P
                // buffer); they leave in chunks of 16 as they are ready.  Returns the row's partial sum.
                auto emit = [&](float m, auto with_max) -> float {
                    const float m_ref = m == -INFINITY ? 0.f : m;
                    const uint64_t sc2 = pack2(scale_log2, scale_log2), nm2 = pack2(-m_ref, -m_ref);
                    uint64_t acc01 = 0ull, acc23 = 0ull;  // two packed pairs of partial row sums
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t packed[8];
#pragma unroll
                        for (int u = 0; u < 16; u += 4) {
                            const int i = c * 16 + u;
                            float x0, x1, x2, x3;
                            unpack2(fma2(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sc2, nm2), x0, x1);
                            unpack2(fma2(pack2(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])), sc2, nm2), x2, x3);
                            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1), p2 = fast_exp2(x2), p3 = fast_exp2(x3);
                            if constexpr (decltype(with_max)::value) {
                                mxa[(i >> 1) & 7] = max3(mxa[(i >> 1) & 7], __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                                mxa[((i >> 1) + 1) & 7] = max3(mxa[((i >> 1) + 1) & 7], __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                            }
                            acc01 = add2(acc01, pack2(p0, p1));
                            acc23 = add2(acc23, pack2(p2, p3));
                            __nv_bfloat162 pa = __floats2bfloat162_rn(p0, p1), pb = __floats2bfloat162_rn(p2, p3);
                            packed[u >> 1] = *reinterpret_cast<uint32_t*>(&pa);
                            packed[(u >> 1) + 1] = *reinterpret_cast<uint32_t*>(&pb);
                        }
                        tc_st8(p_st + c * 8, packed);
                    }
                    float s0, s1;
                    unpack2(add2(acc01, acc23), s0, s1);
                    return s0 + s1;
                };
                // P buffer kt & 1 was last read by the P V of tile kt - 2 (long complete as a rule)
                if (kt >= 2) {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar.pv_done(sb), ((kt >> 1) & 1) ^ 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                }
                // The reference hardly ever moves, so the tile is computed against the current reference at once,
                // without waiting for the partner's maximum; the meeting follows the arithmetic, and only if some
                // row's reference did move is the tile computed and stored again.
                float ls = emit(m_used, std::true_type{});
                publish();
                ok = meet();
                if (!ok) break;
                const bool moved = __any_sync(0xffffffffu, m_new != m_used);  // some row of this warp changed its reference
                if (moved) ls = emit(m_new, std::false_type{});
                l_run = l_run * corr + ls;
                m_used = m_new;
                // Rescaling touches the O accumulators, so the previous tile's P V must be complete first; a warp
                // whose rows all keep their reference (the usual case after the first tiles) has nothing to wait
                // for.  Skipping the wait cannot confuse the barrier's phase parity: the P V of tile kt - 3 (same
                // barrier, previous phase) was awaited before P(kt - 1) was written.
                if (j > 0 && moved) {  // (after the first tile a moved reference always comes with a factor other than 1)
                    ok = __all_sync(0xffffffffu, mbar_wait(bar.pv_done((kt - 1) & 1), ((kt - 1) >> 1) & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    for (int g = 0; g < n_members; ++g) {  // this thread rescales its half of the columns of each O
                        const uint32_t o_addr = lane_addr + O_COL0 + g * HD + half * (HD / 2);
                        if constexpr (HD == 128) tc_ld64_wait(o_addr, r);
                        else tc_ld32_wait(o_addr, r);
#pragma unroll
                        for (int i = 0; i < HD / 2; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * corr);
                        tc_st32(o_addr, r);
                        if constexpr (HD == 128) tc_st32(o_addr + 32, r + 32);
                    }
                }
                tc_wait_st();          // P (and any rescaled O) is in tensor memory
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar.p_full(sb));
            }
            // hand the item to the epilogue warps: row sums of both halves and where the output goes
            ok = __all_sync(0xffffffffu, ok && mbar_wait(bar.epi_empty(), (ei & 1) ^ 1, abort_flag));
            if (!ok) break;
            lsum[half * BM + row] = l_run;
            if (tid == 64) {
                Item& ep = items[2];
                ep = item;
                ep.n_kv = kt - 1;  // global index of the item's last key tile (its P V completion is awaited)
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.epi_full());
            ++ei;
            ++it;
        }
        // tell the epilogue warps that nothing more will come
        if (__all_sync(0xffffffffu, mbar_wait(bar.epi_empty(), (ei & 1) ^ 1, abort_flag))) {
            if (tid == 64) items[2].n_members = -1;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.epi_full());
        }
        if (!ok) asm volatile("bar.arrive %0, 64;" ::"r"(quad + 1) : "memory");  // release a partner that may be waiting to meet
    } else {
        // ---------------- epilogue: O_g / l -> bf16 -> global, one thread per query row ----------------
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const float* lsum = reinterpret_cast<const float*>(smem + OFF_LSUM);
        for (int ei = 0;; ++ei) {
            bool ok = __all_sync(0xffffffffu, mbar_wait(bar.epi_full(), ei & 1, abort_flag));
            if (!ok) break;
            const Item ep = items[2];
            const float l = lsum[row] + lsum[BM + row];
            if (ep.n_members < 0) break;
            const int last = ep.n_kv;
            ok = __all_sync(0xffffffffu, mbar_wait(bar.pv_done(last & 1), (last >> 1) & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar.epi_empty());  // the hand-over area is in registers (all lanes: __syncwarp above)
            const int row_abs = ep.q0 + row;
            const float inv = l > 0.f ? 1.f / l : 0.f;
            const uint64_t inv2 = pack2(inv, inv);
            // The accumulators leave in pieces of 32 columns through two register buffers: the load of the next
            // piece is in flight while the current one is scaled, rounded and stored, and a member's
            // accumulator is released as soon as its last piece is in registers.
            constexpr int NSUB = HD / 32;
            const int n_sub = ep.n_members * NSUB;
            uint32_t ra[32], rb[32];
            tc_ld32(lane_addr + O_COL0, ra);
            tc_wait_ld32(ra);
#pragma unroll
            for (int c = 0; c < GM * NSUB; ++c) {
                if (c >= n_sub) break;
                uint32_t* cur = (c & 1) ? rb : ra;
                uint32_t* nxt = (c & 1) ? ra : rb;
                const int g = c / NSUB, sc = c % NSUB;
                if (c + 1 < n_sub) tc_ld32(lane_addr + O_COL0 + (c + 1) * 32, nxt);  // (members' accumulators are contiguous)
                if (sc == NSUB - 1) {  // this row of the member's accumulator is in registers
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(bar.o_free(g));
                        if (g == ep.n_members - 1)  // keep the phases of the unused members' barriers in step
                            for (int x = ep.n_members; x < GM; ++x) mbar_arrive(bar.o_free(x));
                    }
                }
                if constexpr (QKV) {
                    // the cluster's row goes to every head of the cluster: the warp finds them 32 heads at a time
                    uint32_t w[16];
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        float y0, y1;
                        unpack2(mul2(pack2(__uint_as_float(cur[2 * x]), __uint_as_float(cur[2 * x + 1])), inv2), y0, y1);
                        __nv_bfloat162 pk = __floats2bfloat162_rn(y0, y1);
                        w[x] = *reinterpret_cast<uint32_t*>(&pk);
                    }
                    const int bq = ep.o_plane[0] / H, cq = ep.o_plane[0] % H;
                    const bool row_live = row_abs >= q_start && row_abs < T_len;
                    for (int h0 = 0; h0 < Hq; h0 += 32) {
                        const int hh = h0 + lane;
                        unsigned members = __ballot_sync(0xffffffffu, hh < Hq && __ldg(qkv_membership + (size_t)bq * Hq + hh) == cq);
                        while (members) {
                            const int h = h0 + __ffs(members) - 1;
                            members &= members - 1;
                            if (row_live) {
                                __nv_bfloat16* orow = out + (((size_t)bq * Hq + h) * T_len + row_abs) * HD + sc * 32;
                                st_global_32B(orow, w);
                                st_global_32B(orow + 16, w + 8);
                            }
                        }
                    }
                } else if (row_abs >= q_start && row_abs < T_len) {  // rows before q_start belong to the caller
                    __nv_bfloat16* orow = out + ((size_t)ep.o_plane[g] * T_len + row_abs) * HD + sc * 32;
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        uint32_t w[8];
#pragma unroll
                        for (int x = 0; x < 8; ++x) {
                            float y0, y1;
                            unpack2(mul2(pack2(__uint_as_float(cur[16 * u + 2 * x]), __uint_as_float(cur[16 * u + 2 * x + 1])), inv2), y0, y1);
                            __nv_bfloat162 pk = __floats2bfloat162_rn(y0, y1);
                            w[x] = *reinterpret_cast<uint32_t*>(&pk);
                        }
                        st_global_32B(orow + u * 16, w);
                    }
                }
                if (c + 1 < n_sub) tc_wait_ld32(nxt);
            }
        }
    }

    // teardown: every tcgen05 operation of this CTA has completed or been abandoned after a timeout
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag) atomicExch(&hdr->status, CHAI_ERR_TIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [planes, T, 128] bf16 viewed as a 4-D tensor (innermost first): 64 columns, T rows, 2 column halves, planes;
// box = 64 x 128 x 2 x 1, i.e. a whole 128 x 128 tile per copy, stored as two swizzled 64-column blocks.
// [planes, T, 128] bf16 seen as (64 columns, T rows, 2 column halves, planes); one copy moves box_rows rows of
// both halves, which land as two consecutive blocks of 128-byte swizzled rows.
static bool make_map_rows(CUtensorMap* map, const void* base, int planes, int T, int box_rows, int HD) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    const cuuint32_t halves = (cuuint32_t)(HD / 64);  // head_dim 64: one 64-column block per row
    cuuint64_t dims[4] = {64, (cuuint64_t)T, halves, (cuuint64_t)planes};
    cuuint64_t strides[3] = {(cuuint64_t)HD * 2, 128, (cuuint64_t)T * HD * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)box_rows, halves, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
static bool make_map(CUtensorMap* map, const void* base, int planes, int T, int HD) { return make_map_rows(map, base, planes, T, BN, HD); }

}  // namespace tc
}  // namespace chai

extern "C" int chai_prefill_attention_simt_from(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                                const int32_t* reps, void* out, int B, int H, int k, int T, int q_start,
                                                int D, float scale, int causal, int dtype, void* workspace,
                                                size_t workspace_bytes, void* stream);

namespace chai {

// Plan of CHAI-QKV prefill: one group per usable cluster (cluster c, its representative among the Hq heads, one
// "member": the cluster itself), then zero-fill groups of up to gmax heads for the heads that name no usable cluster.
// grid B, block 128, k ints of shared memory.
static __global__ void __launch_bounds__(128)
prefill_plan_qkv_kernel(const int32_t* __restrict__ membership, const int32_t* __restrict__ reps, WsHeader* __restrict__ hdr,
                        int* __restrict__ n_groups, int* __restrict__ bad_out, GroupEntry* __restrict__ groups, int Hq, int k,
                        int gmax, int group_stride) {
    extern __shared__ __align__(16) int s_live[];
    const int b = blockIdx.x, tid = threadIdx.x;
    dependent_grid_sync();
    if (b == 0)
        for (int i = tid; i < 60; i += blockDim.x) hdr->pad[i] = 0;
    const int32_t* mem = membership + (size_t)b * Hq;
    for (int c = tid; c < k; c += blockDim.x) {
        const int r = reps[(size_t)b * k + c];
        s_live[c] = (r >= 0 && r < Hq && mem[r] == c) ? r : -1;
    }
    __syncthreads();
    if (tid != 0) return;
    GroupEntry* out = groups + (size_t)b * group_stride;
    int ng = 0;
    for (int c = 0; c < k; ++c)
        if (s_live[c] >= 0) {
            int4* dst = reinterpret_cast<int4*>(out + ng++);
            dst[0] = make_int4(c, s_live[c], 1, 0);
            dst[1] = make_int4(c, c, c, c);
        }
    int cnt = 0, first_bad = -1, hd[kGroupMax] = {0, 0, 0, 0};
    for (int h = 0; h < Hq; ++h) {
        const int c = mem[h];
        if (c >= 0 && c < k && s_live[c] >= 0) continue;
        if (first_bad < 0) first_bad = h;
        if (cnt == 0)
            for (int x = 0; x < kGroupMax; ++x) hd[x] = h;
        for (int x = 0; x < kGroupMax; ++x)
            if (x == cnt) hd[x] = h;
        if (++cnt == gmax) {
            int4* dst = reinterpret_cast<int4*>(out + ng++);
            dst[0] = make_int4(-1, -1, cnt, 0);
            dst[1] = make_int4(hd[0], hd[1], hd[2], hd[3]);
            cnt = 0;
        }
    }
    if (cnt > 0) {
        int4* dst = reinterpret_cast<int4*>(out + ng++);
        dst[0] = make_int4(-1, -1, cnt, 0);
        dst[1] = make_int4(hd[0], hd[1], hd[2], hd[3]);
    }
    n_groups[b] = ng;
    bad_out[b] = first_bad + 1;
}

// Launches the tensor-core kernel on a plan that lies in `ws` (layout L).  H: heads per request that the items'
// value and output planes count (the clusters, for CHAI-QKV); qkv_membership / Hq: see the kernel.
static int prefill_tc_launch(const char* fn, const void* q, int q_planes, const void* k_rep, const void* v, int v_planes,
                             void* out, int B, int H, int k, int T, int q_start, int D, float scale, int causal, char* ws,
                             const PrefillLayout& L, int group_stride, const int32_t* qkv_membership, int Hq, cudaStream_t s) {
    CUtensorMap mq, mk, mv;
    CHAI_REQUIRE(tc::make_map(&mq, q, q_planes, T, D) && tc::make_map(&mk, k_rep, B * k, T, D) && tc::make_map(&mv, v, v_planes, T, D),
                 CHAI_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed", fn);
    // per device, once: SM count, and the kernels' opt-in to their shared-memory size
    static PerDeviceOnce once;
    static int sms_of_device[kMaxDevices] = {};
    int dev = 0;
    cudaError_t de = cudaGetDevice(&dev);
    if (de != cudaSuccess) return cuda_fail(de, "prefill_tc_kernel set-up");
    CHAI_REQUIRE(dev >= 0 && dev < kMaxDevices, CHAI_ERR_UNSUPPORTED, "%s: device index %d out of range", fn, dev);
    int rc = once.run(dev, [&]() -> int {
        int count = 0;
        cudaError_t e = cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(tc::prefill_tc_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(tc::prefill_tc_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(tc::prefill_tc_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(tc::prefill_tc_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES);
        if (e != cudaSuccess) return cuda_fail(e, "prefill_tc_kernel set-up");
        sms_of_device[dev] = count;
        return CHAI_OK;
    });
    if (rc != CHAI_OK) return rc;
    const int n_sms = sms_of_device[dev];
    const int n_qtiles = (T + tc::BM - 1) / tc::BM;
    const bool qkv = qkv_membership != nullptr;
    CHAI_LOG_CALL("%s: B=%d H=%d k=%d T=%d q_start=%d D=%d causal=%d tensor-core kernel%s, %d CTAs x %d threads, "
                  "%d query tiles, %d launch(es), members per item <= %d", fn, B, qkv ? Hq : H, k, T, q_start, D, causal,
                  qkv ? " (one item per cluster, rows written to all members)" : "", n_sms, tc::THREADS,
                  n_qtiles - q_start / tc::BM, (B + tc::MAX_B - 1) / tc::MAX_B, qkv ? 1 : (D == 128 ? 2 : 4));
    // one persistent CTA per SM; requests are processed in chunks of MAX_B (the per-request group counts of
    // a chunk are kept in shared memory), each chunk with its own work counter in the workspace header
    for (int b0 = 0, chunk = 0; b0 < B; b0 += tc::MAX_B, ++chunk) {
        const int nb = B - b0 < tc::MAX_B ? B - b0 : tc::MAX_B;
        // launched as a programmatic dependent of the planning kernel: the set-up of this kernel's CTAs
        // overlaps the planner's run, and the kernel itself waits for the planner before it reads the plan
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(n_sms);
        cfg.blockDim = dim3(tc::THREADS);
        cfg.dynamicSmemBytes = tc::SMEM_BYTES;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const int* ng = reinterpret_cast<const int*>(ws + L.off_ngroups);
        const GroupEntry* gr = reinterpret_cast<const GroupEntry*>(ws + L.off_groups);
        __nv_bfloat16* o = static_cast<__nv_bfloat16*>(out);
        WsHeader* hdr = reinterpret_cast<WsHeader*>(ws);
        const int* bad = reinterpret_cast<const int*>(ws + L.off_bad);
        const float scale_log2 = scale * 1.4426950408889634f;
        auto kernel = D == 128 ? (qkv ? tc::prefill_tc_kernel<128, true> : tc::prefill_tc_kernel<128, false>)
                               : (qkv ? tc::prefill_tc_kernel<64, true> : tc::prefill_tc_kernel<64, false>);
        cudaError_t le = cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, ng, gr, o, hdr, bad, B, b0, nb, H, k, T, q_start, scale_log2,
                                            causal, n_qtiles, chunk, qkv_membership, Hq, group_stride);
        if (le != cudaSuccess) return cuda_fail(le, "prefill_tc_kernel launch");
        CHAI_LAUNCH_CHECK("prefill_tc_kernel launch");
    }
    return CHAI_OK;
}

// CHAI-QKV prefill on the tensor-core kernel (bf16, head_dim 64 or 128, at most 60 * 64 requests, positive finite
// scale); kDecodeNotLaunched-style -1 when the call is outside that range and the caller should take the general path.
int prefill_qkv_tc(const void* q, const void* k_rep, const void* v_rep, const int32_t* membership, const int32_t* reps,
                   void* out, int B, int H, int k, int T, int q_start, int D, float scale, int causal, int dtype, void* workspace,
                   size_t workspace_bytes, cudaStream_t s) {
    if (dtype != CHAI_BF16 || (D != 128 && D != 64) || B > 60 * tc::MAX_B || !(scale > 0.f) || !(scale <= 3.0e38f)) return -1;
    const PrefillLayout L = prefill_layout(B, H + k);
    if (workspace_bytes < L.total || (size_t)k * sizeof(int) > 48 * 1024) return -1;
    char* ws = static_cast<char*>(workspace);
    CHAI_LAUNCH_DEPENDENT("prefill_plan_qkv_kernel launch", prefill_plan_qkv_kernel, dim3(B), dim3(128), sizeof(int) * (size_t)k, s,
                          membership, reps, reinterpret_cast<WsHeader*>(ws), reinterpret_cast<int*>(ws + L.off_ngroups),
                          reinterpret_cast<int*>(ws + L.off_bad), reinterpret_cast<GroupEntry*>(ws + L.off_groups), H, k,
                          D == 128 ? 2 : 4, H + k);
    return prefill_tc_launch("chai_prefill_attention_qkv", q, B * H, k_rep, v_rep, B * k, out, B, k, k, T, q_start, D, scale, causal,
                             ws, L, H + k, membership, H, s);
}

}  // namespace chai

extern "C" int chai_prefill_attention_from(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                           const int32_t* reps, void* out, int B, int H, int k, int T, int q_start, int D,
                                           float scale, int causal, int dtype, void* workspace, size_t workspace_bytes,
                                           void* stream) {
    using namespace chai;
    // The tensor-core kernel takes a row's largest raw score and scales it afterwards, which is the largest scaled
    // score only for a positive, finite scale; anything else goes to the CUDA-core kernel, which scales first.
    if (dtype != CHAI_BF16 || (D != 128 && D != 64) || B > 60 * tc::MAX_B || !(scale > 0.f) || !(scale <= 3.0e38f))
        return chai_prefill_attention_simt_from(q, k_rep, v, membership, reps, out, B, H, k, T, q_start, D, scale, causal,
                                                dtype, workspace, workspace_bytes, stream);
    int rc = prefill_check_args("chai_prefill_attention", q, k_rep, v, membership, reps, out, B, H, k, T, D, dtype,
                                workspace, workspace_bytes);
    if (rc != CHAI_OK) return rc;
    CHAI_REQUIRE(q_start >= 0 && q_start < T, CHAI_ERR_INVALID_ARG,
                 "chai_prefill_attention: need 0 <= q_start < T (q_start=%d, T=%d)", q_start, T);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    rc = prefill_run_plan(membership, reps, B, H, k, D == 128 ? 2 : 4, ws, s);
    if (rc != CHAI_OK) return rc;
    return prefill_tc_launch("chai_prefill_attention", q, B * H, k_rep, v, B * H, out, B, H, k, T, q_start, D, scale, causal, ws,
                             prefill_layout(B, H), H, nullptr, H, s);
}

extern "C" int chai_prefill_attention(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                      const int32_t* reps, void* out, int B, int H, int k, int T, int D, float scale,
                                      int causal, int dtype, void* workspace, size_t workspace_bytes, void* stream) {
    return chai_prefill_attention_from(q, k_rep, v, membership, reps, out, B, H, k, T, 0, D, scale, causal, dtype,
                                       workspace, workspace_bytes, stream);
}
