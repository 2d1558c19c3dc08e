// Clustered causal prefill attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// One CTA = (request, member group of <= 2 heads of one cluster, tile of 128 query rows).  The
// representative's Q tile and K tiles and the members' V tiles arrive by TMA (128-byte swizzle);
// S = Q K^T and O_g += P V_g are tcgen05.mma instructions issued by one thread with fp32
// accumulators in tensor memory (two S buffers of 128 columns, one O accumulator of 128 columns
// per member: 512 columns).  Four warps own one query row per thread: they read S from tensor
// memory, keep the running maximum and sum of the softmax (rescaling O only when the maximum grew
// by more than 2^8, which leaves the result exact because p and l use the same reference), write
// P as bf16 into shared memory in the operand layout, and at the end scale O by 1/l and store it.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (also owns the TMEM allocation),
// warps 2..9 = softmax / correction / epilogue, two threads per query row (TMEM lane quadrant = warp
// index mod 4; warps 2..5 take columns 0..63 of a tile, warps 6..9 columns 64..127).
// Every mbarrier wait is bounded: on expiry the CTA records CHAI_ERR_TIMEOUT in the workspace
// status word, skips the rest of its work, frees its tensor memory and returns.
#include <cuda.h>

#include "prefill_plan.cuh"

namespace chai {

int prefill_check_args(const char* fn, const void* q, const void* k_rep, const void* v, const int32_t* membership,
                       const int32_t* reps, void* out, int B, int H, int k, int T, int D, int dtype, void* workspace,
                       size_t workspace_bytes);
int prefill_run_plan(const int32_t* membership, const int32_t* reps, int B, int H, int k, int gmax, char* ws,
                     cudaStream_t s);

namespace tc {

// stage timestamps (SM clock) of CTA (0,0,0), per key tile: debugging aid read by chai_debug_prefill_stats
__device__ long long g_pf_stats[64][8];
// (smid, start ns, end ns, key tiles) of every working CTA of the last launch
__device__ long long g_pf_cta[4096][4];
__device__ int g_pf_cta_n;

constexpr int BM = 128;            // query rows per CTA
constexpr int BN = 128;            // keys per tile
constexpr int HD = 128;            // head dimension
constexpr int G = 2;               // member heads per CTA
constexpr int KST = 2;             // K tile stages
constexpr int VST = 4;             // V tile slots: two key tiles' worth of member tiles in flight
constexpr int TILE_BYTES = BN * HD * 2;        // 32 KB: one 128 x 128 bf16 tile = two 64-column boxes
constexpr int HALF_BYTES = TILE_BYTES / 2;     // 16 KB: one 128-row x 64-column swizzled box
constexpr int SOFTMAX_WARPS = 8;    // two per TMEM lane quadrant: each thread owns half a row (64 columns)
constexpr int THREADS = 64 + SOFTMAX_WARPS * 32;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t S_COL0 = 0, O_COL0 = 256;   // S buffers at columns 0 and 128, O_g at 256 + 128 g
constexpr long long TIMEOUT_CYCLES = 2000000000ll;  // about a second

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + TILE_BYTES;
constexpr int OFF_V = OFF_K + KST * TILE_BYTES;
constexpr int OFF_BAR = OFF_V + VST * TILE_BYTES;
constexpr int NUM_BARS = 1 + 2 * KST + 2 * VST + 2 + 2;
constexpr int OFF_XCH = OFF_BAR + 8 * NUM_BARS + 16;               // after the barriers and the tmem slot / abort word
constexpr int XCH_BYTES = 2 * BM * 4;                              // row maxima / sums exchanged between the two halves
constexpr int SMEM_BYTES = OFF_XCH + XCH_BYTES + 1024;             // + alignment slack

// ---- PTX wrappers ---------------------------------------------------------------------------------
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
// Bounded wait: false when the barrier did not complete in time or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > TIMEOUT_CYCLES) {
            *abort_flag = 1;
            return false;
        }
    }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A operand from tensor memory (the bf16 probabilities written by the softmax warps)
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor (tcgen05): 128-byte swizzle, descriptor version 1.
//   K-major operand (rows of 64 bf16 = 128 B, 8-row groups 1024 B apart): lbo unused, sbo = 1024.
//   MN-major operand (V: rows = keys, 64 head-dim columns per box): lbo = distance between the two
//   64-column boxes, sbo = 1024 (8 keys).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, M = 128, N = 128.
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// mbarrier addresses, computed rather than stored so that stage indices stay in registers
struct Bars {
    uint32_t base;
    __device__ __forceinline__ uint32_t q_full() const { return base; }
    __device__ __forceinline__ uint32_t k_full(int i) const { return base + 8 * (1 + i); }
    __device__ __forceinline__ uint32_t k_empty(int i) const { return base + 8 * (1 + KST + i); }
    __device__ __forceinline__ uint32_t v_full(int i) const { return base + 8 * (1 + 2 * KST + i); }
    __device__ __forceinline__ uint32_t v_empty(int i) const { return base + 8 * (1 + 2 * KST + VST + i); }
    __device__ __forceinline__ uint32_t s_full(int i) const { return base + 8 * (1 + 2 * KST + 2 * VST + i); }
    __device__ __forceinline__ uint32_t p_full() const { return base + 8 * (3 + 2 * KST + 2 * VST); }
    __device__ __forceinline__ uint32_t pv_done() const { return base + 8 * (4 + 2 * KST + 2 * VST); }
};

__global__ void __launch_bounds__(THREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const int* __restrict__ n_groups,
                  const GroupEntry* __restrict__ groups, __nv_bfloat16* __restrict__ out, WsHeader* __restrict__ hdr,
                  int H, int k, int T_len, float scale_log2, int causal, int n_qtiles) {
    const int b = blockIdx.z, slot = blockIdx.y;
    if (slot >= n_groups[b]) return;
    const GroupEntry e = groups[(size_t)b * H + slot];
    const int qt = n_qtiles - 1 - (int)blockIdx.x;  // heaviest query tiles first
    const int q0 = qt * BM;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool dbg = blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;

    if (e.cluster < 0) {  // unresolved heads: zero rows
        for (int g = 0; g < e.n; ++g) {
            uint4* o = reinterpret_cast<uint4*>(out + (((size_t)b * H + e.heads[g]) * T_len + q0) * HD);
            const int rows = min(BM, T_len - q0);
            for (int idx = tid; idx < rows * (HD / 8); idx += THREADS) o[idx] = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    const int n_members = min(e.n, G);
    long long cta_t0 = 0;
    if (tid == 0) asm volatile("mov.u64 %0, %globaltimer;" : "=l"(cta_t0));
    const int n_kv = causal ? min(qt + 1, (T_len + BN - 1) / BN) : (T_len + BN - 1) / BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 8 * NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const Bars bar{sbase + OFF_BAR};

    if (tid == 0) {
        mbar_init(bar.q_full(), 1);
        for (int i = 0; i < KST; ++i) { mbar_init(bar.k_full(i), 1); mbar_init(bar.k_empty(i), 1); }
        for (int i = 0; i < VST; ++i) { mbar_init(bar.v_full(i), 1); mbar_init(bar.v_empty(i), 1); }
        for (int i = 0; i < 2; ++i) mbar_init(bar.s_full(i), 1);
        mbar_init(bar.p_full(), SOFTMAX_WARPS * 32);
        mbar_init(bar.pv_done(), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_proxy();
    }
    if (warp == 1) {  // whole warp: allocate all 512 TMEM columns (one CTA per SM by shared-memory size)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const int q_plane = b * H + e.rep, k_plane = b * k + e.cluster;
            mbar_expect_tx(bar.q_full(), TILE_BYTES);
            tma_load_3d(sbase + OFF_Q, &map_q, 0, q0, q_plane, bar.q_full());
            tma_load_3d(sbase + OFF_Q + HALF_BYTES, &map_q, 64, q0, q_plane, bar.q_full());
            bool ok = true;
            auto load_k = [&](int j) -> bool {
                const int ks = j % KST;
                if (!mbar_wait(bar.k_empty(ks), ((j / KST) & 1) ^ 1, abort_flag)) return false;
                mbar_expect_tx(bar.k_full(ks), TILE_BYTES);
                tma_load_3d(sbase + OFF_K + ks * TILE_BYTES, &map_k, 0, j * BN, k_plane, bar.k_full(ks));
                tma_load_3d(sbase + OFF_K + ks * TILE_BYTES + HALF_BYTES, &map_k, 64, j * BN, k_plane, bar.k_full(ks));
                return true;
            };
            // order of need: K(0), K(1), V(0,*), K(2), V(1,*), ...  (S of tile j+1 is computed before P V of tile j)
            ok = load_k(0);
            for (int j = 0; j < n_kv && ok; ++j) {
                if (dbg && j < 16) g_pf_stats[48 + j][0] = clock64();
                if (j + 1 < n_kv) ok = load_k(j + 1);
                if (dbg && j < 16) g_pf_stats[48 + j][1] = clock64();
                for (int g = 0; g < n_members && ok; ++g) {
                    const int t = j * n_members + g, vs = t % VST;
                    ok = mbar_wait(bar.v_empty(vs), ((t / VST) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    if (dbg && j < 16 && g < 2) g_pf_stats[48 + j][2 + g] = clock64();
                    const int v_plane = b * H + e.heads[g];
                    mbar_expect_tx(bar.v_full(vs), TILE_BYTES);
                    tma_load_3d(sbase + OFF_V + vs * TILE_BYTES, &map_v, 0, j * BN, v_plane, bar.v_full(vs));
                    tma_load_3d(sbase + OFF_V + vs * TILE_BYTES + HALF_BYTES, &map_v, 64, j * BN, v_plane, bar.v_full(vs));
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t IDESC_QK = make_idesc(false), IDESC_PV = make_idesc(true);
            // Descriptors are built once; inside the loops only the 14-bit start-address field (low word)
            // moves, by compile-time offsets, so issuing an MMA costs the thread an add and the instruction.
            const uint64_t dq = make_desc(sbase + OFF_Q, 16, 1024);
            const uint64_t dk = make_desc(sbase + OFF_K, 16, 1024);
            const uint64_t dv = make_desc(sbase + OFF_V, HALF_BYTES, 1024);
            const uint32_t hi_k = (uint32_t)(dq >> 32), hi_v = (uint32_t)(dv >> 32);
            const uint32_t q_lo = (uint32_t)dq, k_lo = (uint32_t)dk, v_lo = (uint32_t)dv;
            auto desc = [](uint32_t hi, uint32_t lo) { return ((uint64_t)hi << 32) | lo; };
            bool ok = mbar_wait(bar.q_full(), 0, abort_flag);
            auto issue_qk = [&](int j) -> bool {
                const int ks = j % KST, sb = j & 1;
                if (!mbar_wait(bar.k_full(ks), (j / KST) & 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t d = tmem_base + S_COL0 + sb * BN;
                const uint32_t kb = k_lo + ks * (TILE_BYTES >> 4);
#pragma unroll
                for (int s = 0; s < HD / 16; ++s) {
                    const uint32_t off = ((s >> 2) * HALF_BYTES + (s & 3) * 32) >> 4;
                    tc_mma(d, desc(hi_k, q_lo + off), desc(hi_k, kb + off), IDESC_QK, s > 0);
                }
                tc_commit(bar.k_empty(ks));
                tc_commit(bar.s_full(sb));
                return true;
            };
            if (ok) ok = issue_qk(0);
            for (int j = 0; j < n_kv && ok; ++j) {
                if (j + 1 < n_kv) ok = issue_qk(j + 1);
                if (!ok) break;
                if (dbg && j < 64) g_pf_stats[j][5] = clock64();
                ok = mbar_wait(bar.p_full(), j & 1, abort_flag);
                if (dbg && j < 16) g_pf_stats[32 + j][0] = clock64();
                for (int g = 0; g < n_members && ok; ++g) {
                    const int t = j * n_members + g;
                    ok = mbar_wait(bar.v_full(t % VST), (t / VST) & 1, abort_flag);
                }
                if (!ok) break;
                tc_fence_after();
                if (dbg && j < 64) g_pf_stats[j][6] = clock64();
                const uint32_t p_addr = tmem_base + S_COL0 + (j & 1) * BN;  // P(j): first 64 columns of S(j)
                for (int g = 0; g < n_members; ++g) {
                    const int vs = (j * n_members + g) % VST;
                    const uint32_t d = tmem_base + O_COL0 + g * HD;
                    const uint32_t vb = v_lo + vs * (TILE_BYTES >> 4);
#pragma unroll
                    for (int s = 0; s < BN / 16; ++s)  // 16 keys per step: 8 TMEM columns of P, 2048 bytes of V
                        tc_mma_ts(d, p_addr + s * 8, desc(hi_v, vb + s * (2048 >> 4)), IDESC_PV, (j > 0 || s > 0) ? 1u : 0u);
                    tc_commit(bar.v_empty(vs));
                }
                if (!ok) break;
                tc_commit(bar.pv_done());
                if (dbg && j < 64) g_pf_stats[j][7] = clock64();
            }
        }
    } else {
        // ---------------- softmax / correction / epilogue: two threads per query row ----------------
        // Warps 2..5 own columns 0..63 of their rows, warps 6..9 columns 64..127; the two threads of a row
        // sit in different warps of the same TMEM lane quadrant and meet once per tile at a 64-thread
        // named barrier, where they exchange their half-row maxima.  By then both have their 64 scores in
        // registers, so writing P over the S buffer afterwards cannot clobber anything still needed.
        const int quad = warp & 3;               // TMEM lanes this warp may touch
        const int half = (warp - 2) >> 2;        // which 64 columns of the tile
        const int row = quad * 32 + lane;        // row of the tile
        const int row_abs = q0 + row;
        const int cbase = half * 64;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        float* xch = reinterpret_cast<float*>(smem + OFF_XCH);  // [half][row]
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + quad) : "memory"); };
        float m_used = -INFINITY, l_run = 0.f;
        bool ok = true;
        uint32_t r[64];
        for (int j = 0; j < n_kv && ok; ++j) {
            const int sb = j & 1;
            const bool rec = dbg && tid == 64 && j < 64;
            if (rec) g_pf_stats[j][0] = clock64();
            ok = __all_sync(0xffffffffu, mbar_wait(bar.s_full(sb), (j >> 1) & 1, abort_flag));
            if (!ok) break;  // warp-uniform: the tcgen05 loads below are warp-collective
            if (rec) g_pf_stats[j][1] = clock64();
            tc_fence_after();
            const uint32_t s_addr = lane_addr + S_COL0 + sb * BN;
            const int col0 = j * BN;
            // columns of this thread's half that the row may see: col_abs < T and (causal: col_abs <= row_abs)
            int vis = T_len - col0;
            if (causal) vis = min(vis, row_abs - col0 + 1);
            vis = max(0, min(vis - cbase, 64));
            // the whole tile is visible to every row unless it is the diagonal tile or runs past T
            const bool full_tile = col0 + BN <= T_len && (!causal || col0 + BN - 1 <= q0);
            tc_ld32(s_addr + cbase, r);
            tc_ld32(s_addr + cbase + 32, r + 32);
            tc_wait_ld();
            float mx0 = -INFINITY, mx1 = -INFINITY;
            if (full_tile) {
#pragma unroll
                for (int i = 0; i < 64; i += 2) {
                    mx0 = fmaxf(mx0, __uint_as_float(r[i]));
                    mx1 = fmaxf(mx1, __uint_as_float(r[i + 1]));
                }
            } else {
#pragma unroll
                for (int i = 0; i < 64; ++i)
                    if (i < vis) mx0 = fmaxf(mx0, __uint_as_float(r[i]));
            }
            float mx = fmaxf(mx0, mx1);
            xch[half * BM + row] = mx;
            pair_sync();
            mx = fmaxf(mx, xch[(half ^ 1) * BM + row]);
            pair_sync();  // both values read before either slot is written again
            if (rec) g_pf_stats[j][2] = clock64();
            const float m_tile = mx * scale_log2;
            float m_new = m_used, corr = 1.f;
            if (m_tile > m_used + 8.f) {  // lazy rescale: only when the reference would be off by > 2^8
                m_new = m_tile;
                corr = fast_exp2(m_used - m_new);  // 0 on the first tile (m_used = -inf)
            }
            const float m_ref = m_new == -INFINITY ? 0.f : m_new;
            // probabilities, rounded to bf16, two per 32-bit column, written over the first half of the S
            // buffer: the layout of an A operand in tensor memory.  S columns 64 h + c map to P column 32 h + c / 2.
            float ls0 = 0.f, ls1 = 0.f, ls2 = 0.f, ls3 = 0.f;
            uint32_t packed[32];
            if (full_tile) {
#pragma unroll
                for (int i = 0; i < 64; i += 4) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(r[i]), scale_log2, -m_ref));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(r[i + 1]), scale_log2, -m_ref));
                    const float p2 = fast_exp2(fmaf(__uint_as_float(r[i + 2]), scale_log2, -m_ref));
                    const float p3 = fast_exp2(fmaf(__uint_as_float(r[i + 3]), scale_log2, -m_ref));
                    ls0 += p0;
                    ls1 += p1;
                    ls2 += p2;
                    ls3 += p3;
                    __nv_bfloat162 pa = __floats2bfloat162_rn(p0, p1), pb = __floats2bfloat162_rn(p2, p3);
                    packed[i >> 1] = *reinterpret_cast<uint32_t*>(&pa);
                    packed[(i >> 1) + 1] = *reinterpret_cast<uint32_t*>(&pb);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 64; i += 2) {
                    float p0 = fast_exp2(fmaf(__uint_as_float(r[i]), scale_log2, -m_ref));
                    float p1 = fast_exp2(fmaf(__uint_as_float(r[i + 1]), scale_log2, -m_ref));
                    if (i >= vis) p0 = 0.f;
                    if (i + 1 >= vis) p1 = 0.f;
                    ls0 += p0;
                    ls1 += p1;
                    __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                    packed[i >> 1] = *reinterpret_cast<uint32_t*>(&pk);
                }
            }
            tc_st16(s_addr + half * 32, packed);
            tc_st16(s_addr + half * 32 + 16, packed + 16);
            l_run = l_run * corr + ((ls0 + ls1) + (ls2 + ls3));
            m_used = m_new;
            if (rec) g_pf_stats[j][3] = clock64();
            // the previous tile's PV must be complete before the O accumulators are rescaled
            if (j > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar.pv_done(), (j - 1) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                if (__any_sync(0xffffffffu, corr != 1.f)) {  // this thread rescales its 64 columns of each O
                    for (int g = 0; g < n_members; ++g) {
                        const uint32_t o_addr = lane_addr + O_COL0 + g * HD + cbase;
                        tc_ld32(o_addr, r);
                        tc_ld32(o_addr + 32, r + 32);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 64; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * corr);
                        tc_st32(o_addr, r);
                        tc_st32(o_addr + 32, r + 32);
                    }
                }
            }
            tc_wait_st();          // P (and any rescaled O) is in tensor memory
            tc_fence_before();
            mbar_arrive(bar.p_full());
            if (rec) g_pf_stats[j][4] = clock64();
            if (dbg && j < 16) atomicMax(reinterpret_cast<unsigned long long*>(&g_pf_stats[32 + j][2]), (unsigned long long)clock64());
        }
        // epilogue: O_g / l -> bf16 -> global; the row sum is the sum of the two halves' sums
        if (ok) ok = mbar_wait(bar.pv_done(), (n_kv - 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        {
            xch[half * BM + row] = l_run;
            pair_sync();
            l_run += xch[(half ^ 1) * BM + row];
        }
        if (ok) {
            tc_fence_after();
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            for (int g = 0; g < n_members; ++g) {
                __nv_bfloat16* orow = out + (((size_t)b * H + e.heads[g]) * T_len + row_abs) * HD + cbase;
                tc_ld32(lane_addr + O_COL0 + g * HD + cbase, r);
                tc_ld32(lane_addr + O_COL0 + g * HD + cbase + 32, r + 32);
                tc_wait_ld();
                if (row_abs < T_len) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        uint32_t w[4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            __nv_bfloat162 pk = __floats2bfloat162_rn(__uint_as_float(r[8 * u + 2 * x]) * inv,
                                                                      __uint_as_float(r[8 * u + 2 * x + 1]) * inv);
                            w[x] = *reinterpret_cast<uint32_t*>(&pk);
                        }
                        *reinterpret_cast<uint4*>(orow + u * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
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
    if (tid == 0) {
        long long t1;
        unsigned smid;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
        asm volatile("mov.u32 %0, %smid;" : "=r"(smid));
        const int idx = atomicAdd(&g_pf_cta_n, 1);
        if (idx < 4096) {
            g_pf_cta[idx][0] = smid;
            g_pf_cta[idx][1] = cta_t0;
            g_pf_cta[idx][2] = t1;
            g_pf_cta[idx][3] = n_kv;
        }
    }
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

// [planes, T, 128] bf16 viewed as a 3-D tensor (innermost first); box = 64 columns x 128 rows x 1 plane.
static bool make_map(CUtensorMap* map, const void* base, int planes, int T) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {(cuuint64_t)HD, (cuuint64_t)T, (cuuint64_t)planes};
    cuuint64_t strides[2] = {(cuuint64_t)HD * 2, (cuuint64_t)T * HD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)BN, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace chai

extern "C" int chai_prefill_attention(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                                      const int32_t* reps, void* out, int B, int H, int k, int T, int D, float scale,
                                      int causal, int dtype, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace chai;
    if (dtype != CHAI_BF16 || D != tc::HD)
        return chai_prefill_attention_simt(q, k_rep, v, membership, reps, out, B, H, k, T, D, scale, causal, dtype,
                                           workspace, workspace_bytes, stream);
    int rc = prefill_check_args("chai_prefill_attention", q, k_rep, v, membership, reps, out, B, H, k, T, D, dtype,
                                workspace, workspace_bytes);
    if (rc != CHAI_OK) return rc;
    CUtensorMap mq, mk, mv;
    CHAI_REQUIRE(tc::make_map(&mq, q, B * H, T) && tc::make_map(&mk, k_rep, B * k, T) && tc::make_map(&mv, v, B * H, T),
                 CHAI_ERR_CUDA, "chai_prefill_attention: cuTensorMapEncodeTiled failed");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    rc = prefill_run_plan(membership, reps, B, H, k, tc::G, ws, s);
    if (rc != CHAI_OK) return rc;
    const PrefillLayout L = prefill_layout(B, H);
    cudaError_t e = cudaFuncSetAttribute(tc::prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES);
    if (e != cudaSuccess) return cuda_fail(e, "prefill_tc_kernel shared-memory opt-in");
    const int n_qtiles = (T + tc::BM - 1) / tc::BM;
    tc::prefill_tc_kernel<<<dim3(n_qtiles, H, B), tc::THREADS, tc::SMEM_BYTES, s>>>(
        mq, mk, mv, reinterpret_cast<const int*>(ws + L.off_ngroups),
        reinterpret_cast<const GroupEntry*>(ws + L.off_groups), static_cast<__nv_bfloat16*>(out),
        reinterpret_cast<WsHeader*>(ws), H, k, T, scale * 1.4426950408889634f, causal, n_qtiles);
    CHAI_LAUNCH_CHECK("prefill_tc_kernel launch");
    return CHAI_OK;
}

// Debugging aid (not part of the public interface): stage timestamps of one CTA of the last tensor-core prefill.
extern "C" int chai_debug_prefill_ctas(long long* host_out, int max_ctas, int* n_out) {
    if (host_out == nullptr || n_out == nullptr || max_ctas <= 0 || max_ctas > 4096) return CHAI_ERR_INVALID_ARG;
    int zero = 0;
    cudaError_t e = cudaMemcpyFromSymbol(n_out, chai::tc::g_pf_cta_n, sizeof(int));
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(host_out, chai::tc::g_pf_cta, sizeof(long long) * 4 * max_ctas);
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(chai::tc::g_pf_cta_n, &zero, sizeof(int));
    return e == cudaSuccess ? CHAI_OK : chai::cuda_fail(e, "chai_debug_prefill_ctas");
}

extern "C" int chai_debug_prefill_stats(long long* host_out) {
    if (host_out == nullptr) return CHAI_ERR_INVALID_ARG;
    cudaError_t e = cudaMemcpyFromSymbol(host_out, chai::tc::g_pf_stats, sizeof(long long) * 64 * 8);
    return e == cudaSuccess ? CHAI_OK : chai::cuda_fail(e, "chai_debug_prefill_stats");
}
