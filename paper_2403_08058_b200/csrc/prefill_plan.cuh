// Work list of clustered prefill attention: (cluster, member group) entries per request.
//
// A prefill CTA keeps one output accumulator per member head while it walks the key tiles of a
// representative, so a cluster's members are cut into groups of at most `gmax` heads (sizes as even
// as possible); each group recomputes the representative's scores.  Groups are listed largest
// first so that the heaviest CTAs start first.  Heads whose membership data are inconsistent are
// collected into groups with cluster = -1, whose CTAs only write zeros.
#pragma once

#include "chai_common.cuh"

namespace chai {

constexpr int kGroupMax = 4;  // capacity of one entry; kernels use gmax <= kGroupMax

struct GroupEntry {
    int cluster;  // -1: zero-fill group
    int rep;      // representative head (query rows and K slot owner)
    int n;        // heads in this group
    int pad;
    int heads[kGroupMax];
};
static_assert(sizeof(GroupEntry) == 32, "GroupEntry is 32 bytes");

struct PrefillLayout {
    size_t off_ngroups, off_bad, off_groups, total;
};

inline PrefillLayout prefill_layout(int B, int H) {
    PrefillLayout L;
    size_t off = sizeof(WsHeader);
    L.off_ngroups = off;
    off = round_up(off + sizeof(int) * (size_t)B, 256);
    L.off_bad = off;
    off = round_up(off + sizeof(int) * (size_t)B, 256);
    L.off_groups = off;
    off = round_up(off + sizeof(GroupEntry) * (size_t)B * H, 256);
    L.total = off;
    return L;
}

// grid B, block 128.  Shared memory: H + k ints, k * ceil(H / 32) mask words, 2 * k ints (see prefill_plan_smem).
// Outputs per request: n_groups[b], bad[b] (first unresolved head + 1, or 0) and the group entries.  Block 0
// also clears the work counters in the workspace header (words pad[0..59]) for the attention kernel that
// follows on the stream; the status word itself is written by that kernel from the bad[] flags, so no
// separate clearing pass is needed and no flag can be lost to a race.
// The kernel sits between two attention calls on the critical path, so it is built for latency: the members
// of every cluster are found with one warp-wide match per 32 heads (a bit mask per cluster), group sizes and
// slots follow from population counts and a warp scan, and each cluster's thread writes its entries straight
// to global memory.
inline size_t prefill_plan_smem(int H, int k) {
    return sizeof(int) * ((size_t)H + 3 * (size_t)k + (size_t)k * ((H + 31) / 32));
}

static __global__ void __launch_bounds__(128)
prefill_plan_kernel(const int32_t* __restrict__ membership, const int32_t* __restrict__ reps, WsHeader* __restrict__ hdr,
                    int* __restrict__ n_groups, int* __restrict__ bad_out, GroupEntry* __restrict__ groups, int H, int k,
                    int gmax) {
    extern __shared__ __align__(16) int s_plan[];
    const int W = (H + 31) >> 5;             // 32-head words per mask
    int* mem = s_plan;                       // [H] membership of this request
    int* rep = mem + H;                      // [k] representative of each cluster, -1 if the cluster is unusable
    int* ngrp = rep + k;                     // [k] groups of the cluster
    int* slot = ngrp + k;                    // [k] first group slot of the cluster
    unsigned* mask = reinterpret_cast<unsigned*>(slot + k);  // [k][W] members of each usable cluster
    __shared__ int s_total, s_first_bad, s_nbad;
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    // a kernel launched as a programmatic dependent may start its own set-up now; it still waits for this
    // grid to finish (griddepcontrol.wait) before it reads anything written here
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // launched as a programmatic dependent itself, the planner may be here while its predecessor still runs
    // (and still uses the workspace): wait for it before the first access to global memory
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (b == 0)
        for (int i = tid; i < 60; i += nt) hdr->pad[i] = 0;
    for (int h = tid; h < H; h += nt) mem[h] = membership[(size_t)b * H + h];
    for (int c = tid; c < k; c += nt) rep[c] = reps[(size_t)b * k + c];
    for (int i = tid; i < k * W; i += nt) mask[i] = 0u;
    if (tid == 0) {
        s_first_bad = H;
        s_nbad = 0;
    }
    __syncthreads();
    // a cluster is usable when its representative is a head of that very cluster
    for (int c = tid; c < k; c += nt) {
        const int r = rep[c];
        if (!(r >= 0 && r < H && mem[r] == c)) rep[c] = -1;
    }
    __syncthreads();
    // member masks: the heads of a 32-head word that share a cluster find each other with one match
    for (int h0 = (tid >> 5) << 5; h0 < H; h0 += nt) {  // (whole warps walk the words: h0 is warp-uniform)
        const int h = h0 + lane;
        int c = -2;                                       // lanes past H
        if (h < H) {
            c = mem[h];
            if (c < 0 || c >= k || rep[c] < 0) c = -1;    // unresolved head
        }
        const unsigned peers = __match_any_sync(0xffffffffu, c);
        if (c >= 0 && lane == __ffs(peers) - 1) mask[c * W + (h0 >> 5)] = peers;
        if (c == -1) {
            atomicMin(&s_first_bad, h);
            if (lane == __ffs(peers) - 1) atomicAdd(&s_nbad, __popc(peers));
        }
    }
    __syncthreads();
    // groups per cluster (sizes as even as possible) and their slots, in cluster order: warp 0 scans
    if (tid < 32) {
        int carry = 0;
        for (int c0 = 0; c0 < k; c0 += 32) {
            const int c = c0 + lane;
            int n = 0;
            if (c < k && rep[c] >= 0)
                for (int w = 0; w < W; ++w) n += __popc(mask[c * W + w]);
            const int ng = (n + gmax - 1) / gmax;
            int incl = ng;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            if (c < k) {
                ngrp[c] = ng;
                slot[c] = carry + incl - ng;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) s_total = carry;
    }
    __syncthreads();
    GroupEntry* out = groups + (size_t)b * H;
    // every usable cluster writes its own groups, members in ascending head order
    for (int c = tid; c < k; c += nt) {
        const int ng = ngrp[c];
        if (ng <= 0) continue;
        int n = 0;
        for (int w = 0; w < W; ++w) n += __popc(mask[c * W + w]);
        const int base = n / ng, rem = n % ng;
        int gi = 0, filled = 0, size = rem > 0 ? base + 1 : base;
        int hd[kGroupMax];
        for (int w = 0; w < W; ++w) {
            unsigned m = mask[c * W + w];
            while (m) {
                const int h = (w << 5) + __ffs(m) - 1;
                m &= m - 1;
                if (filled == 0) {
#pragma unroll
                    for (int x = 0; x < kGroupMax; ++x) hd[x] = h;  // unused slots repeat the first head
                }
#pragma unroll
                for (int x = 0; x < kGroupMax; ++x)
                    if (x == filled) hd[x] = h;
                if (++filled == size) {
                    int4* dst = reinterpret_cast<int4*>(out + slot[c] + gi);
                    dst[0] = make_int4(c, rep[c], size, 0);
                    dst[1] = make_int4(hd[0], hd[1], hd[2], hd[3]);
                    filled = 0;
                    ++gi;
                    size = gi < rem ? base + 1 : base;
                }
            }
        }
    }
    // zero-fill groups for unresolved heads (rare): one thread, after the usable clusters' slots; like every
    // other group they hold at most gmax heads, which is all an attention CTA looks at
    const int total = s_total, nbad = s_nbad;
    if (tid == 0) {
        if (nbad > 0) {
            int cnt = 0, hd[kGroupMax];
            for (int h = 0; h < H; ++h) {
                const int c = mem[h];
                if (!(c < 0 || c >= k || rep[c] < 0)) continue;
                if (cnt % gmax == 0) {
#pragma unroll
                    for (int x = 0; x < kGroupMax; ++x) hd[x] = h;
                }
#pragma unroll
                for (int x = 0; x < kGroupMax; ++x)
                    if (x == cnt % gmax) hd[x] = h;
                ++cnt;
                if (cnt % gmax == 0 || cnt == nbad) {
                    int4* dst = reinterpret_cast<int4*>(out + total + (cnt - 1) / gmax);
                    dst[0] = make_int4(-1, -1, (cnt - 1) % gmax + 1, 0);
                    dst[1] = make_int4(hd[0], hd[1], hd[2], hd[3]);
                }
            }
        }
        n_groups[b] = total + (nbad + gmax - 1) / gmax;
        bad_out[b] = nbad > 0 ? s_first_bad + 1 : 0;
    }
}

// Status word from the planner's per-request flags (run by one thread of the attention kernel that follows).
__device__ __forceinline__ void publish_plan_status(WsHeader* hdr, const int* bad, int B) {
    int st = CHAI_OK, bb = -1, bh = -1;
    for (int b = 0; b < B; ++b)
        if (bad[b] != 0) {
            st = CHAI_ERR_BAD_MEMBERSHIP;
            bb = b;
            bh = bad[b] - 1;
            break;
        }
    hdr->status = st;
    hdr->bad_b = bb;
    hdr->bad_h = bh;
}

}  // namespace chai
