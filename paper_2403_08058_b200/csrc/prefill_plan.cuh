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

// grid B, block 128.  Shared memory: 2*k + 2*H ints (rounded up to 4) + H group entries.
// Outputs per request: n_groups[b], bad[b] (first unresolved head + 1, or 0) and the group entries.  Block 0
// also clears the work counters in the workspace header (words pad[0..59]) for the attention kernel that
// follows on the stream; the status word itself is written by that kernel from the bad[] flags, so no
// separate clearing pass is needed and no flag can be lost to a race.
static __global__ void __launch_bounds__(128)
prefill_plan_kernel(const int32_t* __restrict__ membership, const int32_t* __restrict__ reps, WsHeader* __restrict__ hdr,
                    int* __restrict__ n_groups, int* __restrict__ bad_out, GroupEntry* __restrict__ groups, int H, int k,
                    int gmax) {
    extern __shared__ __align__(16) int s_plan[];
    int* cnt = s_plan;        // [k] members of a valid cluster, -1 for an unusable slot
    int* slot = cnt + k;      // [k] first group slot of the cluster
    int* mem = slot + k;      // [H] membership of this request
    int* bad = mem + H;       // [H] 1 if the head cannot be resolved
    GroupEntry* ent = reinterpret_cast<GroupEntry*>(s_plan + ((2 * k + 2 * H + 3) & ~3));  // [H], 16-byte aligned
    __shared__ int s_next, s_nbad;
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    // a kernel launched as a programmatic dependent may start its own set-up now; it still waits for this
    // grid to finish (griddepcontrol.wait) before it reads anything written here
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // launched as a programmatic dependent itself, the planner may be here while its predecessor still runs
    // (and still uses the workspace): wait for it before the first access to global memory
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (b == 0)
        for (int i = tid; i < 60; i += nt) hdr->pad[i] = 0;
    for (int h = tid; h < H; h += nt) mem[h] = membership[(size_t)b * H + h];
    __syncthreads();
    for (int c = tid; c < k; c += nt) {
        const int r = reps[(size_t)b * k + c];
        int n = -1;
        if (r >= 0 && r < H && mem[r] == c) {
            n = 0;
            for (int h = 0; h < H; ++h) n += (mem[h] == c);
        }
        cnt[c] = n;
    }
    __syncthreads();
    int my_bad = 0;
    for (int h = tid; h < H; h += nt) {
        const int c = mem[h];
        bad[h] = (c < 0 || c >= k || cnt[c] < 0) ? 1 : 0;
        my_bad |= bad[h];
    }
    const int any_bad = __syncthreads_or(my_bad);
    if (tid == 0) {
        // a cluster of n heads is cut into ng = ceil(n / gmax) groups of near-equal size, in cluster order
        int next = 0;
        for (int c = 0; c < k; ++c) {
            slot[c] = next;
            if (cnt[c] > 0) next += (cnt[c] + gmax - 1) / gmax;
        }
        int nbad = 0, first_bad = -1;
        if (any_bad) {  // zero-fill groups for unresolved heads
            for (int h = 0; h < H; ++h) {
                if (!bad[h]) continue;
                if (first_bad < 0) first_bad = h;
                GroupEntry* e = ent + next + nbad / kGroupMax;
                if (nbad % kGroupMax == 0) {
                    e->cluster = -1;
                    e->rep = -1;
                    e->n = 0;
                    e->pad = 0;
                }
                e->heads[e->n++] = h;
                ++nbad;
            }
            for (int i = next; i < next + (nbad + kGroupMax - 1) / kGroupMax; ++i)
                for (int x = ent[i].n; x < kGroupMax; ++x) ent[i].heads[x] = ent[i].heads[0];
        }
        s_next = next + (nbad + kGroupMax - 1) / kGroupMax;
        s_nbad = first_bad + 1;
    }
    __syncthreads();
    // every valid cluster fills its own groups, members in ascending head order
    for (int c = tid; c < k; c += nt) {
        const int n = cnt[c];
        if (n <= 0) continue;
        const int ng = (n + gmax - 1) / gmax, base = n / ng, rem = n % ng;
        const int r = reps[(size_t)b * k + c];
        int gi = 0, filled = 0, size = rem > 0 ? base + 1 : base;
        GroupEntry e;
        for (int h = 0; h < H; ++h) {
            if (mem[h] != c) continue;
            if (filled == 0) {
                size = gi < rem ? base + 1 : base;
                e.cluster = c;
                e.rep = r;
                e.n = size;
                e.pad = 0;
                for (int x = 0; x < kGroupMax; ++x) e.heads[x] = h;
            }
            e.heads[filled++] = h;
            if (filled == size) {
                ent[slot[c] + gi] = e;
                filled = 0;
                ++gi;
            }
        }
    }
    __syncthreads();
    const int total = s_next;
    const uint4* src = reinterpret_cast<const uint4*>(ent);
    uint4* dst = reinterpret_cast<uint4*>(groups + (size_t)b * H);
    for (int i = tid; i < total * 2; i += nt) dst[i] = src[i];
    if (tid == 0) {
        n_groups[b] = total;
        bad_out[b] = s_nbad;
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
