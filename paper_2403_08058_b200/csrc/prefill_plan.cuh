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
    size_t off_ngroups, off_groups, total;
};

inline PrefillLayout prefill_layout(int B, int H) {
    PrefillLayout L;
    size_t off = sizeof(WsHeader);
    L.off_ngroups = off;
    off = round_up(off + sizeof(int) * (size_t)B, 256);
    L.off_groups = off;
    off = round_up(off + sizeof(GroupEntry) * (size_t)B * H, 256);
    L.total = off;
    return L;
}

// grid B, block 128.  Shared memory: 3*k + H ints.  The caller clears the workspace header first.
static __global__ void __launch_bounds__(128)
prefill_plan_kernel(const int32_t* __restrict__ membership, const int32_t* __restrict__ reps, WsHeader* __restrict__ hdr,
                    int* __restrict__ n_groups, GroupEntry* __restrict__ groups, int H, int k, int gmax) {
    extern __shared__ int s_plan[];
    int* cnt = s_plan;        // [k] members of a valid cluster, -1 for an unusable slot
    int* slot0 = cnt + k;     // [k] first slot of the cluster's larger groups
    int* slot1 = slot0 + k;   // [k] first slot of the cluster's smaller groups
    int* bad = slot1 + k;     // [H] 1 if the head cannot be resolved
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    const int32_t* mem = membership + (size_t)b * H;
    GroupEntry* g = groups + (size_t)b * H;

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
    for (int h = tid; h < H; h += nt) {
        const int c = mem[h];
        bad[h] = (c < 0 || c >= k || cnt[c] < 0) ? 1 : 0;
    }
    __syncthreads();
    if (tid == 0) {
        // group sizes present: for a cluster of n heads cut into ng = ceil(n/gmax) groups, `rem` groups
        // have base+1 heads and the rest have base heads.  Slots are handed out by size, largest first.
        int next = 0;
        for (int size = gmax; size >= 1; --size) {
            for (int c = 0; c < k; ++c) {
                const int n = cnt[c];
                if (n <= 0) continue;
                const int ng = (n + gmax - 1) / gmax, base = n / ng, rem = n % ng;
                if (rem > 0 && base + 1 == size) {
                    slot0[c] = next;
                    next += rem;
                }
                if (base == size) {
                    slot1[c] = next;
                    next += ng - rem;
                }
            }
        }
        // zero-fill groups for unresolved heads
        int nbad = 0, first_bad = -1;
        for (int h = 0; h < H; ++h) {
            if (!bad[h]) continue;
            if (first_bad < 0) first_bad = h;
            GroupEntry* e = g + next + nbad / kGroupMax;
            if (nbad % kGroupMax == 0) {
                e->cluster = -1;
                e->rep = -1;
                e->n = 0;
                e->pad = 0;
            }
            e->heads[e->n++] = h;
            ++nbad;
        }
        if (nbad > 0) flag_bad_membership(hdr, b, first_bad);
        next += (nbad + kGroupMax - 1) / kGroupMax;
        n_groups[b] = next;
    }
    __syncthreads();
    // every valid cluster fills its own groups, members in ascending head order
    for (int c = tid; c < k; c += nt) {
        const int n = cnt[c];
        if (n <= 0) continue;
        const int ng = (n + gmax - 1) / gmax, base = n / ng, rem = n % ng;
        const int r = reps[(size_t)b * k + c];
        int gi = 0, filled = 0;
        GroupEntry* e = nullptr;
        for (int h = 0; h < H; ++h) {
            if (mem[h] != c) continue;
            if (filled == 0) {
                e = g + (gi < rem ? slot0[c] + gi : slot1[c] + (gi - rem));
                e->cluster = c;
                e->rep = r;
                e->pad = 0;
                e->n = gi < rem ? base + 1 : base;
            }
            e->heads[filled++] = h;
            if (filled == e->n) {
                filled = 0;
                ++gi;
            }
        }
    }
}

}  // namespace chai
