// Workspace layout shared by the two decode implementations (split kernels and persistent kernel).
#pragma once

#include "chai_common.cuh"

namespace chai {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kStepsK = 8;   // independent 16-byte loads per thread in flight, score kernel
constexpr int kStepsV = 16;  // rows per thread in a value chunk (two batches of 8 loads)
constexpr int kTileBytes = 32768;     // persistent kernel: one ring slot = TR cache rows ...
constexpr int kTileBytesFp8 = 16384;  // ... of half the size for one-byte elements (same number of elements per tile)
inline int decode_tile_bytes(int dtype) { return dtype == CHAI_FP8_E4M3 ? kTileBytesFp8 : kTileBytes; }

// Long contexts: a head's item partials are added in groups of this many, then the group sums (a fixed tree,
// so the result does not depend on who adds).
constexpr int kCombineGroup = 16;

struct DecodeLayout {
    int CK, CV, nK, nV;  // split kernels: rows per key / value chunk and chunks per plane
    int TR;              // persistent kernel: rows per 16 KB tile
    int capK, capV;      // entries per plane reserved for chunk maxima / partials (either implementation)
    int capG;            // groups of kCombineGroup value items per head (tickets of the two-level combine)
    size_t off_counters, off_gcnt, off_flags, off_scores, off_cmax, off_pmax, off_lpart, off_opart, total;
};

// off_flags: 64-bit words of the persistent kernel: [0] carries the launch token once the layer's first key tile
// is done (status and work counter are reset by then); [2 + p] carries it once every key tile of plane p is
// done and off_pmax[p] holds the plane's largest score; [2 + B*k + p] counts plane p's finished key tiles.

inline bool decode_layout(int B, int H, int k, int T, int D, int dtype, DecodeLayout* L) {
    const int es = (int)elem_size(dtype);
    const int epv = 16 / es;
    if (D != 64 && D != 128) return false;
    const int lpr = D / epv, rpw = 32 / lpr, rps = kDecWarps * rpw;
    L->CK = rps * kStepsK;
    L->CV = rps * kStepsV;
    L->nK = (T + L->CK - 1) / L->CK;
    L->nV = (T + L->CV - 1) / L->CV;
    L->TR = decode_tile_bytes(dtype) / (D * es);
    // the persistent kernel deals key work tile by tile and value work in items of 2 tiles
    const int pk = (T + L->TR - 1) / L->TR, pv = (T + 2 * L->TR - 1) / (2 * L->TR);
    L->capK = pk > L->nK ? pk : L->nK;
    L->capV = pv > L->nV ? pv : L->nV;
    size_t off = sizeof(WsHeader);
    L->off_counters = off;
    off = round_up(off + sizeof(int) * (size_t)B * H, 256);
    L->capG = (L->capV + kCombineGroup - 1) / kCombineGroup;
    L->off_gcnt = off;
    off = round_up(off + sizeof(int) * (size_t)B * H * L->capG, 256);
    L->off_flags = off;
    off = round_up(off + sizeof(unsigned long long) * (2 * (size_t)B * k + 2), 256);
    L->off_scores = off;
    off = round_up(off + sizeof(float) * (size_t)B * k * T, 256);
    L->off_cmax = off;
    off = round_up(off + sizeof(float) * (size_t)B * k * L->capK, 256);
    L->off_pmax = off;
    off = round_up(off + sizeof(float) * (size_t)B * k, 256);
    L->off_lpart = off;
    off = round_up(off + sizeof(float) * (size_t)B * H * L->capV, 256);
    L->off_opart = off;
    off = round_up(off + sizeof(float) * (size_t)B * H * L->capV * D, 256);
    L->total = off;
    return true;
}

// Persistent decode kernel (decode_persist.cu).  Returns CHAI_OK, an error, or kDecodeNotLaunched
// when the device cannot run it (no cooperative launch), in which case the caller uses the split kernels.
constexpr int kDecodeNotLaunched = -1;
// seq_lens: per-request context lengths on the device (null: every request has T positions; otherwise T is
// the upper bound the workspace was sized for).  k_batch_stride: elements between two requests' first
// representative plane in k_rep (k * T_cap * D for a dense representative cache, H * T_cap * D for a cache
// compacted in place).
int launch_decode_persistent(const void* q, const void* k_rep, const void* v, const int32_t* membership,
                             const int32_t* reps, const int32_t* seq_lens, void* out, int B, int H, int k, int T,
                             int T_cap, int D, size_t k_batch_stride, float scale, int dtype, char* ws,
                             const DecodeLayout& L, cudaStream_t s, const float* k_scale = nullptr,
                             const float* v_scale = nullptr,  // scales: fp8 caches only (dtype CHAI_FP8_E4M3)
                             // CHAI-QKV: H = k heads (the clusters), reps names representatives among the Hq heads of
                             // q / out, and out_membership [B,Hq] says which heads receive each cluster's row
                             const int32_t* out_membership = nullptr, int Hq = 0);

}  // namespace chai
