"""Seeded synthetic inputs shaped like the paper's workloads.

The paper evaluates LLaMA-7B, LLaMA-33B and OPT-66B on C4 and five zero-shot
suites (Section 4); none of those weights or datasets is used here.  These
generators borrow only the shapes (heads, layers, head_dim 128, sequence 2048 of
Fig. 10) and the qualitative structure the paper reports: heads of one cluster
are strongly correlated (Fig. 2(b)), the number of clusters varies per layer
(Section 3.2) and cluster sizes are skewed, with one dominant cluster (Fig. 11).

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only draws random tensors and random
partitions.  Structure (cluster counts, partitions) comes from numpy generators,
tensor values from a torch.Generator on the requested device; parity tests
create the values once and hand the same bits to both sides.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str          # "f32" | "bf16"
    layers: int
    B: int
    H: int
    D: int
    T: int
    k_choices: tuple    # per-layer cluster count is drawn from these
    partition: str      # "even" | "uneven"
    sigma: float        # value scale of Q/K/V entries
    compaction: bool = False


WORKLOADS = {
    1: Workload("config1-fp32-single-layer", "f32", 1, 1, 32, 128, 256, (8,), "even", 1.0),
    2: Workload("config2-llama7b-decode", "bf16", 32, 16, 32, 128, 2048, (4, 8, 16, 32), "even", 0.5),
    3: Workload("config3-llama33b-decode", "bf16", 60, 8, 52, 128, 4096, (4, 13, 26, 52), "uneven", 0.5),
    4: Workload("config4-opt66b-decode", "bf16", 64, 4, 72, 128, 2048, tuple(range(12, 37)), "uneven",
                0.5, True),
    5: Workload("config5-llama7b-prefill", "bf16", 1, 4, 32, 128, 2048, (8,), "even", 0.5),
}

TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}


def _rng(*key) -> np.random.Generator:
    return np.random.default_rng([int(x) & 0x7FFFFFFF for x in key])


def _tgen(device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(_rng(*key).integers(0, 2**62)))
    return g


def layer_k(cfg_id: int, layer: int, seed: int = 0) -> int:
    """Cluster count of one layer, drawn by seed from the workload's choices."""
    w = WORKLOADS[cfg_id]
    choices = w.k_choices
    return int(choices[int(_rng(seed, cfg_id, layer, 11).integers(0, len(choices)))])


def canonical_labels(labels: np.ndarray):
    """Renumber cluster labels by lowest member index; return (labels [H], reps [k_eff])."""
    labels = np.asarray(labels)
    new = {}
    reps = []
    out = np.empty_like(labels, dtype=np.int32)
    for h, lab in enumerate(labels.tolist()):
        if lab not in new:
            new[lab] = len(new)
            reps.append(h)
        out[h] = new[lab]
    return out, np.asarray(reps, dtype=np.int32)


def make_partition(H: int, k: int, kind: str, rng: np.random.Generator):
    """One partition of H heads into k non-empty clusters, canonical labels.

    even:   a random permutation cut into k groups of near-equal size.
    uneven: every cluster gets one head; each remaining head joins cluster 0 with
            probability 1/2, otherwise a uniformly drawn other cluster.
    Returns (membership [H] int32, reps [k] int32 = lowest member of each cluster).
    """
    assert 1 <= k <= H
    perm = rng.permutation(H)
    labels = np.empty(H, dtype=np.int64)
    if kind == "even":
        for g, chunk in enumerate(np.array_split(perm, k)):
            labels[chunk] = g
    elif kind == "uneven":
        labels[perm[:k]] = np.arange(k)
        for h in perm[k:]:
            if k == 1 or rng.random() < 0.5:
                labels[h] = 0
            else:
                labels[h] = int(rng.integers(1, k))
    else:
        raise ValueError(kind)
    membership, reps = canonical_labels(labels)
    assert len(reps) == k
    return membership, reps


def batch_partitions(B: int, H: int, k: int, kind: str, *key):
    """Independent partitions for the B requests of a batch: (membership [B,H], reps [B,k])."""
    mem = np.empty((B, H), dtype=np.int32)
    reps = np.empty((B, k), dtype=np.int32)
    for b in range(B):
        mem[b], reps[b] = make_partition(H, k, kind, _rng(*key, b, 23))
    return mem, reps


def _randn(shape, sigma, dtype, device, gen):
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if sigma != 1.0:
        x.mul_(sigma)
    return x.to(dtype)


def _randn_big(shape, sigma, dtype, device, gen):
    """Like _randn without the fp32 temporary for one layer's whole cache."""
    n0 = shape[0]
    out = torch.empty(shape, device=device, dtype=dtype)
    for i in range(n0):
        out[i] = _randn(shape[1:], sigma, dtype, device, gen)
    return out


def clustered_queries(membership: np.ndarray, k: int, shape_tail, sigma, noise, dtype, device, gen):
    """Q [B,H,*shape_tail]: one base per (request, cluster) ~ sigma*N(0,1); each head =
    its cluster's base + noise*sigma*N(0,1)."""
    B, H = membership.shape
    base = torch.randn((B, k) + tuple(shape_tail), generator=gen, device=device) * sigma
    idx = torch.as_tensor(membership.astype(np.int64), device=device)
    idx = idx.reshape(B, H, *([1] * len(shape_tail))).expand(B, H, *shape_tail)
    q = torch.gather(base, 1, idx)
    q = q + torch.randn(q.shape, generator=gen, device=device) * (noise * sigma)
    return q.to(dtype)


def decode_layer(cfg_id: int, layer: int = 0, seed: int = 0, device="cpu", B=None, H=None, T=None,
                 k=None, T_cap=None, with_k_full=None, peaked: float = 1.0):
    """Inputs of one layer's decode call for workload `cfg_id` (sizes overridable).

    Returns a dict with q [B,H,D], k_rep [B,k,T_cap,D], v [B,H,T_cap,D], membership [B,H],
    reps [B,k] (int32 tensors on `device`), k, T, T_cap, scale and, for the compaction
    workload (or with_k_full=True), k_full [B,H,T_cap,D] of which k_rep is the gather.
    `peaked` multiplies the queries (peaked > 1 makes the softmax far from uniform, which
    gives the parity check discriminating power).
    """
    w = WORKLOADS[cfg_id]
    B = B or w.B
    H = H or w.H
    T = T or w.T
    T_cap = T_cap or T
    D = w.D
    k = k or min(layer_k(cfg_id, layer, seed), H)
    dtype = TORCH_DTYPE[w.dtype]
    if with_k_full is None:
        with_k_full = w.compaction
    mem, reps = batch_partitions(B, H, k, w.partition, seed, cfg_id, layer)
    g = _tgen(device, seed, cfg_id, layer, 37)
    out = dict(cfg=cfg_id, layer=layer, k=k, B=B, H=H, T=T, T_cap=T_cap, D=D, dtype=w.dtype,
               scale=1.0 / float(np.sqrt(D)))
    out["v"] = _randn_big((B, H, T_cap, D), w.sigma, dtype, device, g)
    if with_k_full:
        k_full = _randn_big((B, H, T_cap, D), w.sigma, dtype, device, g)
        out["k_full"] = k_full
        ridx = torch.as_tensor(reps.astype(np.int64), device=device)
        out["k_rep"] = torch.stack([k_full[b].index_select(0, ridx[b]) for b in range(B)])
    else:
        out["k_rep"] = _randn_big((B, k, T_cap, D), w.sigma, dtype, device, g)
    q = clustered_queries(mem, k, (D,), w.sigma, 0.1, torch.float32, device, g)
    out["q"] = (q * peaked).to(dtype)
    out["membership"] = torch.as_tensor(mem, device=device)
    out["reps"] = torch.as_tensor(reps, device=device)
    return out


def blob_features(B: int = 1, H: int = 32, F: int = 64, k: int = 8, seed: int = 0, noise: float = 0.1,
                  kind: str = "even"):
    """Score-feature stand-ins: k well-separated Gaussian blobs (centres ~ N(0,1)^F, points =
    centre + noise*N(0,1)), heads assigned by a seeded partition.
    Returns (features [B,H,F] float32 numpy, planted membership [B,H] int32 canonical, reps [B,k])."""
    mem, reps = batch_partitions(B, H, k, kind, seed, 101, F)
    r = _rng(seed, 103, H, F, k)
    centres = r.standard_normal((B, k, F))
    x = np.take_along_axis(centres, mem[:, :, None].astype(np.int64), axis=1)
    x = x + noise * r.standard_normal((B, H, F))
    return x.astype(np.float32), mem, reps


def prefill_case(seed: int = 0, device="cpu", B=None, H=None, T=None, k=None, noise: float = 0.1,
                 peaked: float = 1.0):
    """Workload 5: a full prompt with planted head clusters.

    Q and K of head h = its group's base (sigma*N(0,1) over all T rows) + noise*sigma*N(0,1);
    V ~ sigma*N(0,1) independently per head.  Returns q_full, k_full, v [B,H,T,D] (bf16), the
    planted membership [B,H] / reps [B,k], and scale.  `peaked` multiplies Q.
    """
    w = WORKLOADS[5]
    B = B or w.B
    H = H or w.H
    T = T or w.T
    k = k or w.k_choices[0]
    D = w.D
    dtype = TORCH_DTYPE[w.dtype]
    mem, reps = batch_partitions(B, H, k, "even", seed, 5, 0)
    g = _tgen(device, seed, 5, 41)
    q = clustered_queries(mem, k, (T, D), w.sigma, noise, torch.float32, device, g)
    kf = clustered_queries(mem, k, (T, D), w.sigma, noise, dtype, device, g)
    v = _randn_big((B, H, T, D), w.sigma, dtype, device, g)
    return dict(q_full=(q * peaked).to(dtype), k_full=kf, v=v, membership=torch.as_tensor(mem, device=device),
                reps=torch.as_tensor(reps, device=device), planted=mem, B=B, H=H, T=T, D=D, k=k,
                scale=1.0 / float(np.sqrt(D)), dtype=w.dtype)
