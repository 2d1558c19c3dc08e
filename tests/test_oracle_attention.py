"""Pins for the attention, feature and compaction oracles (CPU only).

Each check ties the oracle to something other than itself: a library routine
(torch's scaled_dot_product_attention in fp64), a dense masked-matrix restatement
written a different way, closed forms, and invariances of the softmax.
"""
import numpy as np
import pytest
import torch

from oracle import chai_oracle as orc
from paper_2403_08058_b200 import synth

RNG = np.random.default_rng(1234)


def rand_case(B, H, k, Tq, T, D, kind="uneven", seed=0):
    mem, reps = synth.batch_partitions(B, H, k, kind, seed, 900, H, k)
    r = np.random.default_rng(seed + 77)
    q = r.standard_normal((B, H, Tq, D))
    kr = r.standard_normal((B, k, T, D))
    v = r.standard_normal((B, H, T, D))
    return q, kr, v, mem, reps


def dense_reference(q, kr, v, mem, reps, scale, causal):
    """Second, deliberately different statement: full score matrix per head, additive -inf mask."""
    B, H, Tq, D = q.shape
    T = kr.shape[2]
    out = np.zeros_like(q)
    for b in range(B):
        for h in range(H):
            c = mem[b, h]
            r = reps[b, c]
            S = scale * np.einsum("id,jd->ij", q[b, r], kr[b, c])
            if causal:
                ii = np.arange(Tq)[:, None] + (T - Tq)
                jj = np.arange(T)[None, :]
                S = S + np.where(jj > ii, -np.inf, 0.0)
            A = np.exp(S - S.max(axis=1, keepdims=True))
            A = A / A.sum(axis=1, keepdims=True)
            out[b, h] = A @ v[b, h]
    return out


def sdpa(q, k, v, scale, causal):
    o = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=causal, scale=scale)
    return o.numpy()


@pytest.mark.parametrize("causal", [True, False])
def test_singletons_equal_library_mha(causal):
    B, H, T, D = 2, 5, 13, 7            # non-square on purpose: a transposed operand cannot pass
    q = RNG.standard_normal((B, H, T, D))
    k = RNG.standard_normal((B, H, T, D))
    v = RNG.standard_normal((B, H, T, D))
    mem = np.tile(np.arange(H, dtype=np.int32), (B, 1))
    reps = mem.copy()
    scale = 0.37
    got = orc.cha_attention(q, k, v, mem, reps, scale, causal)
    np.testing.assert_allclose(got, sdpa(q, k, v, scale, causal), rtol=0, atol=1e-12)


def test_decode_singletons_equal_library_mha():
    B, H, T, D = 2, 4, 19, 8
    q = RNG.standard_normal((B, H, D))
    k = RNG.standard_normal((B, H, T, D))
    v = RNG.standard_normal((B, H, T, D))
    mem = np.tile(np.arange(H, dtype=np.int32), (B, 1))
    got = orc.cha_attention(q, k, v, mem, mem.copy(), 0.5, causal=False)
    want = sdpa(q[:, :, None, :], k, v, 0.5, False)[:, :, 0, :]
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("shape", [(1, 4, 2, 6, 6, 4), (2, 6, 3, 5, 5, 3), (2, 7, 3, 1, 9, 5), (1, 5, 5, 3, 8, 2)])
def test_matches_dense_masked_restatement(shape, causal):
    B, H, k, Tq, T, D = shape
    q, kr, v, mem, reps = rand_case(B, H, k, Tq, T, D, seed=sum(shape))
    got = orc.cha_attention(q, kr, v, mem, reps, 0.61, causal)
    want = dense_reference(q, kr, v, mem, reps, 0.61, causal)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


def test_identical_heads_in_a_cluster_equal_mha():
    """If every member shares its representative's Q and K, clustering changes nothing (the premise
    of the problem statement in Section 3.1)."""
    B, H, k, T, D = 2, 8, 3, 11, 6
    q, kr, v, mem, reps = rand_case(B, H, k, T, T, D, seed=5)
    q_mha = np.stack([q[b, reps[b, mem[b]]] for b in range(B)])        # each head gets its rep's Q
    k_mha = np.stack([kr[b, mem[b]] for b in range(B)])                # and its cluster's K
    got = orc.cha_attention(q, kr, v, mem, reps, 0.4, True)
    np.testing.assert_allclose(got, sdpa(q_mha, k_mha, v, 0.4, True), rtol=0, atol=1e-12)


def test_member_queries_are_not_read():
    B, H, k, T, D = 1, 6, 2, 7, 4
    q, kr, v, mem, reps = rand_case(B, H, k, T, T, D, seed=9)
    q2 = q.copy()
    for h in range(H):
        if h not in reps[0]:
            q2[0, h] += 100.0
    a = orc.cha_attention(q, kr, v, mem, reps, 1.0, True)
    b = orc.cha_attention(q2, kr, v, mem, reps, 1.0, True)
    assert np.array_equal(a, b)


def test_closed_forms():
    B, H, k, T, D = 1, 4, 2, 6, 6
    q, kr, v, mem, reps = rand_case(B, H, k, T, T, D, seed=3)
    # Q = 0 -> uniform probabilities -> running mean of V
    o = orc.cha_attention(np.zeros_like(q), kr, v, mem, reps, 1.0, True)
    want = np.cumsum(v, axis=2) / np.arange(1, T + 1)[None, None, :, None]
    np.testing.assert_allclose(o, want, atol=1e-13)
    # V = 1 -> O = 1
    o = orc.cha_attention(q, kr, np.ones_like(v), mem, reps, 1.0, True)
    np.testing.assert_allclose(o, 1.0, atol=1e-13)
    # V = I (T = D) -> O rows are the probability rows themselves
    eye = np.broadcast_to(np.eye(T), (B, H, T, T)).copy()
    a = orc.cha_attention(q, kr, eye, mem, reps, 1.0, True)
    assert (a >= 0).all()
    np.testing.assert_allclose(a.sum(-1), 1.0, atol=1e-14)
    assert np.array_equal(np.triu(a, 1), np.zeros_like(a))           # masked entries exactly 0
    for h in range(H):                                               # and they are the rep's scores
        c = mem[0, h]
        s = q[0, reps[0, c]] @ kr[0, c].T
        row = np.exp(s[T - 1] - s[T - 1].max())
        np.testing.assert_allclose(a[0, h, T - 1], row / row.sum(), atol=1e-14)
    # first row sees only key 0
    o = orc.cha_attention(q, kr, v, mem, reps, 1.0, True)
    np.testing.assert_allclose(o[:, :, 0], v[:, :, 0], atol=1e-14)
    # one dominant key
    kr2 = kr.copy()
    qd = q.copy()
    qd[0, reps[0, 0]] = 0.0
    qd[0, reps[0, 0], :, 0] = 1.0
    kr2[0, 0] = 0.0
    kr2[0, 0, 2, 0] = 1000.0
    o = orc.cha_attention(qd, kr2, v, mem, reps, 1.0, False)
    for h in np.nonzero(mem[0] == 0)[0]:
        np.testing.assert_allclose(o[0, h], np.broadcast_to(v[0, h, 2], (T, D)), atol=1e-12)


def test_invariances():
    B, H, k, T, D = 2, 7, 3, 9, 5
    q, kr, v, mem, reps = rand_case(B, H, k, T, T, D, seed=21)
    base = orc.cha_attention(q, kr, v, mem, reps, 0.7, True)
    # softmax shift: the same vector added to every key of a cluster
    u = RNG.standard_normal(D)
    kr2 = kr.copy()
    kr2[:, 1] += u
    np.testing.assert_allclose(orc.cha_attention(q, kr2, v, mem, reps, 0.7, True), base, atol=1e-12)
    # relabelling clusters together with their K slots
    perm = np.array([2, 0, 1])
    mem_p = perm[mem].astype(np.int32)
    reps_p = np.empty_like(reps)
    kr_p = np.empty_like(kr)
    reps_p[:, perm] = reps
    kr_p[:, perm] = kr
    assert np.array_equal(orc.cha_attention(q, kr_p, v, mem_p, reps_p, 0.7, True), base)
    # clusters do not interact
    kr3 = kr.copy()
    kr3[:, 0] = RNG.standard_normal(kr[:, 0].shape)
    o3 = orc.cha_attention(q, kr3, v, mem, reps, 0.7, True)
    for b in range(B):
        other = mem[b] != 0
        assert np.array_equal(o3[b, other], base[b, other])
        assert not np.allclose(o3[b, ~other], base[b, ~other])


def test_decode_is_last_prefill_row():
    B, H, k, T, D = 2, 6, 3, 10, 4
    q, kr, v, mem, reps = rand_case(B, H, k, T, T, D, seed=33)
    full = orc.cha_attention(q, kr, v, mem, reps, 0.3, True)
    dec = orc.cha_attention(q[:, :, -1, :], kr, v, mem, reps, 0.3, False)
    np.testing.assert_allclose(dec, full[:, :, -1, :], atol=1e-14)
    # chunked prefill: the last 3 query rows against the whole cache
    part = orc.cha_attention(q[:, :, -3:, :], kr, v, mem, reps, 0.3, True)
    np.testing.assert_allclose(part, full[:, :, -3:, :], atol=1e-14)


def test_invalid_clusters_give_zero_and_touch_nothing_else():
    B, H, k, T, D = 1, 5, 3, 4, 3
    q, kr, v, mem, reps = rand_case(B, H, k, T, T, D, seed=2)
    base = orc.cha_attention(q, kr, v, mem, reps, 1.0, True)
    reps2 = reps.copy()
    reps2[0, 1] = -1
    o = orc.cha_attention(q, kr, v, mem, reps2, 1.0, True)
    dead = mem[0] == 1
    assert np.array_equal(o[0, dead], np.zeros_like(o[0, dead]))
    assert np.array_equal(o[0, ~dead], base[0, ~dead])


def test_bf16_inputs_are_widened_exactly():
    t = torch.randn(1, 2, 3, 4).to(torch.bfloat16)
    assert np.array_equal(orc._f64(t), t.float().numpy().astype(np.float64))


# ---- features -------------------------------------------------------------------------------

def test_prefix_features_structure_and_cross_check():
    B, H, T, D, P = 2, 3, 9, 8, 5
    q = RNG.standard_normal((B, H, T, D))
    k = RNG.standard_normal((B, H, T, D))
    f = orc.prefix_features(q, k, P, 0.35).reshape(B, H, P, P)
    np.testing.assert_allclose(f.sum(-1), 1.0, atol=1e-14)
    assert np.array_equal(np.triu(f, 1), np.zeros_like(f))
    assert np.array_equal(f[:, :, 0, 0], np.ones((B, H)))
    # cross-check against the attention oracle: MHA (k = H) on the P-token problem with V = I
    mem = np.tile(np.arange(H, dtype=np.int32), (B, 1))
    eye = np.zeros((B, H, P, D))
    eye[:, :, np.arange(P), np.arange(P)] = 1.0
    a = orc.cha_attention(q[:, :, :P], k[:, :, :P], eye, mem, mem.copy(), 0.35, True)
    np.testing.assert_allclose(f, a[..., :P], atol=1e-14)
    # and against the library routine
    a2 = sdpa(q[:, :, :P], k[:, :, :P], eye, 0.35, True)
    np.testing.assert_allclose(f, a2[..., :P], atol=1e-12)


# ---- compaction -----------------------------------------------------------------------------

def test_compaction_is_a_gather_and_byte_closed_form():
    B, H, k, T, D = 2, 6, 3, 5, 4
    kf = RNG.integers(0, 2**16, size=(B, H, T, D), dtype=np.uint16)   # bf16 bit patterns
    _, reps = synth.batch_partitions(B, H, k, "uneven", 1, 2, 3)
    got, (before, after) = orc.compact_k_cache(kf, reps)
    want = np.stack([kf[b, reps[b]] for b in range(B)])
    assert np.array_equal(got, want)
    plane = T * D * 2
    assert before == 2 * B * H * plane and after == B * (H + k) * plane
    assert after / before == (H + k) / (2 * H)
    reps2 = reps.copy()
    reps2[1, 2] = -1
    got2, _ = orc.compact_k_cache(kf, reps2)
    assert not got2[1, 2].any() and np.array_equal(got2[0], want[0])


def test_kv_saving_matches_the_papers_figure():
    """Section 4.3: 21.4 % of K+V saved with keys only dropped <=> mean k/H = 0.572."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "kv_saving.txt")
    saving, ratio = [float(x) for x in open(path).read().split("\n")[2].split()]
    H, T, D = 32, 8, 4
    kf = np.zeros((1, H, T, D), dtype=np.uint16)
    fr = []
    for k in range(1, H + 1):
        reps = np.arange(k, dtype=np.int32)[None]
        _, (before, after) = orc.compact_k_cache(kf, reps)
        fr.append(1 - after / before)
    fr = np.array(fr)
    np.testing.assert_allclose(fr, (1 - np.arange(1, H + 1) / H) / 2, atol=1e-15)
    assert abs((1 - ratio) / 2 - saving) < 1e-9
    assert fr.max() < 0.5          # values are kept, so the saving can never reach one half


def test_attention_on_compacted_cache_equals_direct():
    B, H, k, T, D = 1, 6, 3, 7, 4
    q, _, v, mem, reps = rand_case(B, H, k, T, T, D, seed=8)
    kf = RNG.standard_normal((B, H, T, D))
    krep, _ = orc.compact_k_cache(kf, reps)
    direct = np.stack([kf[b, reps[b]] for b in range(B)])
    a = orc.cha_attention(q, krep, v, mem, reps, 1.0, True)
    b = orc.cha_attention(q, direct, v, mem, reps, 1.0, True)
    assert np.array_equal(a, b)


# ---- serving-shaped helpers: pinned against brute force written out independently ----------------------

def _brute_decode(q, k_rep, v, membership, reps, n, scale):
    """Direct loops over one request: softmax over the first n positions, then the weighted sum of V."""
    H, D = q.shape
    out = np.zeros((H, D))
    for h in range(H):
        c = int(membership[h])
        r = int(reps[c])
        s = np.array([scale * float(np.dot(q[r], k_rep[c, t])) for t in range(n)])
        p = np.exp(s - s.max())
        p /= p.sum()
        for t in range(n):
            out[h] += p[t] * v[h, t]
    return out


def test_ragged_decode_matches_brute_force_per_request():
    rng = np.random.default_rng(12)
    B, H, k, T_cap, D = 3, 6, 3, 40, 16
    membership = np.array([[0, 1, 0, 2, 1, 2], [0, 0, 1, 1, 2, 2], [0, 1, 2, 0, 1, 2]], dtype=np.int32)
    reps = np.array([[0, 1, 3], [0, 2, 4], [0, 1, 2]], dtype=np.int32)
    q = rng.normal(size=(B, H, D))
    k_rep = rng.normal(size=(B, k, T_cap, D))
    v = rng.normal(size=(B, H, T_cap, D))
    lens = np.array([40, 7, 0])
    scale = 0.31
    got = orc.decode_attention_ragged(q, k_rep, v, membership, reps, lens, scale)
    for b in range(B):
        want = _brute_decode(q[b], k_rep[b], v[b], membership[b], reps[b], int(lens[b]), scale) if lens[b] else 0.0
        assert np.allclose(got[b], want, rtol=1e-12, atol=1e-13)
    # rows beyond a request's length must not matter
    k2, v2 = k_rep.copy(), v.copy()
    k2[1, :, 7:] = 1e6
    v2[1, :, 7:] = -1e6
    assert np.array_equal(orc.decode_attention_ragged(q, k2, v2, membership, reps, lens, scale), got)


def test_append_then_decode_equals_decode_on_longer_cache():
    """Appending a token and decoding over n + 1 positions = decoding on a cache that already held the token."""
    rng = np.random.default_rng(13)
    B, H, k, T_cap, D = 2, 4, 2, 12, 8
    membership = np.array([[0, 1, 0, 1], [0, 0, 1, 1]], dtype=np.int32)
    reps = np.array([[0, 1], [0, 2]], dtype=np.int32)
    k_full = rng.normal(size=(B, H, T_cap, D))
    v = rng.normal(size=(B, H, T_cap, D))
    lens = np.array([5, 9])
    k_rep, _ = orc.compact_k_cache(k_full, reps)
    k_new, v_new = rng.normal(size=(B, H, D)), rng.normal(size=(B, H, D))
    k_rep2, v2, lens2 = orc.append_kv(k_new, v_new, k_rep, v, reps, lens)
    assert lens2.tolist() == [6, 10]
    for b in range(B):
        p = int(lens[b])
        assert np.array_equal(v2[b, :, p], v_new[b])
        for c in range(k):
            assert np.array_equal(k_rep2[b, c, p], k_new[b, reps[b, c]])
        # nothing else moved
        mask = np.ones(T_cap, bool)
        mask[p] = False
        assert np.array_equal(v2[b][:, mask], v[b][:, mask]) and np.array_equal(k_rep2[b][:, mask], k_rep[b][:, mask])
    # a full cache skips the request
    k3, v3, lens3 = orc.append_kv(k_new, v_new, k_rep, v, reps, np.array([T_cap, 2]))
    assert lens3.tolist() == [T_cap, 3] and np.array_equal(v3[0], v[0]) and np.array_equal(k3[0], k_rep[0])


def test_inplace_compaction_definition():
    rng = np.random.default_rng(14)
    k_full = rng.integers(0, 2 ** 16, size=(2, 5, 9, 4)).astype(np.uint16)
    reps = np.array([[0, 2, 4], [0, 1, -1]], dtype=np.int32)
    got = orc.compact_k_cache_inplace(k_full, reps, 6)
    assert got.shape == (2, 3, 6, 4)
    for b in range(2):
        for c in range(3):
            if reps[b, c] >= 0:
                assert np.array_equal(got[b, c], k_full[b, reps[b, c], :6])


def test_qkv_variant_member_rows_equal_the_representatives_plain_attention():
    """In CHAI-QKV a member's output is the representative's own single-head attention output."""
    rng = np.random.default_rng(15)
    B, H, k, T, D = 2, 6, 3, 9, 8
    membership = np.array([[0, 1, 0, 2, 1, 2], [0, 0, 1, 1, 2, 2]], dtype=np.int32)
    reps = np.array([[0, 1, 3], [0, 2, 4]], dtype=np.int32)
    q = rng.normal(size=(B, H, T, D))
    k_rep = rng.normal(size=(B, k, T, D))
    v_rep = rng.normal(size=(B, k, T, D))
    scale = 0.4
    got = orc.cha_attention_qkv(q, k_rep, v_rep, membership, reps, scale, True)
    for b in range(B):
        for h in range(H):
            c = membership[b, h]
            r = reps[b, c]
            s = scale * q[b, r] @ k_rep[b, c].T
            s = np.where(np.tril(np.ones((T, T), bool)), s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            assert np.allclose(got[b, h], p @ v_rep[b, c], rtol=1e-12, atol=1e-13)
            assert np.array_equal(got[b, h], got[b, r])


def test_e4m3_table_and_quantiser():
    vals = orc.e4m3_values()
    assert vals[0] == 0.0 and vals[0x38] == 1.0 and vals[0x7E] == 448.0 and vals[0x01] == 2.0 ** -9
    assert vals[0x08] == 2.0 ** -6 and vals[0x40] == 2.0 and vals[0xB8] == -1.0 and np.isnan(vals[0x7F])
    finite = vals[:127]
    assert np.all(np.diff(finite) > 0)                       # bytes 0..126 ascend
    # a plane whose largest magnitude is 448 has scale 1: representable values map to themselves, midpoints to even
    x = np.zeros((1, 4, 8), dtype=np.float32)
    x[0, 0] = [448.0, -1.0, 1.0625, 1.1875, 0.0, 1e-4, -448.0, 17.0]
    q, s = orc.quantize_cache_fp8(x, 4)
    assert s.tolist() == [1.0]
    got = vals[q[0, 0]]
    # 1.0625 is halfway between 1.0 (mantissa 0) and 1.125 (mantissa 1) -> 1.0; 1.1875 between 1.125 and 1.25 -> 1.25;
    # 1e-4 is below half the smallest subnormal (2^-10) -> 0; 17 lies halfway between 16 and 18 -> 16 (even mantissa)
    assert got.tolist() == [448.0, -1.0, 1.0, 1.25, 0.0, 0.0, -448.0, 16.0]
    # scale: absmax / 448; rows beyond T do not count and stay zero
    y = np.zeros((2, 3, 2), dtype=np.float32)
    y[0, :2] = [[2.0, -4.0], [1.0, 0.5]]
    y[0, 2] = [100.0, 100.0]
    q, s = orc.quantize_cache_fp8(y, 2)
    assert s[0] == np.float32(4.0) / np.float32(448.0) and s[1] == 1.0
    assert np.allclose(vals[q[0, :2]] * s[0], y[0, :2], rtol=2 ** -4) and not q[0, 2].any() and not q[1].any()


@pytest.mark.parametrize("amax", [448.0, 56.0, 1656.0])   # plane scales 1, 2^-3 and 3.696... (not a power of two)
def test_quantiser_equals_the_library_cast_on_every_bf16_value(amax):
    """Every finite bf16 bit pattern of magnitude <= amax in one plane (so the plane's scale is amax / 448):
    the quantiser's byte must be the one PyTorch's float32 -> float8_e4m3fn cast gives for float32(x) / scale,
    an independent implementation of round-to-nearest-even onto the same grid (no input exceeds 448 after
    scaling, so saturation is not involved; NaN and infinity are not cache contents and are left out).  The
    256-entry value table is checked against the library's decoding of the same bytes."""
    import torch
    table = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    vals = orc.e4m3_values()
    assert np.array_equal(np.isnan(table), np.isnan(vals)) and np.array_equal(table[~np.isnan(table)], vals[~np.isnan(vals)])
    bits = torch.arange(65536, dtype=torch.int32).to(torch.int16)
    x = bits.view(torch.bfloat16).float()
    x = x[torch.isfinite(x) & (x.abs() <= amax)]
    assert x.numel() > 30000 and float(x.abs().max()) == amax        # both signs, zeros and subnormals included
    D = 128
    pad = (-x.numel()) % D
    plane = torch.cat([x, torch.zeros(pad)]).reshape(1, -1, D).numpy()
    q, s = orc.quantize_cache_fp8(plane, plane.shape[1])
    scale = np.float32(amax) / np.float32(448.0)
    assert s.tolist() == [scale]
    want = (torch.from_numpy(plane) / torch.tensor(scale)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(q, want), f"{int((q != want).sum())} of {q.size} bytes differ"


def test_fp8_decode_is_the_decode_definition_on_what_the_bytes_stand_for():
    """Values chosen from the e4m3 grid (built here from the format's definition, not from the oracle's table):
    with scale 1 the byte caches stand for exactly the original numbers, so the fp8 decode must equal plain
    clustered attention on them; scaling a plane's bytes' scale by 2 must equal doubling that plane."""
    rng = np.random.default_rng(5)
    grid = np.array([0.0] + [m / 8 * 2.0 ** -6 for m in range(1, 8)] +
                    [(1 + m / 8) * 2.0 ** (e - 7) for e in range(1, 16) for m in range(8)][:-1])   # up to 448
    assert grid[-1] == 448.0 and len(grid) == 127
    B, H, k, T, D = 2, 4, 2, 9, 8
    mem = np.array([[0, 1, 0, 1], [0, 0, 0, 1]], dtype=np.int32)
    reps = np.array([[0, 1], [0, 3]], dtype=np.int32)
    pick = lambda shape: (grid[rng.integers(0, 60, size=shape)] * rng.choice([-1.0, 1.0], size=shape)).astype(np.float32)
    k_rep, v = pick((B, k, T, D)), pick((B, H, T, D))
    k_rep[:, :, 0, 0] = 448.0          # every plane's largest magnitude is 448: scale 1
    v[:, :, 0, 0] = -448.0
    q = rng.standard_normal((B, H, D)).astype(np.float32)
    k8, ks = orc.quantize_cache_fp8(k_rep, T)
    v8, vs = orc.quantize_cache_fp8(v, T)
    assert np.all(ks == 1.0) and np.all(vs == 1.0)
    lens = [T, 5]
    got = orc.decode_attention_fp8(q, k8, v8, ks, vs, mem, reps, lens, 0.3)
    want = orc.decode_attention_ragged(q, k_rep, v, mem, reps, lens, 0.3)
    assert np.abs(got - want).max() <= 1e-12
    # plane scales are plain multipliers of the plane
    vs2 = vs.copy()
    vs2[1, 2] = 2.0
    v2 = v.copy()
    v2[1, 2] *= 2.0
    got2 = orc.decode_attention_fp8(q, k8, v8, ks, vs2, mem, reps, lens, 0.3)
    assert np.abs(got2 - orc.decode_attention_ragged(q, k_rep, v2, mem, reps, lens, 0.3)).max() <= 1e-12
    ks2 = ks.copy()
    ks2[0, 1] = 0.5
    k2 = k_rep.copy()
    k2[0, 1] *= 0.5
    got3 = orc.decode_attention_fp8(q, k8, v8, ks2, vs, mem, reps, lens, 0.3)
    assert np.abs(got3 - orc.decode_attention_ragged(q, k2, v, mem, reps, lens, 0.3)).max() <= 1e-12
