"""GPU parity of the serving-shaped steps: ragged decode, cache append, in-place compaction, prefill that
starts after the plain-attention prefix.  Each CUDA result is compared with the CPU oracle on the same bits."""
import numpy as np
import pytest
import torch

from oracle import chai_oracle as orc
from paper_2403_08058_b200 import chai, synth
from parity import assert_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def bits(t: torch.Tensor) -> np.ndarray:
    """Bit pattern of a tensor as an integer numpy array (bf16 has no numpy dtype)."""
    t = t.detach().cpu().contiguous()
    return t.view(torch.int16).numpy() if t.dtype == torch.bfloat16 else t.view(torch.int32).numpy()


def ragged_case(cfg, seed, B, H, k, T_cap, D=128):
    case = synth.decode_layer(cfg, seed=seed, B=B, H=H, T=T_cap, T_cap=T_cap, k=k, with_k_full=True)
    if D == 64:
        for n in ("q", "k_rep", "v", "k_full"):
            case[n] = case[n][..., :64].contiguous()
        case["scale"] = 0.125
    return case


@pytest.mark.parametrize("cfg,D", [(1, 128), (2, 128), (2, 64)])
@pytest.mark.parametrize("lens", [[700, 1, 129, 0, 333], [128, 256, 384, 512, 640], [5, 5, 5, 5, 5], [0, 0, 0, 0, 1]])
def test_ragged_decode(cfg, D, lens, guard):
    case = ragged_case(cfg, sum(lens), 5, 12, 3, 700, D)
    seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
    q = case["q"].to(DEV)
    out = chai.chai_decode_attention_ragged(q, case["k_rep"].to(DEV), case["v"].to(DEV),
                                            case["membership"].to(DEV), case["reps"].to(DEV), seq, case["scale"],
                                            T_max=max(max(lens), 1), out=guard.empty_like(q))
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    ref = orc.decode_attention_ragged(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], lens,
                                      case["scale"])
    assert np.isfinite(got).all()
    assert_parity(got, ref, case["dtype"], f"ragged decode cfg {cfg} D {D} lens {lens}")
    for b, n in enumerate(lens):
        if n == 0:
            assert not got[b].any()


def test_ragged_decode_never_reads_beyond_a_request(guard):
    """Rows at or after seq_lens[b] hold NaN: the output must not notice."""
    lens = [300, 17, 129]
    case = ragged_case(2, 4, 3, 8, 4, 300)
    k_rep, v = case["k_rep"].clone(), case["v"].clone()
    for b, n in enumerate(lens):
        k_rep[b, :, n:] = float("nan")
        v[b, :, n:] = float("nan")
    seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
    q = case["q"].to(DEV)
    out = chai.chai_decode_attention_ragged(q, k_rep.to(DEV), v.to(DEV), case["membership"].to(DEV),
                                            case["reps"].to(DEV), seq, case["scale"], T_max=300, out=guard.empty_like(q))
    got = out.float().cpu().numpy()
    ref = orc.decode_attention_ragged(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], lens,
                                      case["scale"])
    assert np.isfinite(got).all()
    assert_parity(got, ref, "bf16", "ragged decode with poisoned tails")


@pytest.mark.parametrize("cfg", [1, 2])
def test_inplace_compaction_then_decode_and_append(cfg, guard):
    """The whole serving hand-over on one buffer: compaction in place, decode from the strided cache, append a
    token (representatives' keys only, every head's values), decode again over one more position."""
    B, H, k, T_cap = 3, 12, 4, 260
    lens = [200, 259, 64]
    case = ragged_case(cfg, 21, B, H, k, T_cap)
    reps = case["reps"]
    assert all(int(reps[b, c]) >= c for b in range(B) for c in range(k))
    cache = guard.empty_like(case["k_full"].to(DEV))   # the caches are written in place: they get guard bands too
    cache.copy_(case["k_full"])
    before = bits(cache)
    ws = chai.new_workspace(256, DEV)
    chai.chai_compact_k_cache_inplace(cache, reps.to(DEV), T=T_cap, workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_OK
    after = bits(cache)
    want = orc.compact_k_cache_inplace(bits(case["k_full"]), reps, T_cap)
    assert np.array_equal(after[:, :k], want)                       # bit copy of the representatives
    seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
    d = {n: case[n].to(DEV) for n in ("q", "v", "membership", "reps")}
    v = guard.empty_like(d["v"])
    v.copy_(d["v"])
    out = chai.chai_decode_attention_ragged(d["q"], cache, v, d["membership"], d["reps"], seq, case["scale"],
                                            T_max=T_cap, out=guard.empty_like(d["q"]))
    ref = orc.decode_attention_ragged(case["q"], case["k_rep"], case["v"], case["membership"], reps, lens, case["scale"])
    assert_parity(out.float().cpu().numpy(), ref, case["dtype"], "decode from a cache compacted in place")
    # append one token per request
    g = torch.Generator().manual_seed(3)
    k_new = (torch.randn(B, H, case["q"].shape[-1], generator=g) * 0.5).to(case["q"].dtype)
    v_new = (torch.randn(B, H, case["q"].shape[-1], generator=g) * 0.5).to(case["q"].dtype)
    chai.chai_append_kv(k_new.to(DEV), v_new.to(DEV), cache, v, d["reps"], seq, advance=True, workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_OK
    assert seq.cpu().tolist() == [n + 1 for n in lens]
    k_ref, v_ref, lens_ref = orc.append_kv(bits(k_new), bits(v_new), bits(case["k_rep"]), bits(case["v"]), reps, lens)
    assert np.array_equal(bits(cache)[:, :k], k_ref) and np.array_equal(bits(v), v_ref)
    assert np.array_equal(bits(cache)[:, k:], after[:, k:])          # dead planes are not touched by the append
    out2 = chai.chai_decode_attention_ragged(d["q"], cache, v, d["membership"], d["reps"], seq, case["scale"],
                                             T_max=T_cap, out=guard.empty_like(d["q"]))
    kf, vf = case["k_rep"].clone(), case["v"].clone()
    for b, n in enumerate(lens):
        vf[b, :, n] = v_new[b]
        for c in range(k):
            kf[b, c, n] = k_new[b, int(reps[b, c])]
    ref2 = orc.decode_attention_ragged(case["q"], kf, vf, case["membership"], reps, lens_ref, case["scale"])
    assert_parity(out2.float().cpu().numpy(), ref2, case["dtype"], "decode after append")
    assert before.shape == after.shape


def test_append_full_cache_is_reported_and_skipped():
    B, H, k, T_cap, D = 2, 4, 2, 8, 128
    reps = torch.tensor([[0, 1], [0, 2]], dtype=torch.int32, device=DEV)
    k_rep = torch.zeros(B, k, T_cap, D, dtype=torch.bfloat16, device=DEV)
    v = torch.zeros(B, H, T_cap, D, dtype=torch.bfloat16, device=DEV)
    new = torch.ones(B, H, D, dtype=torch.bfloat16, device=DEV)
    seq = torch.tensor([T_cap, 3], dtype=torch.int32, device=DEV)
    ws = chai.new_workspace(256, DEV)
    chai.chai_append_kv(new, new, k_rep, v, reps, seq, advance=True, workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_ERR_CACHE_FULL
    assert seq.cpu().tolist() == [T_cap, 4]
    assert not k_rep[0].any() and not v[0].any()
    assert v[1, :, 3].eq(1).all() and k_rep[1, :, 3].eq(1).all() and v[1].sum() == H * D


def test_inplace_compaction_refuses_unordered_reps():
    B, H, k, T, D = 2, 6, 3, 16, 128
    g = torch.Generator().manual_seed(0)
    cache = torch.randn(B, H, T, D, generator=g).to(torch.bfloat16).to(DEV)
    before = bits(cache)
    reps = torch.tensor([[0, 2, 4], [3, 1, 5]], dtype=torch.int32, device=DEV)   # request 1 is not ascending
    ws = chai.new_workspace(256, DEV)
    chai.chai_compact_k_cache_inplace(cache, reps, workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_ERR_BAD_MEMBERSHIP
    after = bits(cache)
    assert np.array_equal(after[1], before[1])                         # left untouched
    assert np.array_equal(after[0, 1], before[0, 2]) and np.array_equal(after[0, 2], before[0, 4])


@pytest.mark.parametrize("fn_name", ["chai_prefill_attention_from", "chai_prefill_attention_simt_from"])
@pytest.mark.parametrize("T,q_start,D", [(300, 5, 128), (300, 128, 128), (300, 131, 128), (64, 5, 128), (129, 128, 128),
                                         (640, 257, 128), (300, 5, 64), (300, 131, 64)])
def test_prefill_from_q_start(fn_name, T, q_start, D, guard):
    """Rows from q_start on equal the full clustered prefill; earlier rows of the output are not written."""
    B, H, k = 2, 6, 2
    r = synth.batch_partitions(B, H, k, "uneven", T, 79, q_start)
    g = torch.Generator().manual_seed(T + q_start)
    q = (torch.randn(B, H, T, D, generator=g) * 2.0).to(torch.bfloat16)
    kr = (torch.randn(B, k, T, D, generator=g) * 0.5).to(torch.bfloat16)
    v = (torch.randn(B, H, T, D, generator=g) * 0.5).to(torch.bfloat16)
    mem, reps = torch.as_tensor(r[0]), torch.as_tensor(r[1])
    scale = 1.0 / np.sqrt(D)
    out = guard.empty((B, H, T, D), torch.bfloat16)
    out.fill_(7.0)
    getattr(chai, fn_name)(q.to(DEV), kr.to(DEV), v.to(DEV), mem.to(DEV), reps.to(DEV), scale, q_start, True, out=out)
    got = out.float().cpu().numpy()
    ref = orc.cha_attention(q, kr, v, mem, reps, scale, True)
    assert (got[:, :, :q_start] == 7.0).all()
    assert_parity(got[:, :, q_start:], ref[:, :, q_start:], "bf16", f"{fn_name} T {T} q_start {q_start}")


# ---- variants: CHAI-QKV and CHAI-static ---------------------------------------------------------------

@pytest.mark.parametrize("cfg,ragged", [(1, False), (2, False), (2, True)])
def test_decode_qkv(cfg, ragged):
    B, H, k, T_cap = 4, 12, 3, 300
    case = ragged_case(cfg, 31, B, H, k, T_cap)
    reps = case["reps"]
    v_rep = torch.stack([case["v"][b, reps[b].long()] for b in range(B)]).contiguous()
    lens = [300, 1, 129, 77] if ragged else [T_cap] * B
    seq = torch.tensor(lens, dtype=torch.int32, device=DEV) if ragged else None
    out = chai.chai_decode_attention_qkv(case["q"].to(DEV), case["k_rep"].to(DEV), v_rep.to(DEV),
                                         case["membership"].to(DEV), reps.to(DEV), case["scale"], seq_lens=seq)
    got = out.float().cpu().numpy()
    ref = np.zeros_like(got, dtype=np.float64)
    for b, n in enumerate(lens):
        ref[b] = orc.cha_attention_qkv(case["q"][b:b + 1], case["k_rep"][b:b + 1, :, :n], v_rep[b:b + 1, :, :n],
                                       case["membership"][b:b + 1], reps[b:b + 1], case["scale"], False)[0]
    assert_parity(got, ref, case["dtype"], f"QKV decode cfg {cfg} ragged {ragged}")
    mem = case["membership"]
    for b in range(B):
        for h in range(H):
            assert np.array_equal(got[b, h], got[b, int(reps[b, int(mem[b, h])])])   # a member's row IS its representative's


@pytest.mark.parametrize("T,q_start,dtype", [(300, 0, "bf16"), (300, 5, "bf16"), (200, 0, "f32")])
def test_prefill_qkv(T, q_start, dtype):
    B, H, k, D = 2, 8, 3, 128
    r = synth.batch_partitions(B, H, k, "uneven", T, 80, q_start)
    g = torch.Generator().manual_seed(T)
    td = synth.TORCH_DTYPE[dtype]
    q = (torch.randn(B, H, T, D, generator=g) * 2.0).to(td)
    kr = (torch.randn(B, k, T, D, generator=g) * 0.5).to(td)
    vr = (torch.randn(B, k, T, D, generator=g) * 0.5).to(td)
    mem, reps = torch.as_tensor(r[0]), torch.as_tensor(r[1])
    scale = 1.0 / np.sqrt(D)
    out = torch.full((B, H, T, D), 7.0, dtype=td, device=DEV)
    chai.chai_prefill_attention_qkv(q.to(DEV), kr.to(DEV), vr.to(DEV), mem.to(DEV), reps.to(DEV), scale, True, q_start,
                                    out=out)
    got = out.float().cpu().numpy()
    ref = orc.cha_attention_qkv(q, kr, vr, mem, reps, scale, True)
    assert (got[:, :, :q_start] == 7.0).all()
    assert_parity(got[:, :, q_start:], ref[:, :, q_start:], dtype, f"QKV prefill T {T} q_start {q_start} {dtype}")


@pytest.mark.parametrize("B,H,k,T,D,causal", [(2, 72, 9, 450, 128, True),    # more than 32 heads: members found word by word
                                               (3, 40, 8, 300, 64, True), (1, 12, 12, 260, 128, True),
                                               (2, 33, 2, 200, 128, False)])
def test_prefill_qkv_shapes(B, H, k, T, D, causal, guard):
    """CHAI-QKV prefill on the tensor-core kernel: clusters of many members, singletons, head_dim 64, not causal."""
    r = synth.batch_partitions(B, H, k, "uneven", T, 81, H)
    g = torch.Generator().manual_seed(T + H)
    q = (torch.randn(B, H, T, D, generator=g) * 2.0).to(torch.bfloat16)
    kr = (torch.randn(B, k, T, D, generator=g) * 0.5).to(torch.bfloat16)
    vr = (torch.randn(B, k, T, D, generator=g) * 0.5).to(torch.bfloat16)
    mem, reps = torch.as_tensor(r[0]), torch.as_tensor(r[1])
    scale = 1.0 / np.sqrt(D)
    out = guard.empty((B, H, T, D), torch.bfloat16)
    chai.chai_prefill_attention_qkv(q.to(DEV), kr.to(DEV), vr.to(DEV), mem.to(DEV), reps.to(DEV), scale, causal, 0, out=out)
    got = out.float().cpu().numpy()
    ref = orc.cha_attention_qkv(q, kr, vr, mem, reps, scale, causal)
    assert_parity(got, ref, "bf16", f"QKV prefill B {B} H {H} k {k} T {T} D {D} causal {causal}")
    for b in range(B):
        for h in range(H):
            assert np.array_equal(got[b, h], got[b, int(reps[b, int(mem[b, h])])])   # a member's rows ARE its representative's


def test_prefill_qkv_bad_membership_is_reported():
    """Heads that name no cluster, a cluster without a usable representative: zero rows and the status word; the
    other heads are untouched by it."""
    B, H, k, T, D = 2, 10, 3, 200, 128
    r = synth.batch_partitions(B, H, k, "uneven", 3, 82, T)
    g = torch.Generator().manual_seed(9)
    q = (torch.randn(B, H, T, D, generator=g) * 2.0).to(torch.bfloat16)
    kr = (torch.randn(B, k, T, D, generator=g) * 0.5).to(torch.bfloat16)
    vr = (torch.randn(B, k, T, D, generator=g) * 0.5).to(torch.bfloat16)
    mem, reps = torch.as_tensor(r[0]).clone(), torch.as_tensor(r[1]).clone()
    ref = orc.cha_attention_qkv(q, kr, vr, mem, reps, 1.0 / np.sqrt(D), True)
    non_reps = [h for h in range(H) if h not in reps[0].tolist()]
    mem[0, non_reps[0]] = 77                     # no such cluster
    lost = [h for h in range(H) if int(mem[1, h]) == 1]
    reps[1, 1] = -1                              # cluster 1 of request 1 has no representative
    ws = chai.new_workspace(int(chai.load().chai_prefill_qkv_workspace_bytes(B, H, k, T, D, chai.CHAI_BF16)), DEV)
    out = torch.full((B, H, T, D), 7.0, dtype=torch.bfloat16, device=DEV)
    chai.chai_prefill_attention_qkv(q.to(DEV), kr.to(DEV), vr.to(DEV), mem.to(DEV), reps.to(DEV), 1.0 / np.sqrt(D), True, 0,
                                    out=out, workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_ERR_BAD_MEMBERSHIP
    got = out.float().cpu().numpy()
    bad = {(0, non_reps[0])} | {(1, h) for h in lost}
    for b in range(B):
        for h in range(H):
            if (b, h) in bad:
                assert not got[b, h].any()
            else:
                assert_parity(got[b, h], ref[b, h], "bf16", f"head ({b},{h}) beside unresolved ones")


def test_qkv_bad_membership_is_reported():
    B, H, k, T = 1, 6, 2, 64
    case = ragged_case(2, 5, B, H, k, T)
    v_rep = torch.stack([case["v"][b, case["reps"][b].long()] for b in range(B)]).contiguous()
    mem = case["membership"].clone()
    hbad = [h for h in range(H) if h not in case["reps"][0].tolist()][0]
    mem[0, hbad] = 9
    ws = chai.new_workspace(int(chai.load().chai_decode_qkv_workspace_bytes(B, H, k, T, 128, chai.CHAI_BF16)), DEV)
    out = chai.chai_decode_attention_qkv(case["q"].to(DEV), case["k_rep"].to(DEV), v_rep.to(DEV), mem.to(DEV),
                                         case["reps"].to(DEV), case["scale"], workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_ERR_BAD_MEMBERSHIP
    assert not out[0, hbad].float().abs().sum().item()


def test_static_membership_broadcast_equals_per_request_arrays():
    B, H, k, T = 3, 8, 4, 200
    case = ragged_case(2, 8, B, H, k, T)
    m0, r0 = case["membership"][0].contiguous(), case["reps"][0].contiguous()
    mem, reps = chai.chai_broadcast_membership(m0.to(DEV), r0.to(DEV), B)
    assert mem.cpu().tolist() == [m0.tolist()] * B and reps.cpu().tolist() == [r0.tolist()] * B
    k_rep = torch.stack([case["k_full"][b, r0.long()] for b in range(B)]).contiguous()
    out = chai.chai_decode_attention(case["q"].to(DEV), k_rep.to(DEV), case["v"].to(DEV), mem, reps, case["scale"])
    ref = orc.cha_attention(case["q"], k_rep, case["v"], mem.cpu(), reps.cpu(), case["scale"], False)
    assert_parity(out.float().cpu().numpy(), ref, "bf16", "static membership")


def test_select_representatives_matches_oracle():
    B, H, F, k = 3, 40, 25, 6
    feats, planted, _ = synth.blob_features(B, H, F, k, seed=2)
    feats = torch.as_tensor(feats, dtype=torch.float32)
    mem, _, _, _ = chai.chai_cluster_heads(feats.to(DEV), k, 20, 1)
    got = chai.chai_select_representatives(feats.to(DEV), mem, k).cpu().numpy()
    want = orc.closest_representatives(feats.numpy(), mem.cpu().numpy(), k)
    assert np.array_equal(got, want)
    m = mem.cpu().numpy()
    for b in range(B):
        for c in range(k):
            assert got[b, c] >= c and m[b, got[b, c]] == c           # a member of its own cluster
    # exact ties (duplicated heads) and an empty cluster
    f2 = torch.tensor([[[0.0], [1.0], [10.0], [4.0], [3.0]]])
    m2 = torch.tensor([[0, 1, 0, 0, 1]], dtype=torch.int32)
    assert chai.chai_select_representatives(f2.to(DEV), m2.to(DEV), 3).cpu().tolist() == [[3, 1, -1]]


@pytest.mark.parametrize("k_true,H,F", [(4, 32, 25), (8, 32, 25), (13, 52, 64)])
def test_cluster_sweep_matches_oracle_and_finds_the_planted_count(k_true, H, F):
    feats, _, _ = synth.blob_features(3, H, F, k_true, seed=k_true + 1, noise=0.05)
    curve, knee = chai.chai_cluster_sweep(torch.as_tensor(feats).to(DEV), H, 20, 0)
    ref_curve, ref_knee = orc.cluster_sweep(feats, H, 20, 0)
    got = curve.cpu().numpy()
    assert np.allclose(got, ref_curve, rtol=1e-12, atol=1e-18)
    assert knee.cpu().tolist() == ref_knee.tolist() == [k_true] * 3
    # column k-1 of the sweep is what a single clustering call with k clusters reports
    _, _, _, inertia = chai.chai_cluster_heads(torch.as_tensor(feats).to(DEV), k_true, 20, 0)
    assert np.array_equal(inertia.cpu().numpy(), got[:, k_true - 1])


def test_cluster_sweep_on_unstructured_features():
    rng = np.random.default_rng(9)
    feats = rng.normal(size=(2, 24, 10)).astype(np.float32)
    curve, knee = chai.chai_cluster_sweep(torch.as_tensor(feats).to(DEV), 24, 20, 3)
    ref_curve, ref_knee = orc.cluster_sweep(feats, 24, 20, 3)
    assert np.allclose(curve.cpu().numpy(), ref_curve, rtol=1e-12, atol=1e-18)
    assert knee.cpu().tolist() == ref_knee.tolist()


@pytest.mark.parametrize("k", [8, 16])
def test_decode_qkv_at_workload_2_layer_shape(k):
    """CHAI-QKV decode at the shape and launch configuration its bench leg times (B 16, H 32, T 2048, D 128; one launch
    with the clusters as heads): every output element against the oracle."""
    w = synth.WORKLOADS[2]
    c = synth.decode_layer(2, 4, 5, B=w.B, H=w.H, T=w.T, k=k)
    reps = c["reps"]
    v_rep = torch.stack([c["v"][b].index_select(0, reps[b].long()) for b in range(w.B)]).contiguous()
    out = chai.chai_decode_attention_qkv(c["q"].to(DEV), c["k_rep"].to(DEV), v_rep.to(DEV), c["membership"].to(DEV),
                                         reps.to(DEV), c["scale"])
    got = out.float().cpu().numpy()
    ref = orc.cha_attention_qkv(c["q"], c["k_rep"], v_rep, c["membership"], reps, c["scale"], False)
    assert_parity(got, ref, "bf16", f"QKV decode, workload 2 layer shape, k {k}")


def test_prefill_qkv_at_workload_5_shape_sampled_rows():
    """CHAI-QKV prefill at workload 5's shape (B 4, T 2048, H 32, k 8; one launch, a work item per cluster): run-to-run
    bitwise identical; first rows, rows across a query-tile boundary and last rows against the oracle."""
    case = synth.prefill_case(seed=3, device=DEV)
    B, H, k, T = case["B"], case["H"], case["k"], case["T"]
    k_rep = chai.chai_compact_k_cache(case["k_full"], case["reps"])
    v_rep = torch.stack([case["v"][b].index_select(0, case["reps"][b].long()) for b in range(B)]).contiguous()
    run = lambda: chai.chai_prefill_attention_qkv(case["q_full"], k_rep, v_rep, case["membership"], case["reps"],
                                                  case["scale"], True, 0)
    out, out2 = run(), run()
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    q, kr, vr = case["q_full"].cpu(), k_rep.cpu(), v_rep.cpu()
    mem, reps = case["membership"].cpu(), case["reps"].cpu()
    head = orc.cha_attention_qkv(q[:, :, :192], kr[:, :, :192], vr[:, :, :192], mem, reps, case["scale"], True)
    assert_parity(out[:, :, :192].float().cpu().numpy(), head, "bf16", "QKV prefill first rows")
    lo, hi = 992, 1056
    mid = orc.cha_attention_qkv(q[:, :, :hi], kr[:, :, :hi], vr[:, :, :hi], mem, reps, case["scale"], True)
    assert_parity(out[:, :, lo:hi].float().cpu().numpy(), mid[:, :, lo:hi], "bf16", "QKV prefill middle rows")
    tail = orc.cha_attention_qkv(q[:, :, T - 64:], kr, vr, mem, reps, case["scale"], True)
    assert_parity(out[:, :, T - 64:].float().cpu().numpy(), tail, "bf16", "QKV prefill last rows")


def test_ragged_decode_at_the_serving_bench_shape(guard):
    """The ragged decode call its bench leg times: workload 2's layer shape (B 16, H 32, k 8, D 128, capacity 2048),
    lengths spread over 1/4..1 of the capacity, keys read from a cache compacted in place (strided planes).  Every
    output element against the oracle."""
    w = synth.WORKLOADS[2]
    k, B, H, T_cap = 8, w.B, w.H, w.T
    c = synth.decode_layer(2, 0, 1, B=B, H=H, T=T_cap, k=k, with_k_full=True)
    rng = np.random.default_rng(7)
    lens = rng.integers(T_cap // 4, T_cap, size=B).astype(np.int32)
    lens[0] = T_cap - 1
    cache = c["k_full"].to(DEV).clone()
    chai.chai_compact_k_cache_inplace(cache, c["reps"].to(DEV), T=T_cap)
    q = c["q"].to(DEV)
    out = chai.chai_decode_attention_ragged(q, cache, c["v"].to(DEV), c["membership"].to(DEV), c["reps"].to(DEV),
                                            torch.as_tensor(lens, device=DEV), c["scale"], T_max=T_cap, k_planes=k,
                                            out=guard.empty_like(q))
    torch.cuda.synchronize()
    ref = orc.decode_attention_ragged(c["q"], c["k_rep"], c["v"], c["membership"], c["reps"], [int(n) for n in lens],
                                      c["scale"])
    assert_parity(out.float().cpu().numpy(), ref, "bf16", "ragged decode at the serving bench shape")
