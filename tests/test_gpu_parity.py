"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same bits."""
import numpy as np
import pytest
import torch

from oracle import chai_oracle as orc
from paper_2403_08058_b200 import chai, synth
from parity import assert_parity, errors, gate_ok

pytestmark = pytest.mark.gpu
DEV = "cuda"


def to_dev(case, names=("q", "k_rep", "v", "membership", "reps", "k_full", "q_full")):
    return {n: (case[n].to(DEV) if n in case and torch.is_tensor(case[n]) else case.get(n)) for n in names}


def oracle_decode(case, T=None):
    T = T or case["T"]
    return orc.cha_attention(case["q"], case["k_rep"][:, :, :T], case["v"][:, :, :T], case["membership"],
                             case["reps"], case["scale"], causal=False)


def run_decode(case, T=None, guard=None, **kw):
    d = to_dev(case)
    if guard is not None:            # output inside guard bands (the workspace always is: see conftest)
        kw["out"] = guard.empty_like(d["q"])
    out = chai.chai_decode_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"],
                                     T=T or case["T"], **kw)
    torch.cuda.synchronize()
    return out.float().cpu().numpy()


# ---- decode ---------------------------------------------------------------------------------------

def test_decode_config1_fp32():
    case = synth.decode_layer(1)
    got = run_decode(case)
    e = assert_parity(got, oracle_decode(case), "f32", "config 1 decode")
    assert e["max_rel"] <= 1e-5


@pytest.mark.parametrize("T", [1, 2, 5, 127, 128, 129, 255, 256, 257, 700])
@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_decode_ragged_lengths(cfg, T, guard):
    """Lengths around the 64/128/256-row chunk edges, capacity larger than the length."""
    case = synth.decode_layer(cfg, layer=T % 7, seed=T, B=2, H=12 if cfg != 1 else 8, T=T, T_cap=T + 3, k=3)
    got = run_decode(case, guard=guard)
    assert_parity(got, oracle_decode(case), case["dtype"], f"cfg {cfg} T {T}")


@pytest.mark.parametrize("cfg,D,H,k", [(2, 64, 8, 2), (1, 64, 6, 6), (2, 128, 52, 13), (3, 128, 72, 36),
                                       (3, 128, 9, 1)])
def test_decode_shapes(cfg, D, H, k):
    case = synth.decode_layer(cfg, seed=5, B=3, H=H, T=300, k=k)
    if D == 64:
        for n in ("q", "k_rep", "v"):
            case[n] = case[n][..., :64].contiguous()
        case["scale"] = 0.125
    got = run_decode(case)
    assert_parity(got, oracle_decode(case), case["dtype"], f"cfg {cfg} D {D} H {H} k {k}")


@pytest.mark.parametrize("cfg", [2, 3])
def test_decode_peaked_and_negative_controls(cfg):
    """A peaked softmax gives the gate power; wrong membership / reps / K slots must fail it."""
    case = synth.decode_layer(cfg, seed=3, B=2, H=16, T=1024, k=4, peaked=8.0)
    ref = oracle_decode(case)
    got = run_decode(case)
    assert_parity(got, ref, "bf16", "peaked decode")
    # shuffled membership (still a consistent partition, but the wrong one)
    wrong = dict(case)
    perm = torch.roll(torch.arange(16), 5)
    mem = case["membership"][:, perm].contiguous()
    labels = [synth.canonical_labels(m.numpy()) for m in mem]
    wrong["membership"] = torch.as_tensor(np.stack([l[0] for l in labels]))
    wrong["reps"] = torch.as_tensor(np.stack([l[1] for l in labels]))
    assert not gate_ok(run_decode(wrong), ref, "bf16")
    # K slots swapped
    wrong = dict(case)
    wrong["k_rep"] = case["k_rep"][:, [1, 0, 2, 3]].contiguous()
    assert not gate_ok(run_decode(wrong), ref, "bf16")
    # the oracle itself distinguishes them too
    assert not gate_ok(oracle_decode(wrong), ref, "bf16")


def test_decode_full_size_layers():
    """One layer of each decode workload at full size, every output element against the oracle
    (the oracle is cheap for a single query row), in the launch configuration the bench uses."""
    for cfg, layer in ((2, 0), (2, 3), (3, 1), (4, 2)):
        case = synth.decode_layer(cfg, layer=layer, seed=0, device=DEV, with_k_full=False)
        ws = chai.new_workspace(chai.chai_decode_workspace_bytes(case["B"], case["H"], case["k"], case["T"], 128,
                                                                 chai.CHAI_BF16), DEV)
        out = chai.chai_decode_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"],
                                         case["scale"], workspace=ws)
        out2 = chai.chai_decode_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"],
                                          case["scale"], workspace=ws)
        torch.cuda.synchronize()
        assert chai.chai_device_status(ws) == chai.CHAI_OK
        assert torch.equal(out, out2)                      # run-to-run bitwise identical
        got = out.float().cpu().numpy()
        for b in range(case["B"]):
            sl = {n: case[n][b:b + 1].cpu() for n in ("q", "k_rep", "v", "membership", "reps")}
            ref = orc.cha_attention(sl["q"], sl["k_rep"], sl["v"], sl["membership"], sl["reps"], case["scale"],
                                    causal=False)
            assert_parity(got[b:b + 1], ref, "bf16", f"cfg {cfg} layer {layer} b {b}")
        del case, out, out2, ws
        torch.cuda.empty_cache()


@pytest.mark.parametrize("B,H,k,T", [(2, 8, 3, 100003),     # long context: hundreds of tiles per plane, ragged tail
                                      (1500, 4, 2, 40),        # many short requests: far more heads than the head table holds
                                      (1, 1, 1, 1)])           # the smallest problem there is
def test_decode_extreme_shapes(B, H, k, T, guard):
    case = synth.decode_layer(2, layer=1, seed=5, device=DEV, B=B, H=H, T=T, k=k, with_k_full=False, peaked=4.0)
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(B, H, k, T, 128, chai.CHAI_BF16), DEV)
    out = chai.chai_decode_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"],
                                     case["scale"], out=guard.empty_like(case["q"]), workspace=ws)
    out2 = chai.chai_decode_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"],
                                      case["scale"], out=guard.empty_like(case["q"]), workspace=ws)
    torch.cuda.synchronize()
    assert chai.chai_device_status(ws) == chai.CHAI_OK
    assert torch.equal(out, out2)
    got = out.float().cpu().numpy()
    step = max(1, B // 6)                                      # every request when B is small, a spread of them otherwise
    for b in list(range(0, B, step)) + [B - 1]:
        sl = {n: case[n][b:b + 1].cpu() for n in ("q", "k_rep", "v", "membership", "reps")}
        ref = orc.cha_attention(sl["q"], sl["k_rep"], sl["v"], sl["membership"], sl["reps"], case["scale"], causal=False)
        assert_parity(got[b:b + 1], ref, "bf16", f"B {B} H {H} k {k} T {T} request {b}")


def test_decode_ragged_long_contexts_mix_one_pass_and_grouped_sums(guard):
    """Requests of very different lengths in one call: a head's item partials are added in one pass for the
    short ones and group by group for the long ones (with a last group that is not full); one request is empty."""
    B, H, k, T = 4, 4, 2, 70001
    case = synth.decode_layer(2, layer=2, seed=9, device=DEV, B=B, H=H, T=T, k=k, with_k_full=False, peaked=4.0)
    lens = np.array([T, 40000, 20000, 0], np.int32)
    seq = torch.as_tensor(lens, device=DEV)
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(B, H, k, T, 128, chai.CHAI_BF16), DEV)
    outs = [chai.chai_decode_attention_ragged(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], seq,
                                              case["scale"], T_max=T, out=guard.empty_like(case["q"]), workspace=ws)
            for _ in range(2)]
    torch.cuda.synchronize()
    assert chai.chai_device_status(ws) == chai.CHAI_OK
    assert torch.equal(outs[0], outs[1])
    c = {n: case[n].cpu() for n in ("q", "k_rep", "v", "membership", "reps")}
    ref = orc.decode_attention_ragged(c["q"], c["k_rep"], c["v"], c["membership"], c["reps"], lens, case["scale"])
    assert_parity(outs[0].float().cpu().numpy(), ref, "bf16", "ragged long contexts")
    assert not outs[0][3].float().abs().max().item()  # the empty request's rows are zero


def test_decode_bad_membership_is_reported_not_faulted():
    case = synth.decode_layer(2, seed=1, B=2, H=8, T=200, k=4)
    ref = oracle_decode(case)
    d = to_dev(case)
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(2, 8, 4, 200, 128, chai.CHAI_BF16), DEV)
    canary = torch.full((2, 8, 128), 7.0, device=DEV, dtype=torch.bfloat16)

    def run(mem, reps):
        out = canary.clone()
        chai.chai_decode_attention(d["q"], d["k_rep"], d["v"], mem, reps, case["scale"], out=out, workspace=ws)
        return out.float().cpu().numpy(), chai.chai_device_status(ws)

    got, st = run(d["membership"], d["reps"])
    assert st == chai.CHAI_OK and gate_ok(got, ref, "bf16")
    # cluster id out of range for one head
    mem = d["membership"].clone()
    mem[1, 5] = 99
    got, st = run(mem, d["reps"])
    assert st == chai.CHAI_ERR_BAD_MEMBERSHIP
    # head 5 of request 1 is zero; heads that did not depend on it are untouched
    assert not got[1, 5].any()
    assert gate_ok(got[0], ref[0], "bf16")
    # a cluster without representative: its members get zeros
    reps = d["reps"].clone()
    reps[0, 2] = -1
    got, st = run(d["membership"], reps)
    assert st == chai.CHAI_ERR_BAD_MEMBERSHIP
    dead = (case["membership"][0] == 2).numpy()
    assert not got[0, dead].any() and gate_ok(got[0, ~dead], ref[0, ~dead], "bf16")
    # representative outside its own cluster
    reps = d["reps"].clone()
    reps[0, 1] = int(case["reps"][0, 0])
    got, st = run(d["membership"], reps)
    assert st == chai.CHAI_ERR_BAD_MEMBERSHIP
    # and a good call afterwards clears the word
    got, st = run(d["membership"], d["reps"])
    assert st == chai.CHAI_OK and gate_ok(got, ref, "bf16")


def test_decode_host_entry_point():
    case = synth.decode_layer(2, seed=2, B=2, H=8, T=300, k=4)
    d = to_dev(case)
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(2, 8, 4, 300, 128, chai.CHAI_BF16), DEV)
    qh = case["q"].pin_memory()
    oh = torch.empty_like(case["q"]).pin_memory()
    chai.chai_decode_attention_host(qh, oh, torch.empty_like(d["q"]), torch.empty_like(d["q"]), d["k_rep"], d["v"],
                                    d["membership"], d["reps"], case["scale"], ws)
    assert_parity(oh.float().numpy(), oracle_decode(case), "bf16", "host entry")
    # the enqueue-only form: two calls share the staging buffers, one synchronisation at the end
    oh1, oh2 = torch.zeros_like(oh).pin_memory(), torch.zeros_like(oh).pin_memory()
    qs, os_ = torch.empty_like(d["q"]), torch.empty_like(d["q"])
    for o in (oh1, oh2):
        chai.chai_decode_attention_host_async(qh, o, qs, os_, d["k_rep"], d["v"], d["membership"], d["reps"],
                                              case["scale"], ws)
    torch.cuda.current_stream().synchronize()
    assert torch.equal(oh1, oh) and torch.equal(oh2, oh)
    # the three-stream form: three calls in flight, each with its own staging buffers and events
    s_comp, s_up, s_down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    outs = [torch.zeros_like(oh).pin_memory() for _ in range(3)]
    stages = [(torch.empty_like(d["q"]), torch.empty_like(d["q"])) for _ in range(3)]
    events = [(torch.cuda.Event(), torch.cuda.Event()) for _ in range(3)]
    torch.cuda.synchronize()
    for o, (qs3, os3), (e_up, e_k) in zip(outs, stages, events):
        chai.chai_decode_attention_host_streams(qh, o, qs3, os3, d["k_rep"], d["v"], d["membership"], d["reps"],
                                                case["scale"], ws, s_comp, s_up, s_down, e_up, e_k)
    s_down.synchronize()
    s_comp.synchronize()
    s_up.synchronize()
    assert all(torch.equal(o, oh) for o in outs)


# ---- k-means, features, compaction ---------------------------------------------------------------------

def gpu_kmeans(x, k, max_iter=20, seed=0):
    mem, reps, ke, inertia = chai.chai_cluster_heads(torch.as_tensor(x, device=DEV), k, max_iter, seed)
    torch.cuda.synchronize()
    return mem.cpu().numpy(), reps.cpu().numpy(), ke.cpu().numpy(), inertia.cpu().numpy()


def test_kmeans_config1_blobs_every_seed():
    x, planted, planted_reps = synth.blob_features(1, 32, 64, 8, seed=0)
    for seed in range(32):
        mem, reps, ke, inertia = gpu_kmeans(x, 8, 20, seed)
        ref = orc.kmeans(x, 8, 20, seed)
        assert np.array_equal(mem, planted) and np.array_equal(mem, ref["membership"])
        assert np.array_equal(reps, planted_reps) and ke[0] == 8
        assert inertia[0] == ref["inertia"][0]


def test_kmeans_identical_trajectories_on_unstructured_inputs():
    """Same arithmetic in the same order: labels agree bit for bit even where nothing is separated."""
    r = np.random.default_rng(0)
    for trial in range(25):
        B, H, F = 3, int(r.integers(2, 80)), int(r.integers(1, 70))
        k = int(r.integers(1, H + 1))
        x = r.standard_normal((B, H, F)).astype(np.float32)
        it = int(r.integers(1, 30))
        mem, reps, ke, inertia = gpu_kmeans(x, k, it, trial)
        ref = orc.kmeans(x, k, it, trial)
        assert np.array_equal(mem, ref["membership"]), trial
        assert np.array_equal(reps, ref["reps"]) and np.array_equal(ke, ref["k_eff"])
        np.testing.assert_array_equal(inertia, ref["inertia"])


def test_kmeans_degenerate_inputs():
    r = np.random.default_rng(4)
    y = np.repeat(r.standard_normal((1, 3, 5)), 3, axis=1).astype(np.float32)     # 3 distinct points x3
    mem, reps, ke, _ = gpu_kmeans(y, 5, 20, 1)
    ref = orc.kmeans(y, 5, 20, 1)
    assert ke[0] == 3 and np.array_equal(mem, ref["membership"]) and np.array_equal(reps, ref["reps"])
    mem, reps, ke, inertia = gpu_kmeans(np.ones((2, 6, 2), np.float32), 4, 20, 3)
    assert (ke == 1).all() and not mem.any() and (reps[:, 1:] == -1).all() and np.isfinite(inertia).all()
    x = r.standard_normal((1, 72, 25)).astype(np.float32)
    mem, reps, ke, _ = gpu_kmeans(x, 72, 20, 0)                                  # k = H
    assert mem[0].tolist() == list(range(72))
    mem, _, _, _ = gpu_kmeans(x, 1, 20, 0)
    assert not mem.any()


def test_prefix_features():
    for dtype, tol in ((torch.float32, 2e-6), (torch.bfloat16, 2e-6)):
        g = torch.Generator().manual_seed(3)
        q = torch.randn(2, 5, 9, 128, generator=g).to(dtype)
        k = torch.randn(2, 5, 9, 128, generator=g).to(dtype)
        for P in (1, 5, 8):
            f = chai.chai_prefix_features(q.to(DEV), k.to(DEV), P, 0.09).cpu().numpy()
            ref = orc.prefix_features(q, k, P, 0.09)
            assert np.abs(f - ref).max() <= tol
            assert not np.triu(f.reshape(2, 5, P, P), 1).any()


def test_compaction_bit_exact():
    for dtype in (torch.bfloat16, torch.float32):
        B, H, k, T, T_cap, D = 3, 10, 4, 333, 340, 128
        g = torch.Generator().manual_seed(1)
        kf = torch.randn(B, H, T_cap, D, generator=g).to(dtype)
        _, reps = synth.batch_partitions(B, H, k, "uneven", 4, 4)
        reps[2, 3] = -1
        out = torch.full((B, k, T_cap, D), 3.0, dtype=dtype, device=DEV)
        chai.chai_compact_k_cache(kf.to(DEV), torch.as_tensor(reps, device=DEV), T=T, k_rep=out)
        out = out.cpu()
        bits = kf.view(torch.int16 if dtype == torch.bfloat16 else torch.int32).numpy()
        want, _ = orc.compact_k_cache(np.ascontiguousarray(bits[:, :, :T]), reps)
        got = out.view(torch.int16 if dtype == torch.bfloat16 else torch.int32).numpy()
        assert np.array_equal(got[:, :, :T], want)
        assert (out[:, :, T:] == 3.0).all()              # rows beyond T are not written
        assert not got[2, 3, :T].any()


@pytest.mark.parametrize("k", [12, 24, 36])
def test_compaction_bit_exact_at_workload_4_layer_shape(k):
    """The compaction calls the bench leg times (B 4, H 72, T 2048, D 128, k = 12 / 24 / 36), out of place and in place,
    bit for bit against the oracle's gather."""
    w = synth.WORKLOADS[4]
    B, H, T, D = w.B, w.H, w.T, w.D
    g = torch.Generator().manual_seed(k)
    kf = torch.randn(B, H, T, D, generator=g).to(torch.bfloat16)
    _, reps = synth.batch_partitions(B, H, k, "uneven", k, 4)
    reps_t = torch.as_tensor(reps, device=DEV)
    want, _ = orc.compact_k_cache(kf.view(torch.int16).numpy(), reps)
    got = chai.chai_compact_k_cache(kf.to(DEV), reps_t)
    assert np.array_equal(got.cpu().view(torch.int16).numpy(), want)
    cache = kf.to(DEV).clone()
    chai.chai_compact_k_cache_inplace(cache, reps_t)
    assert np.array_equal(cache[:, :k].cpu().view(torch.int16).numpy(), want)


# ---- prefill --------------------------------------------------------------------------------------------

def prefill_inputs(seed, B, H, T, k, dtype="bf16", kind="uneven", peaked=1.0, D=128):
    r = synth.batch_partitions(B, H, k, kind, seed, 77, T)
    g = torch.Generator().manual_seed(seed)
    td = synth.TORCH_DTYPE[dtype]
    sigma = 0.5 if dtype == "bf16" else 1.0
    q = (torch.randn(B, H, T, D, generator=g) * sigma * peaked).to(td)
    kr = (torch.randn(B, k, T, D, generator=g) * sigma).to(td)
    v = (torch.randn(B, H, T, D, generator=g) * sigma).to(td)
    return dict(q=q, k_rep=kr, v=v, membership=torch.as_tensor(r[0]), reps=torch.as_tensor(r[1]),
                scale=1.0 / np.sqrt(D), dtype=dtype)


def run_prefill(case, causal=True, fn=None, guard=None):
    fn = fn or chai.chai_prefill_attention
    d = to_dev(case)
    out = fn(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"], causal,
             out=None if guard is None else guard.empty_like(d["q"]))
    torch.cuda.synchronize()
    return out.float().cpu().numpy()


@pytest.mark.parametrize("fn_name", ["chai_prefill_attention", "chai_prefill_attention_simt"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("T", [1, 5, 31, 33, 64, 100, 128, 129, 200, 257, 300])
def test_prefill_ragged_lengths(fn_name, dtype, T, guard):
    case = prefill_inputs(T, 2, 7, T, 3, dtype, peaked=4.0)
    for causal in (True, False):
        got = run_prefill(case, causal, getattr(chai, fn_name), guard=guard)
        ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"],
                                case["scale"], causal)
        assert_parity(got, ref, dtype, f"{fn_name} {dtype} T {T} causal {causal}")


@pytest.mark.parametrize("H,k,kind", [(8, 8, "even"), (8, 1, "even"), (12, 3, "even"), (16, 2, "uneven"),
                                      (52, 13, "uneven"), (9, 4, "uneven"), (72, 36, "uneven"), (100, 7, "uneven"),
                                      (64, 64, "even"), (33, 2, "uneven")])
def test_prefill_cluster_shapes(H, k, kind):
    """Singletons (plain MHA), one cluster of everything, groups of 1..many members."""
    case = prefill_inputs(H * k, 1, H, 160, k, "bf16", kind, peaked=4.0)
    got = run_prefill(case)
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], True)
    assert_parity(got, ref, "bf16", f"H {H} k {k}")


@pytest.mark.parametrize("direction", ["growing", "shrinking", "late_spike"])
@pytest.mark.parametrize("causal", [True, False])
def test_prefill_reference_moves(direction, causal):
    """Scores that drift by more than 2^8 from one key tile to the next: the running softmax reference has
    to move (and the accumulated output has to be rescaled) in every tile, or never after the first, or
    once near the end: the paths of the online softmax that ordinary random inputs rarely reach."""
    B, H, T, k, D = 1, 6, 640, 2, 128
    r = synth.batch_partitions(B, H, k, "uneven", 11, 78, T)
    g = torch.Generator().manual_seed(5)
    u = torch.randn(D, generator=g)
    u = u / u.norm()
    t = torch.arange(T, dtype=torch.float32)
    if direction == "growing":
        ramp = 0.1 * t                      # log2-domain score grows by ~18 per tile of 128 keys
    elif direction == "shrinking":
        ramp = 0.1 * (T - 1 - t)
    else:
        ramp = torch.where(t >= 600, torch.full_like(t, 40.0), torch.zeros_like(t))
    scale = 1.0 / np.sqrt(D)
    # q . k_t * scale * log2(e) = ramp_t  (up to bf16 rounding), plus a little noise in other directions
    q = (u * 4.0).expand(B, H, T, D) + 0.05 * torch.randn(B, H, T, D, generator=g)
    kr = (ramp[:, None] * u[None, :] / (4.0 * scale * 1.4426950408889634)).expand(B, k, T, D) \
        + 0.05 * torch.randn(B, k, T, D, generator=g)
    v = 0.5 * torch.randn(B, H, T, D, generator=g)
    case = dict(q=q.to(torch.bfloat16), k_rep=kr.to(torch.bfloat16), v=v.to(torch.bfloat16),
                membership=torch.as_tensor(r[0]), reps=torch.as_tensor(r[1]), scale=scale, dtype="bf16")
    got = run_prefill(case, causal)
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], scale, causal)
    assert np.isfinite(got).all()
    assert_parity(got, ref, "bf16", f"reference moves: {direction} causal {causal}")


@pytest.mark.parametrize("T", [1, 33, 128, 129, 150, 300, 700])
@pytest.mark.parametrize("H,k,kind", [(6, 2, "uneven"), (8, 8, "even"), (8, 2, "even")])
def test_prefill_head_dim_64(T, H, k, kind):
    """head_dim 64 on the tensor-core kernel (one 64-column block per tile; pairs of members, single members and
    the moving-reference path all occur), causal and not, against the oracle; the CUDA-core kernel beside it."""
    case = prefill_inputs(9 + T, 2, H, T, k, "bf16", kind, D=64, peaked=4.0)
    for causal in (True, False):
        ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], causal)
        assert_parity(run_prefill(case, causal), ref, "bf16", f"D 64 T {T} H {H} k {k} causal {causal}")
    if T == 150:
        got = run_prefill(case, True, chai.chai_prefill_attention_simt)
        ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], True)
        assert_parity(got, ref, "bf16", "D 64, CUDA-core kernel")


def test_prefill_negative_controls_and_bad_membership():
    case = prefill_inputs(2, 1, 8, 256, 4, "bf16", "even", peaked=8.0)
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], True)
    assert gate_ok(run_prefill(case), ref, "bf16")
    wrong = dict(case)
    wrong["k_rep"] = case["k_rep"][:, [1, 0, 2, 3]].contiguous()
    assert not gate_ok(run_prefill(wrong), ref, "bf16")
    # invalid cluster id on a non-representative head: reported, zero rows, other heads intact
    d = to_dev(case)
    hbad = [h for h in range(8) if h not in case["reps"][0].tolist()][0]
    mem = d["membership"].clone()
    mem[0, hbad] = -5
    ws = chai.new_workspace(chai.chai_prefill_workspace_bytes(1, 8, 4, 256, 128, chai.CHAI_BF16), DEV)
    out = torch.full_like(d["q"], 7.0)
    chai.chai_prefill_attention(d["q"], d["k_rep"], d["v"], mem, d["reps"], case["scale"], True, out=out, workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_ERR_BAD_MEMBERSHIP
    got = out.float().cpu().numpy()
    assert not got[0, hbad].any()
    keep = np.arange(8) != hbad
    assert gate_ok(got[0, keep], ref[0, keep], "bf16")


@pytest.mark.parametrize("fn_name", ["chai_prefill_attention", "chai_prefill_attention_simt"])
def test_prefill_many_unresolved_heads(fn_name):
    """A whole cluster loses its representative and two more heads carry ids out of range: seven heads in all,
    i.e. more than one zero-fill group; the others are untouched."""
    case = prefill_inputs(5, 2, 40, 200, 8, "bf16", "even", peaked=4.0)   # 8 clusters of 5 heads
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], True)
    d = to_dev(case)
    mem, reps = d["membership"].clone(), d["reps"].clone()
    lost = [h for h in range(40) if int(case["membership"][1, h]) == 3]
    reps[1, 3] = -1                                                     # cluster 3 of request 1: no representative
    others = [h for h in range(40) if h not in lost and h not in case["reps"][1].tolist()][:2]
    mem[1, others[0]] = 99
    mem[1, others[1]] = -1
    bad = sorted(lost + others)
    ws = chai.new_workspace(chai.chai_prefill_workspace_bytes(2, 40, 8, 200, 128, chai.CHAI_BF16), DEV)
    out = torch.full_like(d["q"], 7.0)
    getattr(chai, fn_name)(d["q"], d["k_rep"], d["v"], mem, reps, case["scale"], True, out=out, workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_ERR_BAD_MEMBERSHIP
    got = out.float().cpu().numpy()
    assert not got[1, bad].any()
    keep = np.array([h not in bad for h in range(40)])
    assert gate_ok(got[1, keep], ref[1, keep], "bf16")
    assert gate_ok(got[0], ref[0], "bf16")


def test_prefill_more_requests_than_one_launch_holds():
    """70 requests: the tensor-core path walks them in two launches of at most 64, each with its own work counter."""
    case = prefill_inputs(8, 70, 4, 140, 2, "bf16", "uneven", peaked=4.0)
    got = run_prefill(case)
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], True)
    assert_parity(got, ref, "bf16", "B 70")


def test_unused_cluster_slots():
    """k = 5 slots of which only 3 hold a cluster (what clustering returns when it finds fewer distinct points):
    reps = -1 at the end, no head points there; decode and prefill skip the dead planes."""
    B, H, k, T = 2, 8, 5, 200
    case = prefill_inputs(3, B, H, T, 3, "bf16", "even", peaked=4.0)
    mem = case["membership"]
    reps = torch.full((B, k), -1, dtype=torch.int32)
    reps[:, :3] = case["reps"]
    k_rep = torch.zeros(B, k, T, 128, dtype=torch.bfloat16)
    k_rep[:, :3] = case["k_rep"]
    k_rep[:, 3:] = float("nan")                                       # dead planes: never read into a result
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], mem, case["reps"], case["scale"], True)
    d = {n: x.to(DEV) for n, x in (("q", case["q"]), ("k_rep", k_rep), ("v", case["v"]), ("mem", mem), ("reps", reps))}
    for fn in (chai.chai_prefill_attention, chai.chai_prefill_attention_simt):
        ws = chai.new_workspace(chai.chai_prefill_workspace_bytes(B, H, k, T, 128, chai.CHAI_BF16), DEV)
        out = fn(d["q"], d["k_rep"], d["v"], d["mem"], d["reps"], case["scale"], True, workspace=ws)
        assert chai.chai_device_status(ws) == chai.CHAI_OK
        assert_parity(out.float().cpu().numpy(), ref, "bf16", f"{fn.__name__} with unused slots")
    q_last = d["q"][:, :, -1].contiguous()
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(B, H, k, T, 128, chai.CHAI_BF16), DEV)
    dec = chai.chai_decode_attention(q_last, d["k_rep"], d["v"], d["mem"], d["reps"], case["scale"], workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_OK
    assert_parity(dec.float().cpu().numpy(), ref[:, :, -1], "bf16", "decode with unused slots")


def test_prefill_full_size_sampled_rows():
    """Workload 5 at full size: the first 192 rows, 64 rows in the middle of the prompt that straddle a query-tile
    boundary, and the last 64 rows of every request and head (causal attention of a row depends only on the keys
    up to it, so the oracle runs on the prefix that ends with the sampled rows; the last rows see everything)."""
    case = synth.prefill_case(seed=0, device=DEV)
    k_rep = chai.chai_compact_k_cache(case["k_full"], case["reps"])
    out = chai.chai_prefill_attention(case["q_full"], k_rep, case["v"], case["membership"], case["reps"], case["scale"])
    out2 = chai.chai_prefill_attention(case["q_full"], k_rep, case["v"], case["membership"], case["reps"], case["scale"])
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    T = case["T"]
    q, kr, v = case["q_full"].cpu(), k_rep.cpu(), case["v"].cpu()
    mem, reps = case["membership"].cpu(), case["reps"].cpu()
    head = orc.cha_attention(q[:, :, :192], kr[:, :, :192], v[:, :, :192], mem, reps, case["scale"], True)
    assert_parity(out[:, :, :192].float().cpu().numpy(), head, "bf16", "first rows")
    tail = orc.cha_attention(q[:, :, T - 64:], kr, v, mem, reps, case["scale"], True)
    assert_parity(out[:, :, T - 64:].float().cpu().numpy(), tail, "bf16", "last rows")
    lo, hi = 992, 1056                                            # rows 992..1023 end one query tile, 1024..1055 begin the next
    mid = orc.cha_attention(q[:, :, :hi], kr[:, :, :hi], v[:, :, :hi], mem, reps, case["scale"], True)
    assert_parity(out[:, :, lo:hi].float().cpu().numpy(), mid[:, :, lo:hi], "bf16", "middle rows")


def test_prefill_negative_controls_at_workload_5_statistics():
    """The gates must tell a wrong clustering from the right one on the bench workload's own value distribution
    (near-uniform softmax, small outputs), not only on peaked inputs: the same call with the representatives' key
    planes rolled by one cluster, and with every non-representative head moved to the next cluster, must FAIL
    the gates that the correct call passes (first 192 rows of every request and head)."""
    case = synth.prefill_case(seed=0, device=DEV)
    k_rep = chai.chai_compact_k_cache(case["k_full"], case["reps"])
    n = 192
    q, v = case["q_full"][:, :, :n].contiguous(), case["v"][:, :, :n].contiguous()
    kr = k_rep[:, :, :n].contiguous()
    mem, reps = case["membership"], case["reps"]
    ref = orc.cha_attention(q.cpu(), kr.cpu(), v.cpu(), mem.cpu(), reps.cpu(), case["scale"], True)
    run = lambda kk, mm: chai.chai_prefill_attention(q, kk, v, mm, reps, case["scale"]).float().cpu().numpy()
    assert gate_ok(run(kr, mem), ref, "bf16")
    assert not gate_ok(run(torch.roll(kr, 1, dims=1).contiguous(), mem), ref, "bf16")
    is_rep = torch.zeros_like(mem, dtype=torch.bool)
    is_rep.scatter_(1, reps.long(), True)
    moved = torch.where(is_rep, mem, (mem + 1) % case["k"]).to(mem.dtype)   # still consistent: every representative stays put
    ws = chai.new_workspace(chai.chai_prefill_workspace_bytes(case["B"], case["H"], case["k"], n, case["D"], chai.CHAI_BF16), DEV)
    out = chai.chai_prefill_attention(q, kr, v, moved, reps, case["scale"], workspace=ws)
    assert chai.chai_device_status(ws) == chai.CHAI_OK
    assert not gate_ok(out.float().cpu().numpy(), ref, "bf16")


def test_prefill_long_prompt_sampled_rows():
    """A prompt of 40 query tiles plus a ragged one: first rows, rows around a tile boundary in the middle, last rows."""
    B, H, k, T, D = 1, 6, 2, 5003, 128
    r = synth.batch_partitions(B, H, k, "uneven", 3, 77, T)
    gen = torch.Generator().manual_seed(11)
    q = (torch.randn(B, H, T, D, generator=gen) * 2.0).to(torch.bfloat16)
    kr = (torch.randn(B, k, T, D, generator=gen) * 0.5).to(torch.bfloat16)
    v = (torch.randn(B, H, T, D, generator=gen) * 0.5).to(torch.bfloat16)
    mem, reps = torch.as_tensor(r[0]), torch.as_tensor(r[1])
    scale = 1.0 / np.sqrt(D)
    out = chai.chai_prefill_attention(q.to(DEV), kr.to(DEV), v.to(DEV), mem.to(DEV), reps.to(DEV), scale)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    for lo, hi in ((0, 70), (2530, 2600), (T - 45, T)):
        # rows [lo, hi) see keys [0, hi): the oracle runs on that prefix and its last hi - lo rows are compared
        ref = orc.cha_attention(q[:, :, :hi], kr[:, :, :hi], v[:, :, :hi], mem, reps, scale, True)
        assert_parity(got[:, :, lo:hi], ref[:, :, lo:hi], "bf16", f"long prompt rows {lo}..{hi}")


def test_prefill_head_dim_64_full_size_sampled_rows():
    """Workload 5's shape with 64-wide heads (groups of four members on the tensor-core kernel): run-to-run
    bitwise identical, first and last rows against the oracle."""
    B, H, k, T, D = 4, 32, 8, 2048, 64
    case = prefill_inputs(21, B, H, T, k, "bf16", "even", D=D, peaked=4.0)
    d = to_dev(case)
    out = chai.chai_prefill_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"])
    out2 = chai.chai_prefill_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"])
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    q, kr, v, mem, reps = case["q"], case["k_rep"], case["v"], case["membership"], case["reps"]
    head = orc.cha_attention(q[:, :, :192], kr[:, :, :192], v[:, :, :192], mem, reps, case["scale"], True)
    assert_parity(out[:, :, :192].float().cpu().numpy(), head, "bf16", "D 64 first rows")
    tail = orc.cha_attention(q[:, :, T - 64:], kr, v, mem, reps, case["scale"], True)
    assert_parity(out[:, :, T - 64:].float().cpu().numpy(), tail, "bf16", "D 64 last rows")
    lo, hi = 992, 1056                                            # across the boundary between two query tiles
    mid = orc.cha_attention(q[:, :, :hi], kr[:, :, :hi], v[:, :, :hi], mem, reps, case["scale"], True)
    assert_parity(out[:, :, lo:hi].float().cpu().numpy(), mid[:, :, lo:hi], "bf16", "D 64 middle rows")


@pytest.mark.parametrize("B,H,k,T,D,kind", [
    (4, 32, 3, 3000, 64, "even"),      # clusters of 10-11 heads: items of three and four members, T not a tile multiple
    (3, 32, 5, 2048, 64, "uneven"),
    (4, 32, 3, 3000, 128, "even"),
    (2, 16, 2, 1500, 128, "uneven"),
])
def test_prefill_is_bitwise_repeatable_with_full_groups(B, H, k, T, D, kind):
    """Large clusters fill every work item with the most members the kernel takes; a work item's accumulators
    are reused from item to item.  Four runs must agree bit for bit, and the last rows must match the oracle."""
    case = prefill_inputs(40 + k, B, H, T, k, "bf16", kind, D=D, peaked=4.0)
    d = to_dev(case)
    outs = [chai.chai_prefill_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"])
            for _ in range(4)]
    torch.cuda.synchronize()
    for o in outs[1:]:
        assert torch.equal(outs[0], o)
    q, kr, v, mem, reps = case["q"], case["k_rep"], case["v"], case["membership"], case["reps"]
    tail = orc.cha_attention(q[:1, :, T - 32:], kr[:1], v[:1], mem[:1], reps[:1], case["scale"], True)
    assert_parity(outs[0][:1, :, T - 32:].float().cpu().numpy(), tail, "bf16", "last rows")


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("shape", ["all_far_below", "all_far_above", "growing", "shrinking", "growing_in_one_quadrant"])
def test_prefill_scores_far_from_the_softmax_reference(D, shape):
    """Scores whose size forces the kernel's running softmax reference to move: all of a row's scores far below
    or far above zero, and scores that grow (or fall) by hundreds of powers of two along the keys.  One
    coordinate of Q and K carries the offset, so the oracle sees the same stored values."""
    B, H, k, T = 2, 8, 3, 1900
    case = prefill_inputs(60, B, H, T, k, "bf16", "uneven", D=D, peaked=2.0)
    q, kr = case["q"].clone(), case["k_rep"].clone()
    unit = float(np.sqrt(D)) / 1.4427           # a product of this size moves a score by one power of two
    ramp = torch.linspace(0.0, 1.0, T)
    if shape == "all_far_below":                # every score about 2^-100 relative to the reference at zero
        q[..., 0], kr[..., 0] = 10.0, -10.0 * unit
    elif shape == "all_far_above":
        q[..., 0], kr[..., 0] = 10.0, 10.0 * unit
    elif shape == "growing":                    # later keys outweigh earlier ones by up to 2^300
        q[..., 0] = 10.0
        kr[..., 0] = (30.0 * unit * ramp).to(torch.bfloat16)
    elif shape == "growing_in_one_quadrant":    # only rows 32..63 of every 128: their warps recompute and rescale tile
        q[..., 0] = 0.0                         # after tile and fall behind the warps of the other rows
        rows = torch.arange(T)
        q[:, :, (rows % 128 >= 32) & (rows % 128 < 64), 0] = 10.0
        kr[..., 0] = (30.0 * unit * ramp).to(torch.bfloat16)
    else:                                       # the first keys dominate; later tiles lie far below the reference
        q[..., 0] = 10.0
        kr[..., 0] = (-30.0 * unit * ramp).to(torch.bfloat16)
    case["q"], case["k_rep"] = q, kr
    got = run_prefill(case)
    assert np.isfinite(got).all()
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], True)
    assert_parity(got, ref, "bf16", f"scores {shape}, D {D}")


def test_prefill_flow_features_kmeans_compaction_attention():
    """Workload 5's whole flow at reduced length: both sides derive the membership themselves."""
    case = synth.prefill_case(seed=1, B=2, T=192, peaked=4.0)
    d = to_dev(case, ("q_full", "k_full", "v"))
    feats = chai.chai_prefix_features(d["q_full"], d["k_full"], 5, case["scale"])
    mem, reps, ke, _ = chai.chai_cluster_heads(feats, case["k"], 20, 0)
    k_rep = chai.chai_compact_k_cache(d["k_full"], reps)
    out = chai.chai_prefill_attention(d["q_full"], k_rep, d["v"], mem, reps, case["scale"])
    torch.cuda.synchronize()
    o_feats = orc.prefix_features(case["q_full"], case["k_full"], 5, case["scale"])
    o_km = orc.kmeans(o_feats.astype(np.float32), case["k"], 20, 0)
    assert np.array_equal(mem.cpu().numpy(), o_km["membership"])          # bit-exact as a partition
    assert np.array_equal(mem.cpu().numpy(), case["planted"])
    assert np.array_equal(reps.cpu().numpy(), o_km["reps"])
    bits = case["k_full"].view(torch.int16).numpy()
    o_krep, _ = orc.compact_k_cache(bits, o_km["reps"])
    assert np.array_equal(k_rep.cpu().view(torch.int16).numpy(), o_krep)
    ref = orc.cha_attention(case["q_full"], torch.from_numpy(o_krep).view(torch.bfloat16), case["v"],
                            o_km["membership"], o_km["reps"], case["scale"], True)
    assert_parity(out.float().cpu().numpy(), ref, "bf16", "flow")
