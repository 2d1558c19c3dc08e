"""The decode and prefill calls inside a captured CUDA graph: replays must stay correct although every kernel
argument is frozen at capture time (launch tokens, work counters and status words may not rely on the host)."""
import numpy as np
import pytest
import torch

from oracle import chai_oracle as orc
from paper_2403_08058_b200 import chai, synth
from parity import assert_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def capture(fn):
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=s):
        fn()
    return g


def test_decode_graph_replay_with_changing_inputs():
    c = synth.decode_layer(2, seed=3, B=4, H=16, T=1100, T_cap=1100, k=4)
    d = {n: c[n].to(DEV) for n in ("q", "k_rep", "v", "membership", "reps")}
    out = torch.empty_like(d["q"])
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(4, 16, 4, 1100, 128, chai.CHAI_BF16), DEV)
    call = lambda: chai.chai_decode_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], c["scale"],
                                              out=out, workspace=ws)
    call()                                       # eager warm-up (also what a serving engine does before capture)
    g = capture(call)
    gen = torch.Generator().manual_seed(1)
    for it in range(6):
        q_new = (torch.randn(c["q"].shape, generator=gen) * 0.5).to(torch.bfloat16)
        d["q"].copy_(q_new)                      # new queries in the captured buffer
        if it == 3:                              # and a new key cache: the scores of the previous replay are stale
            d["k_rep"].copy_((torch.randn(c["k_rep"].shape, generator=gen) * 0.5).to(torch.bfloat16))
            c["k_rep"] = d["k_rep"].cpu()
        g.replay()
        torch.cuda.synchronize()
        ref = orc.cha_attention(q_new, c["k_rep"], c["v"], c["membership"], c["reps"], c["scale"], False)
        assert_parity(out.float().cpu().numpy(), ref, "bf16", f"graph replay {it}")
        assert chai.chai_device_status(ws) == chai.CHAI_OK
    call()                                       # an eager call on the same workspace afterwards
    ref = orc.cha_attention(d["q"].cpu(), c["k_rep"], c["v"], c["membership"], c["reps"], c["scale"], False)
    assert_parity(out.float().cpu().numpy(), ref, "bf16", "eager after replays")


def test_prefill_graph_replay():
    B, H, k, T, D = 2, 8, 3, 300, 128
    r = synth.batch_partitions(B, H, k, "uneven", 1, 93, T)
    gen = torch.Generator().manual_seed(2)
    q = (torch.randn(B, H, T, D, generator=gen) * 2.0).to(torch.bfloat16).to(DEV)
    kr = (torch.randn(B, k, T, D, generator=gen) * 0.5).to(torch.bfloat16).to(DEV)
    v = (torch.randn(B, H, T, D, generator=gen) * 0.5).to(torch.bfloat16).to(DEV)
    mem, reps = torch.as_tensor(r[0]).to(DEV), torch.as_tensor(r[1]).to(DEV)
    out = torch.empty_like(q)
    ws = chai.new_workspace(chai.chai_prefill_workspace_bytes(B, H, k, T, D, chai.CHAI_BF16), DEV)
    scale = 1.0 / np.sqrt(D)
    call = lambda: chai.chai_prefill_attention(q, kr, v, mem, reps, scale, True, out=out, workspace=ws)
    call()
    g = capture(call)
    for it in range(3):
        q.copy_((torch.randn(B, H, T, D, generator=gen) * 2.0).to(torch.bfloat16))
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        ref = orc.cha_attention(q.cpu(), kr.cpu(), v.cpu(), mem.cpu(), reps.cpu(), scale, True)
        assert_parity(out.float().cpu().numpy(), ref, "bf16", f"prefill graph replay {it}")


def test_whole_flow_in_one_graph():
    """Features, clustering, compaction, prefill, append and a decode step captured as one graph: the kernels
    that are launched as programmatic dependents of one another keep their order inside a graph, and a replay on
    new inputs gives bit for bit what the same calls give eagerly."""
    case = synth.prefill_case(seed=4, B=2, T=300, peaked=4.0)
    k = case["k"]
    q, kf, v = (case[n].to(DEV).clone() for n in ("q_full", "k_full", "v"))
    B, H, T, D = q.shape
    T_cap = T + 8
    v_cache = torch.zeros(B, H, T_cap, D, dtype=v.dtype, device=DEV)
    k_cache = torch.zeros(B, k, T_cap, D, dtype=v.dtype, device=DEV)
    k_new = torch.randn(B, H, D, device=DEV).to(torch.bfloat16)
    v_new = torch.randn(B, H, D, device=DEV).to(torch.bfloat16)
    q_step = torch.randn(B, H, D, device=DEV).to(torch.bfloat16)
    res = {}

    def flow():
        feats = chai.chai_prefix_features(q, kf, 5, case["scale"])
        mem, reps, _, _ = chai.chai_cluster_heads(feats, k, 20, 0)
        k_rep = chai.chai_compact_k_cache(kf, reps)
        res["out"] = chai.chai_prefill_attention(q, k_rep, v, mem, reps, case["scale"])
        v_cache[:, :, :T].copy_(v)
        k_cache[:, :, :T].copy_(k_rep)
        lens = torch.full((B,), T, dtype=torch.int32, device=DEV)
        chai.chai_append_kv(k_new, v_new, k_cache, v_cache, reps, lens)
        res["dec"] = chai.chai_decode_attention_ragged(q_step, k_cache, v_cache, mem, reps, lens, case["scale"], T + 1)
        res["mem"] = mem

    flow()                                          # eager warm-up
    torch.cuda.synchronize()
    g = capture(flow)
    graph_res = dict(res)
    gen = torch.Generator().manual_seed(9)
    for it in range(3):
        other = synth.prefill_case(seed=10 + it, B=2, T=300, peaked=4.0)
        q.copy_(other["q_full"]); kf.copy_(other["k_full"]); v.copy_(other["v"])
        q_step.copy_((torch.randn(B, H, D, generator=gen)).to(torch.bfloat16))
        g.replay()
        torch.cuda.synchronize()
        got = {n: graph_res[n].clone() for n in ("out", "dec", "mem")}
        flow()                                      # the same calls, eagerly, on the same inputs
        torch.cuda.synchronize()
        for n in ("out", "dec", "mem"):
            assert torch.equal(got[n], res[n]), f"replay {it}: {n} differs from the eager result"
        km = orc.kmeans(orc.prefix_features(other["q_full"], other["k_full"], 5, case["scale"]).astype(np.float32), k, 20, 0)
        assert np.array_equal(got["mem"].cpu().numpy(), km["membership"])
        k_rep_ref = torch.stack([other["k_full"][b][torch.as_tensor(km["reps"][b]).long()] for b in range(B)])
        ref = orc.cha_attention(other["q_full"], k_rep_ref, other["v"], km["membership"], km["reps"], case["scale"], True)
        assert_parity(got["out"].float().cpu().numpy(), ref, "bf16", f"flow graph replay {it}")
