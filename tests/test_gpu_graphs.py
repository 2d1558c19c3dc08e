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
