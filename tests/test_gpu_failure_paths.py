"""Failure paths that ordinary runs never take: a device-side wait that runs out.

Nothing here faults or hangs a GPU.  The decode kernel's waits are all bounded by a cycle count that is a launch
parameter; with a limit of one cycle the first thread that has to wait at all gives up, the launch stops taking
work, waits for the copies it has in flight and returns with CHAI_ERR_TIMEOUT recorded.  The tests check that
the call returns, that the status is reported, that the launch that follows on the same workspace is correct,
and that nothing outside the buffers was written.
"""
import numpy as np
import pytest
import torch

from oracle import chai_oracle as orc
from paper_2403_08058_b200 import chai, synth
from parity import assert_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture
def short_waits():
    chai.chai_set_decode_wait_limit_cycles(1)
    yield
    chai.chai_set_decode_wait_limit_cycles(0)      # back to the default, whatever the test did


def decode_case(B, H, k, T, seed):
    case = synth.decode_layer(2, layer=seed % 5, seed=seed, B=B, H=H, T=T, k=k, with_k_full=False, peaked=4.0)
    d = {n: case[n].to(DEV) for n in ("q", "k_rep", "v", "membership", "reps")}
    ref = orc.cha_attention(case["q"], case["k_rep"], case["v"], case["membership"], case["reps"], case["scale"], False)
    return case, d, ref


@pytest.mark.parametrize("B,H,k,T", [(2, 8, 2, 700), (4, 12, 3, 3000)])
def test_decode_wait_that_runs_out_is_reported_and_the_next_launch_is_clean(B, H, k, T, guard, short_waits):
    case, d, ref = decode_case(B, H, k, T, seed=T)
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(B, H, k, T, 128, chai.CHAI_BF16), DEV)
    out = guard.empty_like(d["q"])
    # twice in a row with waits that cannot succeed: every tile has to come from HBM, which takes more than a cycle
    for _ in range(2):
        chai.chai_decode_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"], out=out,
                                   workspace=ws)
        assert chai.chai_device_status(ws) == chai.CHAI_ERR_TIMEOUT      # (the status read synchronises: the call returned)
    chai.chai_set_decode_wait_limit_cycles(0)
    for _ in range(2):                                                    # same workspace, default limit: clean results
        chai.chai_decode_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"], out=out,
                                   workspace=ws)
        assert chai.chai_device_status(ws) == chai.CHAI_OK
        assert_parity(out.float().cpu().numpy(), ref, "bf16", "launch after a timed-out launch")


def test_replayed_graph_recovers_after_a_timed_out_replay(guard):
    """A captured decode call is replayed with the same kernel arguments every time, the wait limit included: the
    launch count kept in the workspace must move on after a launch that gave up too, or the replay that follows
    would meet its own stale flags.  Capture with the default limit; make one EAGER launch time out in between."""
    B, H, k, T = 3, 8, 4, 1500
    case, d, ref = decode_case(B, H, k, T, seed=77)
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(B, H, k, T, 128, chai.CHAI_BF16), DEV)
    out = guard.empty_like(d["q"])
    call = lambda: chai.chai_decode_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"],
                                              out=out, workspace=ws)
    call()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        call()
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    assert chai.chai_device_status(ws) == chai.CHAI_OK
    chai.chai_set_decode_wait_limit_cycles(1)
    try:
        call()
        assert chai.chai_device_status(ws) == chai.CHAI_ERR_TIMEOUT
    finally:
        chai.chai_set_decode_wait_limit_cycles(0)
    for _ in range(2):
        out.zero_()
        graph.replay()
        assert chai.chai_device_status(ws) == chai.CHAI_OK
        assert_parity(out.float().cpu().numpy(), ref, "bf16", "replay after a timed-out launch")
