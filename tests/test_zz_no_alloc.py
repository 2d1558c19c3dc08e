"""The allocation-free decode entry point (collected last on purpose).

chai_decode_attention_static serves callers that have no scratch to give and may not allocate:
it keeps the decode scratch in an 8 MiB array inside the library image.  It must give exactly what
chai_decode_attention gives with a caller-owned workspace, also on a second call that finds the
first call's leftovers in the array, and must refuse problems that do not fit.
"""
import pytest
import torch

from paper_2403_08058_b200 import chai, synth


@pytest.mark.gpu
def test_static_scratch_decode_matches_workspace_decode_twice():
    from oracle import chai_oracle as orc
    from parity import assert_parity
    dev = "cuda"
    # two calls in a row with different shapes: the second one sees stale scratch contents
    for cfg, kw in ((2, dict(seed=11, B=3, H=16, T=700, T_cap=704, k=4)), (3, dict(seed=12, B=2, H=20, T=333, k=7)),
                    (1, dict(seed=13, B=1, H=32, T=256, k=8))):
        case = synth.decode_layer(cfg, **kw)
        d = {n: case[n].to(dev) for n in ("q", "k_rep", "v", "membership", "reps")}
        want = chai.chai_decode_attention(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"],
                                          T=case["T"])
        out = torch.full_like(d["q"], 7.0)
        again = torch.full_like(d["q"], 7.0)
        chai.chai_decode_attention_static(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"],
                                          T=case["T"], out=out)
        # the second call is the one whose footprint is measured: by then the library's module is loaded on this
        # device, so whatever the call itself allocates would show in the driver's count of free bytes and in the
        # framework's count of allocations
        torch.cuda.synchronize()
        free_before, n_alloc_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_stats()["allocation.all.allocated"]
        chai.chai_decode_attention_static(d["q"], d["k_rep"], d["v"], d["membership"], d["reps"], case["scale"],
                                          T=case["T"], out=again)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == n_alloc_before
        # same kernels, same order of operations: the tolerance of the parity tests is met with zero error
        assert torch.equal(out, want) and torch.equal(again, want), (cfg, kw)
        # ... and against the definition itself, not only against the sibling entry point
        T = case["T"]
        ref = orc.cha_attention(case["q"], case["k_rep"][:, :, :T], case["v"][:, :, :T], case["membership"], case["reps"],
                                case["scale"], causal=False)
        assert_parity(again.float().cpu().numpy(), ref, case["dtype"], f"static entry, cfg {cfg}")


def test_static_scratch_rejects_what_does_not_fit():
    """Host-side check only (no launch): a problem whose scratch exceeds the built-in array is refused."""
    import os
    if not os.path.exists(chai.LIB_PATH):
        from paper_2403_08058_b200.build import build_library
        build_library()
    lib = chai.load()
    cap = chai.DECODE_STATIC_SCRATCH_BYTES
    assert cap == 8 << 20
    assert chai.chai_decode_workspace_bytes(16, 32, 32, 2048, 128, chai.CHAI_BF16) <= cap    # workload 2 fits
    need = chai.chai_decode_workspace_bytes(64, 64, 64, 8192, 128, chai.CHAI_BF16)
    assert need > cap
    rc = lib.chai_decode_attention_static(16, 16, 16, 16, 16, 16, 64, 64, 64, 8192, 8192, 128, 1.0, chai.CHAI_BF16, None)
    assert rc == chai.CHAI_ERR_WORKSPACE
    msg = lib.chai_last_error().decode()
    assert str(need) in msg and str(cap) in msg
