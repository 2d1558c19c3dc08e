"""GPU parity of the fp8 (e4m3) cache path: the quantiser bit for bit, the decode step against the oracle on the
numbers the bytes stand for."""
import numpy as np
import pytest
import torch

from oracle import chai_oracle as orc
from paper_2403_08058_b200 import chai, synth
from parity import assert_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def case_for(seed, B, H, k, T_cap, D=128):
    c = synth.decode_layer(2, seed=seed, B=B, H=H, T=T_cap, T_cap=T_cap, k=k, with_k_full=True)
    if D == 64:
        for n in ("q", "k_rep", "v", "k_full"):
            c[n] = c[n][..., :64].contiguous()
        c["scale"] = 0.125
    return c


# D = 128: 16-byte vector path; D = 12 with odd sizes: element-wise path; (2100, 2100): more than one pass per thread
@pytest.mark.parametrize("T,T_cap,D", [(300, 300, 128), (100, 256, 128), (1, 8, 128), (2100, 2100, 128), (33, 35, 12)])
def test_quantiser_bit_exact(T, T_cap, D):
    g = torch.Generator().manual_seed(T)
    x = (torch.randn(2, 5, T_cap, D, generator=g) * torch.tensor([0.01, 0.5, 1.0, 30.0, 0.0])[None, :, None, None])
    x = x.to(torch.bfloat16)
    x[0, 1, 0, :8] = torch.tensor([1.0625, 1.1875, 17.0, -17.0, 2.0 ** -12, 0.0, -0.0, 3.0]).to(torch.bfloat16)
    q8, scales = chai.chai_quantize_cache_fp8(x.to(DEV), T)
    want_q, want_s = orc.quantize_cache_fp8(x.float().numpy(), T)
    assert np.array_equal(scales.cpu().numpy(), want_s)
    got = q8.cpu().numpy()
    # the sign of a value that rounds to zero is not part of the contract: compare magnitudes there
    same = (got == want_q) | (((got | want_q) & 0x7F) == 0)
    assert same.all()
    assert not got[:, :, T:].any()


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("lens", [None, [700, 1, 129, 0], [256, 512, 300, 699]])
def test_decode_fp8(D, lens):
    B, H, k, T_cap = 4, 12, 3, 700
    c = case_for(17 + D, B, H, k, T_cap, D)
    k8, ks = chai.chai_quantize_cache_fp8(c["k_rep"].to(DEV))
    v8, vs = chai.chai_quantize_cache_fp8(c["v"].to(DEV))
    seq = None if lens is None else torch.tensor(lens, dtype=torch.int32, device=DEV)
    out = chai.chai_decode_attention_fp8(c["q"].to(DEV), k8, v8, ks, vs, c["membership"].to(DEV), c["reps"].to(DEV),
                                         c["scale"], seq_lens=seq)
    got = out.float().cpu().numpy()
    ref = orc.decode_attention_fp8(c["q"], k8.cpu().numpy(), v8.cpu().numpy(), ks.cpu().numpy(), vs.cpu().numpy(),
                                   c["membership"], c["reps"], lens if lens is not None else [T_cap] * B, c["scale"])
    assert np.isfinite(got).all()
    assert_parity(got, ref, "bf16", f"fp8 decode D {D} lens {lens}")
    # and the quantised result stays close to the bf16-cache result (sanity of the format, not a parity gate)
    full = orc.decode_attention_ragged(c["q"], c["k_rep"], c["v"], c["membership"], c["reps"],
                                       lens if lens is not None else [T_cap] * B, c["scale"])
    assert np.abs(ref - full).max() < 0.15 * max(np.abs(full).max(), 1e-6) + 0.05


def test_decode_fp8_from_a_cache_compacted_in_place():
    B, H, k, T_cap = 2, 8, 3, 260
    c = case_for(5, B, H, k, T_cap)
    cache = c["k_full"].to(DEV).clone()
    chai.chai_compact_k_cache_inplace(cache, c["reps"].to(DEV))
    k8_full, ks_full = chai.chai_quantize_cache_fp8(cache)            # all H planes; the first k are live
    v8, vs = chai.chai_quantize_cache_fp8(c["v"].to(DEV))
    ks = ks_full[:, :k].contiguous()
    out = chai.chai_decode_attention_fp8(c["q"].to(DEV), k8_full, v8, ks, vs, c["membership"].to(DEV), c["reps"].to(DEV),
                                         c["scale"])
    ref = orc.decode_attention_fp8(c["q"], k8_full[:, :k].cpu().numpy(), v8.cpu().numpy(), ks.cpu().numpy(),
                                   vs.cpu().numpy(), c["membership"], c["reps"], [T_cap] * B, c["scale"])
    assert_parity(out.float().cpu().numpy(), ref, "bf16", "fp8 decode, strided K cache")


@pytest.mark.parametrize("k", [8, 32])
def test_decode_fp8_at_workload_2_layer_shape(k):
    """The shape and launch configuration the fp8 bench leg times (B 16, H 32, T 2048, D 128): every output element
    against the oracle on the numbers the bytes stand for."""
    w = synth.WORKLOADS[2]
    c = synth.decode_layer(2, 3, 2, B=w.B, H=w.H, T=w.T, k=k)
    k8, ks = chai.chai_quantize_cache_fp8(c["k_rep"].to(DEV))
    v8, vs = chai.chai_quantize_cache_fp8(c["v"].to(DEV))
    out = chai.chai_decode_attention_fp8(c["q"].to(DEV), k8, v8, ks, vs, c["membership"].to(DEV), c["reps"].to(DEV),
                                         c["scale"])
    got = out.float().cpu().numpy()
    ref = orc.decode_attention_fp8(c["q"], k8.cpu().numpy(), v8.cpu().numpy(), ks.cpu().numpy(), vs.cpu().numpy(),
                                   c["membership"], c["reps"], [w.T] * w.B, c["scale"])
    assert np.isfinite(got).all()
    assert_parity(got, ref, "bf16", f"fp8 decode, workload 2 layer shape, k {k}")
