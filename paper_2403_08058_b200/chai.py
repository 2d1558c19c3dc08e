"""Thin ctypes binding of libchai.so: same names as include/chai.h, argument marshalling only.

Torch supplies device memory and the current stream; every step of the path runs in the
library's kernels.  There is no fallback: if the library has not been built (or cannot be
loaded) the first call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libchai.so")

CHAI_OK = 0
CHAI_ERR_INVALID_ARG, CHAI_ERR_UNSUPPORTED, CHAI_ERR_WORKSPACE = 1, 2, 3
CHAI_ERR_BAD_MEMBERSHIP, CHAI_ERR_TIMEOUT, CHAI_ERR_CUDA, CHAI_ERR_CACHE_FULL = 4, 5, 6, 7
CHAI_F32, CHAI_BF16 = 0, 1

# every symbol include/chai.h declares
EXPORTS = [
    "chai_prefix_features", "chai_cluster_heads", "chai_compact_k_cache", "chai_decode_attention",
    "chai_decode_workspace_bytes", "chai_decode_attention_host", "chai_decode_attention_host_async", "chai_decode_attention_host_streams", "chai_prefill_attention",
    "chai_prefill_attention_simt", "chai_prefill_workspace_bytes", "chai_device_status",
    "chai_status_string", "chai_last_error", "chai_version", "chai_decode_attention_static",
    "chai_decode_attention_ragged", "chai_append_kv", "chai_compact_k_cache_inplace",
    "chai_prefill_attention_from", "chai_prefill_attention_simt_from",
    "chai_decode_qkv_workspace_bytes", "chai_decode_attention_qkv", "chai_prefill_qkv_workspace_bytes",
    "chai_prefill_attention_qkv", "chai_broadcast_membership", "chai_select_representatives", "chai_cluster_sweep",
    "chai_quantize_cache_fp8", "chai_decode_fp8_workspace_bytes", "chai_decode_attention_fp8",
    "chai_set_decode_wait_limit_cycles",
]
DECODE_STATIC_SCRATCH_BYTES = 8 << 20   # CHAI_DECODE_STATIC_SCRATCH_BYTES

_lib = None


class ChaiError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"libchai status {status}: {text}")
        self.status = status


def load() -> ctypes.CDLL:
    """Load libchai.so from the package directory (raises if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2403_08058_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.chai_prefix_features.argtypes = [vp, vp, ci, ci, ci, ci, ci, cf, ci, vp, vp]
    lib.chai_cluster_heads.argtypes = [vp, ci, ci, ci, ci, ci, ctypes.c_uint64, vp, vp, vp, vp, vp]
    lib.chai_compact_k_cache.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, vp]
    lib.chai_decode_attention.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, vp, sz, vp]
    for name in ("chai_decode_attention_host", "chai_decode_attention_host_async"):
        getattr(lib, name).argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, vp, sz, vp]
    lib.chai_decode_attention_host_streams.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, vp,
                                                       sz, vp, vp, vp, vp, vp]
    for name in ("chai_prefill_attention", "chai_prefill_attention_simt"):
        getattr(lib, name).argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, ci, ci, vp, sz, vp]
    lib.chai_decode_attention_qkv.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, vp, sz, vp]
    lib.chai_prefill_attention_qkv.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, ci, vp, sz, vp]
    lib.chai_broadcast_membership.argtypes = [vp, vp, vp, vp, ci, ci, ci, vp]
    lib.chai_select_representatives.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp]
    lib.chai_quantize_cache_fp8.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp]
    lib.chai_decode_fp8_workspace_bytes.argtypes = [ci, ci, ci, ci, ci]
    lib.chai_decode_fp8_workspace_bytes.restype = sz
    lib.chai_decode_attention_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, sz, cf, vp, sz, vp]
    lib.chai_cluster_sweep.argtypes = [vp, ci, ci, ci, ci, ci, ctypes.c_uint64, vp, vp, vp]
    for name in ("chai_decode_workspace_bytes", "chai_prefill_workspace_bytes", "chai_decode_qkv_workspace_bytes",
                 "chai_prefill_qkv_workspace_bytes"):
        getattr(lib, name).argtypes = [ci, ci, ci, ci, ci, ci]
        getattr(lib, name).restype = sz
    lib.chai_decode_attention_ragged.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, sz, cf, ci, vp, sz, vp]
    lib.chai_append_kv.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, sz, ci, ci, vp, vp]
    lib.chai_compact_k_cache_inplace.argtypes = [vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, vp]
    for name in ("chai_prefill_attention_from", "chai_prefill_attention_simt_from"):
        getattr(lib, name).argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, ci, vp, sz, vp]
    lib.chai_decode_attention_static.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, ci, vp]
    lib.chai_device_status.argtypes = [vp, ctypes.POINTER(ci), vp]
    lib.chai_set_decode_wait_limit_cycles.argtypes = [ctypes.c_longlong]
    lib.chai_set_decode_wait_limit_cycles.restype = None
    lib.chai_status_string.argtypes = [ci]
    lib.chai_status_string.restype = ctypes.c_char_p
    lib.chai_last_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _check(rc: int) -> None:
    if rc != CHAI_OK:
        lib = load()
        text = lib.chai_last_error().decode() or lib.chai_status_string(rc).decode()
        raise ChaiError(rc, text)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return CHAI_F32
    if t.dtype == torch.bfloat16:
        return CHAI_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _dev(*tensors) -> None:
    for t in tensors:
        if t is None:
            continue
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("tensors must be contiguous CUDA tensors")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def chai_version() -> int:
    return int(load().chai_version())


def chai_status_string(status: int) -> str:
    return load().chai_status_string(int(status)).decode()


def chai_decode_workspace_bytes(B, H, k, T, D, dtype) -> int:
    return int(load().chai_decode_workspace_bytes(B, H, k, T, D, dtype))


def chai_prefill_workspace_bytes(B, H, k, T, D, dtype) -> int:
    return int(load().chai_prefill_workspace_bytes(B, H, k, T, D, dtype))


def chai_prefix_features(q_full, k_full, P: int, scale: float, features=None):
    """q_full, k_full [B,H,T_cap,D] -> features [B,H,P*P] fp32."""
    _dev(q_full, k_full, features)
    B, H, T_cap, D = q_full.shape
    if features is None:
        features = torch.empty((B, H, P * P), device=q_full.device, dtype=torch.float32)
    _check(load().chai_prefix_features(_ptr(q_full), _ptr(k_full), B, H, T_cap, D, P, scale, _dt(q_full),
                                       _ptr(features), _stream()))
    return features


def chai_cluster_heads(features, k: int, max_iter: int = 20, seed: int = 0, want_inertia: bool = True):
    """features [B,H,F] fp32 -> (membership [B,H] i32, reps [B,k] i32, k_eff [B] i32, inertia [B] f64|None)."""
    _dev(features)
    if features.dtype != torch.float32:
        raise TypeError("features must be float32")
    B, H, F = features.shape
    dev = features.device
    membership = torch.empty((B, H), device=dev, dtype=torch.int32)
    reps = torch.empty((B, k), device=dev, dtype=torch.int32)
    k_eff = torch.empty((B,), device=dev, dtype=torch.int32)
    inertia = torch.empty((B,), device=dev, dtype=torch.float64) if want_inertia else None
    _check(load().chai_cluster_heads(_ptr(features), B, H, F, k, max_iter, seed, _ptr(membership), _ptr(reps),
                                     _ptr(k_eff), _ptr(inertia), _stream()))
    return membership, reps, k_eff, inertia


def chai_cluster_sweep(features, k_max: int, max_iter: int = 20, seed: int = 0):
    """features [B,H,F] fp32 -> (inertia curve [B,k_max] f64, knee [B] int32): k-means for every k = 1..k_max."""
    _dev(features)
    if features.dtype != torch.float32:
        raise TypeError("features must be float32")
    B, H, F = features.shape
    curve = torch.empty((B, k_max), device=features.device, dtype=torch.float64)
    pick = torch.empty((B,), device=features.device, dtype=torch.int32)
    _check(load().chai_cluster_sweep(_ptr(features), B, H, F, k_max, max_iter, seed, _ptr(curve), _ptr(pick), _stream()))
    return curve, pick


def chai_select_representatives(features, membership, k: int):
    """features [B,H,F] fp32, membership [B,H] -> reps [B,k]: each cluster's member nearest to the cluster mean."""
    _dev(features, membership)
    B, H, F = features.shape
    reps = torch.empty((B, k), device=features.device, dtype=torch.int32)
    _check(load().chai_select_representatives(_ptr(features), _ptr(membership), B, H, F, k, _ptr(reps), _stream()))
    return reps


def chai_compact_k_cache(k_full, reps, T: int | None = None, k_rep=None):
    """k_full [B,H,T_cap,D], reps [B,k] -> k_rep [B,k,T_cap,D] (rows [0,T) of each slot are written)."""
    _dev(k_full, reps, k_rep)
    B, H, T_cap, D = k_full.shape
    k = reps.shape[1]
    T = T_cap if T is None else T
    if k_rep is None:
        k_rep = torch.empty((B, k, T_cap, D), device=k_full.device, dtype=k_full.dtype)
    _check(load().chai_compact_k_cache(_ptr(k_full), _ptr(k_rep), _ptr(reps), B, H, k, T, T_cap, D, _dt(k_full),
                                       _stream()))
    return k_rep


def new_workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty((max(int(nbytes), 256),), device=device, dtype=torch.uint8)


def chai_decode_attention(q, k_rep, v, membership, reps, scale: float, T: int | None = None, out=None,
                          workspace=None):
    """q [B,H,D], k_rep [B,k,T_cap,D], v [B,H,T_cap,D], membership [B,H], reps [B,k] -> out [B,H,D]."""
    _dev(q, k_rep, v, membership, reps, out, workspace)
    B, H, D = q.shape
    k, T_cap = k_rep.shape[1], k_rep.shape[2]
    T = T_cap if T is None else T
    dt = _dt(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(chai_decode_workspace_bytes(B, H, k, T, D, dt), q.device)
    _check(load().chai_decode_attention(_ptr(q), _ptr(k_rep), _ptr(v), _ptr(membership), _ptr(reps), _ptr(out), B,
                                        H, k, T, T_cap, D, scale, dt, _ptr(workspace), workspace.numel(),
                                        _stream()))
    return out


def chai_decode_attention_static(q, k_rep, v, membership, reps, scale: float, T: int | None = None, out=None):
    """Decode step that uses the library's built-in 8 MiB scratch array: for callers that cannot pass
    a workspace and must not allocate (all HBM already committed to a cache pool, or no allocation
    allowed on the hot loop).  Problems needing more scratch raise ChaiError(CHAI_ERR_WORKSPACE).
    `out` must be supplied by such callers; it is created here only for convenience in tests."""
    _dev(q, k_rep, v, membership, reps, out)
    B, H, D = q.shape
    k, T_cap = k_rep.shape[1], k_rep.shape[2]
    T = T_cap if T is None else T
    if out is None:
        out = torch.empty_like(q)
    _check(load().chai_decode_attention_static(_ptr(q), _ptr(k_rep), _ptr(v), _ptr(membership), _ptr(reps),
                                               _ptr(out), B, H, k, T, T_cap, D, scale, _dt(q), _stream()))
    return out


def chai_decode_attention_ragged(q, k_rep, v, membership, reps, seq_lens, scale: float, T_max: int, k_planes=None,
                                 out=None, workspace=None):
    """Ragged batch: seq_lens [B] int32 (device) gives each request's cached positions, T_max bounds them.
    k_rep is [B,k,T_cap,D], or (k_planes=k) a full [B,H,T_cap,D] cache whose first k planes hold the
    representatives (after chai_compact_k_cache_inplace)."""
    _dev(q, k_rep, v, membership, reps, seq_lens, out, workspace)
    B, H, D = q.shape
    k = reps.shape[1] if k_planes is None else k_planes
    T_cap = k_rep.shape[2]
    stride = k_rep.shape[1] * T_cap * D
    dt = _dt(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(chai_decode_workspace_bytes(B, H, k, T_max, D, dt), q.device)
    _check(load().chai_decode_attention_ragged(_ptr(q), _ptr(k_rep), _ptr(v), _ptr(membership), _ptr(reps),
                                               _ptr(seq_lens), _ptr(out), B, H, k, T_max, T_cap, D, stride, scale, dt,
                                               _ptr(workspace), workspace.numel(), _stream()))
    return out


def chai_append_kv(k_new, v_new, k_rep, v, reps, seq_lens, advance: bool = True, workspace=None):
    """One new token per request: k_rep[b][c][seq_lens[b]] = k_new[b][reps[b][c]], v[b][h][seq_lens[b]] = v_new[b][h];
    seq_lens is incremented afterwards when `advance`.  k_rep may be the full cache compacted in place."""
    _dev(k_new, v_new, k_rep, v, reps, seq_lens, workspace)
    B, H, D = k_new.shape
    k, T_cap = reps.shape[1], v.shape[2]
    stride = k_rep.shape[1] * T_cap * D
    _check(load().chai_append_kv(_ptr(k_new), _ptr(v_new), _ptr(k_rep), _ptr(v), _ptr(reps), _ptr(seq_lens), B, H, k,
                                 T_cap, D, stride, _dt(k_new), int(bool(advance)), _ptr(workspace), _stream()))


def chai_compact_k_cache_inplace(k_cache, reps, T: int | None = None, workspace=None):
    """k_cache [B,H,T_cap,D]: planes 0..k-1 of each request receive the representatives' keys (rows [0,T))."""
    _dev(k_cache, reps, workspace)
    B, H, T_cap, D = k_cache.shape
    k = reps.shape[1]
    T = T_cap if T is None else T
    _check(load().chai_compact_k_cache_inplace(_ptr(k_cache), _ptr(reps), B, H, k, T, T_cap, D, _dt(k_cache),
                                               _ptr(workspace), _stream()))
    return k_cache


def _decode_host(fn_name, q_host, out_host, q_stage, out_stage, k_rep, v, membership, reps, scale, workspace, T):
    _dev(q_stage, out_stage, k_rep, v, membership, reps, workspace)
    B, H, D = q_host.shape
    k, T_cap = k_rep.shape[1], k_rep.shape[2]
    T = T_cap if T is None else T
    _check(getattr(load(), fn_name)(q_host.data_ptr(), out_host.data_ptr(), _ptr(q_stage), _ptr(out_stage),
                                    _ptr(k_rep), _ptr(v), _ptr(membership), _ptr(reps), B, H, k, T, T_cap, D, scale,
                                    _dt(q_host), _ptr(workspace), workspace.numel(), _stream()))
    return out_host


def chai_decode_attention_host(q_host, out_host, q_stage, out_stage, k_rep, v, membership, reps, scale: float,
                               workspace, T: int | None = None):
    """Decode step with q / out in (pinned) host memory; returns after the stream has drained."""
    return _decode_host("chai_decode_attention_host", q_host, out_host, q_stage, out_stage, k_rep, v, membership,
                        reps, scale, workspace, T)


def chai_decode_attention_host_async(q_host, out_host, q_stage, out_stage, k_rep, v, membership, reps, scale: float,
                                     workspace, T: int | None = None):
    """As above but only enqueued on the current stream: out_host is valid after the caller synchronises it."""
    return _decode_host("chai_decode_attention_host_async", q_host, out_host, q_stage, out_stage, k_rep, v,
                        membership, reps, scale, workspace, T)


def chai_decode_attention_host_streams(q_host, out_host, q_stage, out_stage, k_rep, v, membership, reps, scale: float,
                                       workspace, stream, upload_stream, download_stream, uploaded_event,
                                       computed_event, T: int | None = None):
    """Host-buffer decode step over three torch streams and two torch events (see the header); nothing is
    synchronised here: out_host is valid once download_stream has drained."""
    _dev(q_stage, out_stage, k_rep, v, membership, reps, workspace)
    B, H, D = q_host.shape
    k, T_cap = k_rep.shape[1], k_rep.shape[2]
    T = T_cap if T is None else T
    # a torch event has no CUDA handle before its first record: record once where it does no harm
    for ev, st in ((uploaded_event, upload_stream), (computed_event, stream)):
        if not ev.cuda_event:
            ev.record(st)
    _check(load().chai_decode_attention_host_streams(
        q_host.data_ptr(), out_host.data_ptr(), _ptr(q_stage), _ptr(out_stage), _ptr(k_rep), _ptr(v), _ptr(membership),
        _ptr(reps), B, H, k, T, T_cap, D, scale, _dt(q_host), _ptr(workspace), workspace.numel(), stream.cuda_stream,
        upload_stream.cuda_stream, download_stream.cuda_stream, uploaded_event.cuda_event, computed_event.cuda_event))
    return out_host


def _prefill(fn_name, q, k_rep, v, membership, reps, scale, causal, out, workspace):
    _dev(q, k_rep, v, membership, reps, out, workspace)
    B, H, T, D = q.shape
    k = k_rep.shape[1]
    dt = _dt(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(chai_prefill_workspace_bytes(B, H, k, T, D, dt), q.device)
    _check(getattr(load(), fn_name)(_ptr(q), _ptr(k_rep), _ptr(v), _ptr(membership), _ptr(reps), _ptr(out), B, H, k,
                                    T, D, scale, int(bool(causal)), dt, _ptr(workspace), workspace.numel(),
                                    _stream()))
    return out


def _prefill_from(fn_name, q, k_rep, v, membership, reps, scale, q_start, causal, out, workspace):
    _dev(q, k_rep, v, membership, reps, out, workspace)
    B, H, T, D = q.shape
    k = k_rep.shape[1]
    dt = _dt(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(chai_prefill_workspace_bytes(B, H, k, T, D, dt), q.device)
    _check(getattr(load(), fn_name)(_ptr(q), _ptr(k_rep), _ptr(v), _ptr(membership), _ptr(reps), _ptr(out), B, H, k,
                                    T, int(q_start), D, scale, int(bool(causal)), dt, _ptr(workspace),
                                    workspace.numel(), _stream()))
    return out


def chai_prefill_attention_from(q, k_rep, v, membership, reps, scale: float, q_start: int, causal: bool = True,
                                out=None, workspace=None):
    """Rows [q_start, T) of the clustered prefill; rows before q_start of `out` are left untouched."""
    return _prefill_from("chai_prefill_attention_from", q, k_rep, v, membership, reps, scale, q_start, causal, out,
                         workspace)


def chai_prefill_attention_simt_from(q, k_rep, v, membership, reps, scale: float, q_start: int, causal: bool = True,
                                     out=None, workspace=None):
    return _prefill_from("chai_prefill_attention_simt_from", q, k_rep, v, membership, reps, scale, q_start, causal, out,
                         workspace)


def chai_prefill_attention(q, k_rep, v, membership, reps, scale: float, causal: bool = True, out=None,
                           workspace=None):
    """q [B,H,T,D], k_rep [B,k,T,D], v [B,H,T,D] -> out [B,H,T,D]."""
    return _prefill("chai_prefill_attention", q, k_rep, v, membership, reps, scale, causal, out, workspace)


def chai_prefill_attention_simt(q, k_rep, v, membership, reps, scale: float, causal: bool = True, out=None,
                                workspace=None):
    return _prefill("chai_prefill_attention_simt", q, k_rep, v, membership, reps, scale, causal, out, workspace)


def chai_decode_attention_qkv(q, k_rep, v_rep, membership, reps, scale: float, T: int | None = None, seq_lens=None,
                              out=None, workspace=None):
    """CHAI-QKV decode: q [B,H,D], k_rep / v_rep [B,k,T_cap,D] -> out [B,H,D] (a member's row = its cluster's)."""
    _dev(q, k_rep, v_rep, membership, reps, seq_lens, out, workspace)
    B, H, D = q.shape
    k, T_cap = k_rep.shape[1], k_rep.shape[2]
    T = T_cap if T is None else T
    dt = _dt(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(int(load().chai_decode_qkv_workspace_bytes(B, H, k, T, D, dt)), q.device)
    _check(load().chai_decode_attention_qkv(_ptr(q), _ptr(k_rep), _ptr(v_rep), _ptr(membership), _ptr(reps),
                                            _ptr(seq_lens), _ptr(out), B, H, k, T, T_cap, D, scale, dt, _ptr(workspace),
                                            workspace.numel(), _stream()))
    return out


def chai_prefill_attention_qkv(q, k_rep, v_rep, membership, reps, scale: float, causal: bool = True, q_start: int = 0,
                               out=None, workspace=None):
    """CHAI-QKV prefill: q [B,H,T,D], k_rep / v_rep [B,k,T,D] -> out [B,H,T,D]."""
    _dev(q, k_rep, v_rep, membership, reps, out, workspace)
    B, H, T, D = q.shape
    k = k_rep.shape[1]
    dt = _dt(q)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(int(load().chai_prefill_qkv_workspace_bytes(B, H, k, T, D, dt)), q.device)
    _check(load().chai_prefill_attention_qkv(_ptr(q), _ptr(k_rep), _ptr(v_rep), _ptr(membership), _ptr(reps), _ptr(out),
                                             B, H, k, T, int(q_start), D, scale, int(bool(causal)), dt, _ptr(workspace),
                                             workspace.numel(), _stream()))
    return out


def chai_broadcast_membership(membership_static, reps_static, B: int):
    """One membership [H] / reps [k] for every request -> ([B,H], [B,k]) int32 (CHAI-static)."""
    _dev(membership_static, reps_static)
    H, k = membership_static.numel(), reps_static.numel()
    dev = membership_static.device
    membership = torch.empty((B, H), device=dev, dtype=torch.int32)
    reps = torch.empty((B, k), device=dev, dtype=torch.int32)
    _check(load().chai_broadcast_membership(_ptr(membership_static), _ptr(reps_static), _ptr(membership), _ptr(reps), B,
                                            H, k, _stream()))
    return membership, reps


def chai_quantize_cache_fp8(cache, T: int | None = None):
    """cache [B,P,T_cap,D] bf16 -> (bytes [B,P,T_cap,D] uint8 in e4m3, scales [B,P] fp32); rows [0,T) are converted."""
    _dev(cache)
    if cache.dtype != torch.bfloat16:
        raise TypeError("the cache must be bfloat16")
    B, P, T_cap, D = cache.shape
    T = T_cap if T is None else T
    q8 = torch.zeros((B, P, T_cap, D), device=cache.device, dtype=torch.uint8)
    scales = torch.empty((B, P), device=cache.device, dtype=torch.float32)
    _check(load().chai_quantize_cache_fp8(_ptr(cache), _ptr(q8), _ptr(scales), B * P, T, T_cap, D, _stream()))
    return q8, scales


def chai_decode_attention_fp8(q, k_rep8, v8, k_scale, v_scale, membership, reps, scale: float, T: int | None = None,
                              seq_lens=None, out=None, workspace=None):
    """Decode on e4m3 caches: q [B,H,D] bf16, k_rep8 [B,k|H,T_cap,D] uint8, v8 [B,H,T_cap,D] uint8, scales fp32."""
    _dev(q, k_rep8, v8, k_scale, v_scale, membership, reps, seq_lens, out, workspace)
    B, H, D = q.shape
    k, T_cap = reps.shape[1], v8.shape[2]
    T = T_cap if T is None else T
    stride = k_rep8.shape[1] * T_cap * D
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(int(load().chai_decode_fp8_workspace_bytes(B, H, k, T, D)), q.device)
    _check(load().chai_decode_attention_fp8(_ptr(q), _ptr(k_rep8), _ptr(v8), _ptr(k_scale), _ptr(v_scale),
                                            _ptr(membership), _ptr(reps), _ptr(seq_lens), _ptr(out), B, H, k, T, T_cap, D,
                                            stride, scale, _ptr(workspace), workspace.numel(), _stream()))
    return out


def chai_set_decode_wait_limit_cycles(cycles: int) -> None:
    """Test hook: cycle limit of the decode kernel's device-side waits for the launches that follow (<= 0: default)."""
    load().chai_set_decode_wait_limit_cycles(int(cycles))


def chai_device_status(workspace) -> int:
    st = ctypes.c_int(0)
    _check(load().chai_device_status(_ptr(workspace), ctypes.byref(st), _stream()))
    return int(st.value)
