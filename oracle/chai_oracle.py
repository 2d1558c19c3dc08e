"""ctypes front end of the CPU oracle (test infrastructure, never the product path).

Compiles ``chai_oracle.c`` with gcc into ``libchai_oracle.so`` next to this file on
first use and exposes numpy-in / numpy-out wrappers.  Stored values (bf16 or fp32
bits) are widened exactly to float64 before they reach the C code.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "chai_oracle.c")
_LIB = os.path.join(_HERE, "libchai_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (fp contraction off, OpenMP on) and return the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.oracle_cha_attention.argtypes = [dp, dp, dp, ip, ip, dp] + [ctypes.c_int] * 6 + [
            ctypes.c_double, ctypes.c_int]
        lib.oracle_cha_attention.restype = ctypes.c_int
        lib.oracle_prefix_features.argtypes = [dp, dp, dp] + [ctypes.c_int] * 5 + [ctypes.c_double]
        lib.oracle_prefix_features.restype = ctypes.c_int
        lib.oracle_kmeans.argtypes = [dp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_uint64, ip, ip, ip, dp, dp, ip]
        lib.oracle_kmeans.restype = ctypes.c_int
        lib.oracle_compact_k_cache.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ip] + [
            ctypes.c_int] * 6 + [ctypes.POINTER(ctypes.c_int64)]
        lib.oracle_compact_k_cache.restype = ctypes.c_int
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def _f64(x) -> np.ndarray:
    """Exact widening to a C-contiguous float64 array (accepts numpy arrays and torch CPU tensors)."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(x, dtype=np.float64)


def _i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ip(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def cha_attention(q, k_rep, v, membership, reps, scale: float, causal: bool) -> np.ndarray:
    """Clustered-head attention.  q [B,H,Tq,D] (or [B,H,D] for decode), k_rep [B,k,T,D],
    v [B,H,T,D], membership [B,H], reps [B,k]  ->  float64 output shaped like q."""
    q = _f64(q)
    decode = q.ndim == 3
    if decode:
        q = q[:, :, None, :]
    k_rep, v = _f64(k_rep), _f64(v)
    membership, reps = _i32(membership), _i32(reps)
    B, H, Tq, D = q.shape
    k, T = k_rep.shape[1], k_rep.shape[2]
    assert k_rep.shape == (B, k, T, D) and v.shape == (B, H, T, D)
    assert membership.shape == (B, H) and reps.shape == (B, k)
    out = np.empty((B, H, Tq, D), dtype=np.float64)
    rc = _load().oracle_cha_attention(_dp(q), _dp(k_rep), _dp(v), _ip(membership), _ip(reps),
                                      _dp(out), B, H, k, Tq, T, D, float(scale), int(bool(causal)))
    if rc != 0:
        raise ValueError("oracle_cha_attention rejected its arguments")
    return out[:, :, 0, :] if decode else out


def prefix_features(q_full, k_full, P: int, scale: float) -> np.ndarray:
    """q_full, k_full [B,H,T,D] -> features [B,H,P*P] float64."""
    q_full, k_full = _f64(q_full), _f64(k_full)
    B, H, T, D = q_full.shape
    out = np.empty((B, H, P * P), dtype=np.float64)
    rc = _load().oracle_prefix_features(_dp(q_full), _dp(k_full), _dp(out), B, H, T, D, int(P),
                                        float(scale))
    if rc != 0:
        raise ValueError("oracle_prefix_features rejected its arguments")
    return out


def kmeans(features, k: int, max_iter: int = 20, seed: int = 0):
    """features [B,H,F] (or [H,F]) -> dict(membership [B,H], reps [B,k], k_eff [B], inertia [B],
    trace [B,max_iter], init_idx [B,k]); every request is clustered independently."""
    x = _f64(features)
    single = x.ndim == 2
    if single:
        x = x[None]
    B, H, F = x.shape
    membership = np.empty((B, H), dtype=np.int32)
    reps = np.empty((B, k), dtype=np.int32)
    k_eff = np.empty((B,), dtype=np.int32)
    inertia = np.empty((B,), dtype=np.float64)
    trace = np.empty((B, max_iter), dtype=np.float64)
    init_idx = np.empty((B, k), dtype=np.int32)
    lib = _load()
    for b in range(B):
        xb = np.ascontiguousarray(x[b])
        rc = lib.oracle_kmeans(_dp(xb), H, F, int(k), int(max_iter), ctypes.c_uint64(int(seed)),
                               _ip(membership[b]), _ip(reps[b]), _ip(k_eff[b:b + 1]),
                               _dp(inertia[b:b + 1]), _dp(trace[b]), _ip(init_idx[b]))
        if rc != 0:
            raise ValueError("oracle_kmeans rejected its arguments")
    res = dict(membership=membership, reps=reps, k_eff=k_eff, inertia=inertia, trace=trace,
               init_idx=init_idx)
    if single:
        res = {n: a[0] for n, a in res.items()}
    return res


def compact_k_cache(k_full: np.ndarray, reps) -> tuple[np.ndarray, tuple[int, int]]:
    """k_full [B,H,T,D] of any fixed-size dtype (pass bf16 as its uint16 bit pattern) ->
    (k_rep [B,k,T,D] same dtype, (kv_bytes_before, kv_bytes_after))."""
    k_full = np.ascontiguousarray(k_full)
    reps = _i32(reps)
    B, H, T, D = k_full.shape
    k = reps.shape[1]
    out = np.empty((B, k, T, D), dtype=k_full.dtype)
    nbytes = np.zeros(2, dtype=np.int64)
    rc = _load().oracle_compact_k_cache(k_full.ctypes.data_as(ctypes.c_void_p),
                                        out.ctypes.data_as(ctypes.c_void_p), _ip(reps), B, H, k, T,
                                        D, k_full.dtype.itemsize,
                                        nbytes.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)))
    if rc != 0:
        raise ValueError("oracle_compact_k_cache rejected its arguments")
    return out, (int(nbytes[0]), int(nbytes[1]))


# ---- serving-shaped steps (Section 3.5 / 4.3): each is the plain definition applied request by request ----

def decode_attention_ragged(q, k_rep, v, membership, reps, seq_lens, scale: float) -> np.ndarray:
    """Decode step of a ragged batch: request b attends to its first seq_lens[b] cached positions only.
    q [B,H,D], k_rep [B,k,T_cap,D], v [B,H,T_cap,D] -> float64 [B,H,D]; a request with length 0 gets zeros."""
    q, k_rep, v = _f64(q), _f64(k_rep), _f64(v)
    membership, reps = _i32(membership), _i32(reps)
    B, H, D = q.shape
    out = np.zeros((B, H, D), dtype=np.float64)
    for b in range(B):
        n = int(seq_lens[b])
        if n <= 0:
            continue
        out[b] = cha_attention(q[b:b + 1], k_rep[b:b + 1, :, :n], v[b:b + 1, :, :n], membership[b:b + 1],
                               reps[b:b + 1], scale, False)[0]
    return out


def append_kv(k_new, v_new, k_rep, v, reps, seq_lens):
    """One new token per request, written at row seq_lens[b]: the representatives' keys and every head's
    values.  Arrays of any dtype (bit copies); returns (k_rep', v', seq_lens + 1) as new arrays."""
    k_rep, v = np.array(k_rep, copy=True), np.array(v, copy=True)
    reps = _i32(reps)
    lens = np.array(seq_lens, dtype=np.int64, copy=True)
    B, k = reps.shape
    for b in range(B):
        pos = int(lens[b])
        if not 0 <= pos < v.shape[2]:
            continue  # no room: the request is skipped
        v[b, :, pos] = v_new[b]
        for c in range(k):
            r = int(reps[b, c])
            if 0 <= r < v.shape[1]:
                k_rep[b, c, pos] = k_new[b, r]
        lens[b] = pos + 1
    return k_rep, v, lens


def compact_k_cache_inplace(k_full: np.ndarray, reps, T: int) -> np.ndarray:
    """What the first k planes of each request hold after in-place compaction: the gather of
    compact_k_cache over rows [0,T).  Returns [B,k,T,D]; slots with reps = -1 are returned as zeros and are
    not compared (the in-place call leaves them as they were)."""
    k_rep, _ = compact_k_cache(k_full[:, :, :T], reps)
    return k_rep


# ---- variants the paper evaluates (Table 4, Section 3.5) -----------------------------------------------

def cha_attention_qkv(q, k_rep, v_rep, membership, reps, scale: float, causal: bool) -> np.ndarray:
    """CHAI-QKV: the values of non-representative heads are dropped too, i.e. every member head uses its
    representative's values.  Written as the main definition with V expanded accordingly:
    v[b][h] = v_rep[b][membership[b][h]]."""
    v_rep = _f64(v_rep)
    membership = _i32(membership)
    B, H = membership.shape
    v = np.stack([v_rep[b, membership[b]] for b in range(B)])
    return cha_attention(q, k_rep, v, membership, reps, scale, causal)


def closest_representatives(features, membership, k: int) -> np.ndarray:
    """Alternative to 'lowest member': per cluster the member nearest (squared Euclidean, fp64) to the mean of
    the cluster's members; ties to the lowest head index; -1 for an empty cluster.  features [B,H,F],
    membership [B,H] -> reps [B,k].  Sums run in ascending head / feature order, one rounding per operation."""
    x = _f64(features)
    membership = _i32(membership)
    B, H, F = x.shape
    reps = np.full((B, k), -1, dtype=np.int32)
    for b in range(B):
        for c in range(k):
            members = [h for h in range(H) if membership[b, h] == c]
            if not members:
                continue
            mean = np.zeros(F)
            for h in members:
                mean = mean + x[b, h]
            mean = mean / float(len(members))
            best, best_d = -1, 0.0
            for h in members:
                d = 0.0
                for f in range(F):
                    t = x[b, h, f] - mean[f]
                    d = d + t * t
                if best < 0 or d < best_d:
                    best, best_d = h, d
            reps[b, c] = best
    return reps


def knee_of_curve(e) -> int:
    """Knee of a decreasing error curve e[0..n-1] (entry i = error with i + 1 clusters): with the cluster count
    scaled to x in [0,1] and the error to y in [0,1], the count farthest below the line from (0,1) to (1,0),
    i.e. the maximiser of 1 - x - y; ties to the smaller count; a flat curve gives 1."""
    e = np.asarray(e, dtype=np.float64)
    n = len(e)
    lo, hi = float(e.min()), float(e.max())
    if n < 2 or not hi > lo:
        return 1
    best, best_v = 1, None
    for i in range(n):
        x = float(i) / float(n - 1)
        y = (float(e[i]) - lo) / (hi - lo)
        v = (1.0 - x) - y
        if best_v is None or v > best_v:
            best, best_v = i + 1, v
    return best


def cluster_sweep(features, k_max: int, max_iter: int = 20, seed: int = 0):
    """Clustering error for every k = 1..k_max (Section 3.2) and the knee of each curve.
    features [B,H,F] -> (curve [B,k_max] float64, knee [B] int32)."""
    x = _f64(features)
    B = x.shape[0]
    curve = np.empty((B, k_max), dtype=np.float64)
    for k in range(1, k_max + 1):
        curve[:, k - 1] = kmeans(x, k, max_iter, seed)["inertia"]
    return curve, np.array([knee_of_curve(curve[b]) for b in range(B)], dtype=np.int32)


# ---- fp8 (e4m3) caches: the number format written out, and the decode step on dequantised values ---------

def e4m3_values() -> np.ndarray:
    """The 256 numbers an e4m3 byte stands for: sign bit, 4 exponent bits (bias 7), 3 mantissa bits; exponent
    field 0 is subnormal (m/8 * 2^-6); there are no infinities and only exponent 15 with mantissa 7 is NaN."""
    out = np.empty(256, dtype=np.float64)
    for byte in range(256):
        sign = -1.0 if byte & 0x80 else 1.0
        e, m = (byte >> 3) & 0xF, byte & 0x7
        if e == 15 and m == 7:
            out[byte] = np.nan
        elif e == 0:
            out[byte] = sign * (m / 8.0) * 2.0 ** -6
        else:
            out[byte] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return out


def quantize_cache_fp8(cache_f32: np.ndarray, T: int):
    """cache [planes..., T_cap, D] (values exactly representable in float32, e.g. widened bf16) ->
    (bytes uint8 same shape, scales float32 [planes...]).  Per plane: scale = float32(max|x| over rows [0,T)) /
    float32(448) in float32 (1 if the plane is zero); element = float32(x) / scale in float32, rounded to the
    nearest e4m3 value, ties to the even mantissa, saturated to +-448.  Rows >= T are left zero."""
    x = np.asarray(cache_f32, dtype=np.float32)
    lead = x.shape[:-2]
    flat = x.reshape((-1,) + x.shape[-2:])
    vals = e4m3_values()
    pos = vals[:127]                      # bytes 0..126: the finite non-negative values in ascending order
    q = np.zeros(flat.shape, dtype=np.uint8)
    scales = np.empty(flat.shape[0], dtype=np.float32)
    for p in range(flat.shape[0]):
        amax = np.float32(np.max(np.abs(flat[p, :T]))) if T > 0 else np.float32(0)
        scale = np.float32(amax / np.float32(448.0)) if amax > 0 else np.float32(1.0)
        scales[p] = scale
        y = (flat[p, :T] / scale).astype(np.float32).astype(np.float64)
        mag = np.minimum(np.abs(y), 448.0)
        hi = np.searchsorted(pos, mag, side="left")          # first value >= mag
        hi = np.minimum(hi, 126)
        lo = np.maximum(hi - 1, 0)
        d_hi, d_lo = pos[hi] - mag, mag - pos[lo]
        take_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))   # ties: even mantissa = even byte
        code = np.where(take_lo, lo, hi).astype(np.uint8)
        code = np.where(pos[hi] == mag, hi, code).astype(np.uint8)
        q[p, :T] = code | np.where(np.signbit(y), 0x80, 0).astype(np.uint8)
    return q.reshape(x.shape), scales.reshape(lead)


def decode_attention_fp8(q, k8, v8, k_scale, v_scale, membership, reps, seq_lens, scale: float) -> np.ndarray:
    """The ragged decode definition on the numbers the fp8 caches stand for: byte -> e4m3 value * plane scale."""
    vals = e4m3_values()
    k_rep = vals[np.asarray(k8)] * np.asarray(k_scale, dtype=np.float64)[:, :, None, None]
    v = vals[np.asarray(v8)] * np.asarray(v_scale, dtype=np.float64)[:, :, None, None]
    return decode_attention_ragged(q, k_rep, v, membership, reps, seq_lens, scale)
