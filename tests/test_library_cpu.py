"""CPU-side checks of the C-ABI library: it loads, exports what include/chai.h declares, and its
host-side argument validation refuses bad calls before touching CUDA.  No kernel is launched."""
import ctypes
import os
import re

import pytest

from paper_2403_08058_b200 import chai

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(chai.LIB_PATH):
        from paper_2403_08058_b200.build import build_library
        build_library()
    return chai.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "chai.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(chai_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(chai.EXPORTS) == names


def test_version_and_status_strings(lib):
    assert chai.chai_version() >= 100
    assert chai.chai_status_string(0) == "ok"
    assert "workspace" in chai.chai_status_string(chai.CHAI_ERR_WORKSPACE)
    assert chai.chai_status_string(99) == "unknown status"


def test_workspace_sizes(lib):
    small = chai.chai_decode_workspace_bytes(1, 32, 8, 256, 128, chai.CHAI_F32)
    big = chai.chai_decode_workspace_bytes(16, 32, 32, 2048, 128, chai.CHAI_BF16)
    assert 256 < small < big < 64 << 20
    assert chai.chai_decode_workspace_bytes(1, 32, 8, 256, 96, chai.CHAI_F32) == 0     # head_dim unsupported
    assert chai.chai_decode_workspace_bytes(0, 32, 8, 256, 128, chai.CHAI_F32) == 0
    assert chai.chai_prefill_workspace_bytes(4, 32, 8, 2048, 128, chai.CHAI_BF16) >= 256 + 4 * 32 * 32


def test_host_validation_refuses_before_any_launch(lib):
    buf = (ctypes.c_char * 4096)()
    p = ctypes.addressof(buf)
    p16 = (p + 15) // 16 * 16
    ok = [p16] * 6
    # null pointer
    rc = lib.chai_decode_attention(None, p16, p16, p16, p16, p16, 1, 4, 2, 8, 8, 128, 1.0, 0, p16, 1 << 20, None)
    assert rc == chai.CHAI_ERR_INVALID_ARG and b"null" in lib.chai_last_error()
    # misaligned pointer
    rc = lib.chai_decode_attention(p16 + 4, *ok[1:], 1, 4, 2, 8, 8, 128, 1.0, 0, p16, 1 << 20, None)
    assert rc == chai.CHAI_ERR_INVALID_ARG and b"aligned" in lib.chai_last_error()
    # k > H, T > T_cap, bad sizes
    assert lib.chai_decode_attention(*ok, 1, 4, 5, 8, 8, 128, 1.0, 0, p16, 1 << 20, None) == chai.CHAI_ERR_INVALID_ARG
    assert lib.chai_decode_attention(*ok, 1, 4, 2, 9, 8, 128, 1.0, 0, p16, 1 << 20, None) == chai.CHAI_ERR_INVALID_ARG
    assert lib.chai_decode_attention(*ok, 0, 4, 2, 8, 8, 128, 1.0, 0, p16, 1 << 20, None) == chai.CHAI_ERR_INVALID_ARG
    # unsupported head_dim / dtype
    assert lib.chai_decode_attention(*ok, 1, 4, 2, 8, 8, 96, 1.0, 0, p16, 1 << 20, None) == chai.CHAI_ERR_UNSUPPORTED
    assert lib.chai_decode_attention(*ok, 1, 4, 2, 8, 8, 128, 1.0, 7, p16, 1 << 20, None) == chai.CHAI_ERR_UNSUPPORTED
    # workspace too small
    rc = lib.chai_decode_attention(*ok, 1, 4, 2, 8, 8, 128, 1.0, 0, p16, 16, None)
    assert rc == chai.CHAI_ERR_WORKSPACE and b"needed" in lib.chai_last_error()
    # prefill
    for fn in (lib.chai_prefill_attention, lib.chai_prefill_attention_simt):
        assert fn(None, *ok[1:], 1, 4, 2, 8, 128, 1.0, 1, 0, p16, 1 << 20, None) == chai.CHAI_ERR_INVALID_ARG
        assert fn(*ok, 1, 4, 9, 8, 128, 1.0, 1, 0, p16, 1 << 20, None) == chai.CHAI_ERR_INVALID_ARG
        assert fn(*ok, 1, 4, 2, 8, 128, 1.0, 1, 0, p16, 8, None) == chai.CHAI_ERR_WORKSPACE
        assert fn(*ok, 1, 4, 2, 8, 80, 1.0, 1, 0, p16, 1 << 20, None) == chai.CHAI_ERR_UNSUPPORTED
    # k-means, features, compaction
    assert lib.chai_cluster_heads(p16, 1, 4, 8, 5, 20, 0, p16, p16, p16, None, None) == chai.CHAI_ERR_INVALID_ARG
    assert lib.chai_cluster_heads(p16, 1, 4, 8, 2, 0, 0, p16, p16, p16, None, None) == chai.CHAI_ERR_INVALID_ARG
    assert lib.chai_cluster_heads(p16, 1, 1024, 64, 8, 20, 0, p16, p16, p16, None, None) == chai.CHAI_ERR_UNSUPPORTED
    assert lib.chai_prefix_features(p16, p16, 1, 4, 3, 128, 5, 1.0, 0, p16, None) == chai.CHAI_ERR_INVALID_ARG
    assert lib.chai_prefix_features(p16, p16, 1, 4, 64, 128, 33, 1.0, 0, p16, None) == chai.CHAI_ERR_UNSUPPORTED
    assert lib.chai_compact_k_cache(p16, p16, p16, 1, 4, 2, 8, 8, 128, 0, None) == chai.CHAI_ERR_INVALID_ARG  # overlap
    assert lib.chai_compact_k_cache(p16, None, p16, 1, 4, 2, 8, 8, 128, 0, None) == chai.CHAI_ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(chai, "_lib", None)
    monkeypatch.setattr(chai, "LIB_PATH", str(tmp_path / "libchai.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        chai.chai_version()


def test_product_code_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2403_08058_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower().replace(
                    "cpu oracle", ""), f


def header_prototypes():
    """name -> list of C parameter declarations, from include/chai.h (comments removed)."""
    text = open(os.path.join(ROOT, "include", "chai.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    protos = {}
    for m in re.finditer(r"\b(chai_[a-z0-9_]+)\s*\(([^;{]*?)\)\s*;", text, flags=re.S):
        params = [p.strip() for p in m.group(2).replace("\n", " ").split(",")]
        protos[m.group(1)] = [] if params == ["void"] else params
    return protos


def test_binding_signatures_match_the_header(lib):
    """Every entry point that takes arguments has ctypes argtypes of the header's arity, with pointers where the
    header has pointers, 64-bit integers for size_t / uint64_t and a float for float (a mismatch would corrupt the
    call silently)."""
    protos = header_prototypes()
    assert set(protos) == set(chai.EXPORTS)
    for name, params in protos.items():
        fn = getattr(lib, name)
        if not params:
            continue
        assert fn.argtypes is not None, f"{name}: no argtypes declared in the binding"
        assert len(fn.argtypes) == len(params), f"{name}: header has {len(params)} parameters, binding {len(fn.argtypes)}"
        for i, (decl, ct) in enumerate(zip(params, fn.argtypes)):
            where = f"{name} parameter {i} ({decl})"
            if "*" in decl:
                assert ct in (ctypes.c_void_p, ctypes.c_char_p) or issubclass(ct, ctypes._Pointer), where
            elif decl.startswith(("size_t", "uint64_t", "long long")):
                assert ctypes.sizeof(ct) == 8 and ct not in (ctypes.c_void_p, ctypes.c_double), where
            elif decl.startswith("float"):
                assert ct is ctypes.c_float, where
            else:
                assert ct is ctypes.c_int, where


def test_chai_log_prints_one_line_per_call():
    """CHAI_LOG=1: an entry point writes a line with its shapes and launch plan to stderr before it launches (here
    the launch itself cannot happen without a device; the pointers are never dereferenced on the host)."""
    import subprocess
    import sys
    code = (
        "import sys; sys.path.insert(0, %r)\n"
        "from paper_2403_08058_b200 import chai\n"
        "lib = chai.load()\n"
        "lib.chai_cluster_heads(256, 2, 32, 64, 8, 20, 7, 256, 256, 256, None, None)\n" % ROOT)
    for flag, expect in (("1", True), ("0", False)):
        r = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, CHAI_LOG=flag), capture_output=True, text=True)
        assert r.returncode == 0, r.stderr
        assert ("[chai] chai_cluster_heads: B=2 H=32 F=64 k=8 max_iter=20 seed=7" in r.stderr) == expect, r.stderr
