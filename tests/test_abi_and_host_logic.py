"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, sizes its workspace sensibly and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2011_06495_b200 import binding as B
from paper_2011_06495_b200 import build as BUILD

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADERS = sorted(os.path.join(ROOT, "include", f) for f in os.listdir(os.path.join(ROOT, "include")) if f.endswith(".h"))


@pytest.fixture(scope="module")
def lib():
    BUILD.build()                       # nvcc cross-compiles for sm_100a without a GPU
    return B.load()


def declared_functions():
    names = set()
    for header in HEADERS:
        text = re.sub(r"/\*.*?\*/", "", open(header).read(), flags=re.S)
        names |= set(re.findall(r"\b(mv_[a-z_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"mv_sparse_step", "mv_vote", "mv_select", "mv_aggregate", "mv_workspace_bytes", "mv_create",
            "mv_destroy", "mv_sparse_step_host", "mv_pos_encode", "mv_pos_decode", "mv_quantize",
            "mv_dequantize"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"


def test_status_strings(lib):
    for code in (0, -1, -2, -3, 99):
        assert B.status_string(code)
    assert "workspace" in B.status_string(B.MV_ERR_WORKSPACE)


def test_workspace_bytes_ranges(lib):
    assert B.workspace_bytes(0, 10, 1) == 0            # N out of range
    assert B.workspace_bytes(256, 10, 1) == 0
    assert B.workspace_bytes(4, 0, 1) == 0             # d out of range
    assert B.workspace_bytes(4, 1 << 31, 1) == 0
    assert B.workspace_bytes(4, 10, 0) == 0            # K out of range
    assert B.workspace_bytes(4, 10, 11) == 0
    small = B.workspace_bytes(4, 10_000, 100)
    big = B.workspace_bytes(10, 11_173_962, 111_739)
    assert 0 < small < big < 200e6
    assert B.workspace_bytes(64, 1 << 27, 1_342_177) < 9e9
    assert small % 256 == 0 and big % 256 == 0


def _fake_ctx(lib, nbytes):
    handle = ctypes.c_void_p()
    rc = lib.mv_create(ctypes.byref(handle), None, ctypes.c_void_p(0x10000), nbytes)   # never dereferenced
    assert rc == B.MV_OK
    return handle


def test_create_rejects_bad_workspace(lib):
    handle = ctypes.c_void_p()
    assert lib.mv_create(ctypes.byref(handle), None, None, 1024) == B.MV_ERR_INVALID_ARG
    assert lib.mv_create(ctypes.byref(handle), None, ctypes.c_void_p(0x10001), 1024) == B.MV_ERR_INVALID_ARG
    assert lib.mv_create(None, None, ctypes.c_void_p(0x10000), 1024) == B.MV_ERR_INVALID_ARG


def test_argument_checks_happen_before_any_launch(lib):
    """No GPU here: every call below must fail in validation, not in the CUDA runtime."""
    N, d, K = 4, 10_000, 100
    need = B.workspace_bytes(N, d, K)
    ctx = _fake_ctx(lib, need)
    p = lambda a: ctypes.c_void_p(a)
    g, e, oi, ov = 0x100000, 0x200000, 0x300000, 0x400000
    step = lib.mv_sparse_step
    assert step(None, p(g), p(e), N, d, K, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG
    assert step(ctx, None, p(e), N, d, K, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG
    assert step(ctx, p(g), p(e), N, d, K, None, p(ov)) == B.MV_ERR_INVALID_ARG
    assert step(ctx, p(g + 4), p(e), N, d, K, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG       # misaligned
    assert step(ctx, p(g), p(g + 16), N, d, K, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG      # grads overlaps err
    assert step(ctx, p(g), p(e), 0, d, K, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG
    assert step(ctx, p(g), p(e), 256, d, K, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG
    assert step(ctx, p(g), p(e), N, d, d + 1, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG
    assert step(ctx, p(g), p(e), N, d, 0, p(oi), p(ov)) == B.MV_ERR_INVALID_ARG
    assert step(ctx, p(g), p(e), N, 100 * d, K, p(oi), p(ov)) == B.MV_ERR_WORKSPACE       # sized for a smaller d
    assert lib.mv_vote(ctx, p(g), p(e), N, d, K, p(oi + 4), None, None, None) == B.MV_ERR_INVALID_ARG
    assert lib.mv_select(ctx, None, N, d, K, p(oi), None) == B.MV_ERR_INVALID_ARG
    assert lib.mv_aggregate(ctx, p(e), N, d, K, None, p(ov)) == B.MV_ERR_INVALID_ARG
    assert lib.mv_set_mode(ctx, 7) == B.MV_ERR_INVALID_ARG
    assert lib.mv_set_mode(ctx, B.MV_MODE_GENERAL) == B.MV_OK
    assert lib.mv_destroy(ctx) == B.MV_OK
    assert lib.mv_destroy(None) == B.MV_ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        B.load()


def test_wire_host_arithmetic_and_argument_checks(lib):
    """Stream sizes are host arithmetic (Eq. 14 when K = d / B), bad arguments are refused before any launch."""
    assert B.pos_offset_bits(1) == 0 and B.pos_offset_bits(100) == 7 and B.pos_offset_bits(128) == 7 and B.pos_offset_bits(129) == 8
    assert B.pos_stream_bits(12, 4, 3) == 12
    assert B.pos_stream_bits(128 * 1000, 128, 1000) == 1000 * 9            # log2(1/phi) + 2 bits per position
    assert B.pos_stream_bits(11_173_962, 100, 111_739) == 111_739 * 8 + 111_740
    assert B.pos_stream_bits(10, 11, 1) == -1 and B.pos_stream_bits(10, 2, 11) == -1 and B.pos_stream_bits(0, 1, 0) == -1
    assert B.quant_stream_words(10, 4) == 2 + 8 and B.quant_stream_words(0, 1) == 1
    assert B.quant_stream_words(10, 0) == -1 and B.quant_stream_words(10, 9) == -1
    assert B.pos_decode_workspace_bytes(2048 * 3 + 1, 128) >= 4 * (8 * 4 + 4 + 8 + 8)
    assert B.quant_workspace_bytes(4) > 0 and B.quant_workspace_bytes(9) == 0
    p = ctypes.c_void_p(0x10000)
    assert lib.mv_pos_encode(None, p, 3, 10, 11, p) == B.MV_ERR_INVALID_ARG          # B > d
    assert lib.mv_pos_encode(None, None, 3, 10, 2, p) == B.MV_ERR_INVALID_ARG         # idx missing
    assert lib.mv_pos_decode(None, p, 12, 12, 4, p, 3, p, p, 0) == B.MV_ERR_WORKSPACE
    assert lib.mv_pos_decode(None, p, 12, 12, 4, p, 3, None, p, 1 << 20) == B.MV_ERR_INVALID_ARG
    assert lib.mv_quantize(None, p, 10, 9, p, None, p, 1 << 20) == B.MV_ERR_INVALID_ARG
    assert lib.mv_quantize(None, p, 10, 4, p, None, p, 8) == B.MV_ERR_WORKSPACE
    assert lib.mv_dequantize(None, None, 10, 4, p) == B.MV_ERR_INVALID_ARG
