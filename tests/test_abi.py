"""The C-ABI library loads, exports every symbol the header declares, and validates arguments on the
host before touching the GPU (no compute call is made here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "nova_attn.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2608_00029_b200 import build, nova_attn
    build.build()
    return nova_attn.load()


def _declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nova_attn_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_symbols()
    assert {"nova_attn_fwd", "nova_attn_bwd_preprocess", "nova_attn_bwd", "nova_attn_bwd_workspace_bytes",
            "nova_attn_status_string", "nova_attn_poll_device_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in nova_attn.h but not exported"


def test_loss_head_header_symbols_and_validation(lib):
    """include/nova_lmhead.h: every declared entry point is exported, and bad arguments are rejected on the host."""
    from paper_2608_00029_b200 import nova_attn as na, nova_lmhead as lm
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "nova_lmhead.h")).read(), flags=re.S)
    names = sorted(set(re.findall(r"\b(nova_lmhead_[a-z_0-9]+)\s*\(", text)))
    assert names == ["nova_lmhead_fwd", "nova_lmhead_workspace_bytes"]
    for n in names:
        assert hasattr(lib, n), f"{n} declared in nova_lmhead.h but not exported"
    assert lm.nova_lmhead_workspace_bytes(8192, 50304, 768) == 393 * 8192 * 8 + 8192 * 4
    assert lm.nova_lmhead_workspace_bytes(1, 8, 8) == 256
    assert lm.nova_lmhead_workspace_bytes(8, 12, 8) == 0 and lm.nova_lmhead_workspace_bytes(8, 16, 12) == 0
    p = ctypes.c_void_p(0x1000)
    f = lm._lib().nova_lmhead_fwd
    assert f(None, p, p, p, p, p, 8, 8, 8, p, 1 << 20, None) == na.ERR_NULL
    assert f(p, p, p, None, p, None, 8, 8, 8, p, 1 << 20, None) == na.ERR_NULL      # loss is required, logits are not
    assert f(p, p, p, p, p, p, 0, 8, 8, p, 1 << 20, None) == na.ERR_SHAPE
    assert f(p, p, p, p, p, p, 8, 12, 8, p, 1 << 20, None) == na.ERR_SHAPE           # N not a multiple of 8
    assert f(p, p, p, p, p, p, 8, 8, 4, p, 1 << 20, None) == na.ERR_SHAPE
    assert f(p, ctypes.c_void_p(0x1008), p, p, p, p, 8, 8, 8, p, 1 << 20, None) == na.ERR_ALIGNMENT
    assert f(p, p, p, p, p, p, 8, 8, 8, None, 0, None) == na.ERR_WORKSPACE
    assert f(p, p, p, p, p, p, 8, 8, 8, p, 16, None) == na.ERR_WORKSPACE


def test_status_strings(lib):
    from paper_2608_00029_b200 import nova_attn as na
    assert na.nova_attn_status_string(0) == "ok"
    seen = {na.nova_attn_status_string(c) for c in range(-8, 1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert na.nova_attn_status_string(-99) == "unknown status"


def test_workspace_query(lib):
    from paper_2608_00029_b200 import nova_attn as na
    assert na.nova_attn_bwd_workspace_bytes(8, 12, 1024, 64) == 8 * 12 * 1024 * 64 * 4
    assert na.nova_attn_bwd_workspace_bytes(2, 12, 8192, 128) == 2 * 12 * 8192 * 128 * 4
    assert na.nova_attn_bwd_workspace_bytes(1, 1, 1, 64) == 256
    assert na.nova_attn_bwd_workspace_bytes(1, 1, 1, 96) == 0      # unsupported head dim
    assert na.nova_attn_bwd_workspace_bytes(0, 1, 1, 64) == 0


def test_host_side_validation_rejects_before_launch(lib):
    from paper_2608_00029_b200 import nova_attn as na
    p = ctypes.c_void_p(0x1000)       # aligned, never dereferenced: every case fails validation first
    odd = ctypes.c_void_p(0x1008)
    f = lib.nova_attn_fwd
    assert f(None, p, p, p, p, 1, 1, 1, 64, 1.0, 1, None) == na.ERR_NULL
    assert f(p, p, p, p, p, 0, 1, 1, 64, 1.0, 1, None) == na.ERR_SHAPE
    assert f(p, p, p, p, p, 1, 1, -5, 64, 1.0, 1, None) == na.ERR_SHAPE
    assert f(p, p, p, p, p, 1, 1, 16, 96, 1.0, 1, None) == na.ERR_UNSUPPORTED
    assert f(p, odd, p, p, p, 1, 1, 16, 64, 1.0, 1, None) == na.ERR_ALIGNMENT
    assert f(p, p, p, p, p, 1, 1, 16, 64, 0.0, 1, None) == na.ERR_SCALE
    assert f(p, p, p, p, p, 1, 1, 16, 64, float("nan"), 1, None) == na.ERR_SCALE
    assert f(p, p, p, p, p, 1, 1, 16, 64, float("inf"), 1, None) == na.ERR_SCALE
    g = lib.nova_attn_bwd_preprocess
    assert g(p, None, p, 1, 1, 1, 64, None) == na.ERR_NULL
    assert g(p, p, p, 1, 1, 1, 32, None) == na.ERR_UNSUPPORTED
    b = lib.nova_attn_bwd
    args = [p] * 10
    assert b(*args, 1, 1, 16, 64, 1.0, 1, None, 0, None) == na.ERR_WORKSPACE
    assert b(*args, 1, 1, 16, 64, 1.0, 1, p, 16, None) == na.ERR_WORKSPACE      # too small
    assert b(*args, 1, 1, 16, 64, -1.0, 1, p, 1 << 20, None) == na.ERR_SCALE
    args[3] = None                                                              # O may be NULL: it is ignored
    assert b(*args, 1, 1, 16, 64, 1.0, 1, p, 16, None) == na.ERR_WORKSPACE
    e = lib.nova_attn_bwd_preprocess_exact
    assert e(p, p, p, p, None, p, 1, 1, 16, 64, 1.0, 1, None) == na.ERR_NULL
    assert e(p, p, p, p, p, p, 1, 1, 16, 64, -2.0, 1, None) == na.ERR_SCALE


def test_deterministic_backward_validates_without_a_workspace(lib):
    from paper_2608_00029_b200 import nova_attn as na
    p = ctypes.c_void_p(0x1000)
    odd = ctypes.c_void_p(0x1004)
    d = lib.nova_attn_bwd_deterministic
    ptrs = [p] * 9
    assert d(*ptrs, 0, 1, 16, 64, 1.0, 1, None) == na.ERR_SHAPE
    assert d(*ptrs, 1, 1, 16, 80, 1.0, 1, None) == na.ERR_UNSUPPORTED
    assert d(*ptrs, 1, 1, 16, 64, float("nan"), 1, None) == na.ERR_SCALE
    bad = list(ptrs)
    bad[6] = None                                        # dQ
    assert d(*bad, 1, 1, 16, 64, 1.0, 1, None) == na.ERR_NULL
    bad[6] = odd
    assert d(*bad, 1, 1, 16, 64, 1.0, 1, None) == na.ERR_ALIGNMENT


def test_static_scratch_backward_reports_argument_errors_before_the_size_limit(lib):
    """A NULL pointer, an unsupported head dimension or a bad scale is reported as such even when the
    problem would also be too large for the built-in array; only a valid, oversized problem gets the
    workspace error.  None of these calls reaches the GPU."""
    from paper_2608_00029_b200 import nova_attn as na
    p = ctypes.c_void_p(0x1000)
    s = lib.nova_attn_bwd_static_scratch
    ptrs = [p] * 10
    big = (3, 12, 4096)                                   # 9.4 Mi elements at D=64: more than the array holds
    assert s(*ptrs, *big, 64, 1.0, 1, None) == na.ERR_WORKSPACE
    assert s(*ptrs, *big, 96, 1.0, 1, None) == na.ERR_UNSUPPORTED
    assert s(*ptrs, *big, 64, -1.0, 1, None) == na.ERR_SCALE
    bad = list(ptrs)
    bad[7] = None                                         # dQ
    assert s(*bad, *big, 64, 1.0, 1, None) == na.ERR_NULL
    bad[7] = ctypes.c_void_p(0x1004)
    assert s(*bad, *big, 64, 1.0, 1, None) == na.ERR_ALIGNMENT
    bad = list(ptrs)
    bad[3] = None                                         # O is ignored, as in nova_attn_bwd
    assert s(*bad, *big, 64, 1.0, 1, None) == na.ERR_WORKSPACE


def test_strided_entry_points_validate_strides(lib):
    from paper_2608_00029_b200 import nova_attn as na
    p = ctypes.c_void_p(0x1000)
    S = na.Strides
    good = S(16 * 3 * 2 * 64, 64, 3 * 2 * 64)            # the Q slice of a fused [B, T, 3, H=2, D=64] buffer
    f = lib.nova_attn_fwd_strided
    base = (p, p, p, p, p, 1, 2, 16, 64)
    assert f(*base, None, good, good, good, 1.0, 1, None) == na.ERR_NULL
    assert f(*base, good, S(100, 64, 384), good, good, 1.0, 1, None) == na.ERR_ALIGNMENT   # 100 % 8 != 0
    assert f(*base, good, good, S(6144, 64, 32), good, 1.0, 1, None) == na.ERR_SHAPE        # token stride < D
    assert f(*base, good, good, good, S(6144, 0, 384), 1.0, 1, None) == na.ERR_SHAPE
    assert f(*base, good, good, good, S(1 << 40, 64, 384), 1.0, 1, None) == na.ERR_SHAPE
    assert f(*base, good, good, good, good, 0.0, 1, None) == na.ERR_SCALE
    g = lib.nova_attn_bwd_preprocess_strided
    assert g(p, p, p, 1, 2, 16, 64, good, None, None) == na.ERR_NULL
    assert g(p, p, p, 1, 2, 16, 64, good, S(6144, 64, 380), None) == na.ERR_ALIGNMENT
    b = lib.nova_attn_bwd_strided
    ptrs = [p] * 9
    seven = [good] * 7
    assert b(*ptrs, 1, 2, 16, 64, *seven, 1.0, 1, None, 0, None) == na.ERR_WORKSPACE
    seven[4] = S(6144, 64, 8)
    assert b(*ptrs, 1, 2, 16, 64, *seven, 1.0, 1, p, 1 << 20, None) == na.ERR_SHAPE


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2608_00029_b200 import nova_attn as na
    monkeypatch.setattr(na, "_lib", None)
    monkeypatch.setattr(na, "LIB_PATH", str(tmp_path / "libnova_attn.so"))
    with pytest.raises(ImportError):
        na.load()
