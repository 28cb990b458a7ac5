"""ctypes binding of libnova_attn.so: same names as the C ABI, argument marshalling only.

Every step of the attention path runs inside the CUDA library; PyTorch is used here for device
memory and streams.  There is no CPU fallback: if the shared library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnova_attn.so")
_lib = None

OK = 0
ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_SCALE, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(-1, -9, -1)


class Strides(ctypes.Structure):
    """nova_attn_strides: element strides of a tensor addressed (b, h, t, d), d contiguous."""
    _fields_ = [("batch", ctypes.c_longlong), ("head", ctypes.c_longlong), ("token", ctypes.c_longlong)]


class NovaAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib = load()
        msg = lib.nova_attn_status_string(status).decode()
        extra = f" (cuda error {lib.nova_attn_last_cuda_error()})" if status == ERR_CUDA else ""
        super().__init__(f"{where}: {msg}{extra} [status {status}]")


def load():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} not found: build it with `python -m paper_2608_00029_b200.build` "
            "(there is no CPU fallback for this library)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, fp, i, f, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.nova_attn_fwd.argtypes = [vp, vp, vp, vp, fp, i, i, i, i, f, i, vp]
    lib.nova_attn_fwd.restype = i
    lib.nova_attn_bwd_preprocess.argtypes = [vp, vp, fp, i, i, i, i, vp]
    lib.nova_attn_bwd_preprocess.restype = i
    lib.nova_attn_bwd_preprocess_exact.argtypes = [vp, vp, vp, vp, fp, fp, i, i, i, i, f, i, vp]
    lib.nova_attn_bwd_preprocess_exact.restype = i
    lib.nova_attn_bwd_workspace_bytes.argtypes = [i, i, i, i]
    lib.nova_attn_bwd_workspace_bytes.restype = sz
    lib.nova_attn_bwd.argtypes = [vp] * 5 + [fp, fp, vp, vp, vp, i, i, i, i, f, i, vp, sz, vp]
    lib.nova_attn_bwd.restype = i
    lib.nova_attn_bwd_steps.argtypes = [vp] * 5 + [fp, fp, vp, vp, vp, i, i, i, i, f, i, vp, sz, vp, i]
    lib.nova_attn_bwd_steps.restype = i
    sp = ctypes.POINTER(Strides)
    lib.nova_attn_fwd_strided.argtypes = [vp, vp, vp, vp, fp, i, i, i, i, sp, sp, sp, sp, f, i, vp]
    lib.nova_attn_fwd_strided.restype = i
    lib.nova_attn_bwd_preprocess_strided.argtypes = [vp, vp, fp, i, i, i, i, sp, sp, vp]
    lib.nova_attn_bwd_preprocess_strided.restype = i
    lib.nova_attn_bwd_strided.argtypes = [vp] * 4 + [fp, fp, vp, vp, vp, i, i, i, i] + [sp] * 7 + [f, i, vp, sz, vp]
    lib.nova_attn_bwd_strided.restype = i
    lib.nova_attn_bwd_deterministic.argtypes = [vp] * 4 + [fp, fp, vp, vp, vp, i, i, i, i, f, i, vp]
    lib.nova_attn_bwd_deterministic.restype = i
    lib.nova_attn_status_string.argtypes = [i]
    lib.nova_attn_status_string.restype = ctypes.c_char_p
    lib.nova_attn_last_cuda_error.argtypes = []
    lib.nova_attn_last_cuda_error.restype = i
    lib.nova_attn_poll_device_status.argtypes = [vp]
    lib.nova_attn_poll_device_status.restype = i
    lib.nova_attn_bwd_static_scratch.argtypes = [vp] * 5 + [fp, fp, vp, vp, vp, i, i, i, i, f, i, vp]
    lib.nova_attn_bwd_static_scratch.restype = i
    lib.nova_attn_static_scratch_bytes.argtypes = []
    lib.nova_attn_static_scratch_bytes.restype = sz
    lib.nova_attn_test_configure_waits.argtypes = [ctypes.c_longlong, i]
    lib.nova_attn_test_configure_waits.restype = i
    lib.nova_attn_bwd_work_list.argtypes = [i, ctypes.c_longlong, i, i, i, i, ctypes.c_void_p, i, ctypes.c_void_p]
    lib.nova_attn_bwd_work_list.restype = i
    _lib = lib
    return lib


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _check_bf16(name, t, shape=None):
    if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA bf16 tensor")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")


def _view_strides(name, t, shape=None) -> Strides:
    """Strides of a [B,H,T,D]-shaped bf16 CUDA view whose last dimension is contiguous (the view may be a
    slice / permutation of a larger buffer, e.g. of a fused projection output)."""
    if t.dtype != torch.bfloat16 or not t.is_cuda or t.dim() != 4 or t.stride(3) != 1:
        raise TypeError(f"{name} must be a 4-D CUDA bf16 view [B,H,T,D] with a contiguous last dimension")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")
    return Strides(t.stride(0), t.stride(1), t.stride(2))


def _check_f32(name, t, shape):
    if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise TypeError(f"{name} must be a contiguous CUDA fp32 tensor of shape {tuple(shape)}")


def nova_attn_status_string(status: int) -> str:
    return load().nova_attn_status_string(int(status)).decode()


def nova_attn_bwd_workspace_bytes(B: int, H: int, T: int, D: int) -> int:
    return int(load().nova_attn_bwd_workspace_bytes(B, H, T, D))


def nova_attn_fwd(Q, K, V, O, LSE, scale: float, causal: bool = True, stream=None) -> None:
    """O, LSE <- attention(Q, K, V); tensors are [B,H,T,D] bf16, LSE [B,H,T] fp32, all preallocated."""
    _check_bf16("Q", Q)
    B, H, T, D = Q.shape
    for n, t in (("K", K), ("V", V), ("O", O)):
        _check_bf16(n, t, Q.shape)
    _check_f32("LSE", LSE, (B, H, T))
    rc = load().nova_attn_fwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), B, H, T, D, float(scale),
                              int(bool(causal)), _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_fwd")


def nova_attn_bwd_preprocess(O, dO, Delta, stream=None) -> None:
    """Delta <- rowsum(dO * O)."""
    _check_bf16("O", O)
    _check_bf16("dO", dO, O.shape)
    B, H, T, D = O.shape
    _check_f32("Delta", Delta, (B, H, T))
    rc = load().nova_attn_bwd_preprocess(_ptr(O), _ptr(dO), _ptr(Delta), B, H, T, D, _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_bwd_preprocess")


def nova_attn_bwd_preprocess_exact(Q, K, V, dO, LSE, Delta, scale: float, causal: bool = True, stream=None) -> None:
    """Delta <- sum_j P_ij (dO_i . V_j) with P rebuilt from LSE: independent of the rounding of O."""
    _check_bf16("Q", Q)
    B, H, T, D = Q.shape
    for n, t in (("K", K), ("V", V), ("dO", dO)):
        _check_bf16(n, t, Q.shape)
    _check_f32("LSE", LSE, (B, H, T))
    _check_f32("Delta", Delta, (B, H, T))
    rc = load().nova_attn_bwd_preprocess_exact(_ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(LSE), _ptr(Delta), B, H, T,
                                               D, float(scale), int(bool(causal)), _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_bwd_preprocess_exact")


BWD_STEP_ZERO, BWD_STEP_MAIN, BWD_STEP_CONVERT = 1, 2, 4
BWD_STEP_ALL = 7


def nova_attn_bwd(Q, K, V, O, dO, LSE, Delta, dQ, dK, dV, scale: float, causal: bool = True, workspace=None,
                  stream=None, steps: int = BWD_STEP_ALL) -> None:
    """dQ, dK, dV <- gradients of sum(O*dO); `workspace` is a CUDA byte/float tensor of at least
    nova_attn_bwd_workspace_bytes(B,H,T,D) bytes (allocated here if omitted).  `steps` other than
    BWD_STEP_ALL goes through nova_attn_bwd_steps (a timing aid)."""
    _check_bf16("Q", Q)
    B, H, T, D = Q.shape
    for n, t in (("K", K), ("V", V), ("O", O), ("dO", dO), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        _check_bf16(n, t, Q.shape)
    _check_f32("LSE", LSE, (B, H, T))
    _check_f32("Delta", Delta, (B, H, T))
    if workspace is None:
        workspace = torch.empty(nova_attn_bwd_workspace_bytes(B, H, T, D), dtype=torch.uint8, device=Q.device)
    ws_bytes = workspace.numel() * workspace.element_size()
    args = (_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(LSE), _ptr(Delta), _ptr(dQ), _ptr(dK), _ptr(dV),
            B, H, T, D, float(scale), int(bool(causal)), _ptr(workspace), ws_bytes, _stream_ptr(stream))
    if steps == BWD_STEP_ALL:
        rc = load().nova_attn_bwd(*args)
    else:
        rc = load().nova_attn_bwd_steps(*args, int(steps))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_bwd")


def nova_attn_static_scratch_bytes() -> int:
    """Size of the library's built-in dQ accumulator (bytes)."""
    return int(load().nova_attn_static_scratch_bytes())


def nova_attn_bwd_static_scratch(Q, K, V, O, dO, LSE, Delta, dQ, dK, dV, scale: float, causal: bool = True,
                                 stream=None) -> None:
    """nova_attn_bwd for callers that cannot allocate: no workspace argument, nothing is allocated here
    or in the library.  The dQ accumulator is a fixed 32 MiB array inside the library, shared by all
    calls on the device, so B*H*T*D must not exceed 8 Mi elements and calls must not overlap on the
    GPU.  Make the first call on a device before any stream capture."""
    _check_bf16("Q", Q)
    B, H, T, D = Q.shape
    for n, t in (("K", K), ("V", V), ("O", O), ("dO", dO), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        _check_bf16(n, t, Q.shape)
    _check_f32("LSE", LSE, (B, H, T))
    _check_f32("Delta", Delta, (B, H, T))
    rc = load().nova_attn_bwd_static_scratch(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(LSE), _ptr(Delta),
                                             _ptr(dQ), _ptr(dK), _ptr(dV), B, H, T, D, float(scale),
                                             int(bool(causal)), _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_bwd_static_scratch")


def nova_attn_test_configure_waits(limit_cycles: int = 0, inject: int = 0) -> None:
    """Test aid: cycle limit of the device-side waits of kernels launched from now on (0 = default) and,
    with inject=1, a forward whose loader leaves out one K-tile request so that a wait runs out."""
    rc = load().nova_attn_test_configure_waits(int(limit_cycles), int(inject))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_test_configure_waits")


def nova_attn_bwd_work_list(BH: int, T: int, D: int, causal: bool, n_ctas: int, cta: int):
    """Host-side view of the backward kernel's work distribution: ([(key tile, head), ...] of CTA `cta` in
    processing order, (heads per chunk, chunks, passes per full chunk, passes of the last chunk)).  No GPU."""
    lib = load()
    plan = (ctypes.c_int * 4)()
    n = lib.nova_attn_bwd_work_list(int(BH), int(T), int(D), int(bool(causal)), int(n_ctas), int(cta), None, 0, plan)
    if n < 0:
        raise NovaAttnError(n, "nova_attn_bwd_work_list")
    buf = (ctypes.c_int * (2 * max(n, 1)))()
    m = lib.nova_attn_bwd_work_list(int(BH), int(T), int(D), int(bool(causal)), int(n_ctas), int(cta), buf, n, plan)
    if m != n:
        raise NovaAttnError(ERR_SHAPE if m >= 0 else m, "nova_attn_bwd_work_list")
    return [(buf[2 * k], buf[2 * k + 1]) for k in range(n)], tuple(plan)


def nova_attn_poll_device_status(stream=None) -> int:
    """Synchronises the stream and returns the device status (0 = ok); raises on a recorded timeout."""
    rc = load().nova_attn_poll_device_status(_stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_poll_device_status")
    return rc


def nova_attn_fwd_strided(Q, K, V, O, LSE, scale: float, causal: bool = True, stream=None) -> None:
    """nova_attn_fwd on [B,H,T,D]-shaped VIEWS: strides are taken from the tensors, so Q, K, V may be slices
    of a fused projection output and O a permuted view of a [B,T,H,D] buffer.  LSE is contiguous [B,H,T]."""
    sq = _view_strides("Q", Q)
    B, H, T, D = Q.shape
    sk, sv, so = (_view_strides(n, t, Q.shape) for n, t in (("K", K), ("V", V), ("O", O)))
    _check_f32("LSE", LSE, (B, H, T))
    rc = load().nova_attn_fwd_strided(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), B, H, T, D, sq, sk, sv, so,
                                      float(scale), int(bool(causal)), _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_fwd_strided")


def nova_attn_bwd_preprocess_strided(O, dO, Delta, stream=None) -> None:
    """nova_attn_bwd_preprocess on [B,H,T,D]-shaped views."""
    so = _view_strides("O", O)
    sdo = _view_strides("dO", dO, O.shape)
    B, H, T, D = O.shape
    _check_f32("Delta", Delta, (B, H, T))
    rc = load().nova_attn_bwd_preprocess_strided(_ptr(O), _ptr(dO), _ptr(Delta), B, H, T, D, so, sdo,
                                                 _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_bwd_preprocess_strided")


def nova_attn_bwd_strided(Q, K, V, dO, LSE, Delta, dQ, dK, dV, scale: float, causal: bool = True, workspace=None,
                          stream=None) -> None:
    """nova_attn_bwd on [B,H,T,D]-shaped views (dQ, dK, dV may be slices of one fused gradient buffer)."""
    sq = _view_strides("Q", Q)
    B, H, T, D = Q.shape
    rest = [_view_strides(n, t, Q.shape) for n, t in (("K", K), ("V", V), ("dO", dO), ("dQ", dQ), ("dK", dK), ("dV", dV))]
    _check_f32("LSE", LSE, (B, H, T))
    _check_f32("Delta", Delta, (B, H, T))
    need = nova_attn_bwd_workspace_bytes(B, H, T, D)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=Q.device)
    rc = load().nova_attn_bwd_strided(_ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(LSE), _ptr(Delta), _ptr(dQ), _ptr(dK),
                                      _ptr(dV), B, H, T, D, sq, *rest, float(scale), int(bool(causal)),
                                      _ptr(workspace), workspace.numel() * workspace.element_size(),
                                      _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_bwd_strided")


def nova_attn_bwd_deterministic(Q, K, V, dO, LSE, Delta, dQ, dK, dV, scale: float, causal: bool = True,
                                stream=None) -> None:
    """dQ, dK, dV by the two-kernel backward: bitwise reproducible, no workspace, slower than nova_attn_bwd."""
    _check_bf16("Q", Q)
    B, H, T, D = Q.shape
    for n, t in (("K", K), ("V", V), ("dO", dO), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        _check_bf16(n, t, Q.shape)
    _check_f32("LSE", LSE, (B, H, T))
    _check_f32("Delta", Delta, (B, H, T))
    rc = load().nova_attn_bwd_deterministic(_ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(LSE), _ptr(Delta), _ptr(dQ),
                                            _ptr(dK), _ptr(dV), B, H, T, D, float(scale), int(bool(causal)),
                                            _stream_ptr(stream))
    if rc != OK:
        raise NovaAttnError(rc, "nova_attn_bwd_deterministic")
