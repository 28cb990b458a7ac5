"""ctypes binding of the loss-head entry points of libnova_attn.so (include/nova_lmhead.h): same names as the
C ABI, argument marshalling only.  No CPU fallback: a missing library or a failed call raises."""
from __future__ import annotations

import ctypes

import torch

from . import nova_attn as _na

_ready = False


def _lib():
    global _ready
    lib = _na.load()
    if not _ready:
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        lib.nova_lmhead_workspace_bytes.argtypes = [i, i, i]
        lib.nova_lmhead_workspace_bytes.restype = sz
        lib.nova_lmhead_fwd.argtypes = [vp] * 6 + [i, i, i, vp, sz, vp]
        lib.nova_lmhead_fwd.restype = i
        _ready = True
    return lib


def nova_lmhead_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(_lib().nova_lmhead_workspace_bytes(M, N, K))


def nova_lmhead_fwd(X, W, targets, logits, lse, loss, workspace=None, stream=None) -> None:
    """lse, loss (and logits unless None) <- loss head of X [M,K] against W [N,K] with int32 targets [M].
    X, W, logits are contiguous CUDA bf16 tensors, lse and loss fp32 [M]; `workspace` is a CUDA byte tensor of
    at least nova_lmhead_workspace_bytes(M, N, K) bytes (allocated here if omitted)."""
    for name, t in (("X", X), ("W", W)):
        if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or t.dim() != 2:
            raise TypeError(f"{name} must be a contiguous 2-D CUDA bf16 tensor")
    M, K = X.shape
    N = W.shape[0]
    if W.shape[1] != K:
        raise ValueError("X [M,K] and W [N,K] must agree in K")
    if targets.dtype != torch.int32 or not targets.is_cuda or tuple(targets.shape) != (M,):
        raise TypeError("targets must be a CUDA int32 tensor [M]")
    if logits is not None and (logits.dtype != torch.bfloat16 or not logits.is_cuda or not logits.is_contiguous()
                               or tuple(logits.shape) != (M, N)):
        raise TypeError("logits must be a contiguous CUDA bf16 tensor [M,N] or None")
    for name, t in (("lse", lse), ("loss", loss)):
        if t.dtype != torch.float32 or not t.is_cuda or tuple(t.shape) != (M,):
            raise TypeError(f"{name} must be a CUDA fp32 tensor [M]")
    if workspace is None:
        workspace = torch.empty(nova_lmhead_workspace_bytes(M, N, K), dtype=torch.uint8, device=X.device)
    rc = _lib().nova_lmhead_fwd(_na._ptr(X), _na._ptr(W), _na._ptr(targets), _na._ptr(logits), _na._ptr(lse),
                                _na._ptr(loss), M, N, K, _na._ptr(workspace),
                                workspace.numel() * workspace.element_size(), _na._stream_ptr(stream))
    if rc != _na.OK:
        raise _na.NovaAttnError(rc, "nova_lmhead_fwd")
