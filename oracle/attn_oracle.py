"""ctypes front end of the C oracle (``attn_oracle.c``): numpy float64 in, numpy float64 out.

TEST INFRASTRUCTURE ONLY.  The arithmetic lives in ``attn_oracle.c`` (the definition of masked softmax
attention and its gradients, Section 4.2 of the paper restated as plain sums); this file only
marshals arrays.  Tensors are ``[B, H, T, D]`` C-contiguous float64; row vectors ``[B, H, T]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_attn.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP, no fast-math) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i, d = ctypes.c_int, ctypes.c_double
        lib.oracle_attn_fwd.argtypes = [_dp, _dp, _dp, _dp, _dp, i, i, i, i, d, i]
        lib.oracle_attn_fwd.restype = i
        lib.oracle_attn_bwd.argtypes = [_dp] * 8 + [i, i, i, i, d, i]
        lib.oracle_attn_bwd.restype = i
        lib.oracle_attn_probs.argtypes = [_dp, _dp, _dp, i, i, d, i]
        lib.oracle_attn_probs.restype = i
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = i
        _lib = lib
    return _lib


def _as4(x, name):
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    if a.ndim != 4:
        raise ValueError(f"{name} must be [B,H,T,D], got shape {a.shape}")
    return a


def _ptr(a):
    return a.ctypes.data_as(_dp)


def num_threads() -> int:
    """OpenMP threads the oracle will use (heads are spread over them)."""
    return int(_load().oracle_num_threads())


def attn_fwd(Q, K, V, scale: float, causal: bool = True):
    """O [B,H,T,D] and natural-log LSE [B,H,T] of softmax(scale*Q K^T, masked) V."""
    Q, K, V = _as4(Q, "Q"), _as4(K, "K"), _as4(V, "V")
    if not (Q.shape == K.shape == V.shape):
        raise ValueError("Q, K, V must have the same shape")
    B, H, T, D = Q.shape
    O = np.empty_like(Q)
    LSE = np.empty((B, H, T), dtype=np.float64)
    rc = _load().oracle_attn_fwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE), B, H, T, D,
                                 float(scale), int(bool(causal)))
    if rc != 0:
        raise RuntimeError(f"oracle_attn_fwd failed with {rc}")
    return O, LSE


def attn_bwd(Q, K, V, dO, scale: float, causal: bool = True):
    """(dQ, dK, dV, Delta): gradient of sum(O*dO) w.r.t. Q, K, V and the Jacobian row term Delta."""
    Q, K, V, dO = _as4(Q, "Q"), _as4(K, "K"), _as4(V, "V"), _as4(dO, "dO")
    if not (Q.shape == K.shape == V.shape == dO.shape):
        raise ValueError("Q, K, V, dO must have the same shape")
    B, H, T, D = Q.shape
    dQ, dK, dV = np.empty_like(Q), np.empty_like(Q), np.empty_like(Q)
    Delta = np.empty((B, H, T), dtype=np.float64)
    rc = _load().oracle_attn_bwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV),
                                 _ptr(Delta), B, H, T, D, float(scale), int(bool(causal)))
    if rc != 0:
        raise RuntimeError(f"oracle_attn_bwd failed with {rc}")
    return dQ, dK, dV, Delta


def attn_probs(q, k, scale: float, causal: bool = True):
    """Dense probability matrix [T,T] of ONE head (q, k are [T,D]); zeros where masked."""
    q = np.ascontiguousarray(np.asarray(q, dtype=np.float64))
    k = np.ascontiguousarray(np.asarray(k, dtype=np.float64))
    T, D = q.shape
    P = np.empty((T, T), dtype=np.float64)
    rc = _load().oracle_attn_probs(_ptr(q), _ptr(k), _ptr(P), T, D, float(scale), int(bool(causal)))
    if rc != 0:
        raise RuntimeError(f"oracle_attn_probs failed with {rc}")
    return P
