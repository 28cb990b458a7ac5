"""ctypes front end of the C oracle of the language-model loss head (``lmhead_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The arithmetic lives in ``lmhead_oracle.c`` (logits = X W^T, log-sum-exp over the
vocabulary, cross-entropy against integer targets: Section 4.1 of the paper, the loss-head case study,
restated as plain sums); this file only marshals arrays.  X is ``[M, K]``, W ``[N, K]``, targets ``[M]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lmhead_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_lmhead.so")
_lib = None
_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP, no fast-math) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_lmhead_fwd.argtypes = [_dp, _dp, _ip, _dp, _dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        lib.oracle_lmhead_fwd.restype = ctypes.c_int
        _lib = lib
    return _lib


def lmhead_fwd(X, W, targets, want_logits: bool = False):
    """(lse [M], loss [M]) or (logits [M,N], lse, loss): natural-log LSE of X W^T over the vocabulary and the
    cross-entropy of each row against its target (0 for targets outside [0, N))."""
    X = np.ascontiguousarray(np.asarray(X, dtype=np.float64))
    W = np.ascontiguousarray(np.asarray(W, dtype=np.float64))
    t = np.ascontiguousarray(np.asarray(targets, dtype=np.int32))
    if X.ndim != 2 or W.ndim != 2 or X.shape[1] != W.shape[1] or t.shape != (X.shape[0],):
        raise ValueError("X must be [M,K], W [N,K], targets [M]")
    M, K = X.shape
    N = W.shape[0]
    logits = np.empty((M, N), dtype=np.float64) if want_logits else None
    lse = np.empty(M, dtype=np.float64)
    loss = np.empty(M, dtype=np.float64)
    rc = _load().oracle_lmhead_fwd(X.ctypes.data_as(_dp), W.ctypes.data_as(_dp), t.ctypes.data_as(_ip),
                                   logits.ctypes.data_as(_dp) if want_logits else None, lse.ctypes.data_as(_dp),
                                   loss.ctypes.data_as(_dp), M, N, K)
    if rc != 0:
        raise RuntimeError(f"oracle_lmhead_fwd failed with {rc}")
    return (logits, lse, loss) if want_logits else (lse, loss)
