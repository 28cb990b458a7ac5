"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding, run the oracle
on the same seeded inputs (optionally on a sample of heads), compare element by element."""
import numpy as np
import torch

import oracle
from paper_2608_00029_b200 import nova_attn, workloads as W

import tolerance as tol

GUARD = 64  # guard-band elements around every output buffer


def _guarded(shape, dtype, dev, fill):
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), fill, dtype=dtype, device=dev)
    return buf, buf[GUARD:GUARD + n].view(shape)


def run_gpu(Q, K, V, dO, scale, causal=True, O_in=None, LSE_in=None, check_guards=True, exact_delta=False):
    """Forward + preprocess + backward on cuda:0.  Returns CPU tensors.  If O_in/LSE_in are given the
    backward consumes them instead of the forward's own results.  `exact_delta` selects
    nova_attn_bwd_preprocess_exact (Delta from P and dO V^T) instead of rowsum(dO * O)."""
    dev = torch.device("cuda:0")
    q, k, v, do = (x.to(dev).contiguous() for x in (Q, K, V, dO))
    B, H, T, D = q.shape
    bufs = {}
    views = {}
    for name in ("O", "dQ", "dK", "dV"):
        bufs[name], views[name] = _guarded((B, H, T, D), torch.bfloat16, dev, 7.0)
    for name in ("LSE", "Delta"):
        bufs[name], views[name] = _guarded((B, H, T), torch.float32, dev, 7.0)
    nova_attn.nova_attn_fwd(q, k, v, views["O"], views["LSE"], scale, causal)
    o_b = views["O"] if O_in is None else O_in.to(dev)
    lse_b = views["LSE"] if LSE_in is None else LSE_in.to(dev)
    if exact_delta:
        nova_attn.nova_attn_bwd_preprocess_exact(q, k, v, do, lse_b, views["Delta"], scale, causal)
    else:
        nova_attn.nova_attn_bwd_preprocess(o_b, do, views["Delta"])
    nova_attn.nova_attn_bwd(q, k, v, o_b, do, lse_b, views["Delta"], views["dQ"], views["dK"], views["dV"],
                            scale, causal)
    nova_attn.nova_attn_poll_device_status()
    if check_guards:
        for name, buf in bufs.items():
            g = torch.cat([buf[:GUARD], buf[-GUARD:]]).float().cpu()
            assert (g == 7.0).all(), f"{name}: write outside the output buffer"
    return {n: t.cpu() for n, t in views.items()}


def run_oracle(Q, K, V, dO, scale, causal=True, heads=None):
    """Oracle on all heads, or on a list of (b, h) pairs; returns float64 arrays [n,1,T,D]/[n,1,T]."""
    if heads is not None:
        sel = lambda x: torch.stack([x[b, h] for b, h in heads]).unsqueeze(1)
        Q, K, V, dO = (sel(x) for x in (Q, K, V, dO))
    Qd, Kd, Vd, dOd = (W.widen(x) for x in (Q, K, V, dO))
    O, LSE = oracle.attn_fwd(Qd, Kd, Vd, scale, causal)
    dQ, dK, dV, Delta = oracle.attn_bwd(Qd, Kd, Vd, dOd, scale, causal)
    return {"O": O, "LSE": LSE, "dQ": dQ, "dK": dK, "dV": dV, "Delta": Delta, "dO_in": dOd}


def select_heads(got, heads):
    if heads is None:
        return {n: W.widen(t) for n, t in got.items()}
    return {n: W.widen(torch.stack([t[b, h] for b, h in heads]).unsqueeze(1)) for n, t in got.items()}


def compare(got, ref, label="", rms=True, dO=None, bwd_factor=1.0):
    """Element-wise bounds: O, LSE 1e-2 + 1e-2|ref|; dQ, dK, dV 2e-2 + 2e-2|ref|; plus relative RMS
    bounds.  Delta is a D-term dot product of dO with the bf16 O the forward wrote, so its bound is the
    forward bound pushed through that sum: 1e-2 + 1e-2 * sum_d |dO_d| |O_d|  (needs dO [.., T, D] as
    float64; without it Delta is only checked by relative RMS).  Returns the max abs errors."""
    out = {}
    for name in ("O", "LSE"):
        out[name] = tol.assert_close(got[name], ref[name], tol.FWD_ATOL, tol.FWD_RTOL, f"{label}{name}",
                                     tol.FWD_REL_RMS if rms else None)
    derr = np.abs(np.asarray(got["Delta"], dtype=np.float64) - ref["Delta"])
    assert np.isfinite(got["Delta"]).all()
    if dO is not None:
        bound = tol.FWD_ATOL + tol.FWD_RTOL * (np.abs(dO) * np.abs(ref["O"])).sum(-1)
        assert (derr <= bound).all(), f"{label}Delta: max|err|={derr.max():.3e} exceeds the propagated forward bound"
    assert tol.rel_rms(got["Delta"], ref["Delta"]) <= tol.FWD_REL_RMS, f"{label}Delta relative RMS"
    out["Delta"] = float(derr.max())
    for name in ("dQ", "dK", "dV"):
        out[name] = tol.assert_close(got[name], ref[name], bwd_factor * tol.BWD_ATOL, bwd_factor * tol.BWD_RTOL,
                                     f"{label}{name}",
                                     tol.BWD_REL_RMS if rms else None)
    return out
