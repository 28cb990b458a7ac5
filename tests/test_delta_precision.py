"""Arithmetic behind the two Delta routes, on CPU only.

Delta_i = rowsum(dO_i * O_i) uses the bf16 O the forward stored.  With sharply peaked softmax rows
(the large-batch configuration: Q, K ~ 2 N(0,1)) the rounding of O alone, with every other step in
float64, already moves some dQ/dK elements past 2e-2 + 2e-2|ref|; with the exact Delta the same
emulation stays inside.  This is why the library also exports nova_attn_bwd_preprocess_exact and why
the GPU test of that configuration uses it.
"""
import numpy as np
import torch

import oracle
from paper_2608_00029_b200 import workloads as W


def _bf16(x):
    return torch.tensor(x).to(torch.bfloat16).double().numpy()


def test_rowsum_delta_from_bf16_O_exceeds_bound_on_peaked_rows():
    cfg = W.CONFIGS["gpt2_small_large_batch"].replace(B=1, H=4)
    Q, K, V, dO = (W.widen(x) for x in W.make_inputs(cfg))
    scale = cfg.scale
    O, LSE = oracle.attn_fwd(Q, K, V, scale, True)
    dQ, dK, dV, Delta = oracle.attn_bwd(Q, K, V, dO, scale, True)
    mask = np.tril(np.ones((cfg.T, cfg.T), bool))
    P = np.where(mask, np.exp(scale * np.einsum("bhid,bhjd->bhij", Q, K) - LSE[..., None]), 0.0)
    dP = np.einsum("bhid,bhjd->bhij", dO, V)

    def grads(delta):
        dS = P * (dP - delta[..., None])
        return (scale * np.einsum("bhij,bhjd->bhid", dS, K), scale * np.einsum("bhij,bhid->bhjd", dS, Q))

    def worst(got, ref):
        return float((np.abs(got - ref) - (2e-2 + 2e-2 * np.abs(ref))).max())

    # float64 everywhere except the rounding of O to bf16 inside Delta
    delta_rowsum = (dO * _bf16(O)).sum(-1)
    dq_r, dk_r = grads(delta_rowsum)
    assert worst(dq_r, dQ) > 0 or worst(dk_r, dK) > 0
    # identical emulation with the exact Delta: indistinguishable from the oracle
    dq_e, dk_e = grads(Delta)
    assert worst(dq_e, dQ) < -1.9e-2 and worst(dk_e, dK) < -1.9e-2
    # the size of the Delta error matches the bf16 half-ulp model 2^-9 * sum|dO O| (loose factor 1)
    assert np.abs(delta_rowsum - Delta).max() <= 2.0 ** -9 * (np.abs(dO) * np.abs(O)).sum(-1).max()
