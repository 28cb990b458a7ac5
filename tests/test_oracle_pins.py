"""Pins for the fp64 CPU oracle: each test fixes it to something other than itself.

The paper prints no worked numeric example for attention, so the pins are analytic: a hand-worked
two-key case (tests/golden), closed forms, finite differences of the scalar L = sum(O*dO), a library
routine used as a black box (torch CPU float64 SDPA + autograd), brute force in pure Python loops, and
invariants (row sums, causality, shift invariance, zero-sum of dK).
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def rand(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


# ---------------------------------------------------------------------------------------------
# hand-worked example (tests/golden/two_key_worked_example.txt)
def _read_golden(path):
    vals = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, *nums = line.split()
            vals[name] = np.array([float(x) for x in nums]).reshape(1, 1, len(nums), 1)
    return vals


def test_hand_worked_two_key_example():
    g = _read_golden(os.path.join(HERE, "golden", "two_key_worked_example.txt"))
    O, LSE = oracle.attn_fwd(g["Q"], g["K"], g["V"], 1.0, causal=True)
    dQ, dK, dV, Delta = oracle.attn_bwd(g["Q"], g["K"], g["V"], g["dO"], 1.0, causal=True)
    np.testing.assert_allclose(O, g["O"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(LSE, g["LSE"][..., 0], rtol=0, atol=1e-14)
    np.testing.assert_allclose(Delta, g["Delta"][..., 0], rtol=0, atol=1e-13)
    np.testing.assert_allclose(dQ, g["dQ"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(dK, g["dK"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(dV, g["dV"], rtol=0, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# brute force: pure-Python loops over the definition, dense T x T, tiny sizes
def _brute(Q, K, V, dO, scale, causal):
    B, H, T, D = Q.shape
    O = np.zeros_like(Q); LSE = np.zeros((B, H, T))
    dQ = np.zeros_like(Q); dK = np.zeros_like(Q); dV = np.zeros_like(Q); Delta = np.zeros((B, H, T))
    for b in range(B):
        for h in range(H):
            P = [[0.0] * T for _ in range(T)]
            for i in range(T):
                keys = range(i + 1) if causal else range(T)
                s = {j: scale * sum(Q[b, h, i, d] * K[b, h, j, d] for d in range(D)) for j in keys}
                z = sum(math.exp(v) for v in s.values())          # no max subtraction: tiny inputs
                LSE[b, h, i] = math.log(z)
                for j in keys:
                    P[i][j] = math.exp(s[j]) / z
                for d in range(D):
                    O[b, h, i, d] = sum(P[i][j] * V[b, h, j, d] for j in keys)
            for i in range(T):
                dP = [sum(dO[b, h, i, d] * V[b, h, j, d] for d in range(D)) for j in range(T)]
                Delta[b, h, i] = sum(P[i][j] * dP[j] for j in range(T))
                for j in range(T):
                    dS = P[i][j] * (dP[j] - Delta[b, h, i])
                    for d in range(D):
                        dV[b, h, j, d] += P[i][j] * dO[b, h, i, d]
                        dQ[b, h, i, d] += scale * dS * K[b, h, j, d]
                        dK[b, h, j, d] += scale * dS * Q[b, h, i, d]
    return O, LSE, dQ, dK, dV, Delta


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("shape", [(1, 1, 5, 3), (2, 2, 7, 4), (1, 1, 16, 8)])
def test_brute_force_dense(shape, causal):
    Q, K, V, dO = (rand(shape, s) for s in (1, 2, 3, 4))
    scale = 0.37
    ref = _brute(Q, K, V, dO, scale, causal)
    O, LSE = oracle.attn_fwd(Q, K, V, scale, causal)
    dQ, dK, dV, Delta = oracle.attn_bwd(Q, K, V, dO, scale, causal)
    for got, want in zip((O, LSE, dQ, dK, dV, Delta), ref):
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# finite differences of L(Q,K,V) = sum(O * dO)
@pytest.mark.parametrize("causal", [True, False])
def test_gradients_match_central_differences(causal):
    shape = (1, 2, 6, 4)
    Q, K, V, dO = (rand(shape, s) for s in (10, 11, 12, 13))
    scale = 0.5
    dQ, dK, dV, _ = oracle.attn_bwd(Q, K, V, dO, scale, causal)

    def loss(q, k, v):
        O, _ = oracle.attn_fwd(q, k, v, scale, causal)
        return float((O * dO).sum())

    h = 1e-6
    for which, grad in (("Q", dQ), ("K", dK), ("V", dV)):
        num = np.zeros(shape)
        for idx in np.ndindex(*shape):
            args = {"Q": Q.copy(), "K": K.copy(), "V": V.copy()}
            args[which][idx] += h
            lp = loss(args["Q"], args["K"], args["V"])
            args[which][idx] -= 2 * h
            lm = loss(args["Q"], args["K"], args["V"])
            num[idx] = (lp - lm) / (2 * h)
        np.testing.assert_allclose(grad, num, rtol=2e-7, atol=2e-8, err_msg=f"d{which}")


# ---------------------------------------------------------------------------------------------
# library routine as a black box
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("shape,scale", [((2, 3, 33, 16), 0.25), ((1, 2, 64, 64), 0.125)])
def test_against_torch_sdpa_float64(shape, scale, causal):
    Q, K, V, dO = (rand(shape, s) for s in (20, 21, 22, 23))
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    to = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal, scale=scale)
    gq, gk, gv = torch.autograd.grad(to, (tq, tk, tv), grad_outputs=torch.tensor(dO))
    s = scale * torch.einsum("bhid,bhjd->bhij", tq, tk).detach()
    if causal:
        T = shape[2]
        s = s.masked_fill(torch.triu(torch.ones(T, T, dtype=torch.bool), 1), float("-inf"))
    lse = torch.logsumexp(s, dim=-1)
    O, LSE = oracle.attn_fwd(Q, K, V, scale, causal)
    dQ, dK, dV, _ = oracle.attn_bwd(Q, K, V, dO, scale, causal)
    np.testing.assert_allclose(O, to.detach().numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(LSE, lse.numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dQ, gq.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dK, gk.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dV, gv.numpy(), rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# closed forms
def test_single_token_sequence():
    shape = (2, 3, 1, 8)
    Q, K, V, dO = (rand(shape, s) for s in (30, 31, 32, 33))
    scale = 0.3
    O, LSE = oracle.attn_fwd(Q, K, V, scale, True)
    dQ, dK, dV, Delta = oracle.attn_bwd(Q, K, V, dO, scale, True)
    np.testing.assert_array_equal(O, V)
    np.testing.assert_allclose(LSE, scale * (Q * K).sum(-1), rtol=1e-14, atol=1e-15)
    np.testing.assert_array_equal(dV, dO)
    np.testing.assert_allclose(dQ, 0, atol=1e-15)
    np.testing.assert_allclose(dK, 0, atol=1e-15)
    np.testing.assert_allclose(Delta, (dO * V).sum(-1), rtol=1e-14)


def test_zero_queries_give_uniform_prefix_attention():
    """Q = 0 -> P_ij = 1/(i+1): O is the prefix mean of V and LSE_i = ln(i+1).  Pins the natural-log
    base of LSE and that the diagonal key is kept."""
    B, H, T, D = 1, 2, 9, 5
    K, V, dO = (rand((B, H, T, D), s) for s in (41, 42, 43))
    Q = np.zeros((B, H, T, D))
    scale = 0.7
    O, LSE = oracle.attn_fwd(Q, K, V, scale, True)
    n = np.arange(1, T + 1, dtype=np.float64)
    np.testing.assert_allclose(O, np.cumsum(V, axis=2) / n[None, None, :, None], rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(LSE, np.broadcast_to(np.log(n), (B, H, T)), rtol=1e-14, atol=1e-15)
    dQ, dK, dV, Delta = oracle.attn_bwd(Q, K, V, dO, scale, True)
    w = dO / n[None, None, :, None]
    dV_ref = np.flip(np.cumsum(np.flip(w, 2), axis=2), 2)            # sum_{i>=j} dO_i/(i+1)
    np.testing.assert_allclose(dV, dV_ref, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(dK, 0, atol=1e-15)                    # dK_j = scale * sum_i dS_ij * Q_i
    dQ_ref = np.zeros_like(Q)
    for i in range(T):
        dp = np.einsum("bhd,bhjd->bhj", dO[:, :, i], V[:, :, : i + 1])
        dlt = np.einsum("bhd,bhd->bh", dO[:, :, i], O[:, :, i])
        dQ_ref[:, :, i] = scale / (i + 1) * np.einsum("bhj,bhjd->bhd", dp - dlt[..., None], K[:, :, : i + 1])
    np.testing.assert_allclose(dQ, dQ_ref, rtol=1e-12, atol=1e-13)


def test_noncausal_zero_queries_is_global_mean():
    B, H, T, D = 1, 1, 6, 3
    K, V = rand((B, H, T, D), 51), rand((B, H, T, D), 52)
    O, LSE = oracle.attn_fwd(np.zeros((B, H, T, D)), K, V, 1.0, False)
    np.testing.assert_allclose(O, np.broadcast_to(V.mean(2, keepdims=True), V.shape), rtol=1e-13)
    np.testing.assert_allclose(LSE, math.log(T), rtol=1e-14)


# ---------------------------------------------------------------------------------------------
# invariants
@pytest.mark.parametrize("causal", [True, False])
def test_probability_rows(causal):
    T, D = 37, 8
    q, k = rand((T, D), 60), rand((T, D), 61)
    P = oracle.attn_probs(q, k, 0.4, causal)
    np.testing.assert_allclose(P.sum(1), 1.0, rtol=0, atol=1e-13)
    assert (P >= 0).all() and (P <= 1).all()
    if causal:
        assert (np.triu(P, 1) == 0).all()
        assert (np.diag(P) > 0).all()
    # P V reproduces O, and log-sum-exp reproduces the normaliser
    v = rand((T, D), 62)
    O, LSE = oracle.attn_fwd(q[None, None], k[None, None], v[None, None], 0.4, causal)
    np.testing.assert_allclose(P @ v, O[0, 0], rtol=1e-12, atol=1e-13)
    s = 0.4 * q @ k.T
    for i in (0, 5, T - 1):
        n = i + 1 if causal else T
        np.testing.assert_allclose(np.exp(s[i, :n] - LSE[0, 0, i]), P[i, :n], rtol=1e-12)


def test_jacobian_identities():
    shape = (2, 2, 40, 16)
    Q, K, V, dO = (rand(shape, s) for s in (70, 71, 72, 73))
    O, _ = oracle.attn_fwd(Q, K, V, 0.25, True)
    dQ, dK, dV, Delta = oracle.attn_bwd(Q, K, V, dO, 0.25, True)
    # sum_j dS_ij = 0 per row  =>  sum_j dK_j = 0 per head
    np.testing.assert_allclose(dK.sum(2), 0, atol=1e-12)
    # Delta_i = sum_j P_ij dP_ij = dO_i . O_i
    np.testing.assert_allclose(Delta, (dO * O).sum(-1), rtol=1e-11, atol=1e-13)
    # sum_j dV_j = sum_i dO_i (rows of P sum to one)
    np.testing.assert_allclose(dV.sum(2), dO.sum(2), rtol=1e-11, atol=1e-12)


def test_causality_under_perturbation():
    shape = (1, 2, 24, 8)
    Q, K, V, dO = (rand(shape, s) for s in (80, 81, 82, 83))
    t = 11
    O, LSE = oracle.attn_fwd(Q, K, V, 0.3, True)
    dQ, dK, dV, _ = oracle.attn_bwd(Q, K, V, dO, 0.3, True)
    K2, V2 = K.copy(), V.copy()
    K2[:, :, t + 1:] += rand(K2[:, :, t + 1:].shape, 84)
    V2[:, :, t + 1:] -= rand(V2[:, :, t + 1:].shape, 85)
    O2, LSE2 = oracle.attn_fwd(Q, K2, V2, 0.3, True)
    dQ2, _, _, _ = oracle.attn_bwd(Q, K2, V2, dO, 0.3, True)
    np.testing.assert_array_equal(O[:, :, : t + 1], O2[:, :, : t + 1])
    np.testing.assert_array_equal(LSE[:, :, : t + 1], LSE2[:, :, : t + 1])
    np.testing.assert_array_equal(dQ[:, :, : t + 1], dQ2[:, :, : t + 1])
    assert not np.allclose(O[:, :, t + 1:], O2[:, :, t + 1:])
    # key/value gradients at position j ignore queries before j
    Q3, dO3 = Q.copy(), dO.copy()
    Q3[:, :, :t] += 1.0
    dO3[:, :, :t] *= -2.0
    _, dK3, dV3, _ = oracle.attn_bwd(Q3, K, V, dO3, 0.3, True)
    np.testing.assert_array_equal(dK[:, :, t:], dK3[:, :, t:])
    np.testing.assert_array_equal(dV[:, :, t:], dV3[:, :, t:])


def test_key_shift_invariance():
    shape = (1, 1, 19, 6)
    Q, K, V = (rand(shape, s) for s in (90, 91, 92))
    c = rand((6,), 93)
    scale = 0.41
    O, LSE = oracle.attn_fwd(Q, K, V, scale, True)
    O2, LSE2 = oracle.attn_fwd(Q, K + c, V, scale, True)
    np.testing.assert_allclose(O2, O, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(LSE2 - LSE, scale * (Q @ c), rtol=1e-11, atol=1e-12)


def test_peaked_softmax_is_stable():
    """Scores of magnitude ~50-500: one key dominates, O_i -> V_argmax, LSE -> max score, no NaN."""
    B, H, T, D = 1, 1, 32, 8
    Q, K, V, dO = (rand((B, H, T, D), s, sc) for s, sc in ((100, 20.0), (101, 20.0), (102, 1.0), (103, 1.0)))
    scale = 1.0
    O, LSE = oracle.attn_fwd(Q, K, V, scale, True)
    grads = oracle.attn_bwd(Q, K, V, dO, scale, True)
    assert np.isfinite(O).all() and np.isfinite(LSE).all() and all(np.isfinite(g).all() for g in grads)
    s = scale * Q[0, 0] @ K[0, 0].T
    s[np.triu_indices(T, 1)] = -np.inf
    top = np.sort(s, axis=1)
    gap = top[1:, -1] - top[1:, -2]
    rows = np.where(gap > 40.0)[0] + 1
    assert len(rows) > 5
    am = s.argmax(1)
    np.testing.assert_allclose(O[0, 0, rows], V[0, 0, am[rows]], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(LSE[0, 0, rows], s.max(1)[rows], rtol=1e-14)


def test_thread_count_does_not_change_results():
    shape = (2, 4, 50, 8)
    Q, K, V, dO = (rand(shape, s) for s in (110, 111, 112, 113))
    a = oracle.attn_bwd(Q, K, V, dO, 0.2, True)
    # one head at a time (serial order of heads cannot matter because heads never mix)
    for b in range(2):
        for h in range(4):
            sl = (slice(b, b + 1), slice(h, h + 1))
            one = oracle.attn_bwd(Q[sl], K[sl], V[sl], dO[sl], 0.2, True)
            for x, y in zip(a, one):
                np.testing.assert_array_equal(x[sl], y)
    assert oracle.num_threads() >= 1


# ---------------------------------------------------------------------------------------------
# further invariants: each one fails for a different plausible mistake
def test_scale_can_be_moved_into_the_queries():
    """softmax(scale * q.k) only sees the product: scale 0.5 with Q equals scale 1 with Q/2, in O, LSE and dK, dV;
    dQ picks up the factor of the substitution (dL/dQ = 0.5 * dL/d(Q/2))."""
    Q, K, V, dO = (rand((1, 2, 7, 4), s) for s in (1, 2, 3, 4))
    O1, L1 = oracle.attn_fwd(Q, K, V, 0.5, True)
    O2, L2 = oracle.attn_fwd(0.5 * Q, K, V, 1.0, True)
    np.testing.assert_allclose(O1, O2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(L1, L2, rtol=1e-12, atol=1e-14)
    dQ1, dK1, dV1, D1 = oracle.attn_bwd(Q, K, V, dO, 0.5, True)
    dQ2, dK2, dV2, D2 = oracle.attn_bwd(0.5 * Q, K, V, dO, 1.0, True)
    np.testing.assert_allclose(dQ1, 0.5 * dQ2, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dK1, dK2, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dV1, dV2, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(D1, D2, rtol=1e-11, atol=1e-13)


def test_output_is_linear_in_values_and_dv_is_transposed_probabilities():
    """O = P V with P independent of V: O(aV1 + bV2) = a O(V1) + b O(V2), LSE does not move, and
    dV = P^T dO with the P the oracle reports (a transposed or unnormalised P fails here)."""
    Q, K, V1, V2, dO = (rand((1, 1, 6, 3), s) for s in (11, 12, 13, 14, 15))
    Oa, La = oracle.attn_fwd(Q, K, V1, 0.7, True)
    Ob, Lb = oracle.attn_fwd(Q, K, V2, 0.7, True)
    Oc, Lc = oracle.attn_fwd(Q, K, 2.0 * V1 - 3.0 * V2, 0.7, True)
    np.testing.assert_allclose(Oc, 2.0 * Oa - 3.0 * Ob, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(Lc, La, rtol=0, atol=0)
    P = oracle.attn_probs(Q[0, 0], K[0, 0], 0.7, True)   # [T,T] of the one head
    _, _, dV, _ = oracle.attn_bwd(Q, K, V1, dO, 0.7, True)
    np.testing.assert_allclose(dV[0, 0], P.T @ dO[0, 0], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(Oa[0, 0], P @ V1[0, 0], rtol=1e-12, atol=1e-13)


def test_noncausal_attention_is_equivariant_under_key_permutation():
    """Without the mask the keys are a set: permuting (K, V) rows together leaves O and LSE alone and
    permutes dK, dV the same way (an index mix-up between the key loop and the outputs fails here)."""
    Q, K, V, dO = (rand((1, 2, 9, 5), s) for s in (21, 22, 23, 24))
    perm = np.random.default_rng(5).permutation(9)
    O1, L1 = oracle.attn_fwd(Q, K, V, 0.3, False)
    O2, L2 = oracle.attn_fwd(Q, K[:, :, perm], V[:, :, perm], 0.3, False)
    np.testing.assert_allclose(O1, O2, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(L1, L2, rtol=1e-12, atol=1e-13)
    dQ1, dK1, dV1, _ = oracle.attn_bwd(Q, K, V, dO, 0.3, False)
    dQ2, dK2, dV2, _ = oracle.attn_bwd(Q, K[:, :, perm], V[:, :, perm], dO, 0.3, False)
    np.testing.assert_allclose(dQ1, dQ2, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dK1[:, :, perm], dK2, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dV1[:, :, perm], dV2, rtol=1e-11, atol=1e-13)


def test_lse_is_the_potential_of_the_probabilities():
    """d LSE_i / d k_j = scale * P_ij * q_i (central differences): ties LSE, P and the scale together, and
    fixes the natural-log base of LSE (a base-2 LSE would be off by ln 2)."""
    rng = np.random.default_rng(31)
    Q, K, V = (rng.standard_normal((1, 1, 5, 3)) for _ in range(3))
    scale, h = 0.8, 1e-6
    P = oracle.attn_probs(Q[0, 0], K[0, 0], scale, True)
    for (i, j, d) in ((4, 2, 1), (3, 3, 0), (2, 0, 2), (1, 3, 1)):
        Kp, Km = K.copy(), K.copy()
        Kp[0, 0, j, d] += h
        Km[0, 0, j, d] -= h
        num = (oracle.attn_fwd(Q, Kp, V, scale, True)[1][0, 0, i] - oracle.attn_fwd(Q, Km, V, scale, True)[1][0, 0, i]) / (2 * h)
        ana = scale * P[i, j] * Q[0, 0, i, d]  # zero above the diagonal: the masked key cannot move LSE
        assert abs(num - ana) < 1e-8, (i, j, d, num, ana)


def test_heads_and_batches_are_independent():
    """Every (batch, head) is its own problem: running them together equals running each alone."""
    Q, K, V, dO = (rand((2, 3, 6, 4), s) for s in (41, 42, 43, 44))
    O, L = oracle.attn_fwd(Q, K, V, 0.5, True)
    dQ, dK, dV, D = oracle.attn_bwd(Q, K, V, dO, 0.5, True)
    for b in range(2):
        for hd in range(3):
            sl = (slice(b, b + 1), slice(hd, hd + 1))
            o, l = oracle.attn_fwd(Q[sl], K[sl], V[sl], 0.5, True)
            dq, dk, dv, d = oracle.attn_bwd(Q[sl], K[sl], V[sl], dO[sl], 0.5, True)
            for a, b_ in ((O[sl], o), (L[sl], l), (dQ[sl], dq), (dK[sl], dk), (dV[sl], dv), (D[sl], d)):
                np.testing.assert_array_equal(a, b_)
