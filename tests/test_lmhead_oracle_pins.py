"""Pins of the loss-head oracle (oracle/lmhead_oracle.c) to things other than itself: a hand-worked example,
closed forms, a third-party routine used as a black box, invariants, brute force.  CPU only."""
import math
import os

import numpy as np
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "lm_head_worked_example.txt")


def _golden():
    vals = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, *rest = line.split()
        vals[name] = np.array([float(x) for x in rest])
    return vals


def _random(M, N, K, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((M, K)), scale * rng.standard_normal((N, K)), rng.integers(0, N, M).astype(np.int32)


def test_hand_worked_example():
    g = _golden()
    X, W = g["X"].reshape(2, 2), g["W"].reshape(3, 2)
    logits, lse, loss = oracle.lmhead_fwd(X, W, g["targets"].astype(np.int32), want_logits=True)
    np.testing.assert_allclose(logits.ravel(), g["logits"], rtol=0, atol=1e-15)
    np.testing.assert_allclose(lse, g["LSE"], rtol=0, atol=1e-15)
    np.testing.assert_allclose(loss, g["loss"], rtol=0, atol=1e-15)
    # the printed values themselves: ln 4, ln 5, ln 2, ln(5/3)
    np.testing.assert_allclose(g["LSE"], [math.log(4), math.log(5)], atol=1e-16)
    np.testing.assert_allclose(g["loss"], [math.log(2), math.log(5 / 3)], atol=1e-16)


def test_brute_force_pure_python():
    X, W, t = _random(5, 7, 3, 1)
    lse, loss = oracle.lmhead_fwd(X, W, t)
    for i in range(5):
        z = [sum(float(X[i, k]) * float(W[n, k]) for k in range(3)) for n in range(7)]
        ref = math.log(sum(math.exp(v) for v in z))
        assert abs(lse[i] - ref) < 1e-13
        assert abs(loss[i] - (ref - z[t[i]])) < 1e-13


def test_against_library_cross_entropy_and_matmul():
    """torch (fp64, CPU) as a black box: matmul for the logits, cross_entropy and logsumexp for the rest."""
    X, W, t = _random(33, 211, 17, 2, scale=0.7)
    logits, lse, loss = oracle.lmhead_fwd(X, W, t, want_logits=True)
    z = torch.tensor(X) @ torch.tensor(W).T
    np.testing.assert_allclose(logits, z.numpy(), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(lse, torch.logsumexp(z, dim=1).numpy(), rtol=1e-13, atol=1e-13)
    ce = torch.nn.functional.cross_entropy(z, torch.tensor(t, dtype=torch.long), reduction="none")
    np.testing.assert_allclose(loss, ce.numpy(), rtol=1e-12, atol=1e-12)
    # with_logits and without must agree exactly (the second pass recomputes the same sums)
    lse2, loss2 = oracle.lmhead_fwd(X, W, t)
    assert np.array_equal(lse, lse2) and np.array_equal(loss, loss2)


def test_uniform_logits_give_log_vocabulary_size():
    X, W, t = _random(4, 50, 6, 3)
    lse, loss = oracle.lmhead_fwd(np.zeros_like(X), W, t)
    np.testing.assert_allclose(lse, math.log(50), atol=1e-14)
    np.testing.assert_allclose(loss, math.log(50), atol=1e-14)
    lse, loss = oracle.lmhead_fwd(X, np.zeros_like(W), t)
    np.testing.assert_allclose(loss, math.log(50), atol=1e-14)


def test_shift_invariance():
    """A constant added to every logit of a row (one more input column equal to 1 against a column of W equal to
    c) moves the LSE by c and leaves the loss where it was."""
    X, W, t = _random(6, 40, 5, 4)
    lse, loss = oracle.lmhead_fwd(X, W, t)
    c = 3.25
    X1 = np.concatenate([X, np.ones((6, 1))], axis=1)
    W1 = np.concatenate([W, np.full((40, 1), c)], axis=1)
    lse1, loss1 = oracle.lmhead_fwd(X1, W1, t)
    np.testing.assert_allclose(lse1, lse + c, atol=1e-12)
    np.testing.assert_allclose(loss1, loss, atol=1e-12)


def test_vocabulary_split_merges_by_the_rescaling_rule():
    """The log-sum-exp over the whole vocabulary equals the merge of the log-sum-exps over two parts of it, each
    sum rescaled to the common maximum (the rule the fused kernel's partial statistics rely on), and the order
    of the vocabulary entries does not matter."""
    X, W, t = _random(9, 64, 8, 5, scale=2.0)
    lse, loss = oracle.lmhead_fwd(X, W, t)
    la, _ = oracle.lmhead_fwd(X, W[:20], np.zeros(9, np.int32))
    lb, _ = oracle.lmhead_fwd(X, W[20:], np.zeros(9, np.int32))
    m = np.maximum(la, lb)
    np.testing.assert_allclose(lse, m + np.log(np.exp(la - m) + np.exp(lb - m)), atol=1e-12)
    perm = np.random.default_rng(0).permutation(64)
    inv = np.argsort(perm)
    lse_p, loss_p = oracle.lmhead_fwd(X, W[perm], inv[t].astype(np.int32))
    np.testing.assert_allclose(lse_p, lse, atol=1e-12)
    np.testing.assert_allclose(loss_p, loss, atol=1e-12)


def test_dominant_entry_and_large_logits_stay_finite():
    X, W, t = _random(3, 30, 4, 6)
    W = W.copy()
    W[11] = 0.0
    X = X.copy()
    X[:, 0] = 1.0
    W[11, 0] = 500.0  # one logit towers over the rest: exp(500) would overflow without the maximum
    lse, loss = oracle.lmhead_fwd(X, W, np.full(3, 11, np.int32))
    assert np.isfinite(lse).all()
    np.testing.assert_allclose(loss, 0.0, atol=1e-12)
    z = X @ W.T
    np.testing.assert_allclose(lse, z[:, 11], rtol=1e-12)


def test_targets_outside_the_vocabulary_are_ignored():
    X, W, t = _random(5, 12, 3, 7)
    t = t.copy()
    t[1], t[3] = -1, 12
    lse, loss = oracle.lmhead_fwd(X, W, t)
    assert loss[1] == 0.0 and loss[3] == 0.0 and (loss[[0, 2, 4]] > 0).all()
    assert np.isfinite(lse).all()


def test_gradient_of_the_loss_is_softmax_minus_one_hot():
    """Central differences of the mean loss with respect to the logits' inputs: d loss_i / d X[i,:] =
    (softmax(z_i) - onehot(t_i)) W, which pins the sign and the normalisation of the whole chain."""
    X, W, t = _random(3, 9, 4, 8)
    logits, lse, loss = oracle.lmhead_fwd(X, W, t, want_logits=True)
    P = np.exp(logits - lse[:, None])
    P[np.arange(3), t] -= 1.0
    grad = P @ W
    h = 1e-6
    for i in range(3):
        for k in range(4):
            Xp, Xm = X.copy(), X.copy()
            Xp[i, k] += h
            Xm[i, k] -= h
            fd = (oracle.lmhead_fwd(Xp, W, t)[1][i] - oracle.lmhead_fwd(Xm, W, t)[1][i]) / (2 * h)
            assert abs(fd - grad[i, k]) < 1e-7
