"""GPU parity of the fused loss head (through the C ABI) against the fp64 oracle on the same seeded inputs.

Bounds, stated in the test: the lse and the loss are fp32 reductions of fp32-accumulated bf16 products, so
they are held to 1e-2 relative (1e-2 + 1e-2|ref| element-wise; the measured errors are some 1e-5); the stored
logits carry one bf16 rounding: |got - ref| <= 2^-8 |ref| + 1e-3.
"""
import numpy as np
import pytest
import torch

from paper_2608_00029_b200 import workloads as W

pytestmark = pytest.mark.gpu
GUARD = 64


def _run(cfg, X, Wm, t, want_logits=True):
    from paper_2608_00029_b200 import nova_attn as na, nova_lmhead as lm
    dev = torch.device("cuda:0")
    x, w, tt = X.to(dev), Wm.to(dev), t.to(dev)
    M, N = cfg.M, cfg.N
    buf = torch.full((M * N + 2 * GUARD,), 7.0, dtype=torch.bfloat16, device=dev) if want_logits else None
    logits = buf[GUARD:GUARD + M * N].view(M, N) if want_logits else None
    stat = torch.full((2 * M + 2 * GUARD,), 7.0, dtype=torch.float32, device=dev)
    lse, loss = stat[GUARD:GUARD + M], stat[GUARD + M:GUARD + 2 * M]
    lm.nova_lmhead_fwd(x, w, tt, logits, lse, loss)
    na.nova_attn_poll_device_status()
    assert bool((stat[:GUARD] == 7.0).all()) and bool((stat[-GUARD:] == 7.0).all()), "write outside lse / loss"
    if want_logits:
        g = torch.cat([buf[:GUARD], buf[-GUARD:]]).float()
        assert bool((g == 7.0).all()), "write outside the logits"
    return (logits.cpu() if want_logits else None), lse.cpu(), loss.cpu()


def _check(cfg, X, Wm, t, rows=None, want_logits=True):
    import oracle
    logits, lse, loss = _run(cfg, X, Wm, t, want_logits)
    sel = np.arange(cfg.M) if rows is None else np.asarray(rows)
    ref_logits, ref_lse, ref_loss = oracle.lmhead_fwd(W.widen(X)[sel], W.widen(Wm), t.numpy()[sel], want_logits=True)
    got_lse, got_loss = W.widen(lse)[sel], W.widen(loss)[sel]
    assert np.isfinite(got_lse).all() and np.isfinite(got_loss).all()
    assert (np.abs(got_lse - ref_lse) <= 1e-2 + 1e-2 * np.abs(ref_lse)).all(), np.abs(got_lse - ref_lse).max()
    assert (np.abs(got_loss - ref_loss) <= 1e-2 + 1e-2 * np.abs(ref_loss)).all(), np.abs(got_loss - ref_loss).max()
    # far inside the bound in practice: fp32 statistics of fp32 accumulators
    assert np.abs(got_lse - ref_lse).max() <= 2e-4 * max(1.0, np.abs(ref_lse).max())
    if want_logits:
        got = W.widen(logits)[sel]
        assert (np.abs(got - ref_logits) <= 2.0 ** -8 * np.abs(ref_logits) + 1e-3).all(), np.abs(got - ref_logits).max()
    ignored = (t.numpy()[sel] < 0) | (t.numpy()[sel] >= cfg.N)
    assert (got_loss[ignored] == 0.0).all()
    return float(np.abs(got_lse - ref_lse).max()), float(np.abs(got_loss - ref_loss).max())


def test_tiny_config_all_rows():
    cfg = W.LM_HEAD_CONFIGS["lm_head_tiny"]
    print(_check(cfg, *W.make_lmhead_inputs(cfg)))


SHAPES = [  # M, N, K: single tile, ragged rows, ragged vocabulary (half a tile, a sliver), ragged K, several tiles
    (1, 8, 8), (128, 256, 64), (130, 264, 72), (100, 128, 64), (300, 1000, 200), (257, 520, 768), (64, 2056, 128),
    (1024, 512, 96),
]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_edge_shapes(M, N, K):
    cfg = W.LmHeadConfig("edge", M=M, N=N, K=K, seed=100 + M + N + K, w_factor=0.3, ignored_every=5)
    _check(cfg, *W.make_lmhead_inputs(cfg))


def test_without_logits_and_run_to_run_determinism():
    cfg = W.LmHeadConfig("nolog", M=384, N=3000 // 8 * 8, K=256, seed=5, w_factor=0.1)
    X, Wm, t = W.make_lmhead_inputs(cfg)
    _, lse_a, loss_a = _run(cfg, X, Wm, t, want_logits=False)
    lg, lse_b, loss_b = _run(cfg, X, Wm, t, want_logits=True)
    _, lse_c, loss_c = _run(cfg, X, Wm, t, want_logits=True)
    assert torch.equal(lse_a, lse_b) and torch.equal(loss_a, loss_b)
    assert torch.equal(lse_b, lse_c) and torch.equal(loss_b, loss_c)
    _check(cfg, X, Wm, t, want_logits=False)


def test_large_and_peaked_logits():
    """Logits of magnitude ~100 with one dominant entry per row: the running maximum must carry the sums."""
    cfg = W.LmHeadConfig("peaked", M=256, N=1024, K=64, seed=6, x_factor=4.0, w_factor=3.0)
    _check(cfg, *W.make_lmhead_inputs(cfg))


def test_full_size_on_sampled_rows():
    """The paper's shape, 8192 x 768 x 50304, run at full size on the GPU; the oracle checks 96 sampled rows
    (rows are independent), and properties that hold for every row are checked on all of them."""
    cfg = W.LM_HEAD_CONFIGS["lm_head_gpt2"]
    X, Wm, t = W.make_lmhead_inputs(cfg)
    rows = sorted(set(np.random.default_rng(1).choice(cfg.M, 94, replace=False).tolist()) | {0, cfg.M - 1})
    print(_check(cfg, X, Wm, t, rows=rows, want_logits=True))
    logits, lse, loss = _run(cfg, X, Wm, t, want_logits=True)
    # every row: the loss is lse minus the stored target logit (to the logit's bf16 rounding), lse >= max logit,
    # and lse <= max logit + ln N
    lg = logits.float()
    tl = lg.gather(1, t.long().view(-1, 1)).view(-1)
    assert ((lse - tl) - loss).abs().max() <= 2.0 ** -8 * tl.abs().max() + 1e-3
    mx = lg.max(dim=1).values
    assert bool((lse >= mx - 2.0 ** -7 * mx.abs() - 1e-3).all()) and bool((lse <= mx + np.log(cfg.N) + 1e-2).all())
