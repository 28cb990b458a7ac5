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


def test_both_kernels_agree_and_cuda_graph_replay():
    """M <= 128 runs one CTA per tile, larger M one pair of CTAs per 256-row tile: the same rows must come out the
    same either way (a row's statistics do not depend on its neighbours), also when the calls are captured into
    a CUDA graph once and replayed (cluster launches inside a graph), and on a side stream."""
    from paper_2608_00029_b200 import nova_attn as na, nova_lmhead as lm
    dev = torch.device("cuda:0")
    cfg = W.LmHeadConfig("both", M=640, N=1536, K=192, seed=9, w_factor=0.2, ignored_every=11)
    X, Wm, t = W.make_lmhead_inputs(cfg)
    x, w, tt = X.to(dev), Wm.to(dev), t.to(dev)
    ws = torch.empty(lm.nova_lmhead_workspace_bytes(cfg.M, cfg.N, cfg.K), dtype=torch.uint8, device=dev)
    logits = torch.empty((cfg.M, cfg.N), dtype=torch.bfloat16, device=dev)
    lse, loss = torch.empty(cfg.M, device=dev), torch.empty(cfg.M, device=dev)
    lm.nova_lmhead_fwd(x, w, tt, logits, lse, loss, ws)
    na.nova_attn_poll_device_status()
    # the first 100 rows alone (one tile of rows: the single-CTA kernel)
    l1, s1, o1 = torch.empty((100, cfg.N), dtype=torch.bfloat16, device=dev), torch.empty(100, device=dev), torch.empty(100, device=dev)
    lm.nova_lmhead_fwd(x[:100].contiguous(), w, tt[:100].contiguous(), l1, s1, o1)
    na.nova_attn_poll_device_status()
    assert torch.equal(l1, logits[:100]) and torch.equal(s1, lse[:100]) and torch.equal(o1, loss[:100])
    # captured once, replayed three times on a side stream
    side = torch.cuda.Stream()
    lse2, loss2, logits2 = torch.zeros_like(lse), torch.zeros_like(loss), torch.zeros_like(logits)
    with torch.cuda.stream(side):
        lm.nova_lmhead_fwd(x, w, tt, logits2, lse2, loss2, ws, stream=side)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        lm.nova_lmhead_fwd(x, w, tt, logits2, lse2, loss2, ws, stream=torch.cuda.current_stream())
    for _ in range(3):
        lse2.zero_(); loss2.zero_(); logits2.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        na.nova_attn_poll_device_status()
        assert torch.equal(lse2, lse) and torch.equal(loss2, loss) and torch.equal(logits2, logits)
