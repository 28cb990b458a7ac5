"""Seeded input generator: determinism, shapes, value structure, batch sharding."""
import numpy as np
import pytest
import torch

from paper_2608_00029_b200 import workloads as W


def test_five_configs_match_the_stated_shapes():
    shapes = {n: (c.B, c.H, c.T, c.D, c.seed) for n, c in W.CONFIGS.items()}
    assert shapes == {
        "tiny": (1, 2, 64, 64, 0),
        "gpt2_small": (8, 12, 1024, 64, 1),
        "gpt2_small_large_batch": (32, 12, 1024, 64, 2),
        "gpt2_medium": (8, 16, 1024, 64, 3),
        "long_context": (2, 12, 8192, 128, 4),
    }
    assert W.CONFIGS["gpt2_small"].scale == 0.125
    assert abs(W.CONFIGS["long_context"].scale - 0.088388346) < 1e-8
    assert W.CONFIGS["gpt2_small"].fwd_flops == 2 * 8 * 12 * 1024 * 1024 * 64
    assert W.CONFIGS["gpt2_small"].bwd_flops == 2.5 * W.CONFIGS["gpt2_small"].fwd_flops


def test_generator_is_deterministic_and_bf16():
    cfg = W.CONFIGS["tiny"]
    a, b = W.make_inputs(cfg), W.make_inputs(cfg)
    for x, y in zip(a, b):
        assert x.dtype == torch.bfloat16 and x.shape == (1, 2, 64, 64) and x.is_contiguous()
        assert torch.equal(x, y)
    c = W.make_inputs(cfg, seed=5)
    assert not torch.equal(a[0], c[0])
    # the four tensors are different draws
    assert not torch.equal(a[0], a[1])


def test_value_structure():
    cfg = W.CONFIGS["gpt2_small"].replace(B=1, H=2, T=256)
    Q, K, V, dO = (W.widen(x) for x in W.make_inputs(cfg))
    assert abs(Q.std() - 1) < 0.02 and abs(V.std() - 1) < 0.02
    assert abs(dO.std() - 1e-2) < 3e-4
    cfg3 = W.CONFIGS["gpt2_small_large_batch"].replace(B=1, H=2, T=256)
    Q3, K3, V3, dO3 = (W.widen(x) for x in W.make_inputs(cfg3))
    assert abs(Q3.std() - 2) < 0.04 and abs(K3.std() - 2) < 0.04 and abs(V3.std() - 1) < 0.02


def test_widen_is_exact():
    x = torch.tensor([1.0, 0.333, -2.5e-3], dtype=torch.bfloat16)
    w = W.widen(x)
    assert w.dtype == np.float64
    assert [float(v) for v in w] == [float(v) for v in x.float()]


@pytest.mark.parametrize("B,world", [(8, 1), (8, 2), (8, 8), (7, 2), (3, 4), (32, 8)])
def test_shard_batch_partitions_exactly(B, world):
    spans = [W.shard_batch(B, r, world) for r in range(world)]
    assert spans[0][0] == 0 and spans[-1][1] == B
    for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
        assert a1 == b0 and a0 <= a1
    sizes = [b - a for a, b in spans]
    assert max(sizes) - min(sizes) <= 1
