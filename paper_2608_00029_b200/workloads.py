"""Seeded synthetic inputs for the attention path.  Holds NO attention arithmetic.

The paper's attention microbenchmark (Section 6.1, the attention figure) uses random causal
self-attention inputs of GPT-2-like shapes and no public dataset, so these tensors are the workload
itself.  The same bf16 bit patterns are handed to the CUDA library and, widened exactly to float64,
to the CPU oracle.

Recipe: ``torch.Generator('cpu').manual_seed(seed)``; ``torch.randn([B,H,T,D], float32)`` drawn in
the order Q, K, V, dO; each multiplied by its factor in float32; rounded to bf16 (nearest-even).
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class AttnConfig:
    name: str
    B: int
    H: int
    T: int
    D: int
    seed: int
    qk_factor: float = 1.0
    v_factor: float = 1.0
    do_factor: float = 1.0
    causal: bool = True

    @property
    def scale(self) -> float:
        """Softmax scale 1/sqrt(D) as the float32 value the library receives."""
        return float(torch.tensor(1.0 / math.sqrt(self.D), dtype=torch.float32).item())

    @property
    def fwd_flops(self) -> float:
        """Counted causal FLOPs of the forward: 2*B*H*T^2*D (two contractions over half the square)."""
        return 2.0 * self.B * self.H * self.T * self.T * self.D

    @property
    def bwd_flops(self) -> float:
        """Counted causal FLOPs of the backward: five contractions, 2.5x the forward."""
        return 2.5 * self.fwd_flops

    def replace(self, **kw) -> "AttnConfig":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "tiny": AttnConfig("tiny", B=1, H=2, T=64, D=64, seed=0),
    "gpt2_small": AttnConfig("gpt2_small", B=8, H=12, T=1024, D=64, seed=1, do_factor=1e-2),
    "gpt2_small_large_batch": AttnConfig("gpt2_small_large_batch", B=32, H=12, T=1024, D=64, seed=2,
                                         qk_factor=2.0),
    "gpt2_medium": AttnConfig("gpt2_medium", B=8, H=16, T=1024, D=64, seed=3),
    "long_context": AttnConfig("long_context", B=2, H=12, T=8192, D=128, seed=4),
}
CONFIG_ORDER = ["tiny", "gpt2_small", "gpt2_small_large_batch", "gpt2_medium", "long_context"]


@dataclasses.dataclass(frozen=True)
class LmHeadConfig:
    """Loss head of a language model: hidden states X [M, K] against the vocabulary matrix W [N, K]."""
    name: str
    M: int
    N: int
    K: int
    seed: int
    x_factor: float = 1.0      # hidden states after the final normalisation: unit scale
    w_factor: float = 0.02     # GPT-2's initialisation scale of the (tied) embedding matrix
    ignored_every: int = 0     # every so-many-th row gets the target -1 (a position without a label); 0 = none

    @property
    def flops(self) -> float:
        """FLOPs of the projection: 2*M*N*K."""
        return 2.0 * self.M * self.N * self.K

    def replace(self, **kw) -> "LmHeadConfig":
        return dataclasses.replace(self, **kw)


# The paper measures its fused loss head on 8192 x 768 x 50304 (8 sequences of 1024 tokens, GPT-2-small width,
# vocabulary padded to 50304: Section 6.1, "Fused Loss Head").
LM_HEAD_CONFIGS = {
    "lm_head_tiny": LmHeadConfig("lm_head_tiny", M=200, N=1000, K=64, seed=10, ignored_every=7),
    "lm_head_gpt2": LmHeadConfig("lm_head_gpt2", M=8192, N=50304, K=768, seed=11),
}


def make_lmhead_inputs(cfg: LmHeadConfig, seed: int | None = None):
    """Return (X bf16 [M,K], W bf16 [N,K], targets int32 [M]) as CPU tensors: X, W iid normal times their
    factors, rounded to bf16; targets uniform over the vocabulary."""
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.seed if seed is None else seed)
    X = (torch.randn((cfg.M, cfg.K), dtype=torch.float32, generator=g) * cfg.x_factor).to(torch.bfloat16)
    W = (torch.randn((cfg.N, cfg.K), dtype=torch.float32, generator=g) * cfg.w_factor).to(torch.bfloat16)
    t = torch.randint(0, cfg.N, (cfg.M,), generator=g, dtype=torch.int64).to(torch.int32)
    if cfg.ignored_every > 0:
        t[:: cfg.ignored_every] = -1
    return X, W, t


def make_inputs(cfg: AttnConfig, seed: int | None = None):
    """Return (Q, K, V, dO) as CPU bf16 tensors of shape [B,H,T,D]."""
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.seed if seed is None else seed)
    shape = (cfg.B, cfg.H, cfg.T, cfg.D)
    out = []
    for factor in (cfg.qk_factor, cfg.qk_factor, cfg.v_factor, cfg.do_factor):
        x = torch.randn(shape, dtype=torch.float32, generator=g)
        if factor != 1.0:
            x = x * torch.tensor(factor, dtype=torch.float32)
        out.append(x.to(torch.bfloat16))
    return tuple(out)


def widen(x: torch.Tensor):
    """Exact widening of a (bf16/fp32) tensor to a float64 numpy array."""
    return x.detach().to("cpu").to(torch.float64).numpy()


def shard_batch(B: int, rank: int, world_size: int) -> tuple[int, int]:
    """Contiguous [start, stop) slice of the batch dimension owned by ``rank`` (heads are independent,
    so ranks never exchange data)."""
    if world_size <= 0 or not (0 <= rank < world_size):
        raise ValueError("bad rank/world_size")
    base, rem = divmod(B, world_size)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)
