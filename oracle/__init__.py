"""fp64 CPU oracles: fused causal attention (forward and backward) and the language-model loss head.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the benchmark's CPU
baseline leg.  The CUDA library and its Python binding never import this package, and this package
never imports them.
"""
from .attn_oracle import attn_fwd, attn_bwd, attn_probs, num_threads  # noqa: F401
from .attn_oracle import build as _build_attn
from .lmhead_oracle import lmhead_fwd  # noqa: F401
from .lmhead_oracle import build as _build_lmhead


def build(force: bool = False) -> None:
    """Compile every C oracle."""
    _build_attn(force)
    _build_lmhead(force)
