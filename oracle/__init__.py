"""fp64 CPU oracle for fused causal attention (forward and backward).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the benchmark's CPU
baseline leg.  The CUDA library and its Python binding never import this package, and this package
never imports them.
"""
from .attn_oracle import attn_fwd, attn_bwd, attn_probs, num_threads, build  # noqa: F401
