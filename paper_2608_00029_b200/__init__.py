"""Fused causal multi-head attention (forward + backward) for NVIDIA B200 (sm_100a).

``nova_attn`` is the thin binding over the C-ABI library ``libnova_attn.so``; ``workloads`` holds
the seeded synthetic inputs.  Importing this package does not load the CUDA library; the first call
into ``nova_attn`` does, and fails loudly if it is missing.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "nova_attn"]


def __getattr__(name):
    if name == "nova_attn":
        import importlib
        return importlib.import_module(".nova_attn", __name__)
    raise AttributeError(name)
