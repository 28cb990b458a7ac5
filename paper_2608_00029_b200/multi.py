"""Host-side plumbing for running the attention path on N GPUs of one node.

Every (batch, head) pair is an independent problem in forward, preprocess and backward, so ranks only
split the batch dimension and never exchange tensor data.  The only collectives are the benchmark's
own: a barrier and a MAX over ranks of the measured time.  Works with any torch.distributed backend
(NCCL on GPUs, gloo on CPU for the tests).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist

from .workloads import shard_batch


def env_rank_world() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when not launched by it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init_process_group(backend: str) -> bool:
    """Initialise torch.distributed from the environment if WORLD_SIZE > 1.  Returns True if it did."""
    _, _, world = env_rank_world()
    if world <= 1 or dist.is_initialized():
        return dist.is_initialized()
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    dist.init_process_group(backend=backend)
    return True


def weak_scaling_plan(per_gpu_batch: int, world_size: int, rank: int) -> dict:
    """Weak scaling: every rank owns `per_gpu_batch` sequences of a global batch of per_gpu_batch * N."""
    global_batch = per_gpu_batch * world_size
    start, stop = shard_batch(global_batch, rank, world_size)
    return {"global_batch": global_batch, "start": start, "stop": stop, "local_batch": stop - start}


def max_over_ranks(value: float, device) -> float:
    """MAX all-reduce of one scalar (identity when not distributed)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device) -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
