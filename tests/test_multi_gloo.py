"""World-size-2 gloo run of the multi-GPU host logic (batch sharding, barrier, max/sum over ranks)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_00029_b200 import multi, workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert multi.init_process_group("gloo")
    assert multi.env_rank_world() == (rank, rank, world)
    plan = multi.weak_scaling_plan(8, world, rank)
    # each rank generates only its own slice of the global batch, from a seed that depends on the slice
    cfg = W.CONFIGS["tiny"].replace(B=plan["local_batch"], seed=100 + plan["start"])
    Q, _, _, _ = W.make_inputs(cfg)
    multi.barrier()
    slowest = multi.max_over_ranks(10.0 + rank, "cpu")
    total = multi.sum_over_ranks(float(plan["local_batch"]), "cpu")
    out.put((rank, plan, slowest, total, float(Q.float().sum())))
    dist.destroy_process_group()


def test_two_ranks_shard_batch_and_reduce():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, p0, m0, t0, s0), (r1, p1, m1, t1, s1) = res
    assert (p0["start"], p0["stop"]) == (0, 8) and (p1["start"], p1["stop"]) == (8, 16)
    assert p0["global_batch"] == p1["global_batch"] == 16
    assert m0 == m1 == 11.0          # max over ranks
    assert t0 == t1 == 16.0          # all sequences accounted for exactly once
    assert s0 != s1                  # different slices -> different data


def test_single_process_helpers_are_identities():
    assert multi.max_over_ranks(3.5, "cpu") == 3.5
    assert multi.sum_over_ranks(2.0, "cpu") == 2.0
    multi.barrier()
    assert multi.weak_scaling_plan(8, 1, 0) == {"global_batch": 8, "start": 0, "stop": 8, "local_batch": 8}
