"""Runs the attention hot path a few times on one named configuration: a small, self-contained
command to put under a profiler.

    python -m paper_2608_00029_b200.profile_case [--config gpt2_small] [--iters 3] [--batch B]
"""
from __future__ import annotations

import argparse

import torch

from . import nova_attn as na
from . import workloads as W


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="gpt2_small", choices=W.CONFIG_ORDER)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (0 = the configuration's)")
    ap.add_argument("--exact-delta", action="store_true")
    args = ap.parse_args()
    cfg = W.CONFIGS[args.config]
    if args.batch > 0:
        cfg = cfg.replace(B=args.batch)
    dev = torch.device("cuda:0")
    q, k, v, do = (x.to(dev) for x in W.make_inputs(cfg))
    o, dq, dk, dv = (torch.empty_like(q) for _ in range(4))
    lse = torch.empty((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device=dev)
    delta = torch.empty_like(lse)
    ws = torch.empty(na.nova_attn_bwd_workspace_bytes(cfg.B, cfg.H, cfg.T, cfg.D), dtype=torch.uint8, device=dev)
    for _ in range(args.iters):
        na.nova_attn_fwd(q, k, v, o, lse, cfg.scale, cfg.causal)
        if args.exact_delta:
            na.nova_attn_bwd_preprocess_exact(q, k, v, do, lse, delta, cfg.scale, cfg.causal)
        else:
            na.nova_attn_bwd_preprocess(o, do, delta)
        na.nova_attn_bwd(q, k, v, o, do, lse, delta, dq, dk, dv, cfg.scale, cfg.causal, ws)
    na.nova_attn_poll_device_status()
    print(f"{cfg.name}: {args.iters} iterations ok; checksum {float(dq.float().sum()):.4f}")


if __name__ == "__main__":
    main()
