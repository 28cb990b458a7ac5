"""Times forward and backward over a grid of causal self-attention shapes spanning the ranges of the
paper's attention microbenchmark (Section 6, "Attention": sequence lengths 512 to 2048, 12 to 32
heads, head dimension 64 or 128; the figure with the per-shape values is an image, so the eight points
here are chosen inside those ranges, at batch 16 like the figure's "16x12x64" label).

    python -m paper_2608_00029_b200.grid_case [--batch 16] [--reps 30] [--non-causal] [--fused | --deterministic]

--deterministic times nova_attn_bwd_deterministic (the paper's two-kernel backward) as the backward.

--fused times the strided entry points on the fused-projection layout instead: Q, K, V read in place from
a [B, T, 3, H, D] buffer, O and dO as [B, T, H, D], dQ, dK, dV written into a [B, T, 3, H, D] buffer.

Prints one markdown table row per shape: milliseconds and counted TFLOP/s (forward 2*B*H*T^2*D for the
causal case, backward 2.5x that; twice as much without the mask) of nova_attn_fwd and of
nova_attn_bwd_preprocess + nova_attn_bwd, each timed back to back with CUDA events.
"""
from __future__ import annotations

import argparse

import torch

from . import nova_attn as na
from . import workloads as W

GRID = [  # (T, H, D)
    (512, 12, 64), (1024, 12, 64), (2048, 12, 64), (1024, 16, 64),
    (1024, 20, 64), (512, 32, 128), (1024, 32, 128), (2048, 32, 128),
]


def _time(fn, reps: int) -> float:
    for _ in range(5):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--reps", type=int, default=30)
    ap.add_argument("--non-causal", action="store_true")
    ap.add_argument("--fused", action="store_true")
    ap.add_argument("--deterministic", action="store_true")
    args = ap.parse_args()
    causal = not args.non_causal
    dev = torch.device("cuda:0")
    print("| B | H | T | D | causal | fwd ms | fwd TFLOP/s | bwd ms | bwd TFLOP/s | fwd+bwd ms |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for T, H, D in GRID:
        cfg = W.AttnConfig(f"grid_T{T}_H{H}_D{D}", B=args.batch, H=H, T=T, D=D, seed=5, causal=causal)
        q, k, v, do = (x.to(dev) for x in W.make_inputs(cfg))
        o, dq, dk, dv = (torch.empty_like(q) for _ in range(4))
        lse = torch.empty((cfg.B, H, T), dtype=torch.float32, device=dev)
        delta = torch.empty_like(lse)
        ws = torch.empty(na.nova_attn_bwd_workspace_bytes(cfg.B, H, T, D), dtype=torch.uint8, device=dev)

        if args.fused:
            B = cfg.B
            qkv = torch.empty((B, T, 3, H, D), dtype=torch.bfloat16, device=dev)
            for i, x in enumerate((q, k, v)):
                qkv[:, :, i] = x.permute(0, 2, 1, 3)
            dqkv = torch.empty_like(qkv)
            o_buf = torch.empty((B, T, H, D), dtype=torch.bfloat16, device=dev)
            do_buf = do.permute(0, 2, 1, 3).contiguous()
            q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
            dq, dk, dv = (dqkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
            o, do = o_buf.permute(0, 2, 1, 3), do_buf.permute(0, 2, 1, 3)

            def fwd():
                na.nova_attn_fwd_strided(q, k, v, o, lse, cfg.scale, causal)

            def bwd():
                na.nova_attn_bwd_preprocess_strided(o, do, delta)
                na.nova_attn_bwd_strided(q, k, v, do, lse, delta, dq, dk, dv, cfg.scale, causal, ws)
        else:
            def fwd():
                na.nova_attn_fwd(q, k, v, o, lse, cfg.scale, causal)

            def bwd():
                na.nova_attn_bwd_preprocess(o, do, delta)
                if args.deterministic:
                    na.nova_attn_bwd_deterministic(q, k, v, do, lse, delta, dq, dk, dv, cfg.scale, causal)
                else:
                    na.nova_attn_bwd(q, k, v, o, do, lse, delta, dq, dk, dv, cfg.scale, causal, ws)

        t_f, t_b = _time(fwd, args.reps), _time(bwd, args.reps)
        f_flops = cfg.fwd_flops * (1.0 if causal else 2.0)  # the counted figure covers half the square
        b_flops = 2.5 * f_flops
        na.nova_attn_poll_device_status()
        print(f"| {cfg.B} | {H} | {T} | {D} | {'yes' if causal else 'no'} | {t_f:.4f} | {f_flops / t_f / 1e9:.0f} | "
              f"{t_b:.4f} | {b_flops / t_b / 1e9:.0f} | {t_f + t_b:.4f} |", flush=True)
        del q, k, v, do, o, dq, dk, dv, lse, delta, ws, fwd, bwd
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
