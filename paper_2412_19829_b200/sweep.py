"""Timing sweep of the hybrid layer over the 32 points of the sequence-length / window / head-size
grid (65 536 tokens per launch, H = 16), each with the default head split and with all heads
windowed, half and half, and all heads linear.  Prints a markdown table: microseconds per launch
(CUDA events, median of `--iters` launches after warm-up) and the fraction of the HBM roofline for
the layer's algorithmic bytes (Q, K, V read once, O written once).

    python -m paper_2412_19829_b200.sweep [--iters 10] [--peak-gbs 6533.8]

Inputs are seeded Gaussians generated on the device (timing only; parity is the tests' job)."""
import argparse

import numpy as np
import torch

from . import binding as gf
from . import synth


def time_call(fn, iters, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    evs[0].record()
    for i in range(iters):
        fn()
        evs[i + 1].record()
    torch.cuda.synchronize()
    return float(np.median([evs[i].elapsed_time(evs[i + 1]) * 1e3 for i in range(iters)]))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--peak-gbs", type=float, default=6533.8, help="measured copy bandwidth the fractions refer to")
    args = ap.parse_args()
    print("| N | B | d | w | H0=3 (default) us | frac | H0=16 us | H0=8 us | H0=0 us |")
    print("|---|---|---|---|---|---|---|---|---|")
    for c in synth.sweep_points():
        B, H, N, d, w = c["B"], c["H"], c["N"], c["d"], c["w"]
        g = torch.Generator(device="cuda").manual_seed(c["seed"])
        q, k, v = [torch.randn(B, H, N, d, device="cuda", generator=g).mul_(d ** -0.5).to(torch.bfloat16)
                   for _ in range(3)]
        o = torch.empty_like(q)
        byts = 4 * q.numel() * 2
        cells = []
        for h0 in (gf.default_h_sparse(H), H, H // 2, 0):
            ws = gf.Workspace.for_problem(B, H, N, d, w, h0)
            us = time_call(lambda: gf.hybrid_attn(q, k, v, w, h_sparse=h0, out=o, ws=ws), args.iters)
            if ws.last_device_status() != gf.GF_OK:
                raise SystemExit("device-side wait timed out")
            cells.append(us)
        frac = byts / (cells[0] * 1e-6) / 1e9 / args.peak_gbs
        print(f"| {N} | {B} | {d} | {w} | {cells[0]:.0f} | {frac:.2f} | {cells[1]:.0f} | {cells[2]:.0f} | {cells[3]:.0f} |",
              flush=True)


if __name__ == "__main__":
    main()
