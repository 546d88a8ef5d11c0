"""Number of windowed heads by the balance rule of Algorithm 2, from micro-benchmarks on this GPU.

    python -m paper_2412_19829_b200.partition [--B 1 --H 32 --N 32768 --d 128 --w 512] [--self-layer]

Two micro-benchmarks (every head windowed; every head linear) give the seconds one head of each
kind costs at this problem size.  Algorithm 2, with those as the work per unit and unit rates,
gives the share p' of heads at which both kinds take equally long; the nearest whole number of
heads is reported, with the layer's measured time there.  The FLOP model of Sec. III-D is
evaluated beside it with the rates the micro-benchmarks imply.

On a B200 both kinds of heads run on the same SMs (side by side, not on two engines), so a layer
takes about the sum of its two parts and the balanced split gives each kind half of that time: it
is not the fastest split (that is simply every head of the cheaper kind), and the head split stays
a model-quality choice (Sec. IV-D).  This tool reports what the rule gives.

Inputs are seeded Gaussians generated on the device (timing only)."""
import argparse
import json

import numpy as np
import torch

from . import binding as gf


def time_call(fn, iters, warm=3):
    """Median microseconds of `iters` calls (CUDA events on the current stream, after `warm` calls)."""
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


def measure(B, H, N, d, w, self_layer=False, iters=5, seed=0):
    """Seconds per windowed head and per linear head, the balanced split, the layer's time there."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    q, k, v = [torch.randn(B, H, N, d, device="cuda", generator=g).mul_(d ** -0.5).to(torch.bfloat16) for _ in range(3)]
    o = torch.empty_like(q)
    layer = gf.hybrid_attn_self if self_layer else gf.hybrid_attn

    def layer_us(h0):
        ws = gf.Workspace.for_problem(B, H, N, d, w, h0)
        us = time_call(lambda: layer(q, k, v, w, h_sparse=h0, out=o, ws=ws), iters)
        if ws.last_device_status() != gf.GF_OK:
            raise RuntimeError("device-side wait timed out")
        return us

    t_window = layer_us(H) * 1e-6 / H  # every head windowed
    t_linear = layer_us(0) * 1e-6 / H  # every head linear
    # Algorithm 2 on the measured times, and the section's FLOP model with the rates they imply
    p, h0, perf_sparse, perf_linear = gf.partition_from_times(B, H, N, d, w, t_window, t_linear)
    h0_model, lat_s, lat_l = gf.partition_heads(B, H, N, d, w, perf_sparse, perf_linear)
    return {"B": B, "H": H, "N": N, "d": d, "w": w, "layer": "self" if self_layer else "causal",
            "s_per_window_head": t_window, "s_per_linear_head": t_linear, "p_balanced": p, "h_sparse_balanced": h0,
            "layer_us_at_balanced": layer_us(h0), "layer_us_all_window": t_window * H * 1e6,
            "layer_us_all_linear": t_linear * H * 1e6, "flop_model": {"h_sparse": h0_model, "latency_sparse_s": lat_s,
                                                                      "latency_linear_s": lat_l}}


def main():
    ap = argparse.ArgumentParser()
    for name, default in (("B", 1), ("H", 32), ("N", 32768), ("d", 128), ("w", 512), ("iters", 5)):
        ap.add_argument("--" + name, type=int, default=default)
    ap.add_argument("--self-layer", action="store_true", help="the bidirectional layer instead of the causal one")
    a = ap.parse_args()
    print(json.dumps(measure(a.B, a.H, a.N, a.d, a.w, self_layer=a.self_layer, iters=a.iters)))


if __name__ == "__main__":
    main()
