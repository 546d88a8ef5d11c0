"""Runs one entry point twice on random bf16 inputs (a small driver for profilers).

    python -m paper_2412_19829_b200.run_once {linear|window|hybrid|self} B H N d w

(`self`: the bidirectional layer with all heads linear, i.e. its three linear-attention kernels.)
"""
import sys

import torch

from . import binding as gf


def main(argv):
    kind = argv[0]
    B, H, N, d, w = [int(x) for x in argv[1:6]]
    g = torch.Generator(device="cuda").manual_seed(0)
    q, k, v = [torch.randn(B, H, N, d, device="cuda", generator=g).mul_(d ** -0.5).to(torch.bfloat16) for _ in range(3)]
    o = torch.empty_like(q)
    for _ in range(2):
        if kind == "linear":
            gf.causal_linear_attn(q, k, v, out=o)
        elif kind == "window":
            gf.window_attn(q, k, v, w, out=o)
        elif kind == "self":
            gf.hybrid_attn_self(q, k, v, w, h_sparse=0, out=o)
        else:
            gf.hybrid_attn(q, k, v, w, out=o)
    torch.cuda.synchronize()
    print("done")


if __name__ == "__main__":
    main(sys.argv[1:])
