"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module only draws random numbers and rounds them to the storage dtype; it holds
none of the attention arithmetic, so both the CUDA path and the CPU oracle can be fed
from it without sharing any of the method's code.

Recipe (stands in for the activations of the paper's GPT-Neo-125M / ViT-base shaped
layers, which need datasets and trained weights): Q, K, V are drawn in that order from
one CPU generator as i.i.d. N(0,1) float32 tensors of shape [B, H, N, d], multiplied by
``gain`` (default d**-0.5) in float32, then rounded to the storage dtype (RNE).  The
oracle is given exactly the rounded values.
"""
from __future__ import annotations

import torch

# The five workload shapes of the benchmark contract (config index -> parameters).
CONFIGS = {
    "tiny": dict(B=1, H=2, N=256, d=64, w=32, dtype="f32", seed=0),
    "gpt2s": dict(B=8, H=12, N=2048, d=64, w=128, dtype="bf16", seed=1),
    "long32k": dict(B=1, H=32, N=32768, d=128, w=512, dtype="bf16", seed=2),
    "decode": dict(B=64, H=16, N=4096, d=64, w=256, dtype="bf16", seed=3, steps=256),
}


def sweep_points():
    """Config 5: 65 536 tokens per launch, H=16."""
    pts = []
    idx = 0
    for N in (1024, 4096, 16384, 65536):
        for d in (64, 128):
            for w in (64, 128, 256, 512):
                pts.append(dict(B=65536 // N, H=16, N=N, d=d, w=w, dtype="bf16", seed=4 + idx))
                idx += 1
    return pts


def torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def qkv(B, H, N, d, dtype="bf16", seed=0, gain=None, layout="bhnd"):
    """Returns (q, k, v) CPU tensors of the storage dtype, logically [B, H, N, d].

    With layout="bnhd" the same values are stored [B, N, H, d] and the returned tensors
    are the [B, N, H, d] arrays themselves."""
    g = torch.Generator(device="cpu").manual_seed(int(seed))
    gain = float(d) ** -0.5 if gain is None else float(gain)
    out = []
    for _ in range(3):
        x = torch.randn(B, H, N, d, generator=g, dtype=torch.float32) * gain
        x = x.to(torch_dtype(dtype))
        if layout == "bnhd":
            x = x.permute(0, 2, 1, 3).contiguous()
        out.append(x)
    return tuple(out)


def decode_tokens(steps, B, H, d, dtype="bf16", seed=0, gain=None):
    """Per-step (q, k, v) of shape [steps, B, H, d] for the decode workload."""
    g = torch.Generator(device="cpu").manual_seed(int(seed) + 7919)
    gain = float(d) ** -0.5 if gain is None else float(gain)
    out = []
    for _ in range(3):
        x = torch.randn(steps, B, H, d, generator=g, dtype=torch.float32) * gain
        out.append(x.to(torch_dtype(dtype)))
    return tuple(out)


def favor_projection(heads, d, seed=0, orthogonal=True, dtype="f32"):
    """Projection matrices W [heads, d, d] of the positive random feature map (rows = projection
    vectors): i.i.d. N(0,1) entries drawn from a CPU generator; with orthogonal=True the rows of
    every matrix are made orthogonal (QR of the Gaussian matrix) and given back the norms of
    independent Gaussian vectors, so that each row is still N(0, I) on its own.  Rounded to `dtype`.
    This is the random draw of the method, handed to it as an input."""
    g = torch.Generator(device="cpu").manual_seed(int(seed) + 104729)
    out = []
    for _ in range(heads):
        G = torch.randn(d, d, generator=g, dtype=torch.float64)
        if orthogonal:
            Q, _ = torch.linalg.qr(G.T)            # columns orthonormal -> rows of Q.T orthonormal
            norms = torch.randn(d, d, generator=g, dtype=torch.float64).norm(dim=1)
            # the factorisation fixes the signs of its columns: random signs make every row a
            # direction uniform on the sphere again
            signs = torch.where(torch.rand(d, generator=g, dtype=torch.float64) < 0.5, -1.0, 1.0)
            G = Q.T * (norms * signs)[:, None]
        out.append(G)
    return torch.stack(out).to(torch.float32).to(torch_dtype(dtype))
