"""Oracle of the head-partition rule (TEST INFRASTRUCTURE ONLY).

Algorithm 2 (Sec. III-D) estimates the latency of two engines from the work a split ``p``
gives to each and looks for the split at which the two estimates meet; the FLOP model of
the same section instantiates it for the sparse (windowed) and the linear heads.  This
file takes those steps in the algorithm's order, in fp64, and finds the meeting point by
bisection and by exhaustive search: no closed form appears here, so that the closed forms
the library uses can be checked against it.

Pinned by hand-worked splits, mirror and scale invariants and the sign change of the latency
gap.  The section's own worked example (3 sparse heads of 16 at 4k tokens with rates of 13.37
and 2.31 TFLOP/s) is not what its printed formulas give with those rates (13 to 16 heads for any
window from 16 to 1024), so that example pins nothing: parity unpinned for the example.

Nothing here imports the CUDA package and the CUDA package never imports this.
"""
from __future__ import annotations


def latencies(p, size, flops_per0, flops_per1, perf0, perf1):
    """The two latency estimates of Algorithm 2 for a split p."""
    flops_p0 = p * size * flops_per0
    flops_p1 = (1.0 - p) * size * flops_per1
    latency0 = flops_p0 / perf0
    latency1 = flops_p1 / perf1
    return latency0, latency1


def balance(size, flops_per0, flops_per1, perf0, perf1, iters=200):
    """p' in [0, 1] with latency0 = latency1 (last step of Algorithm 2).

    latency0 - latency1 grows with p, is negative at p = 0 and positive at p = 1: bisect.
    """
    lo, hi = 0.0, 1.0
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        l0, l1 = latencies(mid, size, flops_per0, flops_per1, perf0, perf1)
        if l0 < l1:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def model_latencies(B, H, N, E, W, h_sparse, perf_sparse, perf_linear):
    """(sparse, linear) latency estimates of the FLOP model of Sec. III-D, as printed:

    linear heads  8 B N (H1 E)^2 / perf_linear   with H1 = H - h_sparse,
    sparse heads  5 B H0 N W / perf_sparse       with H0 = h_sparse.
    """
    h1 = H - h_sparse
    linear = 8.0 * B * N * float(h1 * E) ** 2 / perf_linear
    sparse = 5.0 * B * h_sparse * N * W / perf_sparse
    return sparse, linear


def partition_heads(B, H, N, E, W, perf_sparse, perf_linear):
    """Whole number of sparse heads whose two estimates are closest (smallest on a tie):
    every H0 in [0, H] is tried."""
    best_gap, best_h0 = None, 0
    for h0 in range(H + 1):
        s, l = model_latencies(B, H, N, E, W, h0, perf_sparse, perf_linear)
        gap = abs(s - l)
        if best_gap is None or gap < best_gap:
            best_gap, best_h0 = gap, h0
    return best_h0
