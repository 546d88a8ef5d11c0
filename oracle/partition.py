"""Oracle of the head-partition rule (TEST INFRASTRUCTURE ONLY).

Algorithm 2 (Sec. III-D) estimates the latency of two engines from the work a split ``p``
gives to each and looks for the split at which the two estimates meet; the FLOP model of
the same section instantiates it for the sparse (windowed) and the linear heads.  This
file restates the rule as one function, the gap between the two estimates, in fp64, and finds
its zero by bisection and the best whole number of heads by exhaustive search: no closed form
appears here, so that the closed forms the library uses can be checked against it.

Pinned by hand-worked splits, mirror and scale invariants and the sign change of the latency
gap.  The section's own worked example (3 sparse heads of 16 at 4k tokens with rates of 13.37
and 2.31 TFLOP/s) is not what its printed formulas give with those rates (13 to 16 heads for any
window from 16 to 1024), so that example pins nothing: parity unpinned for the example.

Nothing here imports the CUDA package and the CUDA package never imports this.
"""
from __future__ import annotations


def gap(p, size, work0, work1, rate0, rate1):
    """Time engine 0 needs for the share p of the problem minus the time engine 1 needs for the
    rest (Algorithm 2, Sec. III-D: work per unit over rate, times the units each engine gets).
    Negative while engine 0 would finish first."""
    return p * size * work0 / rate0 - (1.0 - p) * size * work1 / rate1


def latencies(p, size, work0, work1, rate0, rate1):
    """The two finishing times whose difference `gap` is: engine 0 on the share p, engine 1 on the rest."""
    return gap(p, size, work0, 0.0, rate0, 1.0), -gap(p, size, 0.0, work1, 1.0, rate1)


def balance(size, work0, work1, rate0, rate1, iters=200):
    """The share p' in [0, 1] at which both engines finish together (Algorithm 2).

    The gap grows with p, is negative at p = 0 and positive at p = 1: bisect on its sign.
    """
    lo, hi = 0.0, 1.0
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        if gap(mid, size, work0, work1, rate0, rate1) < 0.0:
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
