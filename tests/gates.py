"""Parity gates shared by the GPU tests (oracle = fp64 reference on the same rounded inputs)."""
import numpy as np

# absolute gates of the benchmark contract + the stricter per-head relative L2 gate
GATES = {
    "bf16": dict(max_abs=2e-2, mean_abs=2e-3, rel_l2=1e-2),
    "f32": dict(max_abs=1e-4, mean_abs=1e-5, rel_l2=1e-5),
}


def errors(got, ref):
    """got, ref: arrays [B, H, N, d] (or [B, H, d]); returns dict of error measures."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    diff = got - ref
    axes = tuple(range(2, ref.ndim))
    num = np.sqrt((diff ** 2).sum(axis=axes))
    den = np.sqrt((ref ** 2).sum(axis=axes))
    rel = num / np.maximum(den, 1e-300)
    return dict(max_abs=float(np.abs(diff).max()), mean_abs=float(np.abs(diff).mean()),
                rel_l2=float(rel.max()), finite=bool(np.isfinite(got).all()))


def passes(got, ref, kind):
    e = errors(got, ref)
    g = GATES[kind]
    return e["finite"] and e["max_abs"] <= g["max_abs"] and e["mean_abs"] <= g["mean_abs"] and \
        e["rel_l2"] <= g["rel_l2"]


def assert_parity(got, ref, kind, what=""):
    e = errors(got, ref)
    g = GATES[kind]
    assert e["finite"], f"{what}: non-finite output"
    assert e["max_abs"] <= g["max_abs"], f"{what}: max abs {e['max_abs']:.3e} > {g['max_abs']:.1e} ({e})"
    assert e["mean_abs"] <= g["mean_abs"], f"{what}: mean abs {e['mean_abs']:.3e} > {g['mean_abs']:.1e} ({e})"
    assert e["rel_l2"] <= g["rel_l2"], f"{what}: rel L2 {e['rel_l2']:.3e} > {g['rel_l2']:.1e} ({e})"
    return e
