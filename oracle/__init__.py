"""fp64 CPU oracle of the GFormer hybrid attention layer (TEST INFRASTRUCTURE ONLY).

Thin numpy/ctypes front end of ``gformer_oracle.c``: argument marshalling only, the
arithmetic is all in the C file.  Nothing here imports the CUDA package and the CUDA
package never imports this; tests, the smoke check and the benchmark's CPU-baseline
leg are the only callers.

All tensors are numpy float64, C-contiguous, laid out [B, H, N, d] (decode: [B, H, d]).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gformer_oracle.c")
_LIB = os.path.join(_HERE, "libgformer_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP across heads) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.gfo_num_threads.restype = ctypes.c_int
        _lib.gfo_phi.restype = ctypes.c_double
        _lib.gfo_phi.argtypes = [ctypes.c_double]
    return _lib


_dp = ctypes.POINTER(ctypes.c_double)


def _p(a):
    if a is None:
        return ctypes.cast(None, _dp)
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_dp)


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def num_threads() -> int:
    return int(_load().gfo_num_threads())


def phi(x):
    """phi(x) = elu(x) + 1, elementwise (Sec. II-B)."""
    x = _f64(x)
    y = np.empty_like(x)
    _load().gfo_phi_array(_p(x), _p(y), ctypes.c_long(x.size))
    return y


def phi_favor(x, W):
    """Positive random features of the vectors x [..., d] under the projection W [d, d] (rows w_a):
    exp(<w_a, x> - |x|^2 / 2) / sqrt(d)  (Sec. III-A / III-C; the formula is the cited Performer paper's)."""
    x, W = _f64(x), _f64(W)
    d = x.shape[-1]
    assert W.shape == (d, d)
    y = np.empty_like(x)
    xs, ys = x.reshape(-1, d), y.reshape(-1, d)
    lib = _load()
    for i in range(xs.shape[0]):
        lib.gfo_phi_favor(_p(xs[i]), _p(W), ctypes.c_int(d), _p(ys[i]))
    return y


def _proj(W, heads, d):
    """W [heads, d, d] (float64, contiguous) or None: the projection of the linear heads' feature map."""
    if W is None:
        return None
    W = _f64(W)
    assert W.shape == (heads, d, d), (W.shape, (heads, d, d))
    return W


def default_scale(d: int) -> float:
    """Eq. 1 divides the logits by sqrt(D)."""
    return 1.0 / float(np.sqrt(float(d)))


def default_h_sparse(H: int) -> int:
    """Number of windowed heads when the caller gives none: 3 of 16 heads is the
    causal optimum the paper reports (Sec. IV-D), rounded, at least one."""
    return max(1, int(np.floor(3.0 * H / 16.0 + 0.5)))


def window_attn(q, k, v, w: int, scale: float | None = None):
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, N, d = q.shape
    o = np.empty_like(q)
    s = default_scale(d) if scale is None else float(scale)
    _load().gfo_window_attn(_p(q), _p(k), _p(v), _p(o), ctypes.c_long(B), ctypes.c_long(H),
                            ctypes.c_long(N), ctypes.c_int(d), ctypes.c_long(w), ctypes.c_double(s))
    return o


def causal_linear_attn(q, k, v, S=None, z=None, W=None):
    """Returns o; if S [B,H,d,d] / z [B,H,d] are given they are the initial state and are
    overwritten in place with the final state.  W [H, d, d]: positive random features under these
    projections instead of elu + 1."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, N, d = q.shape
    o = np.empty_like(q)
    if (S is None) != (z is None):
        raise ValueError("give both S and z or neither")
    if S is not None:
        assert S.shape == (B, H, d, d) and z.shape == (B, H, d)
    _load().gfo_causal_linear_attn(_p(q), _p(k), _p(v), _p(o), ctypes.c_long(B), ctypes.c_long(H),
                                   ctypes.c_long(N), ctypes.c_int(d), _p(S), _p(z), _p(_proj(W, H, d)))
    return o


def hybrid_attn_self(q, k, v, w: int, h_sparse: int | None = None, scale: float | None = None, W=None):
    """The bidirectional ("self") layer: heads [0, h_sparse) see the keys with |i - j| < w,
    the others run global linear attention phi(Q)(phi(K)^T V) with row normalisation."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, N, d = q.shape
    h0 = default_h_sparse(H) if h_sparse is None else int(h_sparse)
    assert 0 <= h0 <= H
    s = default_scale(d) if scale is None else float(scale)
    o = np.empty_like(q)
    _load().gfo_hybrid_attn_self(_p(q), _p(k), _p(v), _p(o), ctypes.c_long(B), ctypes.c_long(H), ctypes.c_long(N),
                                 ctypes.c_int(d), ctypes.c_long(w), ctypes.c_long(h0), ctypes.c_double(s),
                                 _p(_proj(W, H - h0, d)))
    return o


def window_attn_self(q, k, v, w: int, scale: float | None = None):
    return hybrid_attn_self(q, k, v, w, h_sparse=np.asarray(q).shape[1], scale=scale)


def linear_attn_self(q, k, v, W=None):
    return hybrid_attn_self(q, k, v, 1, h_sparse=0, W=W)


class DecodeState:
    """Ring-buffer KV cache of the windowed heads plus (S, z) of the linear heads."""

    def __init__(self, B, H, d, w, h_sparse):
        self.B, self.H, self.d, self.w, self.h_sparse = B, H, d, w, h_sparse
        H1 = H - h_sparse
        self.k_cache = np.zeros((B, h_sparse, w, d))
        self.v_cache = np.zeros((B, h_sparse, w, d))
        self.S = np.zeros((B, H1, d, d))
        self.z = np.zeros((B, H1, d))
        self.t = 0
        self.W = None  # [H1, d, d]: projections of the positive random features, None: elu + 1


def hybrid_attn(q, k, v, w: int, h_sparse: int | None = None, scale: float | None = None,
                export_state: bool = False, W=None):
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, N, d = q.shape
    h0 = default_h_sparse(H) if h_sparse is None else int(h_sparse)
    assert 0 <= h0 <= H
    s = default_scale(d) if scale is None else float(scale)
    o = np.empty_like(q)
    st = DecodeState(B, H, d, w, h0) if export_state else None
    _load().gfo_hybrid_attn(
        _p(q), _p(k), _p(v), _p(o), ctypes.c_long(B), ctypes.c_long(H), ctypes.c_long(N),
        ctypes.c_int(d), ctypes.c_long(w), ctypes.c_long(h0), ctypes.c_double(s),
        _p(st.k_cache if st else None), _p(st.v_cache if st else None),
        _p(st.S if st else None), _p(st.z if st else None), _p(_proj(W, H - h0, d)))
    if st is not None:
        st.t = N
        st.W = _proj(W, H - h0, d)
        return o, st
    return o


def decode_step(q, k, v, st: DecodeState, scale: float | None = None):
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, d = q.shape
    assert (B, H, d) == (st.B, st.H, st.d)
    s = default_scale(d) if scale is None else float(scale)
    o = np.empty_like(q)
    _load().gfo_decode_step(
        _p(q), _p(k), _p(v), _p(o), _p(st.k_cache), _p(st.v_cache), _p(st.S), _p(st.z),
        ctypes.c_long(st.t), ctypes.c_long(B), ctypes.c_long(H), ctypes.c_int(d),
        ctypes.c_long(st.w), ctypes.c_long(st.h_sparse), ctypes.c_double(s), _p(_proj(st.W, H - st.h_sparse, d)))
    st.t += 1
    return o
