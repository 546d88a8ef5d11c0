"""ctypes binding of libgformer.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the attention path runs in the
library's kernels.  There is no CPU fallback: if the shared library is missing or a call
returns a non-zero status, a GformerError is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

GF_OK, GF_ERR_INVALID_ARG, GF_ERR_UNSUPPORTED, GF_ERR_WORKSPACE, GF_ERR_CUDA, GF_ERR_TIMEOUT = range(6)
GF_F32, GF_BF16 = 0, 1
GF_BHND, GF_BNHD = 0, 1
GF_PHI_ELU1, GF_PHI_FAVOR_POS = 0, 1
GF_TUNE_FORCE_SIMT, GF_TUNE_LINEAR_SPLIT, GF_TUNE_LINEAR_CTAS, GF_TUNE_WAIT_KCYCLES, GF_TUNE_TEST_DROP_FLAG = 0, 1, 2, 3, 4

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgformer.so")


class GformerError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


class DecodeStateC(ctypes.Structure):
    _fields_ = [("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
                ("S", ctypes.c_void_p), ("z", ctypes.c_void_p), ("t", ctypes.c_longlong),
                ("B", ctypes.c_int), ("H", ctypes.c_int), ("d", ctypes.c_int), ("w", ctypes.c_int),
                ("h_sparse", ctypes.c_int), ("dtype", ctypes.c_int)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libgformer.so (built in-tree by paper_2412_19829_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is not built; run `python -m paper_2412_19829_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.gformer_status_string.restype = ctypes.c_char_p
        L.gformer_status_string.argtypes = [i]
        L.gformer_version.restype = i
        L.gformer_launch_count.restype = ctypes.c_ulonglong
        L.gformer_default_h_sparse.restype = i
        L.gformer_default_h_sparse.argtypes = [i]
        L.gformer_set_tuning.restype = i
        L.gformer_set_tuning.argtypes = [i, i]
        L.gformer_linear_plan.restype = i
        L.gformer_linear_plan.argtypes = [i, i, i, i, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
        dbl, pdbl = ctypes.c_double, ctypes.POINTER(ctypes.c_double)
        L.gformer_partition_balance.restype = i
        L.gformer_partition_balance.argtypes = [dbl, dbl, dbl, dbl, pdbl]
        L.gformer_partition_from_times.restype = i
        L.gformer_partition_from_times.argtypes = [i, i, i, i, i, dbl, dbl, pdbl, ctypes.POINTER(ctypes.c_int), pdbl, pdbl]
        L.gformer_partition_heads.restype = i
        L.gformer_partition_heads.argtypes = [i, i, i, i, i, dbl, dbl, ctypes.POINTER(ctypes.c_int), pdbl, pdbl]
        pint = ctypes.POINTER(ctypes.c_int)
        L.gformer_linear_plan_parts.restype = i
        L.gformer_linear_plan_parts.argtypes = [i, i, i, i, pint, pint, pint]
        L.gformer_workspace_bytes.restype = sz
        L.gformer_workspace_bytes.argtypes = [i] * 7
        L.gformer_workspace_bytes_phi.restype = sz
        L.gformer_workspace_bytes_phi.argtypes = [i] * 8
        L.gformer_causal_linear_attn_w.restype = i
        L.gformer_causal_linear_attn_w.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp, i, vp, vp, i, i, vp, sz, vp]
        L.gformer_hybrid_attn_w.restype = i
        L.gformer_hybrid_attn_w.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, f, i, vp, i, i, i,
                                            ctypes.POINTER(DecodeStateC), vp, sz, vp]
        L.gformer_hybrid_attn_self_w.restype = i
        L.gformer_hybrid_attn_self_w.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, f, i, vp, i, i, vp, sz, vp]
        L.gformer_decode_step_w.restype = i
        L.gformer_decode_step_w.argtypes = [vp, vp, vp, vp, ctypes.POINTER(DecodeStateC), f, i, vp, vp]
        L.gformer_last_device_status.restype = i
        L.gformer_last_device_status.argtypes = [vp, vp]
        L.gformer_window_attn.restype = i
        L.gformer_window_attn.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, i, i, vp, sz, vp]
        L.gformer_window_attn_self.restype = i
        L.gformer_window_attn_self.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, i, i, vp, sz, vp]
        L.gformer_hybrid_attn_self.restype = i
        L.gformer_hybrid_attn_self.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, f, i, i, i, vp, sz, vp]
        L.gformer_causal_linear_attn.restype = i
        L.gformer_causal_linear_attn.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, vp, i, i, vp, sz, vp]
        L.gformer_noalloc_scratch_bytes.restype = sz
        L.gformer_noalloc_last_device_status.restype = i
        L.gformer_noalloc_last_device_status.argtypes = [vp]
        L.gformer_causal_linear_attn_noalloc.restype = i
        L.gformer_causal_linear_attn_noalloc.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp, vp, i, i, vp]
        L.gformer_hybrid_attn.restype = i
        L.gformer_hybrid_attn.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, f, i, i, i, i,
                                          ctypes.POINTER(DecodeStateC), vp, sz, vp]
        L.gformer_decode_step.restype = i
        L.gformer_decode_step.argtypes = [vp, vp, vp, vp, ctypes.POINTER(DecodeStateC), f, i, vp]
        L.gformer_decode_step_ragged.restype = i
        L.gformer_decode_step_ragged.argtypes = [vp, vp, vp, vp, ctypes.POINTER(DecodeStateC), vp, f, i, vp]
        L.gformer_decode_step_ragged_w.restype = i
        L.gformer_decode_step_ragged_w.argtypes = [vp, vp, vp, vp, ctypes.POINTER(DecodeStateC), vp, f, i, vp, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().gformer_status_string(int(status)).decode()


def version() -> int:
    return int(lib().gformer_version())


def launch_count() -> int:
    return int(lib().gformer_launch_count())


def default_h_sparse(H: int) -> int:
    return int(lib().gformer_default_h_sparse(int(H)))


def set_tuning(key: int, value: int) -> None:
    rc = lib().gformer_set_tuning(int(key), int(value))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_set_tuning")


def linear_plan(chains: int, N: int, d: int, ctas: int = 0):
    """(segments per chain, chunks of the longest segment) the linear kernel would use."""
    g, l = ctypes.c_int(0), ctypes.c_int(0)
    rc = lib().gformer_linear_plan(int(chains), int(N), int(d), int(ctas), ctypes.byref(g), ctypes.byref(l))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_linear_plan")
    return g.value, l.value


def linear_plan_parts(chains: int, N: int, d: int, ctas: int = 0):
    """(chains left whole, segments per cut chain, chunks of the longest segment)."""
    wh, g, l = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    rc = lib().gformer_linear_plan_parts(int(chains), int(N), int(d), int(ctas), ctypes.byref(wh), ctypes.byref(g),
                                         ctypes.byref(l))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_linear_plan_parts")
    return wh.value, g.value, l.value


def partition_balance(flops_per0: float, flops_per1: float, perf0: float, perf1: float) -> float:
    """Share of the problem for engine 0 at which the two latency estimates of Algorithm 2 meet."""
    p = ctypes.c_double(0.0)
    rc = lib().gformer_partition_balance(float(flops_per0), float(flops_per1), float(perf0), float(perf1),
                                         ctypes.byref(p))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_partition_balance")
    return p.value


def partition_from_times(B: int, H: int, N: int, E: int, W: int, seconds_per_sparse_head: float,
                         seconds_per_linear_head: float):
    """(p', balanced head count, perf_sparse, perf_linear) from measured seconds per head (gformer_partition_from_times)."""
    p, h0 = ctypes.c_double(0.0), ctypes.c_int(0)
    ps, pl = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = lib().gformer_partition_from_times(int(B), int(H), int(N), int(E), int(W), float(seconds_per_sparse_head),
                                            float(seconds_per_linear_head), ctypes.byref(p), ctypes.byref(h0),
                                            ctypes.byref(ps), ctypes.byref(pl))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_partition_from_times")
    return p.value, h0.value, ps.value, pl.value


def partition_heads(B: int, H: int, N: int, E: int, W: int, perf_sparse: float, perf_linear: float):
    """(windowed heads, sparse latency, linear latency) of the FLOP model of Sec. III-D."""
    h0, ls, ll = ctypes.c_int(0), ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = lib().gformer_partition_heads(int(B), int(H), int(N), int(E), int(W), float(perf_sparse),
                                       float(perf_linear), ctypes.byref(h0), ctypes.byref(ls), ctypes.byref(ll))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_partition_heads")
    return h0.value, ls.value, ll.value


def workspace_bytes(B, H, N, d, w, h_sparse, dtype, phi: int = GF_PHI_ELU1) -> int:
    return int(lib().gformer_workspace_bytes_phi(B, H, N, d, w, h_sparse, dtype, phi))


def _phi_args(W, q, heads, d):
    """(phi, pointer) of the linear heads' feature map: W None = elu + 1, else the projections [heads, d, d]
    of the positive random features, a contiguous CUDA tensor of q's dtype."""
    if W is None:
        return GF_PHI_ELU1, None
    if not (W.is_cuda and W.is_contiguous() and W.dtype == q.dtype and tuple(W.shape) == (heads, d, d)):
        raise ValueError(f"W must be a contiguous CUDA tensor [{heads}, {d}, {d}] of dtype {q.dtype}")
    return GF_PHI_FAVOR_POS, W.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GF_F32
    if t.dtype == torch.bfloat16:
        return GF_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _check_qkv(q, k, v):
    for t in (q, k, v):
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("q, k, v must be contiguous CUDA tensors")
        if t.shape != q.shape or t.dtype != q.dtype:
            raise ValueError("q, k, v must agree in shape and dtype")


def _dims(q, layout):
    if q.dim() != 4:
        raise ValueError("expected a 4-D tensor")
    if layout == GF_BNHD:
        B, N, H, d = q.shape
    else:
        B, H, N, d = q.shape
    return int(B), int(H), int(N), int(d)


class Workspace:
    """Caller-owned device scratch for the attention entry points."""

    def __init__(self, nbytes: int = 256, device=None):
        self.buf = torch.empty(max(int(nbytes), 256) + 256, dtype=torch.uint8,
                               device=device if device is not None else "cuda")
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        self.nbytes = self.buf.numel() - off

    @classmethod
    def for_problem(cls, B, H, N, d, w=1, h_sparse=0, dtype=GF_BF16, device=None, phi=GF_PHI_ELU1):
        """Scratch sized by gformer_workspace_bytes_phi for this problem."""
        return cls(workspace_bytes(B, H, N, d, w, h_sparse, dtype, phi), device)

    def last_device_status(self, stream=None) -> int:
        return int(lib().gformer_last_device_status(self.ptr, _stream_ptr(stream)))


_default_ws: dict = {}


def _ws_for(t: torch.Tensor, ws, need: int) -> Workspace:
    if ws is not None:
        return ws
    key = t.device.index
    cur = _default_ws.get(key)
    if cur is None or cur.nbytes < need:
        cur = Workspace(need, t.device)
        _default_ws[key] = cur
    return cur


def window_attn(q, k, v, w: int, scale: float = 0.0, layout: int = GF_BHND, out=None, ws=None, stream=None):
    """gformer_window_attn: causal softmax attention over the w most recent keys."""
    _check_qkv(q, k, v)
    B, H, N, d = _dims(q, layout)
    o = torch.empty_like(q) if out is None else out
    dt = _dtype_code(q)
    W = _ws_for(q, ws, workspace_bytes(B, H, N, d, w, H, dt))
    rc = lib().gformer_window_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, int(w),
                                   float(scale), dt, layout, W.ptr, W.nbytes, _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_window_attn")
    return o


def window_attn_self(q, k, v, w: int, scale: float = 0.0, layout: int = GF_BHND, out=None, ws=None, stream=None):
    """gformer_window_attn_self: softmax attention over the keys with |i - j| < w (no causal mask)."""
    _check_qkv(q, k, v)
    B, H, N, d = _dims(q, layout)
    o = torch.empty_like(q) if out is None else out
    dt = _dtype_code(q)
    W = _ws_for(q, ws, workspace_bytes(B, H, N, d, w, H, dt))
    rc = lib().gformer_window_attn_self(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, int(w),
                                        float(scale), dt, layout, W.ptr, W.nbytes, _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_window_attn_self")
    return o


def hybrid_attn_self(q, k, v, w: int, h_sparse: int = -1, scale: float = 0.0, layout: int = GF_BHND, out=None,
                     ws=None, stream=None, W=None):
    """gformer_hybrid_attn_self(_w): the bidirectional layer (two-sided windowed heads, global linear heads).
    W [H - h_sparse, d, d]: positive random features under these projections instead of elu + 1."""
    _check_qkv(q, k, v)
    B, H, N, d = _dims(q, layout)
    o = torch.empty_like(q) if out is None else out
    dt = _dtype_code(q)
    h0 = default_h_sparse(H) if h_sparse < 0 else h_sparse
    phi, wp = _phi_args(W, q, H - h0, d)
    wsp = _ws_for(q, ws, workspace_bytes(B, H, N, d, w, h_sparse, dt, phi))
    rc = lib().gformer_hybrid_attn_self_w(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, int(w),
                                          int(h_sparse), float(scale), phi, wp, dt, layout, wsp.ptr, wsp.nbytes,
                                          _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_hybrid_attn_self_w")
    return o


def causal_linear_attn(q, k, v, S=None, z=None, chunk: int = 0, layout: int = GF_BHND, out=None, ws=None,
                       stream=None, W=None):
    """gformer_causal_linear_attn(_w): Algorithm 1 with phi = elu + 1, or with the positive random features
    under the projections W [H, d, d]; S, z (fp32) updated in place."""
    _check_qkv(q, k, v)
    B, H, N, d = _dims(q, layout)
    o = torch.empty_like(q) if out is None else out
    dt = _dtype_code(q)
    if S is not None:
        assert S.dtype == torch.float32 and S.is_contiguous() and tuple(S.shape) == (B, H, d, d)
        assert z.dtype == torch.float32 and z.is_contiguous() and tuple(z.shape) == (B, H, d)
    phi, wp = _phi_args(W, q, H, d)
    wsp = _ws_for(q, ws, workspace_bytes(B, H, N, d, 1, 0, dt, phi))
    rc = lib().gformer_causal_linear_attn_w(
        q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, phi, wp, int(chunk),
        S.data_ptr() if S is not None else None, z.data_ptr() if z is not None else None,
        dt, layout, wsp.ptr, wsp.nbytes, _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_causal_linear_attn_w")
    return o


def causal_linear_attn_noalloc(q, k, v, out, S=None, z=None, chunk: int = 0, layout: int = GF_BHND, stream=None):
    """gformer_causal_linear_attn_noalloc: same result as causal_linear_attn, but the kernel's scratch
    is the fixed array inside the library, so nothing is allocated here or there.  The caller brings
    the output tensor; problems whose scratch exceeds the array raise GformerError(GF_ERR_WORKSPACE)."""
    _check_qkv(q, k, v)
    B, H, N, d = _dims(q, layout)
    rc = lib().gformer_causal_linear_attn_noalloc(
        q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), B, H, N, d, GF_PHI_ELU1, int(chunk),
        S.data_ptr() if S is not None else None, z.data_ptr() if z is not None else None,
        _dtype_code(q), layout, _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_causal_linear_attn_noalloc")
    return out


class DecodeState:
    """Device buffers of the decode state (ring KV cache, S, z) plus the host-side struct."""

    def __init__(self, B, H, d, w, h_sparse, dtype=torch.bfloat16, device="cuda"):
        H1 = H - h_sparse
        self.k_cache = torch.zeros(B, max(h_sparse, 1), w, d, dtype=dtype, device=device)
        self.v_cache = torch.zeros(B, max(h_sparse, 1), w, d, dtype=dtype, device=device)
        self.S = torch.zeros(B, max(H1, 1), d, d, dtype=torch.float32, device=device)
        self.z = torch.zeros(B, max(H1, 1), d, dtype=torch.float32, device=device)
        self.c = DecodeStateC(self.k_cache.data_ptr(), self.v_cache.data_ptr(), self.S.data_ptr(),
                              self.z.data_ptr(), 0, B, H, d, w, h_sparse,
                              GF_F32 if dtype == torch.float32 else GF_BF16)

    @property
    def t(self) -> int:
        return int(self.c.t)

    @t.setter
    def t(self, value: int):
        self.c.t = int(value)


def hybrid_attn(q, k, v, w: int, h_sparse: int = -1, scale: float = 0.0, chunk: int = 0,
                layout: int = GF_BHND, state_out: DecodeState | None = None, out=None, ws=None, stream=None, W=None):
    """gformer_hybrid_attn(_w): heads [0, h_sparse) windowed, the rest linear, merged by head.
    W [H - h_sparse, d, d]: positive random features under these projections instead of elu + 1."""
    _check_qkv(q, k, v)
    B, H, N, d = _dims(q, layout)
    o = torch.empty_like(q) if out is None else out
    dt = _dtype_code(q)
    h0 = default_h_sparse(H) if h_sparse < 0 else h_sparse
    phi, wp = _phi_args(W, q, H - h0, d)
    wsp = _ws_for(q, ws, workspace_bytes(B, H, N, d, w, h_sparse, dt, phi))
    rc = lib().gformer_hybrid_attn_w(
        q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, int(w), int(h_sparse), float(scale),
        phi, wp, int(chunk), dt, layout, ctypes.byref(state_out.c) if state_out is not None else None,
        wsp.ptr, wsp.nbytes, _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_hybrid_attn_w")
    return o


def decode_step(q, k, v, st: DecodeState, scale: float = 0.0, out=None, stream=None, W=None):
    """gformer_decode_step(_w): q, k, v are [B, H, d]; st is advanced by one token.  W as in hybrid_attn."""
    for t in (q, k, v):
        if not (t.is_cuda and t.is_contiguous() and t.dim() == 3):
            raise ValueError("q, k, v must be contiguous [B, H, d] CUDA tensors")
    o = torch.empty_like(q) if out is None else out
    phi, wp = _phi_args(W, q, st.c.H - st.c.h_sparse, st.c.d)
    rc = lib().gformer_decode_step_w(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), ctypes.byref(st.c),
                                     float(scale), phi, wp, _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_decode_step_w")
    return o


def decode_step_ragged(q, k, v, st: DecodeState, t_seq: torch.Tensor, scale: float = 0.0, out=None, stream=None,
                       W=None):
    """gformer_decode_step_ragged(_w): sequence b of the batch is at position t_seq[b] (int64 CUDA
    tensor of B entries, negative = idle slot); the positions are advanced on the device.  W as in hybrid_attn."""
    for t in (q, k, v):
        if not (t.is_cuda and t.is_contiguous() and t.dim() == 3):
            raise ValueError("q, k, v must be contiguous [B, H, d] CUDA tensors")
    if not (t_seq.is_cuda and t_seq.dtype == torch.int64 and t_seq.is_contiguous() and t_seq.numel() == q.shape[0]):
        raise ValueError("t_seq must be a contiguous int64 CUDA tensor with one entry per sequence")
    o = torch.empty_like(q) if out is None else out
    phi, wp = _phi_args(W, q, st.c.H - st.c.h_sparse, st.c.d)
    rc = lib().gformer_decode_step_ragged_w(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                            ctypes.byref(st.c), t_seq.data_ptr(), float(scale), phi, wp,
                                            _stream_ptr(stream))
    if rc != GF_OK:
        raise GformerError(rc, "gformer_decode_step_ragged_w")
    return o
