"""B200-native hybrid attention (windowed softmax + causal linear) forward pass.

The arithmetic lives in libgformer.so (CUDA, sm_100a; C ABI in include/gformer.h);
``binding`` marshals torch tensors into it.
"""
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    DecodeState, GformerError, Workspace, causal_linear_attn, decode_step, default_h_sparse,
    hybrid_attn, set_tuning, window_attn,
)
