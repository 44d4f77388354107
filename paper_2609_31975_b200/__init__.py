"""B200-native activation-sparse gated FFN (hand-written CUDA for sm_100a behind a C ABI).

This package is a thin binding: argument marshalling over ``libsparse_ffn.so``.  Every step of the
FFN runs in the library's kernels; there is no CPU or PyTorch fallback, and importing the binding
without the built library raises.
"""
from .binding import (  # noqa: F401
    ACT,
    PATH,
    SFFNError,
    SparseFFN,
    lib_path,
    load_library,
    residual_cast,
    sparse_ffn_forward_static,
    test_set_knob,
)
from .lopa import g_diagonal, g_tiled, touched_bytes, dense_bytes, lopa_approximation  # noqa: F401
