"""CPU oracle for the activation-sparse gated FFN -- TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``sparse_ffn_oracle.cpp`` (plain C++, double accumulation) plus the
closed-form cost helpers of ``cost_model.py``.  Nothing in the CUDA package imports this module and
this module imports nothing from the CUDA package; only the tests, the smoke check and the
benchmark's CPU-baseline legs may use it.

Arrays cross the boundary as numpy arrays: fp32 (``float32``), bf16 (``uint16`` bit patterns) or
``float64``.  The helper :func:`as_oracle_array` converts torch CPU tensors without changing a bit.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

from .cost_model import (  # noqa: F401  (re-exported)
    adaptive_hidden_dim,
    fixed_matrix_dense,
    flop_ratio_lopa,
    flop_ratio_lopa_fixed_h,
    flop_ratio_standard,
    g_diagonal,
    g_padded_identity,
    g_tiled,
)

from . import lopa_cast  # noqa: F401,E402  (the LoPA approximation of Sec. 3.4)

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "sparse_ffn_oracle.cpp"
_LIB = _HERE / "build" / "libsparse_ffn_oracle.so"

ACT = {"relu": 0, "sqrelu": 1, "rsplus": 2, "silu": 3}  # silu: only as act_up (it is not sparse)
_DT = {np.dtype(np.float32): 0, np.dtype(np.uint16): 1, np.dtype(np.float64): 2}


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (no CUDA, no SIMD intrinsics, -O2, OpenMP over tokens only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        _LIB.parent.mkdir(exist_ok=True)
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", str(tmp), str(_SRC)],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        lib.oracle_activation.restype = ctypes.c_double
        lib.oracle_activation.argtypes = [ctypes.c_int, ctypes.c_double]
        lib.oracle_active_set.restype = ctypes.c_int
        lib.oracle_updown.restype = ctypes.c_int
        lib.oracle_ffn_batch.restype = ctypes.c_int
        lib.oracle_gate_standard.restype = None
        lib.oracle_gate_lopa.restype = None
        _lib = lib
    return _lib


def as_oracle_array(t) -> np.ndarray:
    """torch CPU tensor or numpy array -> contiguous numpy array the oracle decodes exactly."""
    if isinstance(t, np.ndarray):
        a = t
    else:
        import torch

        t = t.detach().cpu().contiguous()
        a = t.view(torch.uint16).numpy() if t.dtype == torch.bfloat16 else t.numpy()
    a = np.ascontiguousarray(a)
    if a.dtype not in _DT:
        raise TypeError(f"oracle takes float32, float64 or uint16 (bf16 bits), got {a.dtype}")
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _opt(a, dtype):
    if a is None:
        return None
    if not isinstance(a, np.ndarray):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, dtype=dtype)


def activation(act: str, z: float) -> float:
    """A(z) for one value (activation table of Sec. 3.1; squared RELU from the activation study)."""
    return float(_load().oracle_activation(ACT[act], float(z)))


def gate_standard(W1, x, b_g=None) -> np.ndarray:
    """z = W_1 x + b_g for one token (Eq. 1).  W1 [H,D], x [D]."""
    W1, x = as_oracle_array(W1), as_oracle_array(x)
    H, D = W1.shape
    assert x.shape == (D,)
    b = _opt(b_g, np.float32)
    z = np.empty(H, np.float64)
    _load().oracle_gate_standard(_p(W1), _DT[W1.dtype], _p(x), _DT[x.dtype], _p(b), H, D, _p(z))
    return z


def gate_lopa(V, U, x, g_idx=None, g_sign=None, gamma=None, use_rmsnorm=True, eps=1e-5, b_g=None,
              return_vn=False):
    """z = G x + U RMSNorm(V x) + b_g for one token (Eq. 3 and the practical form of Sec. 3.3)."""
    V, U, x = as_oracle_array(V), as_oracle_array(U), as_oracle_array(x)
    assert V.dtype == U.dtype
    r, D = V.shape
    H = U.shape[0]
    assert U.shape == (H, r) and x.shape == (D,)
    gi, gs = _opt(g_idx, np.int32), _opt(g_sign, np.int8)
    gm, b = _opt(gamma, np.float32), _opt(b_g, np.float32)
    z, v, n = np.empty(H, np.float64), np.empty(r, np.float64), np.empty(r, np.float64)
    _load().oracle_gate_lopa(_p(V), _p(U), _DT[V.dtype], _p(gi), _p(gs), _p(gm), int(use_rmsnorm),
                             ctypes.c_double(eps), r, _p(x), _DT[x.dtype], _p(b), H, D, _p(z),
                             _p(v), _p(n))
    return (z, v, n) if return_vn else z


def active_set(z) -> np.ndarray:
    """Ascending indices of the neurons with A(z_j) != 0, i.e. z_j > 0."""
    z = np.ascontiguousarray(z, np.float64)
    idx = np.empty(z.shape[0], np.int32)
    n = _load().oracle_active_set(_p(z), z.shape[0], _p(idx))
    return idx[:n].copy()


def ffn(x, W_up, W_down, act="relu", *, W_g=None, lopa=None, b_g=None, route="sparse", threads=1, act_up=None):
    """Gated FFN for a batch of independent tokens.

    x [B,D] (or [D]); W_up, W_down [H,D] (W_down = W_2 transposed); either ``W_g`` [H,D] or
    ``lopa`` = dict(V=[r,D], U=[H,r], g_idx=None|[H], g_sign=None|[H], gamma=None|[r],
    use_rmsnorm=bool, eps=float).  ``route`` is "dense" (all H neurons, Eq. 1) or "sparse"
    (only z_j > 0).  ``act_up`` names the activation A_3 on the output of W_3 (double activation,
    Sec. 3.3); None is Eq. 1.  Returns dict(y [B,D] f64, z [B,H] f64, n_act [B], n_gated [B] = number
    of neurons with a nonzero h_j, union_mask [H] bool).
    """
    x = as_oracle_array(x)
    single = x.ndim == 1
    if single:
        x = x[None, :]
    W_up, W_down = as_oracle_array(W_up), as_oracle_array(W_down)
    H, D = W_up.shape
    B = x.shape[0]
    assert W_down.shape == (H, D) and x.shape == (B, D) and W_down.dtype == W_up.dtype
    b = _opt(b_g, np.float32)
    y = np.zeros((B, D), np.float64)
    z = np.zeros((B, H), np.float64)
    n_act = np.zeros(B, np.int32)
    n_gated = np.zeros(B, np.int32)
    mask = np.zeros(H, np.uint8)
    W1 = V = U = gi = gs = gm = None
    kind, use_rms, eps, r = 0, 0, 0.0, 0
    if lopa is None:
        W1 = as_oracle_array(W_g)
        assert W1.shape == (H, D) and W1.dtype == W_up.dtype
    else:
        kind = 1
        V, U = as_oracle_array(lopa["V"]), as_oracle_array(lopa["U"])
        r = V.shape[0]
        assert V.shape == (r, D) and U.shape == (H, r) and V.dtype == U.dtype == W_up.dtype
        gi, gs = _opt(lopa.get("g_idx"), np.int32), _opt(lopa.get("g_sign"), np.int8)
        gm = _opt(lopa.get("gamma"), np.float32)
        use_rms, eps = int(lopa.get("use_rmsnorm", True)), float(lopa.get("eps", 1e-5))
    rc = _load().oracle_ffn_batch(
        kind, _p(W1), _p(V), _p(U), _p(gi), _p(gs), _p(gm), use_rms, ctypes.c_double(eps), r, _p(b),
        _p(W_up), _p(W_down), _DT[W_up.dtype], _p(x), _DT[x.dtype], B, H, D, ACT[act],
        -1 if act_up is None else ACT[act_up], {"dense": 0, "sparse": 1}[route], int(threads), _p(y), _p(z),
        _p(n_act), _p(n_gated), _p(mask))
    if rc != 0:
        raise ValueError("oracle_ffn_batch rejected its arguments")
    out = dict(y=y, z=z, n_act=n_act, n_gated=n_gated, union_mask=mask.astype(bool))
    if single:
        out["y"], out["z"] = y[0], z[0]
    return out


def dequantize_rows(q, scale) -> np.ndarray:
    """The matrix int8 codes stand for under weight-only quantisation with one scale per row (appendix on
    quantisation-aware training: only the weights are turned into int8, at inference time; the paper does not fix the
    granularity, one fp32 scale per output row is the reading taken here): W[j, k] = scale[j] * q[j, k], as float64."""
    if not isinstance(q, np.ndarray):
        q = q.detach().cpu().numpy()
    if not isinstance(scale, np.ndarray):
        scale = scale.detach().cpu().numpy()
    assert q.dtype == np.int8 and q.ndim == 2 and scale.shape == (q.shape[0],)
    return scale.astype(np.float64)[:, None] * q.astype(np.float64)


def dequantize_rows_q4(packed, scale) -> np.ndarray:
    """The matrix that 4-bit codes stand for (the same appendix also stores the weights on four bits and
    fixes no format; reading taken: symmetric two's-complement codes in [-8, 7], two per byte with the even column in
    the low nibble, one fp32 scale per row): W[j, 2b] = scale[j] * low(packed[j, b]), W[j, 2b + 1] = scale[j] *
    high(packed[j, b]), as float64.  ``packed`` is uint8 [rows, cols / 2]."""
    if not isinstance(packed, np.ndarray):
        packed = packed.detach().cpu().numpy()
    if not isinstance(scale, np.ndarray):
        scale = scale.detach().cpu().numpy()
    assert packed.dtype == np.uint8 and packed.ndim == 2 and scale.shape == (packed.shape[0],)
    rows, half = packed.shape
    q = np.empty((rows, 2 * half), np.float64)
    for part, nib in ((0, packed & 0x0F), (1, packed >> 4)):
        nib = nib.astype(np.int16)
        q[:, part::2] = np.where(nib >= 8, nib - 16, nib)   # two's complement on four bits
    return scale.astype(np.float64)[:, None] * q


def ffn_q4(x, W_up, W_down, act="relu", *, W_g=None, lopa=None, **kw):
    """:func:`ffn` on 4-bit weights: every matrix is a dict(q=uint8 [rows, cols / 2], s=fp32 [rows]) and enters Eq. 1
    as its float64 dequantisation (:func:`dequantize_rows_q4`); tokens stay in their own dtype (weight-only)."""
    dq = lambda m: dequantize_rows_q4(m["q"], m["s"])  # noqa: E731
    if lopa is not None:
        lopa = dict(lopa, V=dq(lopa["V"]), U=dq(lopa["U"]))
    return ffn(x, dq(W_up), dq(W_down), act, W_g=None if W_g is None else dq(W_g), lopa=lopa, **kw)


def ffn_q8(x, W_up, W_down, act="relu", *, W_g=None, lopa=None, **kw):
    """:func:`ffn` on int8 weights: every matrix is a dict(q=int8 [rows, cols], s=fp32 [rows]) and enters Eq. 1 as
    its float64 dequantisation (:func:`dequantize_rows`); tokens stay in their own dtype (weight-only)."""
    dq = lambda m: dequantize_rows(m["q"], m["s"])  # noqa: E731
    if lopa is not None:
        lopa = dict(lopa, V=dq(lopa["V"]), U=dq(lopa["U"]))
    return ffn(x, dq(W_up), dq(W_down), act, W_g=None if W_g is None else dq(W_g), lopa=lopa, **kw)
