"""Closed forms and fixed-matrix generators stated in the paper -- oracle side, TEST INFRASTRUCTURE.

Each function restates one formula; the tests pin them to the values the paper prints.
"""
from __future__ import annotations

import numpy as np


def flop_ratio_standard(s: float) -> float:
    """Dense cost 3HD over executed cost HD + 2(1-s)HD (Eq. 2 and the line after it): 3/(3-2s)."""
    return 3.0 / (3.0 - 2.0 * s)


def adaptive_hidden_dim(D: int, H: int, r: int) -> float:
    """H' with r(H'+D) + 2H'D = 3HD (Sec. 3.3, adaptive hidden dimension); not rounded."""
    return D * (3.0 * H - r) / (r + 2.0 * D)


def flop_ratio_lopa(s: float, D: float, H_prime: float, r: float) -> float:
    """Eq. 4: (r(D+H') + 2DH') / (r(D+H') + 2(1-s)DH'); the fixed matrix costs nothing."""
    gate = r * (D + H_prime)
    return (gate + 2.0 * D * H_prime) / (gate + 2.0 * (1.0 - s) * D * H_prime)


def flop_ratio_lopa_fixed_h(s: float, D: float, H: float, r: float) -> float:
    """Architecture casting (Sec. 3.4): H is kept, so the dense baseline 3HD is divided by the
    executed cost r(D+H) + 2(1-s)DH."""
    return 3.0 * H * D / (r * (D + H) + 2.0 * (1.0 - s) * D * H)


def g_diagonal(H: int, D: int) -> np.ndarray:
    """Column of the single 1 in each row of the repeated diagonal G: j = floor(i/k), k = H/D
    (appendix on the W_1 design).  Integer form floor(i*D/H), valid for non-integer k too."""
    i = np.arange(H, dtype=np.int64)
    return ((i * D) // H).astype(np.int32)


def g_tiled(H: int, D: int) -> np.ndarray:
    """Tiled identity T: (Tx)_i = x_{i mod D}."""
    return (np.arange(H, dtype=np.int64) % D).astype(np.int32)


def g_padded_identity(H: int, D: int) -> np.ndarray:
    """I_pad: identity on the first D rows, zero rows below (-1 marks a row with no nonzero).
    Not a LoPA matrix (some rows are empty); kept for the contrast the paper draws."""
    idx = np.full(H, -1, np.int32)
    idx[:D] = np.arange(D, dtype=np.int32)
    return idx


def fixed_matrix_dense(idx: np.ndarray, D: int, sign: np.ndarray | None = None) -> np.ndarray:
    """Materialise the H x D fixed matrix from its index form (rows with idx < 0 stay zero)."""
    H = idx.shape[0]
    M = np.zeros((H, D), np.float64)
    rows = np.nonzero(idx >= 0)[0]
    M[rows, idx[rows]] = 1.0 if sign is None else sign[rows].astype(np.float64)
    return M
