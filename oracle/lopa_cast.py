"""CPU oracle for the LoPA approximation of a full gate matrix (architecture casting) -- TEST INFRASTRUCTURE ONLY.

Sec. 3.4, "LoPA approximation": to replace W in R^{H x D} by M + U V with M in C (entries in {0, -1, +1}, exactly one
nonzero per row), U in R^{H x r}, V in R^{r x D}, minimise || W - M - U V ||_F^2 by alternating two exact half-steps,
starting from U = V = 0 with the M-step first:

  M-step (U, V fixed):  in every row of R = W - U V the +-1 goes to the entry of largest magnitude, with its sign;
  UV-step (M fixed):    U V is the truncated singular value decomposition of W - M at rank r.

Each half-step minimises the objective over its own block, so the objective never increases.  Plain numpy, float64.
"""
from __future__ import annotations

import numpy as np


def objective(W, g_idx, g_sign, U, V) -> float:
    """|| W - M - U V ||_F^2 with M[i, g_idx[i]] = g_sign[i]."""
    R = np.asarray(W, np.float64) - np.asarray(U, np.float64) @ np.asarray(V, np.float64)
    R[np.arange(R.shape[0]), g_idx] -= g_sign
    return float((R * R).sum())


def m_step(W, U, V):
    """Best M for fixed U, V: per row the position of the largest |R_ij| (first one on ties) and the sign of that entry
    (+1 for an exact zero).  Returns (g_idx int32 [H], g_sign int8 [H])."""
    R = np.asarray(W, np.float64) - np.asarray(U, np.float64) @ np.asarray(V, np.float64)
    g_idx = np.argmax(np.abs(R), axis=1).astype(np.int32)
    picked = R[np.arange(R.shape[0]), g_idx]
    g_sign = np.where(picked < 0, -1, 1).astype(np.int8)
    return g_idx, g_sign


def uv_step(W, g_idx, g_sign, r: int):
    """Best U V of rank <= r for fixed M: truncated SVD of W - M.  Returns (U [H, r] = left vectors times singular
    values, V [r, D] = right vectors)."""
    A = np.array(W, np.float64, copy=True)
    A[np.arange(A.shape[0]), g_idx] -= g_sign
    P, s, Qt = np.linalg.svd(A, full_matrices=False)
    return P[:, :r] * s[:r], Qt[:r]


def lopa_approximation(W, r: int, n_iter: int = 4):
    """Alternating minimisation from U = V = 0, M first.  Returns dict(g_idx, g_sign, U, V, trace) where trace lists the
    objective after every half-step (M, UV, M, UV, ...)."""
    W = np.asarray(W, np.float64)
    H, D = W.shape
    U, V = np.zeros((H, r)), np.zeros((r, D))
    trace = []
    for _ in range(n_iter):
        g_idx, g_sign = m_step(W, U, V)
        trace.append(objective(W, g_idx, g_sign, U, V))
        U, V = uv_step(W, g_idx, g_sign, r)
        trace.append(objective(W, g_idx, g_sign, U, V))
    return dict(g_idx=g_idx, g_sign=g_sign, U=U, V=V, trace=trace)
