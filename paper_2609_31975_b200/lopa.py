"""Host helpers of the product side: fixed-matrix index generators for the LoPA gate and the
byte accounting used by the benchmark.  (No FFN arithmetic here; that lives in the CUDA kernels.)"""
from __future__ import annotations

import torch


def g_diagonal(H: int, D: int, device="cpu") -> torch.Tensor:
    """Repeated-diagonal fixed matrix G as an index array: row i has its 1 in column floor(i*D/H)
    (the paper's j = floor(i/k), k = H/D, written so that a non-integer k still hits every column)."""
    i = torch.arange(H, dtype=torch.int64, device=device)
    return torch.div(i * D, H, rounding_mode="floor").to(torch.int32)


def g_tiled(H: int, D: int, device="cpu") -> torch.Tensor:
    """Tiled-identity fixed matrix T as an index array: (Tx)_i = x_{i mod D}."""
    return (torch.arange(H, dtype=torch.int64, device=device) % D).to(torch.int32)


def touched_bytes(D: int, H: int, n_rows: int, esz: int, B: int = 1, r: int | None = None,
                  has_g_idx: bool = True, has_gain: bool = False) -> int:
    """Bytes one sparse call must read or write: the whole gate, the n_rows listed rows of W_up and
    W_down, the tokens, the gate bias and y.  Index lists, partial sums and re-reads of x are
    overhead and not counted."""
    if r is None:
        gate = H * D * esz
    else:
        gate = (r * D + H * r) * esz + (H * 4 if has_g_idx else 0) + (r * 4 if has_gain else 0)
    return gate + 2 * n_rows * D * esz + B * D * esz + H * 4 + B * D * 4


def dense_bytes(D: int, H: int, esz: int, B: int = 1, r: int | None = None) -> int:
    """Bytes of the dense comparator: as touched_bytes with all H rows."""
    return touched_bytes(D, H, H, esz, B, r)


def lopa_approximation(W: torch.Tensor, r: int, n_iter: int = 4) -> dict:
    """Architecture casting (Sec. 3.4, "LoPA approximation"): replaces a full gate matrix W [H, D] (fp32, on the GPU)
    by M + U V with one +-1 per row of M, minimising ||W - M - U V||_F^2 by alternating minimisation from U = V = 0,
    M-step first.  The row-wise and element-wise parts run in this library's kernels (``sffn_lopa_m_step``,
    ``sffn_lopa_residual``); the truncated SVD and the product U V are torch's (cuSOLVER / cuBLAS).

    Returns dict(g_idx int32 [H], g_sign int8 [H], U [H, r], V [r, D], trace): ``trace`` lists the objective after every
    half-step (M, UV, M, UV, ...).  Feed the result to ``sparse_ffn_forward`` as a LoPA gate with ``use_rmsnorm=False``
    (architecture casting has no RMSNorm between U and V), cast to the handle's dtype.
    """
    from .binding import lopa_m_step, lopa_residual

    W = W.contiguous().float()
    H, D = W.shape
    U = torch.zeros((H, r), dtype=torch.float32, device=W.device)
    V = torch.zeros((r, D), dtype=torch.float32, device=W.device)
    P = None
    trace = []
    for _ in range(n_iter):
        g_idx, g_sign, energy, best = lopa_m_step(W, P)
        trace.append(float((energy - 2.0 * best.double() + 1.0).sum()))
        A = lopa_residual(W, g_idx, g_sign)
        Pm, sv, Qt = torch.linalg.svd(A, full_matrices=False)
        U, V = (Pm[:, :r] * sv[:r]).contiguous(), Qt[:r].contiguous()
        P = U @ V
        _, _, energy, _ = lopa_m_step(A, P)      # || (W - M) - U V ||^2 row by row
        trace.append(float(energy.sum()))
    return dict(g_idx=g_idx, g_sign=g_sign, U=U, V=V, trace=trace)
