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
