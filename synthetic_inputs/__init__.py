"""Seeded synthetic inputs for the activation-sparse gated FFN.

Data only: this module draws weights, tokens and gate biases with the shapes and distributions of
the benchmark configurations.  It holds none of the FFN's arithmetic and is the one module that
both the CPU oracle's tests and the CUDA path's tests/benchmarks may share.  A tensor drawn here is
handed to both sides unchanged (the oracle receives a host copy of the very same bits), so the two
never depend on a generator behaving identically on two devices.

Recipe (all configurable):
  weights  W ~ N(0, 1/fan_in) drawn in fp32 then rounded to the storage dtype (bf16: round to
           nearest even by ``Tensor.to``);  tokens x ~ N(0, 1), same rounding;
  gate bias b_g = -Phi^-1(s) * sigma_z, the constant that makes a N(0, sigma_z^2) pre-activation
           negative with probability s;  or a per-neuron bias from a Zipf firing profile.
  int8 weights (weight-only quantisation): codes drawn directly, q = clip(round(N(0, 32^2)), +-127), which is
           what an abs-max quantiser leaves of a Gaussian row of a few thousand entries (max ~ 4 sigma), and
           one fp32 scale per row, s_j = std / 32 * (1 + 0.1 u_j), u_j ~ U(-1, 1); the matrix the codes stand
           for is s_j * q[j, :].  Nothing is quantised here, so no rounding rule is shared with either side.
"""
from __future__ import annotations

import math

import torch

_TAGS = {"W_g": 1, "W_up": 2, "W_down": 3, "V": 4, "U": 5, "x": 6, "perm": 7, "scale": 8}


def _gen(seed: int, tag: str, device, extra: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1_000_003 + _TAGS[tag]) * 1_000_003 + int(extra))
    return g


def normal_quantile(p: float) -> float:
    """Phi^-1(p) of the standard normal."""
    return math.sqrt(2.0) * float(torch.erfinv(torch.tensor(2.0 * p - 1.0, dtype=torch.float64)))


def gate_bias_for_sparsity(s: float, sigma_z: float = 1.0) -> float:
    """Constant gate bias giving P(z <= 0) = s when z - b_g ~ N(0, sigma_z^2)."""
    return -normal_quantile(s) * sigma_z


def normal_tensor(shape, std: float, dtype, seed: int, tag: str, device="cpu", extra: int = 0,
                  chunk_rows: int = 4096) -> torch.Tensor:
    """N(0, std^2) tensor of ``dtype``; drawn in fp32 row-chunks so large matrices need no big temp."""
    out = torch.empty(shape, dtype=dtype, device=device)
    g = _gen(seed, tag, device, extra)
    flat = out.view(shape[0], -1) if len(shape) > 1 else out.view(1, -1)
    for r0 in range(0, flat.shape[0], chunk_rows):
        r1 = min(flat.shape[0], r0 + chunk_rows)
        blk = torch.randn((r1 - r0, flat.shape[1]), generator=g, device=device, dtype=torch.float32)
        flat[r0:r1] = (blk * std).to(dtype)
    return out


def tokens(n: int, D: int, dtype, seed: int, device="cpu", extra: int = 0) -> torch.Tensor:
    """n independent tokens x ~ N(0, 1), [n, D]."""
    return normal_tensor((n, D), 1.0, dtype, seed, "x", device, extra)


def standard_ffn(D: int, H: int, dtype, seed: int, device="cpu", sparsity: float | None = 0.9,
                 extra: int = 0) -> dict:
    """Standard-gated FFN weights: W_g, W_up, W_down [H,D] ~ N(0, 1/D); b_g [H] fp32 constant."""
    std = 1.0 / math.sqrt(D)
    w = {k: normal_tensor((H, D), std, dtype, seed, k, device, extra) for k in ("W_g", "W_up", "W_down")}
    w["b_g"] = None if sparsity is None else torch.full(
        (H,), gate_bias_for_sparsity(sparsity), dtype=torch.float32, device=device)
    return w


def lopa_ffn(D: int, H: int, r: int, dtype, seed: int, device="cpu", sparsity: float | None = 0.9,
             with_fixed_matrix: bool = True, extra: int = 0) -> dict:
    """LoPA-gated FFN weights: V [r,D] ~ N(0,1/D), U [H,r] ~ N(0,1/r), W_up/W_down [H,D] ~ N(0,1/D).

    With RMSNorm and unit gain U n ~ N(0,1); the fixed matrix adds one N(0,1) token entry, so the
    pre-activation has sigma_z = sqrt(2) with it and 1 without; the bias is scaled accordingly.
    The fixed matrix itself (an index array) is supplied by the caller.
    """
    w = {
        "V": normal_tensor((r, D), 1.0 / math.sqrt(D), dtype, seed, "V", device, extra),
        "U": normal_tensor((H, r), 1.0 / math.sqrt(r), dtype, seed, "U", device, extra),
        "W_up": normal_tensor((H, D), 1.0 / math.sqrt(D), dtype, seed, "W_up", device, extra),
        "W_down": normal_tensor((H, D), 1.0 / math.sqrt(D), dtype, seed, "W_down", device, extra),
    }
    sigma = math.sqrt(2.0) if with_fixed_matrix else 1.0
    w["b_g"] = None if sparsity is None else torch.full(
        (H,), gate_bias_for_sparsity(sparsity, sigma), dtype=torch.float32, device=device)
    return w


def q8_matrix(shape, std: float, seed: int, tag: str, device="cpu", extra: int = 0, chunk_rows: int = 4096) -> dict:
    """int8 codes q [rows, cols] and fp32 row scales s [rows] of a matrix whose entries s_j q[j,k] have
    standard deviation ~ std (see the module recipe).  Returns dict(q=int8 tensor, s=float32 tensor)."""
    rows, cols = shape
    q = torch.empty((rows, cols), dtype=torch.int8, device=device)
    g = _gen(seed, tag, device, extra)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        blk = torch.randn((r1 - r0, cols), generator=g, device=device, dtype=torch.float32)
        q[r0:r1] = (blk * 32.0).round().clamp(-127, 127).to(torch.int8)
    u = torch.rand((rows,), generator=_gen(seed, "scale", device, extra * 16 + _TAGS[tag]), device=device,
                   dtype=torch.float32)
    s = (std / 32.0) * (1.0 + 0.1 * (2.0 * u - 1.0))
    return {"q": q, "s": s.float()}


def q4_matrix(shape, std: float, seed: int, tag: str, device="cpu", extra: int = 0, chunk_rows: int = 4096) -> dict:
    """4-bit codes and fp32 row scales of a matrix whose entries s_j q[j,k] have standard deviation ~ std: codes
    clip(round(N(0, 2.5^2)), -7, 7) (what an abs-max quantiser leaves of a Gaussian row on 4 bits), packed two per byte
    with the even column in the low nibble, two's complement; scales (std / 2.5) (1 +- 0.1 u).  Returns
    dict(q=uint8 [rows, cols / 2], s=float32 [rows]).  cols must be even."""
    rows, cols = shape
    assert cols % 2 == 0
    q = torch.empty((rows, cols // 2), dtype=torch.uint8, device=device)
    g = _gen(seed, tag, device, extra)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        blk = torch.randn((r1 - r0, cols), generator=g, device=device, dtype=torch.float32)
        c = (blk * 2.5).round().clamp(-7, 7).to(torch.int16) & 0xF
        q[r0:r1] = (c[:, 0::2] | (c[:, 1::2] << 4)).to(torch.uint8)
    u = torch.rand((rows,), generator=_gen(seed, "scale", device, extra * 16 + _TAGS[tag]), device=device,
                   dtype=torch.float32)
    s = (std / 2.5) * (1.0 + 0.1 * (2.0 * u - 1.0))
    return {"q": q, "s": s.float()}


def standard_ffn_q4(D: int, H: int, seed: int, device="cpu", sparsity: float | None = 0.9, extra: int = 0) -> dict:
    """Standard-gated FFN in 4-bit codes + row scales (see :func:`q4_matrix`); b_g as in :func:`standard_ffn`."""
    std = 1.0 / math.sqrt(D)
    w = {k: q4_matrix((H, D), std, seed, k, device, extra) for k in ("W_g", "W_up", "W_down")}
    w["b_g"] = None if sparsity is None else torch.full(
        (H,), gate_bias_for_sparsity(sparsity), dtype=torch.float32, device=device)
    return w


def lopa_ffn_q4(D: int, H: int, r: int, seed: int, device="cpu", sparsity: float | None = 0.9,
                with_fixed_matrix: bool = True, extra: int = 0) -> dict:
    """LoPA-gated FFN in 4-bit codes + row scales (V [r,D], U [H,r], W_up, W_down [H,D]); b_g as in :func:`lopa_ffn`."""
    w = {
        "V": q4_matrix((r, D), 1.0 / math.sqrt(D), seed, "V", device, extra),
        "U": q4_matrix((H, r), 1.0 / math.sqrt(r), seed, "U", device, extra),
        "W_up": q4_matrix((H, D), 1.0 / math.sqrt(D), seed, "W_up", device, extra),
        "W_down": q4_matrix((H, D), 1.0 / math.sqrt(D), seed, "W_down", device, extra),
    }
    sigma = math.sqrt(2.0) if with_fixed_matrix else 1.0
    w["b_g"] = None if sparsity is None else torch.full(
        (H,), gate_bias_for_sparsity(sparsity, sigma), dtype=torch.float32, device=device)
    return w


def standard_ffn_q8(D: int, H: int, seed: int, device="cpu", sparsity: float | None = 0.9, extra: int = 0) -> dict:
    """Standard-gated FFN in int8 codes + row scales: W_g, W_up, W_down each dict(q [H,D], s [H]); b_g as in
    :func:`standard_ffn`."""
    std = 1.0 / math.sqrt(D)
    w = {k: q8_matrix((H, D), std, seed, k, device, extra) for k in ("W_g", "W_up", "W_down")}
    w["b_g"] = None if sparsity is None else torch.full(
        (H,), gate_bias_for_sparsity(sparsity), dtype=torch.float32, device=device)
    return w


def lopa_ffn_q8(D: int, H: int, r: int, seed: int, device="cpu", sparsity: float | None = 0.9,
                with_fixed_matrix: bool = True, extra: int = 0) -> dict:
    """LoPA-gated FFN in int8 codes + row scales (V [r,D], U [H,r], W_up, W_down [H,D]); b_g as in
    :func:`lopa_ffn`."""
    w = {
        "V": q8_matrix((r, D), 1.0 / math.sqrt(D), seed, "V", device, extra),
        "U": q8_matrix((H, r), 1.0 / math.sqrt(r), seed, "U", device, extra),
        "W_up": q8_matrix((H, D), 1.0 / math.sqrt(D), seed, "W_up", device, extra),
        "W_down": q8_matrix((H, D), 1.0 / math.sqrt(D), seed, "W_down", device, extra),
    }
    sigma = math.sqrt(2.0) if with_fixed_matrix else 1.0
    w["b_g"] = None if sparsity is None else torch.full(
        (H,), gate_bias_for_sparsity(sparsity, sigma), dtype=torch.float32, device=device)
    return w


def zipf_firing_profile(H: int, alpha: float = 1.1, mean_p: float = 0.1, p_max: float = 0.99,
                        seed: int = 4) -> torch.Tensor:
    """Per-neuron firing probabilities p_k = min(p_max, c k^-alpha), c solved so mean(p) = mean_p,
    assigned to neurons through a seeded permutation.  Returns p [H] float64 (CPU)."""
    k = torch.arange(1, H + 1, dtype=torch.float64)
    base = k.pow(-alpha)
    lo, hi = 0.0, float(H)
    for _ in range(200):
        c = 0.5 * (lo + hi)
        if torch.clamp(c * base, max=p_max).mean().item() < mean_p:
            lo = c
        else:
            hi = c
    p = torch.clamp(0.5 * (lo + hi) * base, max=p_max)
    perm = torch.randperm(H, generator=_gen(seed, "perm", "cpu"))
    out = torch.empty(H, dtype=torch.float64)
    out[perm] = p
    return out


def bias_from_firing_profile(p: torch.Tensor, sigma_z: float = 1.0) -> torch.Tensor:
    """b_g[j] = -Phi^-1(1 - p_j) sigma_z, so neuron j fires with probability p_j.  fp32 [H]."""
    q = (1.0 - p.double()).clamp(1e-12, 1 - 1e-12)
    return (-math.sqrt(2.0) * torch.erfinv(2.0 * q - 1.0) * sigma_z).float()


def expected_union_fraction(p: torch.Tensor, B: int) -> float:
    """E|union of B independent active sets| / H = mean(1 - (1 - p_j)^B)."""
    return float((1.0 - (1.0 - p.double()).pow(B)).mean())
