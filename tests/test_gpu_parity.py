"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element, on the
same seeded tensors.  Run with `-m gpu` on a B200."""
import math

import numpy as np
import pytest
import torch

import synthetic_inputs as syn
from parity import assert_active_set, assert_y_close, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def mod():
    import paper_2609_31975_b200 as m
    m.load_library()
    return m


@pytest.fixture(params=["cuda_core_gate", "tensor_core_gate"])
def gate_engine(request, mod):
    """Single-token calls on the fused path with the gate forced onto one engine (where the tensor-core kernel does
    not cover the call, both values run the CUDA-core kernel)."""
    mod.test_set_knob("tensor_gate", 1 if request.param == "tensor_core_gate" else 0)
    yield request.param
    mod.test_set_knob("tensor_gate", -1)


def make_std(D, H, dtype, seed, s):
    w = syn.standard_ffn(D, H, dtype, seed, DEV, sparsity=s)
    return {"W_g": w["W_g"]}, w


def make_lopa(mod, D, H, r, dtype, seed, s, fixed="diag", sign=False, gain=False, rms=True):
    w = syn.lopa_ffn(D, H, r, dtype, seed, DEV, sparsity=s, with_fixed_matrix=fixed is not None)
    gate = {"V": w["V"], "U": w["U"], "use_rmsnorm": rms, "rms_eps": 1e-5, "g_idx": None}
    if fixed == "diag":
        gate["g_idx"] = mod.g_diagonal(H, D, DEV)
    elif fixed == "tiled":
        gate["g_idx"] = mod.g_tiled(H, D, DEV)
    g = torch.Generator().manual_seed(seed)
    if sign:
        gate["g_sign"] = (torch.randint(0, 2, (H,), generator=g) * 2 - 1).to(torch.int8).to(DEV)
    if gain:
        gate["rms_gain"] = (0.5 + torch.rand(r, generator=g)).to(DEV)
    return gate, w


def run_both_paths(mod, ffn, x, gate, w, act, paths, tol=None, what=""):
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
    kw = {} if tol is None else dict(rel_l2=tol, max_abs=tol)
    for path in paths:
        ffn.set_path(path)
        y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert ffn.device_status() == 0, f"{what} [{path}]: status words {ffn.status_words()}"
        assert_y_close(y, ref["y"], what=f"{what} [{path}]", **kw)
        assert_active_set(ffn.last_active(), ref, what=f"{what} [{path}]")
    ffn.set_path("auto")
    return ref


# ------------------------------------------------------------------ config 1: tiny fp32 bring-up
def test_config1_fp32_all_64_tokens(mod):
    D, H = 256, 1024
    gate, w = make_std(D, H, torch.float32, 0, 0.9)
    x = syn.tokens(64, D, torch.float32, 0, DEV)
    ffn = mod.SparseFFN(D, H, torch.float32, B_max=1)
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    for path in ("general", "fused"):
        ffn.set_path(path)
        for t in range(64):
            y = ffn.sparse_ffn_forward(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
            one = dict(y=ref["y"][t], z=ref["z"][t])
            assert_y_close(y, one["y"], rel_l2=1e-5, max_abs=1e-5, what=f"token {t} [{path}]")
            assert_active_set(ffn.last_active(), one, what=f"token {t} [{path}]")
    assert ffn.device_status() == 0


# ------------------------------------------------------------------ shrunken decode shapes, ragged sizes
@pytest.mark.parametrize("D,H", [(512, 1000), (264, 777), (1024, 2049), (2048, 300)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_standard_gate_small_shapes(mod, gate_engine, D, H, dtype):
    ffn = mod.SparseFFN(D, H, dtype, B_max=1)
    for s, act in ((0.5, "relu"), (0.9, "sqrelu"), (0.95, "rsplus")):
        gate, w = make_std(D, H, dtype, 21, s)
        x = syn.tokens(3, D, dtype, 21, DEV)
        for t in range(3):
            run_both_paths(mod, ffn, x[t], gate, w, act, ("general", "fused"), what=f"{D}x{H} s={s} {act}")


@pytest.mark.parametrize("D,H", [(3840, 300), (5120, 200), (8192, 160), (16384, 96)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_wide_rows(mod, gate_engine, D, H, dtype):
    """Rows of 7.5 to 64 KB: one row per gate slot, few ring slots, up to eight chunks per act thread; whatever
    `auto` picks for the shape (the fused kernels where their geometry fits, else the general ones)."""
    if D * (2 if dtype == torch.bfloat16 else 4) > 32768:               # rows above 32 KB are refused, not mangled
        with pytest.raises(mod.SFFNError) as e:
            mod.SparseFFN(D, H, dtype, r_max=64, B_max=2)
        assert e.value.code == 2
        return
    ffn = mod.SparseFFN(D, H, dtype, r_max=64, B_max=2)
    gate, w = make_std(D, H, dtype, 23, 0.8)
    x = syn.tokens(2, D, dtype, 23, DEV)
    run_both_paths(mod, ffn, x[0], gate, w, "relu", ("general", "auto"), what=f"wide {D}x{H}")
    lg, lw = make_lopa(mod, D, H, 64, dtype, 24, 0.8, "tiled")
    run_both_paths(mod, ffn, x[1], lg, lw, "sqrelu", ("general", "auto"), what=f"wide lopa {D}x{H}")
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")      # two tokens
    assert_y_close(y, ref["y"], what=f"wide {D}x{H} B=2")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0


def test_widest_rows_batch_of_four_on_the_cuda_core_path(mod):
    """16384 bf16 elements per row: the CUDA-core gate kernel stages its tokens as fp32 in shared memory and takes
    two tokens per pass there (four would need 256 KB)."""
    D, H = 16384, 96
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=4)
    gate, w = make_std(D, H, torch.bfloat16, 25, 0.8)
    x = syn.tokens(4, D, torch.bfloat16, 25, DEV)
    run_both_paths(mod, ffn, x, gate, w, "relu", ("general",), what="wide 16384 B=4")


@pytest.mark.parametrize("r,fixed,sign,gain,rms", [
    (64, "diag", False, False, True), (128, "tiled", True, True, True),
    (96, None, False, False, False), (256, "diag", True, False, False)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_lopa_gate_small_shapes(mod, r, fixed, sign, gain, rms, dtype):
    D, H = 512, 1531
    ffn = mod.SparseFFN(D, H, dtype, r_max=256, B_max=1)
    gate, w = make_lopa(mod, D, H, r, dtype, 31, 0.9, fixed, sign, gain, rms)
    x = syn.tokens(2, D, dtype, 31, DEV)
    for t in range(2):
        for act in ("relu", "sqrelu"):
            run_both_paths(mod, ffn, x[t], gate, w, act, ("general", "fused"), what=f"lopa r={r} {fixed}")


# ------------------------------------------------------------------ batches: union of active sets
@pytest.mark.parametrize("path", ["general", "mma_sync", "auto"])   # auto = tcgen05 kernels for bf16 batches
@pytest.mark.parametrize("B", [2, 3, 4, 7, 16, 33, 64])
def test_batched_union(mod, B, path):
    D, H = 512, 1200
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=64)
    ffn.set_path(path)
    gate, w = make_std(D, H, torch.bfloat16, 41, 0.9)
    p = syn.zipf_firing_profile(H, 1.1, 0.1, 0.99, seed=4)
    w["b_g"] = syn.bias_from_firing_profile(p).to(DEV)
    x = syn.tokens(B, D, torch.bfloat16, 41, DEV)
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert_y_close(y, ref["y"], what=f"B={B} [{path}]")
    assert_active_set(ffn.last_active(), ref, what=f"B={B} [{path}]")
    y2 = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert torch.equal(y, y2)                                    # run-to-run determinism
    yd = ffn.dense_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    dref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", route="dense")
    assert_y_close(yd, dref["y"], what=f"dense B={B} [{path}]")
    # each token of the batch equals its own single-token call
    for b in (0, B - 1):
        y1 = ffn.sparse_ffn_forward(x[b], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        assert_y_close(y1, ref["y"][b], what=f"B={B} token {b} alone")


@pytest.mark.parametrize("path", ["general", "mma_sync", "auto"])
@pytest.mark.parametrize("B,r,rms", [(5, 128, True), (16, 64, True), (24, 96, False)])
def test_batched_lopa(mod, B, r, rms, path):
    D, H = 512, 1100
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=128, B_max=32)
    ffn.set_path(path)
    gate, w = make_lopa(mod, D, H, r, torch.bfloat16, 43, 0.9, "diag", True, rms, rms)
    x = syn.tokens(B, D, torch.bfloat16, 43, DEV)
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "sqrelu")
    y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "sqrelu")
    assert_y_close(y, ref["y"], what=f"batched lopa [{path}]")
    assert_active_set(ffn.last_active(), ref, what=f"batched lopa [{path}]")


@pytest.mark.parametrize("kind", ["standard", "lopa"])
@pytest.mark.parametrize("B", [65, 96, 130])
def test_batches_of_more_than_64_tokens_run_in_chunks_with_the_union_of_all(mod, kind, B):
    D, H, r = 512, 1200, 128
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=r, B_max=130)
    if kind == "standard":
        gate, w = make_std(D, H, torch.bfloat16, 45, 0.9)
    else:
        gate, w = make_lopa(mod, D, H, r, torch.bfloat16, 45, 0.9, "diag", True, True, True)
    p = syn.zipf_firing_profile(H, 1.1, 0.02, 0.9, seed=5)       # a union that keeps growing with the tokens
    w["b_g"] = syn.bias_from_firing_profile(p).to(DEV)
    x = syn.tokens(B, D, torch.bfloat16, 45, DEV)
    ref = run_both_paths(mod, ffn, x, gate, w, "relu", ("auto", "mma_sync"), what=f"{kind} B={B}")
    last = run_oracle(x[64 * ((B - 1) // 64):], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert last["union_mask"].sum() < ref["union_mask"].sum()    # the list is not just the last chunk's
    yd = ffn.dense_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    dref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", route="dense")
    assert_y_close(yd, dref["y"], what=f"dense {kind} B={B}")
    y1 = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    y2 = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert torch.equal(y1, y2)


@pytest.mark.parametrize("dtype,D", [(torch.float32, 512), (torch.bfloat16, 520), (torch.float32, 776)])
@pytest.mark.parametrize("kind", ["standard", "lopa"])
@pytest.mark.parametrize("B", [2, 5, 70])
def test_batches_without_a_tensor_core_path_run_token_by_token(mod, dtype, D, kind, B):
    # fp32 operands, or bf16 rows of a width the tensor-core batch kernels do not take
    H, r = 1100, 64
    ffn = mod.SparseFFN(D, H, dtype, r_max=r, B_max=70)
    if kind == "standard":
        gate, w = make_std(D, H, dtype, 46, 0.9)
    else:
        gate, w = make_lopa(mod, D, H, r, dtype, 46, 0.9, "diag", True, True, True)
    x = syn.tokens(B, D, dtype, 46, DEV)
    tol = 1e-5 if dtype == torch.float32 else None
    ref = run_both_paths(mod, ffn, x, gate, w, "relu", ("auto", "general"), tol=tol, what=f"{kind} {dtype} B={B}")
    launches0 = ffn.launch_count()
    y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert ffn.launch_count() - launches0 == B                   # one launch per token: the single-token kernel
    for b in (0, B - 1):                                         # and bit for bit what the token gives alone
        y1 = ffn.sparse_ffn_forward(x[b], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        assert torch.equal(y1, y[b])
    yd = ffn.dense_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    dref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", route="dense")
    assert_y_close(yd, dref["y"], what=f"dense {kind} {dtype} B={B}", **({} if tol is None else dict(rel_l2=tol, max_abs=tol)))


# ------------------------------------------------------------------ degenerate cases
@pytest.mark.parametrize("path", ["general", "fused"])
def test_full_and_zero_sparsity(mod, gate_engine, path):
    D, H = 512, 900
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    ffn.set_path(path)
    gate, w = make_std(D, H, torch.bfloat16, 51, None)
    x = syn.tokens(1, D, torch.bfloat16, 51, DEV)[0]
    lo = torch.full((H,), -1e3, device=DEV)
    y = ffn.sparse_ffn_forward(x, gate, lo, w["W_up"], w["W_down"], "relu")
    assert not y.any() and ffn.last_active().numel() == 0        # 100 % sparsity: y == 0 exactly
    hi = torch.full((H,), 1e3, device=DEV)
    y = ffn.sparse_ffn_forward(x, gate, hi, w["W_up"], w["W_down"], "relu")
    assert ffn.last_active().tolist() == list(range(H))           # 0 % sparsity: every row
    yd = ffn.dense_ffn_forward(x, gate, hi, w["W_up"], w["W_down"], "relu")
    assert torch.equal(y, yd)                                      # same rows, same order, same bits
    ref = run_oracle(x, gate, hi, w["W_up"], w["W_down"], "relu", route="dense")
    assert_y_close(y, ref["y"], what="0% sparsity")
    # no bias at all (the paper's form of Eq. 1)
    y = ffn.sparse_ffn_forward(x, gate, None, w["W_up"], w["W_down"], "rsplus")
    ref = run_oracle(x, gate, None, w["W_up"], w["W_down"], "rsplus")
    assert_y_close(y, ref["y"], what="no bias")
    assert_active_set(ffn.last_active(), ref, what="no bias")


@pytest.mark.parametrize("path", ["general", "fused"])
def test_dense_comparator_and_determinism(mod, gate_engine, path):
    D, H = 1024, 3000
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=128, B_max=1)
    ffn.set_path(path)
    for gate, w in (make_std(D, H, torch.bfloat16, 61, 0.8),
                    make_lopa(mod, D, H, 128, torch.bfloat16, 61, 0.8, "diag")):
        x = syn.tokens(1, D, torch.bfloat16, 61, DEV)[0]
        ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", route="dense")
        yd = ffn.dense_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        ys = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        assert_y_close(yd, ref["y"], what="dense comparator")
        assert_y_close(ys, yd.double().cpu().numpy(), rel_l2=1e-5, max_abs=1e-5, what="sparse vs dense (GPU)")
        idx0 = ffn.last_active()
        for _ in range(5):                                           # bitwise run-to-run determinism
            y2 = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
            assert torch.equal(ys, y2) and torch.equal(idx0, ffn.last_active())
    assert ffn.device_status() == 0


def test_host_entry_and_errors(mod):
    D, H = 512, 640
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=2)
    gate, w = make_std(D, H, torch.bfloat16, 71, 0.9)
    x = syn.tokens(2, D, torch.bfloat16, 71, DEV)
    xh = x.cpu().pin_memory()
    yh = torch.empty((2, D), dtype=torch.float32).pin_memory()
    ffn.sparse_ffn_forward_host(xh, gate, w["b_g"], w["W_up"], w["W_down"], "relu", yh)
    torch.cuda.synchronize()
    y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert torch.equal(y.cpu(), yh)
    xp, yp = x.cpu(), torch.full((2, D), float("nan"), dtype=torch.float32)   # pageable memory: copy-engine route
    ffn.sparse_ffn_forward_host(xp, gate, w["b_g"], w["W_up"], w["W_down"], "relu", yp)
    torch.cuda.synchronize()
    assert torch.equal(y.cpu(), yp)
    yh1 = torch.empty(D, dtype=torch.float32).pin_memory()                       # one token: fused kernels
    ffn.sparse_ffn_forward_host(xh[1], gate, w["b_g"], w["W_up"], w["W_down"], "relu", yh1)
    torch.cuda.synchronize()
    assert torch.equal(ffn.sparse_ffn_forward(x[1], gate, w["b_g"], w["W_up"], w["W_down"], "relu").cpu(), yh1)
    n0 = ffn.launch_count()
    ffn.sparse_ffn_forward(x[0], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert ffn.launch_count() > n0
    with pytest.raises(mod.SFFNError) as e:                           # B > B_max
        ffn.sparse_ffn_forward(syn.tokens(3, D, torch.bfloat16, 1, DEV), gate, w["b_g"], w["W_up"], w["W_down"])
    assert e.value.code == 1
    with pytest.raises(mod.SFFNError) as e:                           # misaligned weight pointer
        big = torch.empty(H * D + 8, dtype=torch.bfloat16, device=DEV)
        ffn.sparse_ffn_forward(x[0], gate, w["b_g"], big[1:1 + H * D].view(H, D), w["W_down"])
    assert e.value.code == 2
    ffn.set_path("fused")
    n0 = ffn.launch_count()                                           # the fused kernel is single-token: a batch
    yb = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"])   # runs it once per token
    assert ffn.launch_count() - n0 == x.shape[0]
    assert torch.equal(yb[1], ffn.sparse_ffn_forward(x[1], gate, w["b_g"], w["W_up"], w["W_down"]))
    with pytest.raises(mod.SFFNError):                                # rows must be multiples of 16 bytes
        mod.SparseFFN(260, 64, torch.bfloat16)


@pytest.mark.parametrize("D,H,B,s", [
    (256, 20000, 8, 0.2),    # union = every row: more than 128 rows x 148 CTAs, several tiles per CTA
    (256, 50048, 4, 0.9),    # more flags than the in-kernel compaction takes: separate compaction launch
    (256, 777, 3, 0.9),      # H not a multiple of 8: ragged last tile, byte-wise flag reads
    (512, 1500, 33, 0.95),   # 33 tokens: 48 token columns, three column groups shared by all warps
    (512, 19072, 40, 0.9),   # the same with two tiles for some CTAs: warps that join for the last tile only
    (512, 38000, 20, 0.95),  # three tiles for some CTAs
    (256, 64, 2, 0.5),       # fewer rows than one tile of eight per CTA
])
def test_batched_tcgen05_edge_shapes(mod, D, H, B, s):
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=B)
    gate, w = make_std(D, H, torch.bfloat16, 43, s)
    x = syn.tokens(B, D, torch.bfloat16, 43, DEV)
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", threads=16)
    y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0
    assert_y_close(y, ref["y"], what=f"edge {D}x{H} B={B}")
    assert_active_set(ffn.last_active(), ref, what=f"edge {D}x{H} B={B}")
    y2 = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert torch.equal(y, y2)
    yd = ffn.dense_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    dref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", route="dense", threads=16)
    assert_y_close(yd, dref["y"], what=f"edge dense {D}x{H} B={B}")


def test_batched_empty_and_full_union(mod):
    D, H, B = 256, 1000, 6
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=B)
    gate, w = make_std(D, H, torch.bfloat16, 44, None)
    x = syn.tokens(B, D, torch.bfloat16, 44, DEV)
    lo = torch.full((H,), -1e3, device=DEV)
    y = ffn.sparse_ffn_forward(x, gate, lo, w["W_up"], w["W_down"], "relu")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0
    assert not y.any() and ffn.last_active().numel() == 0        # no neuron fires for any token: y == 0 exactly
    hi = torch.full((H,), 1e3, device=DEV)
    y = ffn.sparse_ffn_forward(x, gate, hi, w["W_up"], w["W_down"], "relu")
    assert ffn.last_active().tolist() == list(range(H))           # every neuron fires: the union is every row
    ref = run_oracle(x, gate, hi, w["W_up"], w["W_down"], "relu", route="dense")
    assert_y_close(y, ref["y"], what="batched, full union")


def test_batched_calls_repeat_bit_for_bit(mod):
    """Back-to-back calls chained by dependent launch, interleaved with other work on the same handle, must
    give the same bits every time (ring phases, bit masks, list and partial buffers are reused across calls)."""
    D, H = 512, 2500
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=64, B_max=33)
    gate, w = make_std(D, H, torch.bfloat16, 45, 0.9)
    gate2, w2 = make_std(D, H, torch.bfloat16, 46, 0.5)
    lg, lw = make_lopa(mod, D, H, 64, torch.bfloat16, 47, 0.9, "diag")
    for B in (33, 5, 1):
        x = syn.tokens(B, D, torch.bfloat16, 45, DEV)
        xs = x if B > 1 else x[0]
        for g_, w_ in ((gate, w), (lg, lw)):
            ref = ffn.sparse_ffn_forward(xs, g_, w_["b_g"], w_["W_up"], w_["W_down"], "relu").clone()
            idx = ffn.last_active().clone()
            for it in range(30):
                if it % 3 == 0:
                    ffn.dense_ffn_forward(xs, gate2, w2["b_g"], w2["W_up"], w2["W_down"], "sqrelu")
                if it % 5 == 0:
                    ffn.sparse_ffn_forward(x[0], gate2, w2["b_g"], w2["W_up"], w2["W_down"], "relu")
                y = ffn.sparse_ffn_forward(xs, g_, w_["b_g"], w_["W_up"], w_["W_down"], "relu")
                assert torch.equal(y, ref), f"B={B} repeat {it}"
            assert torch.equal(ffn.last_active(), idx)
    assert ffn.device_status() == 0


# ------------------------------------------------------------------ double activation (Sec. 3.3)
@pytest.mark.parametrize("act,act_up", [("relu", "relu"), ("sqrelu", "rsplus"), ("rsplus", "sqrelu"), ("relu", "silu")])
def test_double_activation_all_paths(mod, gate_engine, act, act_up):
    D, H = 512, 1100
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=64, B_max=8)
    ffn.set_up_activation(act_up)
    gate, w = make_std(D, H, torch.bfloat16, 61, 0.8)
    x = syn.tokens(8, D, torch.bfloat16, 61, DEV)
    ref1 = run_oracle(x[0], gate, w["b_g"], w["W_up"], w["W_down"], act, act_up=act_up)
    if act_up == "silu":                                                # SILU is not sparse: nothing is removed
        assert ref1["n_gated"][0] == ref1["n_act"][0]
    else:
        assert 0 < ref1["n_gated"][0] < ref1["n_act"][0]                # A_3 really removes neurons
    for path in ("general", "fused"):                                   # one token
        ffn.set_path(path)
        y = ffn.sparse_ffn_forward(x[0], gate, w["b_g"], w["W_up"], w["W_down"], act)
        assert_y_close(y, ref1["y"], what=f"double activation {act}/{act_up} [{path}]")
        assert_active_set(ffn.last_active(), ref1, what=f"double activation [{path}]")   # the list is the gate's
        yd = ffn.dense_ffn_forward(x[0], gate, w["b_g"], w["W_up"], w["W_down"], act)
        assert_y_close(yd, ref1["y"], what=f"double activation dense [{path}]")
    ref8 = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], act, act_up=act_up)
    for path in ("general", "mma_sync", "auto"):                        # a batch: CUDA cores, mma.sync, tcgen05
        ffn.set_path(path)
        y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        assert_y_close(y, ref8["y"], what=f"double activation batch [{path}]")
    # LoPA gate, one token and a batch
    lg, lw = make_lopa(mod, D, H, 64, torch.bfloat16, 62, 0.8, "diag")
    ffn.set_path("auto")
    for xs in (x[1], x[:5]):
        ref = run_oracle(xs, lg, lw["b_g"], lw["W_up"], lw["W_down"], act, act_up=act_up)
        y = ffn.sparse_ffn_forward(xs, lg, lw["b_g"], lw["W_up"], lw["W_down"], act)
        assert_y_close(y, ref["y"], what="double activation, LoPA gate")
    # back to Eq. 1
    ffn.set_up_activation(None)
    y = ffn.sparse_ffn_forward(x[0], gate, w["b_g"], w["W_up"], w["W_down"], act)
    assert_y_close(y, run_oracle(x[0], gate, w["b_g"], w["W_up"], w["W_down"], act)["y"], what="act_up reset")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0


@pytest.mark.parametrize("dtype,D,H,s", [(torch.bfloat16, 512, 1000, 0.9), (torch.float32, 264, 777, 0.8),
                                         (torch.bfloat16, 2048, 300, 0.5), (torch.bfloat16, 4096, 14336, 0.9),
                                         (torch.float32, 4096, 2000, 0.2), (torch.bfloat16, 8192, 4000, 0.9)])
def test_gated_skip_fetches_fewer_rows_and_changes_no_bit(mod, dtype, D, H, s):
    """sffn_set_gated_skip: the W_down row of a fired neuron only where a_j A_3(u_j) != 0 (single token, standard gate)."""
    gate, w = make_std(D, H, dtype, 63, s)
    x = syn.tokens(4, D, dtype, 63, DEV)
    ffn = mod.SparseFFN(D, H, dtype, r_max=64, B_max=4)
    tol = dict(rel_l2=1e-5, max_abs=1e-5) if dtype == torch.float32 else {}
    for act_up in ("relu", "silu", "rsplus", None):
        ffn.set_up_activation(act_up)
        for t in range(4):
            ffn.set_gated_skip(False)
            y0 = ffn.sparse_ffn_forward(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu").clone()
            ffn.set_gated_skip(True)
            y1 = ffn.sparse_ffn_forward(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu").clone()
            torch.cuda.synchronize()
            assert ffn.device_status() == 0, ffn.status_words()
            assert torch.equal(y0, y1), f"act_up={act_up} token {t}"
            if t == 0:
                ref = run_oracle(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu", act_up=act_up)
                assert_y_close(y1, ref["y"], what=f"gated skip act_up={act_up}", **tol)
                assert_active_set(ffn.last_active(), ref, what=f"gated skip act_up={act_up}")   # the list stays the gate's
                if act_up == "relu" and s > 0:
                    assert ref["n_gated"][0] < ref["n_act"][0]                   # there are rows to skip
    # the other kinds of call ignore the setting: a batch, the dense route, a LoPA gate
    ffn.set_up_activation("relu")
    yb = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert_y_close(yb, run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", act_up="relu")["y"], what="batch", **tol)
    yd = ffn.dense_ffn_forward(x[0], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert_y_close(yd, run_oracle(x[0], gate, w["b_g"], w["W_up"], w["W_down"], "relu", act_up="relu", route="dense")["y"],
                   what="dense", **tol)
    lg, lw = make_lopa(mod, D, H, 64, dtype, 64, 0.8, "diag")
    yl = ffn.sparse_ffn_forward(x[1], lg, lw["b_g"], lw["W_up"], lw["W_down"], "relu")
    assert_y_close(yl, run_oracle(x[1], lg, lw["b_g"], lw["W_up"], lw["W_down"], "relu", act_up="relu")["y"], what="lopa", **tol)
    torch.cuda.synchronize()
    assert ffn.device_status() == 0


# ------------------------------------------------------------------ layer loop under a CUDA graph
@pytest.mark.parametrize("kind", ["standard", "lopa"])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_layer_chain_in_cuda_graph(mod, gate_engine, dtype, kind):
    D, H, L, r = 512, 900, 3, 64
    ffn = mod.SparseFFN(D, H, dtype, r_max=r, B_max=1)
    if kind == "standard":
        layers = [syn.standard_ffn(D, H, dtype, 81, DEV, sparsity=0.8, extra=i) for i in range(L)]
        gates = [{"W_g": w["W_g"]} for w in layers]
    else:
        made = [make_lopa(mod, D, H, r, dtype, 81 + i, 0.8, sign=True, gain=True) for i in range(L)]
        gates, layers = [g for g, _ in made], [w for _, w in made]
    resid = syn.tokens(L + 1, D, dtype, 81, DEV)
    xs = torch.zeros((L + 1, D), dtype=dtype, device=DEV)
    ys = torch.zeros((L, D), dtype=torch.float32, device=DEV)
    stream = torch.cuda.Stream(DEV)

    def body():
        xs[0].copy_(resid[0])
        for l, w in enumerate(layers):
            ffn.sparse_ffn_forward(xs[l], gates[l], w["b_g"], w["W_up"], w["W_down"], "relu", ys[l], stream=stream)
            mod.residual_cast(ys[l], resid[l + 1], 0.25, xs[l + 1], stream=stream)

    with torch.cuda.stream(stream):
        body()
        stream.synchronize()
        eager_x, eager_y = xs.clone(), ys.clone()
        # the glue kernel against its definition, and the chain against the oracle layer by layer
        for l in range(L):
            want = (resid[l + 1].float() + 0.25 * eager_y[l]).to(dtype)
            assert torch.equal(eager_x[l + 1], want)
            ref = run_oracle(eager_x[l], gates[l], layers[l]["b_g"], layers[l]["W_up"], layers[l]["W_down"], "relu")
            assert_y_close(eager_y[l], ref["y"], what=f"chain layer {l}")
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            body()
        # a captured launch is replayed with the arguments of its capture: nothing in them may count calls
        for _ in range(4):
            xs.zero_(); ys.zero_()
            graph.replay()
            stream.synchronize()
            assert torch.equal(xs, eager_x) and torch.equal(ys, eager_y)   # bit for bit the eager run, every replay
        body()                                                             # and eager calls after the replays
        stream.synchronize()
        assert torch.equal(ys, eager_y)
    assert ffn.device_status() == 0


# ------------------------------------------------------------------ full-size configurations
@pytest.mark.parametrize("s,ntok", [(0.9, 8), (0.5, 1), (0.7, 2), (0.8, 2), (0.95, 1)])
def test_config2_full_size_decode(mod, gate_engine, s, ntok):
    D, H = 4096, 14336
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    gate, w = make_std(D, H, torch.bfloat16, 2, s)
    x = syn.tokens(ntok, D, torch.bfloat16, 2, DEV)
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", threads=16)
    assert abs(1 - ref["n_act"].mean() / H - s) < 0.03
    for path in ("general", "fused"):
        ffn.set_path(path)
        for t in range(ntok if path == "fused" else min(ntok, 2)):
            y = ffn.sparse_ffn_forward(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
            one = dict(y=ref["y"][t], z=ref["z"][t])
            assert_y_close(y, one["y"], what=f"config2 s={s} token {t} [{path}]")
            assert_active_set(ffn.last_active(), one, what=f"config2 s={s} token {t} [{path}]")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0


def test_config2_full_size_rsplus(mod, gate_engine):
    D, H = 4096, 14336
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    gate, w = make_std(D, H, torch.bfloat16, 2, 0.9)
    x = syn.tokens(1, D, torch.bfloat16, 7, DEV)[0]
    run_both_paths(mod, ffn, x, gate, w, "rsplus", ("general", "fused"), what="config2 R-S+")


@pytest.mark.parametrize("r", [256, 512, 1024])
@pytest.mark.parametrize("act", ["relu", "sqrelu"])
def test_config3_full_size_lopa(mod, r, act):
    D, H = 4096, 14336
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=1024, B_max=1)
    gate, w = make_lopa(mod, D, H, r, torch.bfloat16, 3, 0.9, "diag")
    x = syn.tokens(1, D, torch.bfloat16, 3, DEV)[0]
    ref = run_both_paths(mod, ffn, x, gate, w, act, ("general", "fused"), what=f"config3 r={r} {act}")
    assert abs(1 - ref["n_act"][0] / H - 0.9) < 0.03


@pytest.mark.parametrize("B", [4, 16, 64])
def test_config4_full_size_batched_zipf(mod, B):
    D, H = 4096, 14336
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=B)
    gate, w = make_std(D, H, torch.bfloat16, 4, None)
    p = syn.zipf_firing_profile(H, 1.1, 0.1, 0.99, seed=4)
    w["b_g"] = syn.bias_from_firing_profile(p).to(DEV)
    x = syn.tokens(B, D, torch.bfloat16, 4, DEV)
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu", threads=16)
    y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert_y_close(y, ref["y"], what=f"config4 B={B}")
    assert_active_set(ffn.last_active(), ref, what=f"config4 B={B}")
    frac = ref["union_mask"].mean()
    assert abs(frac - syn.expected_union_fraction(p, B)) < 0.05


@pytest.mark.parametrize("s", [0.9, 0.8, 0.95])
def test_config5_full_size_stress_layer0(mod, gate_engine, s):
    """8192 x 28672, squared RELU, standard and LoPA r = 1024 gates, one token and a batch of eight (the batch:
    the tcgen05 gate GEMM with K = 8192 and several 128-row tiles per CTA, gather4 over the union)."""
    D, H = 8192, 28672
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=1024, B_max=8)
    gate, w = make_std(D, H, torch.bfloat16, 5, s)
    x8 = syn.tokens(8, D, torch.bfloat16, 5, DEV, extra=1)
    ntok = 8 if s == 0.9 else 2                     # the other sparsities: two tokens of the batch are checked
    ref = run_oracle(x8[:ntok], gate, w["b_g"], w["W_up"], w["W_down"], "sqrelu", threads=16)
    assert abs(1 - ref["n_act"].mean() / H - s) < 0.03
    for path in ("general", "fused") if s == 0.9 else ("fused",):
        ffn.set_path(path)
        y = ffn.sparse_ffn_forward(x8[0], gate, w["b_g"], w["W_up"], w["W_down"], "sqrelu")
        one = dict(y=ref["y"][0], z=ref["z"][0])
        assert_y_close(y, one["y"], what=f"config5 standard s={s} [{path}]")
        assert_active_set(ffn.last_active(), one, what=f"config5 standard s={s} [{path}]")
    ffn.set_path("auto")
    y = ffn.sparse_ffn_forward(x8[:ntok], gate, w["b_g"], w["W_up"], w["W_down"], "sqrelu")
    assert_y_close(y, ref["y"], what=f"config5 standard s={s} B={ntok}")
    assert_active_set(ffn.last_active(), ref, what=f"config5 standard s={s} B={ntok}")
    if s != 0.9:
        return
    del gate["W_g"], w["W_g"]
    lg, lw = make_lopa(mod, D, H, 1024, torch.bfloat16, 5, 0.9, "diag")
    lw["W_up"], lw["W_down"] = w["W_up"], w["W_down"]
    run_both_paths(mod, ffn, x8[0], lg, lw, "sqrelu", ("general", "fused"), what="config5 lopa")
    ref = run_oracle(x8, lg, lw["b_g"], lw["W_up"], lw["W_down"], "sqrelu", threads=16)
    y = ffn.sparse_ffn_forward(x8, lg, lw["b_g"], lw["W_up"], lw["W_down"], "sqrelu")
    assert_y_close(y, ref["y"], what="config5 lopa B=8")
    assert_active_set(ffn.last_active(), ref, what="config5 lopa B=8")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0


def test_two_handles_on_two_streams_overlap_and_agree(mod):
    # Two standard-gate single-token calls in flight at once (different handles, different streams): each wants every SM
    # and its last CTAs wait for the rest, but at most 64 + 64 CTAs sit waiting for partial results, so both complete -- and bit for bit with
    # what they give one after the other.
    D, H = 4096, 14336
    sets = [syn.standard_ffn(D, H, torch.bfloat16, 90 + i, DEV, sparsity=0.9) for i in range(2)]
    x = syn.tokens(40, D, torch.bfloat16, 90, DEV)
    ffns = [mod.SparseFFN(D, H, torch.bfloat16, B_max=1) for _ in range(2)]
    streams = [torch.cuda.Stream(DEV) for _ in range(2)]
    want = [torch.empty((40, D), device=DEV) for _ in range(2)]
    for i in range(2):
        for t in range(40):
            ffns[i].sparse_ffn_forward(x[t], {"W_g": sets[i]["W_g"]}, sets[i]["b_g"], sets[i]["W_up"], sets[i]["W_down"],
                                       "relu", want[i][t])
        torch.cuda.synchronize()
    got = [torch.zeros((40, D), device=DEV) for _ in range(2)]
    for t in range(40):
        for i in range(2):
            ffns[i].sparse_ffn_forward(x[t], {"W_g": sets[i]["W_g"]}, sets[i]["b_g"], sets[i]["W_up"], sets[i]["W_down"],
                                       "relu", got[i][t], stream=streams[i])
    torch.cuda.synchronize()
    for i in range(2):
        assert ffns[i].device_status() == 0
        assert torch.equal(got[i], want[i])


def test_gate_engine_setting_and_a_long_chain_of_mixed_calls(mod):
    # The public engine setting (parity under each value), then 6000 calls back to back on one stream that switch
    # engine, weights and sparse / dense every few calls: no wait runs out, and every call repeats its first result
    # bit for bit (the calls of a chain overlap at their edges; nothing of one call may leak into the next).
    D, H = 4096, 14336
    sets = [syn.standard_ffn(D, H, torch.bfloat16, 70 + i, DEV, sparsity=sp) for i, sp in enumerate((0.9, 0.6, 0.97))]
    x = syn.tokens(6, D, torch.bfloat16, 70, DEV)
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    assert ffn.lib.sffn_set_gate_engine(ffn._h, 3) == 1          # no such engine: SFFN_ERR_INVALID_ARG
    ref = run_oracle(x[0], {"W_g": sets[0]["W_g"]}, sets[0]["b_g"], sets[0]["W_up"], sets[0]["W_down"], "relu", threads=16)
    for engine in ("cuda_core", "tensor_core", "auto"):
        ffn.set_gate_engine(engine)
        for dense in (False, True):
            fn = ffn.dense_ffn_forward if dense else ffn.sparse_ffn_forward
            y = fn(x[0], {"W_g": sets[0]["W_g"]}, sets[0]["b_g"], sets[0]["W_up"], sets[0]["W_down"], "relu")
            assert_y_close(y, ref["y"], what=f"engine {engine}, dense {dense}")
    engines = ("cuda_core", "tensor_core", "auto")
    kinds = [(e, w, dense) for e in range(3) for w in range(3) for dense in (False, True)]
    first = torch.empty((len(kinds), 6, D), device=DEV)
    out = torch.empty((len(kinds), 6, D), device=DEV)
    for rounds, dst in ((1, first), (55, out)):
        for rnd in range(rounds):
            for k, (e, w, dense) in enumerate(kinds):
                ffn.set_gate_engine(engines[e])
                fn = ffn.dense_ffn_forward if dense else ffn.sparse_ffn_forward
                for t in range(6):
                    fn(x[t], {"W_g": sets[w]["W_g"]}, sets[w]["b_g"], sets[w]["W_up"], sets[w]["W_down"], "relu", dst[k, t])
    torch.cuda.synchronize()
    assert ffn.device_status() == 0
    assert torch.equal(first, out)


def test_lopa_act_groups_keep_their_ring_slots(mod):
    # 16 KB rows leave the LoPA kernel few act slots; its two act groups must each keep their own (a slot that went back
    # and forth between them let a group read the other's row when that row was late: rare timeouts, once a fault).
    # Every call is followed by a synchronisation -- all CTAs then start at once, which is what provoked it -- and must
    # repeat the first result bit for bit.
    D, H, r = 8192, 4096, 1024
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=r, B_max=1)
    lg, lw = make_lopa(mod, D, H, r, torch.bfloat16, 61, 0.8, "diag")
    x = syn.tokens(2, D, torch.bfloat16, 61, DEV)
    ref = run_both_paths(mod, ffn, x[0], lg, lw, "relu", ("fused",), what="lopa 8192 r=1024")
    assert 0 < ref["n_act"][0] < H
    ffn.set_path("fused")
    first = [ffn.sparse_ffn_forward(x[t], lg, lw["b_g"], lw["W_up"], lw["W_down"], "relu").clone() for t in range(2)]
    for rep in range(40):
        y = ffn.sparse_ffn_forward(x[rep % 2], lg, lw["b_g"], lw["W_up"], lw["W_down"], "relu")
        torch.cuda.synchronize()
        assert ffn.device_status() == 0, f"rep {rep}: status words {ffn.status_words()}"
        assert torch.equal(y, first[rep % 2]), f"rep {rep}"


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_fused_path_agrees_with_the_cuda_core_path(mod, seed):
    # Seeded random geometries (row widths, neuron counts that leave ragged slabs, LoPA ranks, storage types, both
    # gate engines, repeated calls): the single-token kernels against the plain CUDA-core kernels, which share none
    # of their code; both within the usual tolerance of each other, no wait runs out, and repeats are bit for bit.
    g = torch.Generator().manual_seed(1000 + seed)
    ri = lambda lo, hi: int(torch.randint(lo, hi + 1, (1,), generator=g))  # noqa: E731
    for case in range(7):
        dtype = (torch.bfloat16, torch.bfloat16, torch.float32)[ri(0, 2)]
        D = 64 * ri(4, 72) if dtype == torch.bfloat16 else 64 * ri(4, 40)
        H = ri(60, 5000)
        lopa = ri(0, 1) == 1
        r = 32 * ri(1, min(24, D // 64)) if lopa else 0
        s = (0.5, 0.8, 0.9, 0.97)[ri(0, 3)]
        act = ("relu", "sqrelu", "rsplus")[ri(0, 2)]
        what = f"seed {seed} case {case}: D={D} H={H} r={r} {dtype} s={s} {act}"
        ffn = mod.SparseFFN(D, H, dtype, r_max=r, B_max=1)
        if lopa:
            gate, w = make_lopa(mod, D, H, r, dtype, 2000 + 10 * seed + case, s, ("diag", "tiled", None)[ri(0, 2)],
                                sign=ri(0, 1) == 1, gain=ri(0, 1) == 1, rms=ri(0, 1) == 1)
        else:
            gate, w = make_std(D, H, dtype, 2000 + 10 * seed + case, s)
        x = syn.tokens(2, D, dtype, 3000 + seed, DEV)
        ffn.set_path("general")
        want = [ffn.sparse_ffn_forward(x[t], gate, w["b_g"], w["W_up"], w["W_down"], act).clone() for t in range(2)]
        ffn.set_path("auto")
        for engine in ("cuda_core", "tensor_core"):
            ffn.set_gate_engine(engine)
            got = []
            for rep in range(3):
                for t in range(2):
                    y = ffn.sparse_ffn_forward(x[t], gate, w["b_g"], w["W_up"], w["W_down"], act)
                    if rep == 0:
                        got.append(y.clone())
                        assert_y_close(y, want[t].double().cpu().numpy(), rel_l2=2e-3, max_abs=2e-3,
                                       what=f"{what} [{engine}] token {t}")
                    else:
                        assert torch.equal(y, got[t]), f"{what} [{engine}] repeat {rep} token {t}"
            torch.cuda.synchronize()
            assert ffn.device_status() == 0, f"{what} [{engine}]: status words {ffn.status_words()}"


@pytest.mark.parametrize("seed", range(4))
def test_random_shapes_batched_paths_agree_with_the_cuda_core_path(mod, seed):
    # The same for batches: whatever `auto` picks (the tcgen05 kernels where the shape allows) and the mma.sync kernels
    # against the CUDA-core kernels, random batch sizes, widths, neuron counts and LoPA ranks.
    g = torch.Generator().manual_seed(5000 + seed)
    ri = lambda lo, hi: int(torch.randint(lo, hi + 1, (1,), generator=g))  # noqa: E731
    for case in range(6):
        B = ri(2, 64)
        D = 128 * ri(2, 32)
        H = ri(100, 6000)
        lopa = ri(0, 2) == 0
        r = 64 * ri(1, min(8, D // 128)) if lopa else 0
        s = (0.6, 0.8, 0.9, 0.97)[ri(0, 3)]
        act = ("relu", "sqrelu", "rsplus")[ri(0, 2)]
        what = f"seed {seed} case {case}: B={B} D={D} H={H} r={r} s={s} {act}"
        ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=r, B_max=B)
        if lopa:
            gate, w = make_lopa(mod, D, H, r, torch.bfloat16, 6000 + 10 * seed + case, s, ("diag", None)[ri(0, 1)],
                                rms=ri(0, 1) == 1)
        else:
            gate, w = make_std(D, H, torch.bfloat16, 6000 + 10 * seed + case, s)
        x = syn.tokens(B, D, torch.bfloat16, 7000 + seed, DEV)
        ffn.set_path("general")
        want = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], act).double().cpu().numpy()
        n_want = int(ffn.last_active().numel())
        for path in ("auto", "mma_sync"):
            ffn.set_path(path)
            try:
                y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
            except mod.SFFNError as e:            # a shape the mma.sync kernels do not take
                assert path == "mma_sync" and e.code == 2, what
                continue
            # the tensor-core paths round h and the LoPA vector to bf16 pairs: a looser band than fp32 against fp32
            assert_y_close(y, want, rel_l2=1e-2, max_abs=2e-2, what=f"{what} [{path}]")
            assert abs(int(ffn.last_active().numel()) - n_want) <= max(4, n_want // 200), f"{what} [{path}]"
            y2 = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
            assert torch.equal(y, y2), f"{what} [{path}] repeat"
            torch.cuda.synchronize()
            assert ffn.device_status() == 0, f"{what} [{path}]: status words {ffn.status_words()}"
