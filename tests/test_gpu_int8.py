"""GPU parity of the weight-only int8 entry points (int8 codes + one fp32 scale per row, bf16 tokens) against the
CPU oracle on the dequantised matrices, through the C ABI.  Run with `-m gpu` on a B200."""
import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as syn
from parity import assert_active_set, assert_y_close, host

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-3  # codes and tokens decode exactly on both sides; what is left is fp32 accumulation order


@pytest.fixture(scope="module")
def mod():
    import paper_2609_31975_b200 as m
    m.load_library()
    return m


def hq(m):
    return dict(q=host(m["q"]), s=host(m["s"]))


def run_oracle_q8(x, gate, w, act, route="sparse", act_up=None):
    if "W_g" in gate:
        kw = dict(W_g=hq(gate["W_g"]))
    else:
        kw = dict(lopa=dict(V=hq(gate["V"]), U=hq(gate["U"]), g_idx=host(gate.get("g_idx")),
                            g_sign=host(gate.get("g_sign")), gamma=host(gate.get("rms_gain")),
                            use_rmsnorm=gate.get("use_rmsnorm", True), eps=gate.get("rms_eps", 1e-5)))
    return oracle.ffn_q8(host(x), hq(w["W_up"]), hq(w["W_down"]), act, b_g=host(w["b_g"]), route=route, threads=8,
                         act_up=act_up, **kw)


def make_std(D, H, seed, s):
    w = syn.standard_ffn_q8(D, H, seed, DEV, sparsity=s)
    return {"W_g": w["W_g"]}, w


def make_lopa(mod, D, H, r, seed, s, fixed=True, sign=False, gain=False, rms=True):
    w = syn.lopa_ffn_q8(D, H, r, seed, DEV, sparsity=s, with_fixed_matrix=fixed)
    gate = {"V": w["V"], "U": w["U"], "use_rmsnorm": rms, "rms_eps": 1e-5,
            "g_idx": mod.g_diagonal(H, D, DEV) if fixed else None}
    g = torch.Generator().manual_seed(seed)
    if sign:
        gate["g_sign"] = (torch.randint(0, 2, (H,), generator=g) * 2 - 1).to(torch.int8).to(DEV)
    if gain:
        gate["rms_gain"] = (0.5 + torch.rand(r, generator=g)).to(DEV)
    return gate, w


def check(mod, ffn, x, gate, w, act, paths, what, act_up=None):
    ref = run_oracle_q8(x, gate, w, act, act_up=act_up)
    for path in paths:
        ffn.set_path(path)
        y = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert ffn.device_status() == 0
        # a batch on the tensor-core kernels (auto): Hm is rounded to bf16 there, as for bf16 weights -> default tolerance
        kw = {} if path == "auto" and x.ndim == 2 and x.shape[0] > 1 else dict(rel_l2=TOL, max_abs=TOL)
        assert_y_close(y, ref["y"], what=f"{what} [{path}]", **kw)
        assert_active_set(ffn.last_active(), ref, what=f"{what} [{path}]")
        yd = ffn.dense_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert_y_close(yd, ref["y"], what=f"{what} dense [{path}]", **kw)
    ffn.set_path("auto")
    return ref


@pytest.mark.parametrize("D,H", [(512, 1000), (272, 777), (1024, 2049), (2048, 300), (4096, 600)])
def test_int8_standard_gate_one_token(mod, D, H):
    gate, w = make_std(D, H, 11, 0.85)
    x = syn.tokens(3, D, torch.bfloat16, 11, DEV)
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    for t in range(3):
        ref = check(mod, ffn, x[t], gate, w, ("relu", "sqrelu", "rsplus")[t], ("general", "fused"), f"q8 {D}x{H} t{t}")
        assert 0 < ref["n_act"][0] < H


@pytest.mark.parametrize("r,fixed,sign,gain,rms", [
    (64, True, False, False, True), (128, True, True, True, True), (512, False, False, True, True),
    (96, True, True, False, False)])
def test_int8_lopa_gate_one_token(mod, r, fixed, sign, gain, rms):
    D, H = 1024, 3000
    gate, w = make_lopa(mod, D, H, r, 12, 0.9, fixed, sign, gain, rms)
    x = syn.tokens(2, D, torch.bfloat16, 12, DEV)
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=r, B_max=1)
    for t in range(2):
        check(mod, ffn, x[t], gate, w, "relu", ("general", "fused"), f"q8 lopa r={r} t{t}")


def check_batch(mod, ffn, x, gate, w, act, what, act_up=None):
    """auto = the tcgen05 kernels (codes expanded to bf16 on the way to the tensor cores; Hm is rounded to bf16 there
    as for bf16 weights, hence the default tolerance), fused = token by token, general = CUDA-core batch kernels."""
    ref = run_oracle_q8(x, gate, w, act, act_up=act_up)
    dref = run_oracle_q8(x, gate, w, act, route="dense", act_up=act_up)
    ffn.set_up_activation(act_up)
    for path, kw in (("auto", {}), ("fused", dict(rel_l2=TOL, max_abs=TOL)), ("general", dict(rel_l2=TOL, max_abs=TOL))):
        ffn.set_path(path)
        y = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert ffn.device_status() == 0, f"{what} [{path}]: status words {ffn.status_words()}"
        assert_y_close(y, ref["y"], what=f"{what} [{path}]", **kw)
        assert_active_set(ffn.last_active(), ref, what=f"{what} [{path}]")
        yd = ffn.dense_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert_y_close(yd, dref["y"], what=f"{what} dense [{path}]", **kw)
    ffn.set_path("auto")
    ffn.set_up_activation(None)
    return ref


@pytest.mark.parametrize("B", [2, 3, 4, 7, 16, 33, 64, 70])
def test_int8_batches_on_the_tensor_cores_token_by_token_and_on_the_cuda_core_kernels(mod, B):
    D, H = 1024, 2500
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=128, B_max=70)
    gate, w = make_std(D, H, 13, 0.9)
    x = syn.tokens(B, D, torch.bfloat16, 13, DEV)
    ref = check_batch(mod, ffn, x, gate, w, "relu", f"q8 B={B}")
    assert ref["union_mask"].sum() > ref["n_act"].max() or B == 1
    n0 = ffn.launch_count()
    ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert ffn.launch_count() - n0 < B or B <= 4                 # the batch kernels, not one launch per token
    gate, w = make_lopa(mod, D, H, 128, 13, 0.9, sign=True, gain=True)
    check_batch(mod, ffn, x, gate, w, "rsplus", f"q8 lopa B={B}", act_up="silu" if B == 16 else None)
    ffn.set_path("mma_sync")   # the warp-level tensor-core kernels take bf16 weights only
    with pytest.raises(mod.SFFNError) as e:
        ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert e.value.code == 2


@pytest.mark.parametrize("D,H,B,s", [
    (512, 19072, 40, 0.9),    # several tiles per CTA, 48 token columns: the last tile's epilogue is shared by all warps
    (512, 19072, 40, 0.99),   # the same with a short union (gathered rows)
    (256, 20000, 8, 0.2),     # union = every row
    (256, 777, 3, 0.9),       # H not a multiple of 8: ragged last tile
    (4096, 1200, 16, 0.9),    # long rows: 64 K blocks per tile
    (256, 64, 2, 0.5),        # fewer rows than one tile of eight per CTA
])
def test_int8_batches_tcgen05_edge_shapes(mod, D, H, B, s):
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=B)
    gate, w = make_std(D, H, 15, s)
    x = syn.tokens(B, D, torch.bfloat16, 15, DEV)
    ref = run_oracle_q8(x, gate, w, "relu")
    y = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0, ffn.status_words()
    assert_y_close(y, ref["y"], what=f"q8 edge {D}x{H} B={B}")
    assert_active_set(ffn.last_active(), ref, what=f"q8 edge {D}x{H} B={B}")
    y2 = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert torch.equal(y, y2)


@pytest.mark.parametrize("path", ["general", "fused"])
def test_int8_full_and_zero_sparsity_and_double_activation(mod, path):
    D, H = 768, 1500
    gate, w = make_std(D, H, 14, 0.9)
    x = syn.tokens(1, D, torch.bfloat16, 14, DEV)[0]
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    ffn.set_path(path)
    w["b_g"] = torch.full((H,), 50.0, device=DEV)    # everything fires: sparse = dense
    ref = run_oracle_q8(x, gate, w, "relu")
    assert ref["n_act"][0] == H
    y = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert_y_close(y, ref["y"], rel_l2=TOL, max_abs=TOL, what="all fire")
    assert len(ffn.last_active()) == H
    w["b_g"] = torch.full((H,), -50.0, device=DEV)   # nothing fires: y = 0 exactly
    y = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    torch.cuda.synchronize()
    assert not y.any() and len(ffn.last_active()) == 0
    w["b_g"] = torch.full((H,), -1.0, device=DEV)
    for act, act_up in (("relu", "relu"), ("sqrelu", "rsplus")):
        ffn.set_up_activation(act_up)
        ref = run_oracle_q8(x, gate, w, act, act_up=act_up)
        assert 0 < ref["n_gated"][0] < ref["n_act"][0]
        y = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        assert_y_close(y, ref["y"], rel_l2=TOL, max_abs=TOL, what=f"double activation {act}/{act_up}")
    ffn.set_up_activation(None)
    assert ffn.device_status() == 0


def test_int8_repeat_bit_for_bit_and_scales_matter(mod):
    D, H = 2048, 4000
    gate, w = make_std(D, H, 15, 0.9)
    x = syn.tokens(1, D, torch.bfloat16, 15, DEV)[0]
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    y0 = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu").clone()
    for _ in range(5):
        y = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        assert torch.equal(y, y0)
    # doubling the scales of W_down doubles y exactly (a power of two); doubling those of W_up as well: x4
    w2 = dict(w, W_down=dict(q=w["W_down"]["q"], s=w["W_down"]["s"] * 2))
    y2 = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w2["W_up"], w2["W_down"], "relu")
    assert torch.equal(y2, 2 * y0)
    w4 = dict(w2, W_up=dict(q=w["W_up"]["q"], s=w["W_up"]["s"] * 2))
    y4 = ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w4["W_up"], w4["W_down"], "relu")
    assert torch.equal(y4, 4 * y0)


def test_int8_argument_checks(mod):
    D, H = 512, 640
    gate, w = make_std(D, H, 16, 0.9)
    x32 = syn.tokens(1, D, torch.float32, 16, DEV)[0]
    f32 = mod.SparseFFN(D, H, torch.float32, B_max=1)
    with pytest.raises(mod.SFFNError) as e:   # int8 weights meet bf16 tokens only
        f32.sparse_ffn_forward_q8(x32, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert e.value.code == 2
    D2 = 264                                   # rows of 264 bytes: not a multiple of 16
    gate2, w2 = make_std(D2, H, 16, 0.9)
    ffn2 = mod.SparseFFN(D2, H, torch.bfloat16, B_max=1)
    with pytest.raises(mod.SFFNError) as e:
        ffn2.sparse_ffn_forward_q8(syn.tokens(1, D2, torch.bfloat16, 16, DEV)[0], gate2, w2["b_g"], w2["W_up"],
                                   w2["W_down"], "relu")
    assert e.value.code == 2
    with pytest.raises(TypeError):             # scales of the wrong type never reach the library
        bad = dict(q=w["W_up"]["q"], s=w["W_up"]["s"].double())
        mod.SparseFFN(D, H, torch.bfloat16, B_max=1).sparse_ffn_forward_q8(
            syn.tokens(1, D, torch.bfloat16, 16, DEV)[0], gate, w["b_g"], bad, w["W_down"], "relu")


@pytest.mark.parametrize("D,H", [(8192, 300), (16384, 160)])
def test_int8_wide_rows(mod, D, H):
    gate, w = make_std(D, H, 17, 0.8)
    x = syn.tokens(1, D, torch.bfloat16, 17, DEV)[0]
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=2)
    paths = ("general", "fused") if D <= 8192 else ("general", "auto")   # 16 KB rows: CUDA-core kernels only
    check(mod, ffn, x, gate, w, "relu", paths, f"q8 wide {D}")
    if D > 8192:
        ffn.set_path("fused")
        with pytest.raises(mod.SFFNError) as e:
            ffn.sparse_ffn_forward_q8(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        assert e.value.code == 2


def test_int8_widest_rows_batch_of_four(mod):
    """16384 codes per row: the gate kernel stages its tokens as fp32 in shared memory and takes two tokens per pass
    there (four would need 256 KB)."""
    D, H = 16384, 160
    gate, w = make_std(D, H, 18, 0.8)
    x = syn.tokens(4, D, torch.bfloat16, 18, DEV)
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=4)
    check(mod, ffn, x, gate, w, "relu", ("general", "auto"), "q8 wide 16384 B=4")


def test_int8_full_size_decode_and_lopa(mod):
    D, H = 4096, 14336
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=512, B_max=4)
    gate, w = make_std(D, H, 18, 0.9)
    x = syn.tokens(4, D, torch.bfloat16, 18, DEV)
    for t in range(2):
        ref = check(mod, ffn, x[t], gate, w, "relu", ("general", "fused"), f"q8 full size t{t}")
        assert abs(1 - ref["n_act"][0] / H - 0.9) < 0.03
    check(mod, ffn, x, gate, w, "relu", ("auto",), "q8 full size B=4")
    del gate, w
    gate, w = make_lopa(mod, D, H, 512, 18, 0.9, sign=True, gain=True)
    check(mod, ffn, x[0], gate, w, "relu", ("general", "fused"), "q8 full size lopa")


@pytest.mark.parametrize("seed", range(4))
def test_random_shapes_quantised_batches_agree_with_the_single_token_kernel(mod, seed):
    """int8 and int4 rows: the tcgen05 batch kernels (auto) against the single-token kernel run once per token (fused),
    random batch sizes (beyond 64 too: chunks), widths, neuron counts, LoPA ranks and activations."""
    g = torch.Generator().manual_seed(8000 + seed)
    ri = lambda lo, hi: int(torch.randint(lo, hi + 1, (1,), generator=g))  # noqa: E731
    for case in range(6):
        bits = (8, 4)[ri(0, 1)]
        B = ri(2, 40) if ri(0, 3) else ri(65, 100)
        D = 256 * ri(1, 16)
        H = ri(100, 6000) if ri(0, 4) else ri(19000, 24000)
        lopa = ri(0, 2) == 0
        r = 64 * ri(1, min(8, D // 128)) if lopa else 0
        s = (0.6, 0.8, 0.9, 0.97)[ri(0, 3)]
        act = ("relu", "sqrelu", "rsplus")[ri(0, 2)]
        what = f"seed {seed} case {case}: int{bits} B={B} D={D} H={H} r={r} s={s} {act}"
        ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=r, B_max=B)
        sd = 9000 + 10 * seed + case
        if lopa:
            w = (syn.lopa_ffn_q8 if bits == 8 else syn.lopa_ffn_q4)(D, H, r, sd, DEV, sparsity=s, with_fixed_matrix=True)
            gate = {"V": w["V"], "U": w["U"], "use_rmsnorm": ri(0, 1) == 1, "rms_eps": 1e-5, "g_idx": mod.g_diagonal(H, D, DEV)}
        else:
            w = (syn.standard_ffn_q8 if bits == 8 else syn.standard_ffn_q4)(D, H, sd, DEV, sparsity=s)
            gate = {"W_g": w["W_g"]}
        x = syn.tokens(B, D, torch.bfloat16, sd, DEV)
        f = ffn.sparse_ffn_forward_q8 if bits == 8 else ffn.sparse_ffn_forward_q4
        ffn.set_path("fused")
        try:
            want = f(x, gate, w["b_g"], w["W_up"], w["W_down"], act).double().cpu().numpy()
        except mod.SFFNError as e:                 # a shape the single-token kernel does not take
            assert e.code == 2, what
            continue
        n_want = int(ffn.last_active().numel())
        ffn.set_path("auto")
        n0 = ffn.launch_count()
        y = f(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        assert B <= 8 or ffn.launch_count() - n0 < B, what   # the batch kernels ran, not one launch per token
        # the tensor-core path rounds h and the LoPA vector to bf16 pairs: a looser band than fp32 against fp32
        assert_y_close(y, want, rel_l2=1e-2, max_abs=2e-2, what=what)
        assert abs(int(ffn.last_active().numel()) - n_want) <= max(4, n_want // 200), what
        y2 = f(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        assert torch.equal(y, y2), f"{what} repeat"
        torch.cuda.synchronize()
        assert ffn.device_status() == 0, f"{what}: status words {ffn.status_words()}"


@pytest.mark.parametrize("bits", [8, 4])
def test_quantised_rows_with_outliers_in_the_token(mod, bits):
    """The integer routes split the token into int8 limbs: per 16-byte chunk of a row in the single-token kernel, per
    token in the batch kernels.  Entries a thousand times the rest (as activations of language models have) must not
    cost the other entries their precision."""
    D, H = 2048, 3000
    w = (syn.standard_ffn_q8 if bits == 8 else syn.standard_ffn_q4)(D, H, 77, DEV, sparsity=0.8)
    gate = {"W_g": w["W_g"]}
    x = syn.tokens(6, D, torch.bfloat16, 77, DEV).clone()
    x[:, 5] *= 1000.0
    x[1, 777] *= -300.0
    x[2, 1024:] *= 1e-3
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=6)
    oracle_ffn = oracle.ffn_q8 if bits == 8 else oracle.ffn_q4
    f = ffn.sparse_ffn_forward_q8 if bits == 8 else ffn.sparse_ffn_forward_q4
    ref = oracle_ffn(host(x), hq(w["W_up"]), hq(w["W_down"]), "relu", b_g=host(w["b_g"]), threads=8, W_g=hq(gate["W_g"]))
    def same_fired_set(got_idx, z, what):
        # the outliers scale every z by hundreds, so the dead band of the fired-set check is taken relative to max |z|
        z = z if z.ndim == 2 else z[None, :]
        got = np.zeros(z.shape[1], bool)
        got[got_idx.cpu().numpy()] = True
        diff = np.nonzero(got != (z > 0).any(axis=0))[0]
        band = 1e-4 * np.abs(z).max()
        assert all((np.abs(z[:, j]) < band).any() and not (z[:, j] >= band).any() for j in diff), f"{what}: {len(diff)} differ"

    for t in range(3):                                           # one token: integer dot products, limbs per chunk
        y = f(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        assert_y_close(y, ref["y"][t], rel_l2=TOL, max_abs=TOL, what=f"int{bits} outlier token {t}")
        same_fired_set(ffn.last_active(), ref["z"][t], f"int{bits} outlier token {t}")
    y = f(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")     # the batch: int8 MMAs, four limbs per token
    assert_y_close(y, ref["y"], what=f"int{bits} outlier batch")
    same_fired_set(ffn.last_active(), ref["z"], f"int{bits} outlier batch")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0
