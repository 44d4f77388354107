"""GPU parity of the weight-only int4 entry points (packed 4-bit codes + one fp32 scale per row, bf16 tokens) against
the CPU oracle on the dequantised matrices, through the C ABI.  Run with `-m gpu` on a B200."""
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


def run_oracle_q4(x, gate, w, act, route="sparse", act_up=None):
    if "W_g" in gate:
        kw = dict(W_g=hq(gate["W_g"]))
    else:
        kw = dict(lopa=dict(V=hq(gate["V"]), U=hq(gate["U"]), g_idx=host(gate.get("g_idx")),
                            g_sign=host(gate.get("g_sign")), gamma=host(gate.get("rms_gain")),
                            use_rmsnorm=gate.get("use_rmsnorm", True), eps=gate.get("rms_eps", 1e-5)))
    return oracle.ffn_q4(host(x), hq(w["W_up"]), hq(w["W_down"]), act, b_g=host(w["b_g"]), route=route, threads=8,
                         act_up=act_up, **kw)


def make_std(D, H, seed, s):
    w = syn.standard_ffn_q4(D, H, seed, DEV, sparsity=s)
    return {"W_g": w["W_g"]}, w


def make_lopa(mod, D, H, r, seed, s, fixed=True, rms=True):
    w = syn.lopa_ffn_q4(D, H, r, seed, DEV, sparsity=s, with_fixed_matrix=fixed)
    gate = {"V": w["V"], "U": w["U"], "use_rmsnorm": rms, "rms_eps": 1e-5,
            "g_idx": mod.g_diagonal(H, D, DEV) if fixed else None}
    return gate, w


def check(ffn, x, gate, w, act, paths, what, act_up=None):
    ref = run_oracle_q4(x, gate, w, act, act_up=act_up)
    for path in paths:
        ffn.set_path(path)
        y = ffn.sparse_ffn_forward_q4(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert ffn.device_status() == 0
        # a batch on the tensor-core kernels (auto): Hm is rounded to bf16 there, as for bf16 weights -> default tolerance
        kw = {} if path == "auto" and x.ndim == 2 and x.shape[0] > 1 else dict(rel_l2=TOL, max_abs=TOL)
        assert_y_close(y, ref["y"], what=f"{what} [{path}]", **kw)
        assert_active_set(ffn.last_active(), ref, what=f"{what} [{path}]")
        yd = ffn.dense_ffn_forward_q4(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert_y_close(yd, ref["y"], what=f"{what} dense [{path}]", **kw)
    ffn.set_path("auto")
    return ref


@pytest.mark.parametrize("D,H", [(512, 1000), (1024, 2049), (2048, 300), (4096, 1200)])
def test_int4_standard_gate_one_token(mod, D, H):
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    gate, w = make_std(D, H, 31, 0.8)
    x = syn.tokens(3, D, torch.bfloat16, 31, DEV)
    for t in range(3):
        ref = check(ffn, x[t], gate, w, ("relu", "sqrelu", "rsplus")[t], ("general", "fused"), f"q4 {D}x{H} t{t}")
        assert 0 < ref["n_act"][0] < H


@pytest.mark.parametrize("r,fixed,rms", [(64, True, True), (128, False, True), (96, True, False)])
def test_int4_lopa_gate_one_token(mod, r, fixed, rms):
    D, H = 1024, 3000
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=r, B_max=1)
    gate, w = make_lopa(mod, D, H, r, 32, 0.85, fixed, rms)
    x = syn.tokens(2, D, torch.bfloat16, 32, DEV)
    for t in range(2):
        check(ffn, x[t], gate, w, "relu", ("general", "fused"), f"q4 lopa r={r} t{t}")


@pytest.mark.parametrize("B", [2, 5, 16, 40, 70])
def test_int4_batches_on_the_tensor_cores_token_by_token_and_on_the_cuda_core_kernels(mod, B):
    """auto = the tcgen05 kernels (codes expanded to bf16 on the way to the tensor cores; Hm is rounded to bf16 there
    as for bf16 weights, hence the default tolerance), fused = token by token, general = CUDA-core batch kernels."""
    D, H = 1024, 2049
    ffn = mod.SparseFFN(D, H, torch.bfloat16, r_max=64, B_max=B)
    for gate, w, act in (make_std(D, H, 33, 0.8) + ("relu",), make_lopa(mod, D, H, 64, 34, 0.8) + ("rsplus",)):
        x = syn.tokens(B, D, torch.bfloat16, 33, DEV)
        ref = run_oracle_q4(x, gate, w, act)
        for path, kw in (("auto", {}), ("fused", dict(rel_l2=TOL, max_abs=TOL)), ("general", dict(rel_l2=TOL, max_abs=TOL))):
            if path == "general" and B > 16:
                continue                                         # slow, and covered by the smaller batches
            ffn.set_path(path)
            y = ffn.sparse_ffn_forward_q4(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
            torch.cuda.synchronize()
            assert ffn.device_status() == 0, f"q4 B={B} [{path}]: status words {ffn.status_words()}"
            assert_y_close(y, ref["y"], what=f"q4 B={B} {act} [{path}]", **kw)
            assert_active_set(ffn.last_active(), ref, what=f"q4 B={B} {act} [{path}]")
            yd = ffn.dense_ffn_forward_q4(x, gate, w["b_g"], w["W_up"], w["W_down"], act)
            torch.cuda.synchronize()
            assert_y_close(yd, ref["y"], what=f"q4 B={B} {act} dense [{path}]", **kw)
        ffn.set_path("auto")


@pytest.mark.parametrize("D,H,B,s", [
    (512, 19072, 40, 0.9),    # several tiles per CTA, 48 token columns: the last tile's epilogue is shared by all warps
    (256, 20000, 8, 0.2),     # union = every row
    (256, 776, 3, 0.9),       # ragged last tile
    (4096, 1200, 16, 0.9),    # long rows: 64 K blocks per tile
])
def test_int4_batches_tcgen05_edge_shapes(mod, D, H, B, s):
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=B)
    gate, w = make_std(D, H, 35, s)
    x = syn.tokens(B, D, torch.bfloat16, 35, DEV)
    ref = run_oracle_q4(x, gate, w, "relu")
    y = ffn.sparse_ffn_forward_q4(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0, ffn.status_words()
    assert_y_close(y, ref["y"], what=f"q4 edge {D}x{H} B={B}")
    assert_active_set(ffn.last_active(), ref, what=f"q4 edge {D}x{H} B={B}")
    y2 = ffn.sparse_ffn_forward_q4(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert torch.equal(y, y2)


def test_int4_full_size_decode_point_double_activation_and_repeatability(mod):
    D, H = 4096, 14336
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=1)
    gate, w = make_std(D, H, 35, 0.9)
    x = syn.tokens(2, D, torch.bfloat16, 35, DEV)
    ref = check(ffn, x[0], gate, w, "relu", ("fused",), "q4 4096x14336")
    assert abs(ref["n_act"][0] / H - 0.1) < 0.03
    y0 = ffn.sparse_ffn_forward_q4(x[0], gate, w["b_g"], w["W_up"], w["W_down"], "relu").clone()
    for _ in range(3):
        assert torch.equal(ffn.sparse_ffn_forward_q4(x[0], gate, w["b_g"], w["W_up"], w["W_down"], "relu"), y0)
    ffn.set_up_activation("relu")
    ref = run_oracle_q4(x[1], gate, w, "sqrelu", act_up="relu")
    y = ffn.sparse_ffn_forward_q4(x[1], gate, w["b_g"], w["W_up"], w["W_down"], "sqrelu")
    assert_y_close(y, ref["y"], rel_l2=TOL, max_abs=TOL, what="q4 double activation")
    torch.cuda.synchronize()
    assert ffn.device_status() == 0


def test_int4_argument_checks(mod):
    D, H = 1024, 512
    gate, w = make_std(D, H, 36, 0.8)
    x32 = syn.tokens(1, D, torch.float32, 36, DEV)
    with pytest.raises(mod.SFFNError) as e:                       # 4-bit weights meet bf16 tokens only
        mod.SparseFFN(D, H, torch.float32, B_max=1).sparse_ffn_forward_q4(x32[0], gate, w["b_g"], w["W_up"], w["W_down"])
    assert e.value.code == 2
    D2 = 1040                                                     # rows of 520 bytes: not a multiple of 16
    gate2, w2 = make_std(D2, H, 36, 0.8)
    with pytest.raises(mod.SFFNError) as e:
        mod.SparseFFN(D2, H, torch.bfloat16, B_max=1).sparse_ffn_forward_q4(
            syn.tokens(1, D2, torch.bfloat16, 36, DEV)[0], gate2, w2["b_g"], w2["W_up"], w2["W_down"])
    assert e.value.code == 2
