"""Pins for the CPU oracle: everything here runs without a GPU and without the CUDA library.

Each test fixes the oracle to something other than itself: hand-worked numbers, the activation
table, printed closed-form values, brute force on tiny inputs, a library matmul written with W_2 in
its own [D, H] orientation, or an invariant of the mathematics.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as syn

RNG = np.random.default_rng(1234)


# ---------------------------------------------------------------- hand-worked examples (Eq. 1)
W1_EX = np.array([[1.0, 2.0], [-1.0, 0.5], [0.5, 0.5]], np.float32)
W3_EX = np.array([[2.0, 0.0], [1.0, 1.0], [0.0, -1.0]], np.float32)
W2_EX = np.array([[1.0, 10.0, 3.0], [-1.0, 20.0, 0.5]], np.float32)  # [D, H] as in Eq. 1
X_EX = np.array([1.0, -2.0], np.float32)
B_EX = np.array([4.0, 0.0, 1.0], np.float32)


def test_hand_worked_standard_ffn():
    # z = W1 x + b = [1-4+4, -1-1+0, 0.5-1+1] = [1, -2, 0.5];  u = W3 x = [2, -1, 2]
    # RELU: h = [1*2, 0, 0.5*2] = [2, 0, 1];  y = W2 h = [2+0+3, -2+0+0.5] = [5, -1.5]
    for route in ("dense", "sparse"):
        out = oracle.ffn(X_EX, W3_EX, np.ascontiguousarray(W2_EX.T), "relu", W_g=W1_EX, b_g=B_EX,
                         route=route)
        np.testing.assert_array_equal(out["z"], [1.0, -2.0, 0.5])
        np.testing.assert_array_equal(out["y"], [5.0, -1.5])
        assert out["n_act"][0] == 2
        np.testing.assert_array_equal(out["union_mask"], [True, False, True])
        # squared RELU: a = [1, 0, .25]; h = [2, 0, .5]; y = [2+1.5, -2+.25]
        out = oracle.ffn(X_EX, W3_EX, np.ascontiguousarray(W2_EX.T), "sqrelu", W_g=W1_EX, b_g=B_EX,
                         route=route)
        np.testing.assert_array_equal(out["y"], [3.5, -1.75])
    # without the bias (the paper's form): z = [-3, -2, -0.5] -> nothing fires, y = 0
    out = oracle.ffn(X_EX, W3_EX, np.ascontiguousarray(W2_EX.T), "relu", W_g=W1_EX)
    np.testing.assert_array_equal(out["y"], [0.0, 0.0])
    assert out["n_act"][0] == 0


def test_hand_worked_lopa_gate():
    V = np.array([[3.0, 4.0], [1.0, 0.0]], np.float32)        # v = V x = [-5, 1]
    U = np.array([[1.0, 2.0], [-0.2, 0.0], [0.4, -1.0]], np.float32)
    g_idx, g_sign = np.array([0, 0, 1], np.int32), np.array([1, -1, 1], np.int8)
    b = np.array([0.0, 0.0, 5.0], np.float32)
    # no RMSNorm: U v = [-5+2, 1, -2-1] = [-3, 1, -3];  G x = [1, -1, -2];  z = [-2, 0, 0]
    z, v, n = oracle.gate_lopa(V, U, X_EX, g_idx, g_sign, None, False, 0.0, b, return_vn=True)
    np.testing.assert_allclose(v, [-5.0, 1.0], atol=0)
    np.testing.assert_allclose(z, [-2.0, 0.0, 0.0], atol=1e-6)  # U holds fp32(0.2), fp32(0.4)
    # RMSNorm: mean(v^2) = 13, eps = 3 -> rms = 4;  gamma = [2, 4] -> n = [-2.5, 1]
    # U n = [-0.5, 0.5, -2];  z = U n + G x + b = [0.5, -0.5, 1]
    gamma = np.array([2.0, 4.0], np.float32)
    z, v, n = oracle.gate_lopa(V, U, X_EX, g_idx, g_sign, gamma, True, 3.0, b, return_vn=True)
    np.testing.assert_allclose(n, [-2.5, 1.0], atol=1e-15)
    np.testing.assert_allclose(z, [0.5, -0.5, 1.0], atol=1e-6)
    # dropping the fixed matrix leaves U n + b
    z = oracle.gate_lopa(V, U, X_EX, None, None, gamma, True, 3.0, b)
    np.testing.assert_allclose(z, [-0.5, 0.5, 3.0], atol=1e-6)


def test_activation_table(golden):
    for act, x, want in golden("activation_table.txt"):
        assert oracle.activation(act, float(x)) == pytest.approx(float(want), abs=1e-15), (act, x)
    # R-S+ equals SILU on the non-negative side and RELU's zero on the negative side
    for x in np.linspace(0.0, 6.0, 25):
        assert oracle.activation("rsplus", x) == pytest.approx(x / (1 + math.exp(-x)), rel=1e-15)
    for x in (-1e-30, -0.5, -40.0):
        assert oracle.activation("rsplus", x) == 0.0 and oracle.activation("relu", x) == 0.0
    assert oracle.activation("relu", -0.0) == 0.0
    assert oracle.activation("sqrelu", 1e-200) == 0.0   # z*z underflows; activity is decided on z
    # SILU: x * sigmoid(x) on both sides; odd part is x / 2 (silu(x) - silu(-x) = x), minimum near x = -1.2785
    for x in np.linspace(-6.0, 6.0, 49):
        assert oracle.activation("silu", x) == pytest.approx(x / (1 + math.exp(-x)), rel=1e-15, abs=1e-300)
        assert oracle.activation("silu", x) - oracle.activation("silu", -x) == pytest.approx(x, abs=1e-14)
        if x >= 0:
            assert oracle.activation("silu", x) == oracle.activation("rsplus", x)
    assert oracle.activation("silu", -1.2785) == pytest.approx(-0.27846, abs=1e-5)


def test_bf16_inputs_decode_exactly():
    # bf16 bit patterns: 1.0 = 0x3F80, -2.0 = 0xC000, 0.5 = 0x3F00, 3.0 = 0x4040, -1.5 = 0xBFC0
    W = np.array([[0x3F80, 0xC000], [0x3F00, 0x4040]], np.uint16)   # [[1, -2], [0.5, 3]]
    x = np.array([0x4040, 0xBFC0], np.uint16)                        # [3, -1.5]
    np.testing.assert_array_equal(oracle.gate_standard(W, x), [3.0 + 3.0, 1.5 - 4.5])
    t = torch.tensor([[1.0, -2.0], [0.5, 3.0]], dtype=torch.bfloat16)
    np.testing.assert_array_equal(oracle.as_oracle_array(t), W)


# ---------------------------------------------------------------- library routine, other orientation
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("act", ["relu", "sqrelu", "rsplus"])
def test_dense_route_matches_matmul_with_w2_as_D_by_H(dtype, act):
    D, H = 40, 112
    w = syn.standard_ffn(D, H, dtype, seed=11, sparsity=0.5)
    x = syn.tokens(3, D, dtype, seed=11)
    out = oracle.ffn(x, w["W_up"], w["W_down"], act, W_g=w["W_g"], b_g=w["b_g"], route="dense")
    W1, W3 = w["W_g"].double().numpy(), w["W_up"].double().numpy()
    W2 = w["W_down"].double().numpy().T.copy()          # [D, H]: Eq. 1's own orientation
    for b in range(3):
        xb = x[b].double().numpy()
        z = W1 @ xb + w["b_g"].double().numpy()
        a = {"relu": np.maximum(z, 0), "sqrelu": np.maximum(z, 0) ** 2,
             "rsplus": np.where(z >= 0, z / (1 + np.exp(-z)), 0.0)}[act]
        y = W2 @ (a * (W3 @ xb))
        np.testing.assert_allclose(out["z"][b], z, rtol=0, atol=1e-12)
        np.testing.assert_allclose(out["y"][b], y, rtol=1e-11, atol=1e-12)


def test_gate_is_affine_in_x():
    D, H = 33, 70
    W = RNG.standard_normal((H, D)).astype(np.float32)
    x = RNG.standard_normal(D).astype(np.float32)
    b = RNG.standard_normal(H).astype(np.float32)
    z1 = oracle.gate_standard(W, x, b) - b.astype(np.float64)
    z4 = oracle.gate_standard(W, (4.0 * x).astype(np.float32), b) - b.astype(np.float64)
    np.testing.assert_allclose(z4, 4.0 * z1, rtol=1e-13, atol=1e-13)  # scaling by 4 is exact in fp32


# ---------------------------------------------------------------- active set
def test_active_set_brute_force():
    z = RNG.standard_normal(500)
    z[[3, 77, 200]] = [0.0, -0.0, 1e-300]
    for act in ("relu", "sqrelu", "rsplus"):
        # brute force: evaluate A(z_j) for every j and keep the nonzeros; squared RELU underflows at
        # 1e-300, so activity is decided on z (a contributes nothing either way)
        brute = [j for j in range(500) if oracle.activation(act, z[j]) != 0.0 or z[j] > 0]
        got = oracle.active_set(z)
        assert got.tolist() == brute == sorted(brute)
        assert len(got) + int(np.sum(~(z > 0))) == 500
    assert 3 not in got and 77 not in got and 200 in got


def test_config1_sparsity_statistics():
    # tiny bring-up config: D=256, H=1024, fp32, RELU, b_g = -Phi^-1(0.9), 64 tokens, seed 0
    w = syn.standard_ffn(256, 1024, torch.float32, seed=0, sparsity=0.9)
    assert w["b_g"][0].item() == pytest.approx(-1.2815516, abs=1e-6)
    x = syn.tokens(64, 256, torch.float32, seed=0)
    out = oracle.ffn(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=w["b_g"], threads=4)
    sparsity = 1.0 - out["n_act"].mean() / 1024
    assert abs(sparsity - 0.9) < 0.01
    assert np.std(out["z"] - w["b_g"][0].item()) == pytest.approx(1.0, abs=0.03)


# ---------------------------------------------------------------- sparse execution is exact
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sparse_route_is_bit_identical_to_dense_route(dtype):
    D, H = 48, 130
    w = syn.standard_ffn(D, H, dtype, seed=5, sparsity=0.8)
    x = syn.tokens(4, D, dtype, seed=5)
    for act in ("relu", "sqrelu", "rsplus"):
        d = oracle.ffn(x, w["W_up"], w["W_down"], act, W_g=w["W_g"], b_g=w["b_g"], route="dense")
        s = oracle.ffn(x, w["W_up"], w["W_down"], act, W_g=w["W_g"], b_g=w["b_g"], route="sparse")
        assert np.array_equal(d["y"], s["y"]) and np.array_equal(d["z"], s["z"])
        assert 0 < s["n_act"].min() and s["n_act"].max() < H


def test_zero_and_full_sparsity_and_single_neuron():
    D, H = 24, 60
    w = syn.standard_ffn(D, H, torch.float32, seed=6, sparsity=None)
    x = syn.tokens(1, D, torch.float32, seed=6)[0]
    hi, lo = torch.full((H,), 1e3), torch.full((H,), -1e3)
    full = oracle.ffn(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=hi, route="sparse")
    dense = oracle.ffn(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=hi, route="dense")
    assert full["n_act"][0] == H and np.array_equal(full["y"], dense["y"])
    none = oracle.ffn(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=lo, route="sparse")
    assert none["n_act"][0] == 0 and not none["y"].any()
    # exactly one active neuron j: y = a_j u_j W_down[j]
    j = 17
    one = lo.clone()
    one[j] = 1e3
    out = oracle.ffn(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=one)
    xd = x.double().numpy()
    a = float(w["W_g"][j].double().numpy() @ xd + 1e3)
    u = float(w["W_up"][j].double().numpy() @ xd)
    assert out["n_act"][0] == 1
    np.testing.assert_allclose(out["y"], a * u * w["W_down"][j].double().numpy(), rtol=1e-12)


def test_neuron_permutation_invariance():
    D, H = 32, 90
    w = syn.standard_ffn(D, H, torch.float32, seed=7, sparsity=0.7)
    x = syn.tokens(1, D, torch.float32, seed=7)[0]
    perm = torch.randperm(H, generator=torch.Generator().manual_seed(1))
    a = oracle.ffn(x, w["W_up"], w["W_down"], "rsplus", W_g=w["W_g"], b_g=w["b_g"])
    b = oracle.ffn(x, w["W_up"][perm], w["W_down"][perm], "rsplus", W_g=w["W_g"][perm],
                   b_g=w["b_g"][perm])
    np.testing.assert_allclose(a["y"], b["y"], rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(a["z"][perm.numpy()], b["z"])


# ---------------------------------------------------------------- LoPA gate (Eq. 3)
def test_lopa_equals_materialised_gate():
    D, H, r = 12, 30, 5
    V, U = RNG.standard_normal((r, D)), RNG.standard_normal((H, r))
    x = RNG.standard_normal(D)
    b = RNG.standard_normal(H).astype(np.float32)
    for gen in (oracle.g_diagonal, oracle.g_tiled):
        g_idx = gen(H, D)
        sign = RNG.choice([-1, 1], H).astype(np.int8)
        W1 = oracle.fixed_matrix_dense(g_idx, D, sign) + U @ V      # W_1 = G + UV, materialised
        z_mat = oracle.gate_standard(W1, x, b)
        z_lopa = oracle.gate_lopa(V, U, x, g_idx, sign, None, False, 0.0, b)
        np.testing.assert_allclose(z_lopa, z_mat, rtol=1e-12, atol=1e-12)
    z_uv = oracle.gate_lopa(V, U, x, None, None, None, False, 0.0, None)
    np.testing.assert_allclose(z_uv, oracle.gate_standard(U @ V, x), rtol=1e-12, atol=1e-12)
    # whole FFN through the LoPA gate == whole FFN through the materialised W_1
    W3, Wd = RNG.standard_normal((H, D)), RNG.standard_normal((H, D))
    g_idx = oracle.g_diagonal(H, D)
    lopa = dict(V=V, U=U, g_idx=g_idx, use_rmsnorm=False)
    a = oracle.ffn(x, W3, Wd, "relu", lopa=lopa, b_g=b)
    m = oracle.ffn(x, W3, Wd, "relu", W_g=oracle.fixed_matrix_dense(g_idx, D) + U @ V, b_g=b)
    np.testing.assert_allclose(a["y"], m["y"], rtol=1e-10, atol=1e-10)


def test_rmsnorm_properties():
    D, H, r = 20, 16, 8
    V, U = RNG.standard_normal((r, D)), RNG.standard_normal((H, r))
    x = RNG.standard_normal(D)
    _, v, n = oracle.gate_lopa(V, U, x, None, None, None, True, 0.0, None, return_vn=True)
    assert float(n @ n) == pytest.approx(r, rel=1e-12)            # unit RMS at gain 1, eps 0
    np.testing.assert_allclose(n, v / math.sqrt(float(v @ v) / r), rtol=1e-13)
    z1 = oracle.gate_lopa(V, U, x, None, None, None, True, 0.0, None)
    z3 = oracle.gate_lopa(V, U, 3.0 * x, None, None, None, True, 0.0, None)
    np.testing.assert_allclose(z3, z1, rtol=1e-12, atol=1e-12)     # scale-invariant without G
    z0 = oracle.gate_lopa(V, U, x, None, None, None, False, 0.0, None)
    np.testing.assert_allclose(z0, U @ (V @ x), rtol=1e-12)


def test_fixed_matrices_picture(golden):
    rows = {r[0]: np.array(r[1:], np.int32) for r in golden("fixed_matrices_h12_d6.txt")}
    np.testing.assert_array_equal(oracle.g_diagonal(12, 6), rows["diagonal"])
    np.testing.assert_array_equal(oracle.g_tiled(12, 6), rows["tiled_identity"])
    np.testing.assert_array_equal(oracle.g_padded_identity(12, 6), rows["padded_identity"])
    for gen in (oracle.g_diagonal, oracle.g_tiled):
        M = oracle.fixed_matrix_dense(gen(12, 6), 6)
        assert (M.sum(axis=1) == 1).all() and (M.sum(axis=0) == 2).all()   # one per row, all columns hit
    assert (oracle.fixed_matrix_dense(oracle.g_padded_identity(12, 6), 6).sum(axis=1)[6:] == 0).all()
    x = np.arange(6, dtype=np.float64) + 1
    np.testing.assert_array_equal(oracle.fixed_matrix_dense(oracle.g_tiled(12, 6), 6) @ x,
                                  x[np.arange(12) % 6])
    # non-integer H/D (the benchmark shape 14336/4096 = 3.5): still one column per row, all used
    g = oracle.g_diagonal(14336, 4096)
    assert g.min() == 0 and g.max() == 4095 and (np.diff(g) >= 0).all()
    assert set(np.bincount(g).tolist()) == {3, 4}


# ---------------------------------------------------------------- closed forms (Eq. 2, Eq. 4, H')
def test_printed_closed_form_values(golden):
    for row in golden("flop_ratio_values.txt"):
        kind, *args = row
        *args, want, tol = [float(a) for a in args]
        if kind == "standard":
            got = oracle.flop_ratio_standard(args[0])
        elif kind == "hprime":
            got = oracle.adaptive_hidden_dim(*args)
        else:
            alpha, h_over_d, s = args
            D = 1024.0
            hp = oracle.adaptive_hidden_dim(D, h_over_d * D, alpha * D)
            got = oracle.flop_ratio_lopa(s, D, hp, alpha * D)
        assert abs(got - want) <= tol, (row, got)
    # parameter count is preserved by H'
    D, H, r = 2560, 7168, 400
    hp = oracle.adaptive_hidden_dim(D, H, r)
    assert r * (hp + D) + 2 * hp * D == pytest.approx(3 * H * D, rel=1e-12)


def test_casting_table_speedups(golden):
    D, H, r = 1920.0, 5120.0, 240.0
    hp = oracle.adaptive_hidden_dim(D, H, r)
    f = {"base": oracle.flop_ratio_standard,
         "lopa": lambda s: oracle.flop_ratio_lopa(s, D, hp, r),
         "archcast": lambda s: oracle.flop_ratio_lopa_fixed_h(s, D, H, r)}
    for arch, s, printed in golden("casting_table_speedups.txt"):
        s, printed = float(s), float(printed)
        lo, hi = f[arch](max(0.0, s - 0.01)), f[arch](min(1.0, s + 0.01))
        assert lo - 0.006 <= printed <= hi + 0.006, (arch, s, printed, lo, hi)


# ---------------------------------------------------------------- batches and the union of masks
def test_batch_equals_independent_tokens_and_union():
    D, H, B = 36, 100, 5
    w = syn.standard_ffn(D, H, torch.bfloat16, seed=9, sparsity=0.85)
    x = syn.tokens(B, D, torch.bfloat16, seed=9)
    batch = oracle.ffn(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=w["b_g"], threads=3)
    union = np.zeros(H, bool)
    for b in range(B):
        one = oracle.ffn(x[b], w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=w["b_g"])
        assert np.array_equal(one["y"], batch["y"][b]) and np.array_equal(one["z"], batch["z"][b])
        union[oracle.active_set(one["z"])] = True
    np.testing.assert_array_equal(batch["union_mask"], union)
    assert batch["union_mask"].sum() >= batch["n_act"].max()


def test_zipf_profile_recipe():
    H = 14336
    p = syn.zipf_firing_profile(H, 1.1, 0.1, 0.99, seed=4)
    assert float(p.mean()) == pytest.approx(0.1, abs=1e-6)
    assert int((p >= 0.99 - 1e-12).sum()) in range(300, 400) and float(p.min()) == pytest.approx(0.0169, abs=2e-3)
    for B, want in ((4, 0.24), (16, 0.53), (64, 0.88)):
        assert syn.expected_union_fraction(p, B) == pytest.approx(want, abs=0.015)
    b = syn.bias_from_firing_profile(p)
    # a N(0,1) pre-activation plus b_j is positive with probability p_j
    fire = 0.5 * torch.erfc(-b.double() / math.sqrt(2.0))
    np.testing.assert_allclose(fire.numpy(), p.numpy(), atol=1e-6)


# ---------------------------------------------------------------- double activation (Sec. 3.3) and the s_gated site
def test_hand_worked_double_activation():
    # x = [1, 2];  z = W1 x = [1, -2, 3] (RELU: a = [1, 0, 3]);  u = W3 x = [3-2, 2+4, -1+0.5] = [1, 6, -0.5]
    W1 = np.array([[1.0, 0.0], [0.0, -1.0], [1.0, 1.0]], np.float32)
    W3 = np.array([[3.0, -1.0], [2.0, 2.0], [-1.0, 0.25]], np.float32)
    Wd = np.array([[1.0, 1.0], [5.0, 5.0], [2.0, -2.0]], np.float32)   # rows = columns of W_2
    x = np.array([1.0, 2.0], np.float32)
    for route in ("dense", "sparse"):
        # Eq. 1: h = a * u = [1, 0, -1.5];  y = 1*[1,1] - 1.5*[2,-2] = [-2, 4];  two neurons with h != 0
        out = oracle.ffn(x, W3, Wd, "relu", W_g=W1, route=route)
        np.testing.assert_array_equal(out["y"], [-2.0, 4.0])
        assert out["n_act"][0] == 2 and out["n_gated"][0] == 2
        # A_3 = RELU on the W_3 output: A_3(u) = [1, 6, 0];  h = [1, 0, 0];  y = [1, 1];  one gated neuron
        out = oracle.ffn(x, W3, Wd, "relu", W_g=W1, route=route, act_up="relu")
        np.testing.assert_array_equal(out["y"], [1.0, 1.0])
        assert out["n_act"][0] == 2 and out["n_gated"][0] == 1
        # A_3 = squared RELU: A_3(u) = [1, 36, 0] -> the same h;  A = squared RELU too: a = [1, 0, 9], h = [1, 0, 0]
        out = oracle.ffn(x, W3, Wd, "sqrelu", W_g=W1, route=route, act_up="sqrelu")
        np.testing.assert_array_equal(out["y"], [1.0, 1.0])
        # A_3 = R-S+: A_3(1) = sigmoid(1) = 1 / (1 + e^-1)
        out = oracle.ffn(x, W3, Wd, "relu", W_g=W1, route=route, act_up="rsplus")
        np.testing.assert_allclose(out["y"], [1.0 / (1.0 + math.exp(-1.0))] * 2, rtol=1e-15)
        # A_3 = SILU (the uncast activation of the up branch): A_3(u) = [sigmoid(1), 6 sigmoid(6), -0.5 sigmoid(-0.5)];
        # h = [sigmoid(1), 0, -1.5 sigmoid(-0.5)];  y = h_0 [1, 1] + h_2 [2, -2];  both fired neurons keep h != 0
        out = oracle.ffn(x, W3, Wd, "relu", W_g=W1, route=route, act_up="silu")
        h0, h2 = 1.0 / (1.0 + math.exp(-1.0)), -1.5 / (1.0 + math.exp(0.5))
        np.testing.assert_allclose(out["y"], [h0 + 2 * h2, h0 - 2 * h2], rtol=1e-15)
        assert out["n_act"][0] == 2 and out["n_gated"][0] == 2
    with pytest.raises(ValueError):          # SILU is not sparse: it cannot be the gate's activation
        oracle.ffn(x, W3, Wd, "silu", W_g=W1)


def test_double_activation_special_cases():
    D, H, B = 24, 40, 5
    x = np.abs(RNG.standard_normal((B, D))).astype(np.float32)          # x >= 0
    W1 = RNG.standard_normal((H, D)).astype(np.float32)
    Wd = RNG.standard_normal((H, D)).astype(np.float32)
    Wp = np.abs(RNG.standard_normal((H, D))).astype(np.float32)         # W_3 >= 0  =>  u >= 0
    single = oracle.ffn(x, Wp, Wd, "relu", W_g=W1)
    double = oracle.ffn(x, Wp, Wd, "relu", W_g=W1, act_up="relu")
    np.testing.assert_array_equal(double["y"], single["y"])               # RELU is the identity on u >= 0
    np.testing.assert_array_equal(double["n_gated"], single["n_act"])
    neg = oracle.ffn(x, -Wp, Wd, "relu", W_g=W1, act_up="relu")          # u <= 0: A_3(u) = 0 everywhere
    assert not neg["y"].any() and not neg["n_gated"].any()
    np.testing.assert_array_equal(neg["n_act"], single["n_act"])          # the gate is untouched
    # skipping rows never changes y, and the gated set is a subset of the active set
    W3 = RNG.standard_normal((H, D)).astype(np.float32)
    for a3 in ("relu", "sqrelu", "rsplus", "silu"):
        dense = oracle.ffn(x, W3, Wd, "sqrelu", W_g=W1, route="dense", act_up=a3)
        sparse = oracle.ffn(x, W3, Wd, "sqrelu", W_g=W1, route="sparse", act_up=a3)
        np.testing.assert_array_equal(dense["y"], sparse["y"])
        assert (sparse["n_gated"] <= sparse["n_act"]).all()
        # against a library matmul: y = W_2 (A(z) * A_3(u)) with W_2 = Wd^T
        z = x.astype(np.float64) @ W1.astype(np.float64).T
        u = x.astype(np.float64) @ W3.astype(np.float64).T
        a = np.maximum(z, 0.0) ** 2
        g = {"relu": np.maximum(u, 0.0), "sqrelu": np.maximum(u, 0.0) ** 2,
             "rsplus": np.where(u >= 0, u / (1.0 + np.exp(-u)), 0.0), "silu": u / (1.0 + np.exp(-u))}[a3]
        np.testing.assert_allclose(sparse["y"], (a * g) @ Wd.astype(np.float64), rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- weight-only int8 (appendix on quantisation-aware training)
def test_hand_worked_int8_rows():
    # codes with one scale per ROW: W = [[0.5*1, 0.5*-2], [0.25*3, 0.25*4]] = [[0.5, -1], [0.75, 1]]
    q = np.array([[1, -2], [3, 4]], np.int8)
    s = np.array([0.5, 0.25], np.float32)
    np.testing.assert_array_equal(oracle.dequantize_rows(q, s), [[0.5, -1.0], [0.75, 1.0]])
    # x = [2, 1];  z = W1 x = [0, 2.5]: only neuron 1 fires (z > 0);  u = W3 x with W3 = 2*[[1,1],[1,-1]] = [6, 2]
    # y = a_1 u_1 Wd[1] = 2.5 * 2 * (0.5*[4, -6]) = [10, -15]
    W1 = dict(q=q, s=s)
    W3 = dict(q=np.array([[1, 1], [1, -1]], np.int8), s=np.array([2.0, 2.0], np.float32))
    Wd = dict(q=np.array([[100, 100], [4, -6]], np.int8), s=np.array([1.0, 0.5], np.float32))
    x = np.array([2.0, 1.0], np.float32)
    for route in ("dense", "sparse"):
        out = oracle.ffn_q8(x, W3, Wd, "relu", W_g=W1, route=route)
        np.testing.assert_array_equal(out["z"], [0.0, 2.5])
        np.testing.assert_array_equal(out["y"], [10.0, -15.0])
        assert out["n_act"][0] == 1


def test_int8_with_power_of_two_scales_equals_fp32_weights():
    # s_j q_jk is exactly an fp32 number when s_j is a power of two, so the int8 route and the fp32 route see the
    # same real matrices and must agree to the last bit (both accumulate the same products in the same order)
    D, H, r, B = 32, 48, 16, 3
    x = syn.tokens(B, D, torch.bfloat16, 5)

    def mat(rows, cols, tag):
        q = RNG.integers(-127, 128, (rows, cols)).astype(np.int8)
        s = (2.0 ** RNG.integers(-9, -3, rows)).astype(np.float32)
        return dict(q=q, s=s), (s[:, None] * q.astype(np.float32)).astype(np.float32)

    (W1q, W1), (W3q, W3), (Wdq, Wd) = mat(H, D, "g"), mat(H, D, "u"), mat(H, D, "d")
    (Vq, V), (Uq, U) = mat(r, D, "V"), mat(H, r, "U")
    b = np.full(H, -0.3, np.float32)
    a = oracle.ffn_q8(x, W3q, Wdq, "relu", W_g=W1q, b_g=b)
    f = oracle.ffn(x, W3, Wd, "relu", W_g=W1, b_g=b)
    np.testing.assert_array_equal(a["y"], f["y"])
    np.testing.assert_array_equal(a["z"], f["z"])
    gi = RNG.integers(0, D, H).astype(np.int32)
    lq = dict(V=Vq, U=Uq, g_idx=gi, use_rmsnorm=True, eps=1e-5)
    lf = dict(V=V, U=U, g_idx=gi, use_rmsnorm=True, eps=1e-5)
    a = oracle.ffn_q8(x, W3q, Wdq, "rsplus", lopa=lq, b_g=b, act_up="relu")
    f = oracle.ffn(x, W3, Wd, "rsplus", lopa=lf, b_g=b, act_up="relu")
    np.testing.assert_array_equal(a["y"], f["y"])
    assert a["y"].any()


def test_int8_inputs_recipe():
    w = syn.standard_ffn_q8(256, 512, 3)
    for k in ("W_g", "W_up", "W_down"):
        q, s = w[k]["q"], w[k]["s"]
        assert q.dtype == torch.int8 and s.dtype == torch.float32 and q.shape == (512, 256) and s.shape == (512,)
        assert int(q.min()) >= -127 and int(q.max()) <= 127
        assert float(q.float().std()) == pytest.approx(32.0, rel=0.02)
        # dequantised entries have the standard deviation of the bf16 recipe, 1/sqrt(D), within the +-10 % row spread
        W = oracle.dequantize_rows(q, s)
        assert float(W.std()) * 16.0 == pytest.approx(1.0, rel=0.02)
        assert len(torch.unique(s)) > 500                                  # the scales really differ by row
    assert not torch.equal(w["W_g"]["q"], w["W_up"]["q"]) and not torch.equal(w["W_g"]["s"], w["W_up"]["s"])
    # 90 % target sparsity holds on the dequantised gate
    x = syn.tokens(16, 256, torch.bfloat16, 3)
    out = oracle.ffn_q8(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=w["b_g"])
    assert out["n_act"].mean() / 512 == pytest.approx(0.1, abs=0.03)


# ---------------------------------------------------------------- weight-only int4 (same appendix)
def test_hand_worked_int4_nibbles():
    # byte 0x2F: low nibble F = -1 (even column), high nibble 2 = +2 (odd column); byte 0x78: low 8 = -8, high 7 = +7
    packed = np.array([[0x2F, 0x78], [0x10, 0xF9]], np.uint8)
    s = np.array([0.5, 2.0], np.float32)
    np.testing.assert_array_equal(oracle.dequantize_rows_q4(packed, s),
                                  [[-0.5, 1.0, -4.0, 3.5], [0.0, 2.0, -14.0, -2.0]])
    # the same hand-worked FFN as for int8 rows, written in nibbles: W1 = [[0.5,-1],[0.75,1]], W3 = 2*[[1,1],[1,-1]],
    # Wd = [[7,7],[2,-3]];  x = [2,1]: z = [0, 2.5], u = [6, 2], y = 2.5 * 2 * [2,-3] = [10,-15]
    W1 = dict(q=np.array([[0xE1], [0x43]], np.uint8), s=np.array([0.5, 0.25], np.float32))
    W3 = dict(q=np.array([[0x11], [0xF1]], np.uint8), s=np.array([2.0, 2.0], np.float32))
    Wd = dict(q=np.array([[0x77], [0xA4]], np.uint8), s=np.array([1.0, 0.5], np.float32))
    x = np.array([2.0, 1.0], np.float32)
    for route in ("dense", "sparse"):
        out = oracle.ffn_q4(x, W3, Wd, "relu", W_g=W1, route=route)
        np.testing.assert_array_equal(out["z"], [0.0, 2.5])
        np.testing.assert_array_equal(out["y"], [10.0, -15.0])


def test_int4_codes_equal_the_same_codes_stored_as_int8():
    # packing is the only thing the 4-bit route adds: the same integer codes given as int8 go through the pinned int8
    # route and must give the same bits
    D, H, r, B = 32, 40, 16, 3
    x = syn.tokens(B, D, torch.bfloat16, 6)

    def mat(rows, cols):
        q = RNG.integers(-8, 8, (rows, cols)).astype(np.int8)
        s = RNG.uniform(0.01, 0.1, rows).astype(np.float32)
        nib = (q.astype(np.int16) & 0xF).astype(np.uint8)
        return dict(q=(nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8), s=s), dict(q=q, s=s)

    (g4, g8), (u4, u8), (d4, d8), (V4, V8), (U4, U8) = mat(H, D), mat(H, D), mat(H, D), mat(r, D), mat(H, r)
    b = np.full(H, -0.2, np.float32)
    a, f = oracle.ffn_q4(x, u4, d4, "relu", W_g=g4, b_g=b), oracle.ffn_q8(x, u8, d8, "relu", W_g=g8, b_g=b)
    np.testing.assert_array_equal(a["y"], f["y"])
    np.testing.assert_array_equal(a["z"], f["z"])
    assert a["y"].any() and 0 < a["n_act"].mean() < H
    gi = RNG.integers(0, D, H).astype(np.int32)
    l4 = dict(V=V4, U=U4, g_idx=gi, use_rmsnorm=True, eps=1e-5)
    l8 = dict(V=V8, U=U8, g_idx=gi, use_rmsnorm=True, eps=1e-5)
    a = oracle.ffn_q4(x, u4, d4, "sqrelu", lopa=l4, b_g=b, act_up="relu")
    f = oracle.ffn_q8(x, u8, d8, "sqrelu", lopa=l8, b_g=b, act_up="relu")
    np.testing.assert_array_equal(a["y"], f["y"])


def test_int4_inputs_recipe():
    w = syn.standard_ffn_q4(256, 512, 3)
    for k in ("W_g", "W_up", "W_down"):
        q, s = w[k]["q"], w[k]["s"]
        assert q.dtype == torch.uint8 and s.dtype == torch.float32 and q.shape == (512, 128) and s.shape == (512,)
        W = oracle.dequantize_rows_q4(q, s)
        codes = W / s.numpy().astype(np.float64)[:, None]
        assert codes.min() >= -7 and codes.max() <= 7 and np.all(codes == np.round(codes))
        assert float(codes.std()) == pytest.approx(2.5, rel=0.05)
        assert float(W.std()) * 16.0 == pytest.approx(1.0, rel=0.05)
    x = syn.tokens(16, 256, torch.bfloat16, 3)
    out = oracle.ffn_q4(x, w["W_up"], w["W_down"], "relu", W_g=w["W_g"], b_g=w["b_g"])
    assert out["n_act"].mean() / 512 == pytest.approx(0.1, abs=0.03)


# ---------------------------------------------------------------- LoPA approximation of a full gate (Sec. 3.4)
def test_lopa_approximation_m_step_is_the_row_optimum_by_brute_force():
    cast = oracle.lopa_cast
    H, D, r = 7, 5, 2
    W = RNG.standard_normal((H, D))
    U, V = RNG.standard_normal((H, r)) * 0.3, RNG.standard_normal((r, D)) * 0.3
    g_idx, g_sign = cast.m_step(W, U, V)
    R = W - U @ V
    for i in range(H):
        # every admissible row of M: one entry, +1 or -1
        costs = {(j, sg): ((R[i] - sg * np.eye(D)[j]) ** 2).sum() for j in range(D) for sg in (-1, 1)}
        best = min(costs, key=costs.get)
        assert (int(g_idx[i]), int(g_sign[i])) == best
    # hand-worked: R = [[0.2, -3, 1], [0.5, 0.4, -0.1]] -> row 0: column 1, sign -1; row 1: column 0, sign +1
    gi, gs = cast.m_step(np.array([[0.2, -3.0, 1.0], [0.5, 0.4, -0.1]]), np.zeros((2, 1)), np.zeros((1, 3)))
    assert gi.tolist() == [1, 0] and gs.tolist() == [-1, 1]
    # objective of that choice: (0.04 + 4 + 1) + (0.25 + 0.16 + 0.01) = 5.46
    assert cast.objective(np.array([[0.2, -3.0, 1.0], [0.5, 0.4, -0.1]]), gi, gs, np.zeros((2, 1)), np.zeros((1, 3))) \
        == pytest.approx(5.46, abs=1e-12)


def test_lopa_approximation_uv_step_is_the_best_rank_r_matrix():
    cast = oracle.lopa_cast
    H, D, r = 12, 9, 3
    W = RNG.standard_normal((H, D))
    g_idx, g_sign = cast.m_step(W, np.zeros((H, r)), np.zeros((r, D)))
    U, V = cast.uv_step(W, g_idx, g_sign, r)
    A = W.copy()
    A[np.arange(H), g_idx] -= g_sign
    sv = np.linalg.svd(A, compute_uv=False)
    # Eckart-Young: the error of the best rank-r approximation is the energy of the dropped singular values
    assert cast.objective(W, g_idx, g_sign, U, V) == pytest.approx((sv[r:] ** 2).sum(), rel=1e-12)
    assert np.linalg.matrix_rank(U @ V) == r
    # no other rank-r matrix does better (random perturbations of the factors)
    for _ in range(20):
        U2, V2 = U + 0.05 * RNG.standard_normal(U.shape), V + 0.05 * RNG.standard_normal(V.shape)
        assert cast.objective(W, g_idx, g_sign, U2, V2) >= cast.objective(W, g_idx, g_sign, U, V)
    # full rank: nothing is left
    Uf, Vf = cast.uv_step(W, g_idx, g_sign, min(H, D))
    assert cast.objective(W, g_idx, g_sign, Uf, Vf) < 1e-20


def test_lopa_approximation_descends_and_recovers_a_planted_gate():
    cast = oracle.lopa_cast
    H, D, r = 40, 24, 4
    # the objective never increases, half-step by half-step (the guarantee stated with the algorithm)
    W = RNG.standard_normal((H, D)) / np.sqrt(D)
    out = cast.lopa_approximation(W, r, n_iter=5)
    tr = np.array(out["trace"])
    assert (np.diff(tr) <= 1e-12).all() and tr[-1] < tr[0]
    assert tr[0] == pytest.approx(cast.objective(W, out["g_idx"] * 0 + np.argmax(np.abs(W), 1), np.sign(
        W[np.arange(H), np.argmax(np.abs(W), 1)]), np.zeros((H, r)), np.zeros((r, D))))   # first M-step: U = V = 0
    # a matrix that is exactly M0 + U0 V0 with small low-rank part is recovered: first M-step finds M0, the SVD the rest
    gi0 = RNG.integers(0, D, H)
    gs0 = RNG.choice([-1, 1], H)
    U0, V0 = 0.1 * RNG.standard_normal((H, r)), 0.1 * RNG.standard_normal((r, D))
    Wp = U0 @ V0
    Wp[np.arange(H), gi0] += gs0
    rec = cast.lopa_approximation(Wp, r, n_iter=2)
    assert rec["g_idx"].tolist() == gi0.tolist() and rec["g_sign"].tolist() == gs0.tolist()
    assert rec["trace"][-1] < 1e-20
    np.testing.assert_allclose(rec["U"] @ rec["V"], U0 @ V0, atol=1e-12)
    # the result drives the gate of Eq. 3 without RMSNorm: z = M x + U V x equals the materialised matrix times x
    x = RNG.standard_normal(D).astype(np.float32)
    z = oracle.gate_lopa(rec["V"], rec["U"], x, g_idx=rec["g_idx"], g_sign=rec["g_sign"], use_rmsnorm=False)
    np.testing.assert_allclose(z, Wp @ x.astype(np.float64), atol=1e-10)
