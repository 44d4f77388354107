"""GPU parity of the LoPA approximation of a full gate matrix (architecture casting, Sec. 3.4) against the CPU oracle,
through the C ABI, and of the cast gate inside the sparse FFN.  Run with `-m gpu` on a B200."""
import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as syn
from parity import assert_active_set, assert_y_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def mod():
    import paper_2609_31975_b200 as m
    m.load_library()
    return m


@pytest.mark.parametrize("H,D", [(200, 96), (777, 264), (64, 1000), (33, 7)])
def test_m_step_and_residual_match_the_oracle(mod, H, D):
    from paper_2609_31975_b200.binding import lopa_m_step, lopa_residual
    cast = oracle.lopa_cast
    W = syn.normal_tensor((H, D), 1.0, torch.float32, 31, "W_g", DEV)
    r = 5
    U = syn.normal_tensor((H, r), 0.3, torch.float32, 31, "U", DEV)
    V = syn.normal_tensor((r, D), 0.3, torch.float32, 31, "V", DEV)
    for P in (None, (U @ V).contiguous()):
        g_idx, g_sign, energy, best = lopa_m_step(W, P)
        torch.cuda.synchronize()
        Wd = W.cpu().double().numpy()
        Pd = np.zeros_like(Wd) if P is None else P.cpu().double().numpy()     # the same product on both sides
        gi, gs = cast.m_step(Wd - Pd, np.zeros((H, 1)), np.zeros((1, D)))
        R = Wd - Pd
        # the arg max is an integer decided by floating point: both sides see the same fp32 R up to its last bit, so
        # positions agree unless the two largest magnitudes of a row are closer than that
        top2 = np.sort(np.abs(R), axis=1)[:, -2:]
        clear = (top2[:, 1] - top2[:, 0]) > 1e-5 if D > 1 else np.ones(H, bool)
        assert clear.mean() > 0.95
        assert (g_idx.cpu().numpy()[clear] == gi[clear]).all()
        assert (g_sign.cpu().numpy()[clear] == gs[clear]).all()
        np.testing.assert_allclose(energy.cpu().numpy(), (R * R).sum(1), rtol=1e-5)
        np.testing.assert_allclose(best.cpu().numpy(), np.abs(R).max(1), rtol=1e-5, atol=1e-7)
        A = lopa_residual(W, g_idx, g_sign)
        want = W.clone()
        want[torch.arange(H, device=DEV), g_idx.long()] -= g_sign.float()
        assert torch.equal(A, want)
    # ties resolve to the first column, zeros get sign +1
    Wt = torch.zeros((3, 40), device=DEV)
    Wt[0, 5] = Wt[0, 37] = -2.0
    Wt[1, 33] = Wt[1, 2] = 1.5
    g_idx, g_sign, _, _ = lopa_m_step(Wt)
    assert g_idx.tolist() == [5, 2, 0] and g_sign.tolist() == [-1, 1, 1]


def test_alternating_minimisation_matches_the_oracle_and_descends(mod):
    H, D, r = 300, 128, 8
    W = syn.normal_tensor((H, D), 1.0 / np.sqrt(D), torch.float32, 32, "W_g", DEV)
    got = mod.lopa_approximation(W, r, n_iter=4)
    ref = oracle.lopa_cast.lopa_approximation(W.cpu().numpy(), r, n_iter=4)
    tr = np.array(got["trace"])
    assert (np.diff(tr) <= 1e-4 * tr[0]).all() and tr[-1] < tr[0]          # never increases (up to fp32 rounding)
    np.testing.assert_allclose(tr, ref["trace"], rtol=2e-4)
    # same fixed matrix except where a row's two largest residuals are nearly tied
    same = (got["g_idx"].cpu().numpy() == ref["g_idx"]) & (got["g_sign"].cpu().numpy() == ref["g_sign"])
    assert same.mean() > 0.97
    # the low-rank part is unique as a product (the factors are not): compare U V, and the final objective
    UV = (got["U"] @ got["V"]).cpu().double().numpy()
    if same.all():
        np.testing.assert_allclose(UV, ref["U"] @ ref["V"], atol=2e-4)
    final = oracle.lopa_cast.objective(W.cpu().numpy(), got["g_idx"].cpu().numpy(), got["g_sign"].cpu().numpy(),
                                       got["U"].cpu().numpy(), got["V"].cpu().numpy())
    assert final == pytest.approx(ref["trace"][-1], rel=2e-4)


def test_planted_gate_is_recovered_and_drives_the_sparse_ffn(mod):
    # W_g = M0 + U0 V0 exactly: the cast recovers it, and the FFN with the cast LoPA gate (no RMSNorm, signed fixed
    # matrix) equals the FFN with the full matrix
    D, H, r = 256, 900, 16
    g = torch.Generator().manual_seed(33)
    gi0 = torch.randint(0, D, (H,), generator=g)
    gs0 = torch.randint(0, 2, (H,), generator=g) * 2 - 1
    U0 = syn.normal_tensor((H, r), 0.1, torch.float32, 33, "U", DEV)
    V0 = syn.normal_tensor((r, D), 0.1, torch.float32, 33, "V", DEV)
    Wg = (U0 @ V0).contiguous()
    Wg[torch.arange(H, device=DEV), gi0.to(DEV)] += gs0.to(DEV).float()
    got = mod.lopa_approximation(Wg, r, n_iter=2)
    assert got["g_idx"].cpu().tolist() == gi0.tolist() and got["g_sign"].cpu().tolist() == gs0.tolist()
    assert got["trace"][-1] < 1e-6 * got["trace"][0]
    w = syn.standard_ffn(D, H, torch.float32, 33, DEV, sparsity=None)
    b_g = torch.full((H,), -0.8, device=DEV)
    x = syn.tokens(3, D, torch.float32, 33, DEV)
    gate = {"V": got["V"], "U": got["U"], "g_idx": got["g_idx"], "g_sign": got["g_sign"], "use_rmsnorm": False}
    ffn = mod.SparseFFN(D, H, torch.float32, r_max=r, B_max=3)
    ref = oracle.ffn(x.cpu(), w["W_up"].cpu(), w["W_down"].cpu(), "relu", W_g=Wg.cpu(), b_g=b_g.cpu())
    assert 0 < ref["n_act"].min() and ref["n_act"].max() < H
    for t in range(3):
        for path in ("general", "fused"):
            ffn.set_path(path)
            y = ffn.sparse_ffn_forward(x[t], gate, b_g, w["W_up"], w["W_down"], "relu")
            torch.cuda.synchronize()
            assert_y_close(y, ref["y"][t], rel_l2=1e-4, max_abs=1e-4, what=f"cast gate t{t} [{path}]")
            assert_active_set(ffn.last_active(), dict(z=ref["z"][t]), what=f"cast gate t{t} [{path}]")
    assert ffn.device_status() == 0
