"""The allocation-free entry point, checked on a GPU against the CPU oracle and against the handle-based entry.

Some callers cannot allocate device memory when they need an FFN (all of HBM already belongs to the
application's own pool, or an allocation's device-wide synchronisation is not acceptable where they
run).  For them the library carries its scratch inside its own device image.  This file is collected
last on purpose: a run that stops at the first failure has then already run every other test.
"""
import pytest
import torch

import synthetic_inputs as syn
from parity import MAX_ABS, REL_L2, assert_active_set, assert_y_close, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_entry_matches_oracle_and_handle_entry_twice_in_a_row(dtype):
    import paper_2609_31975_b200 as m

    D, H = 1024, 3001                       # odd H: the flag and list tails are ragged
    ffn = m.SparseFFN(D, H, dtype, B_max=1, device=DEV)
    x = syn.tokens(3, D, dtype, 81, DEV)
    # first call: about half the neurons fire; second call: far fewer, other weights -- anything the
    # first call left in the shared scratch (a longer index list, other gate values) must not leak;
    # third call: no bias at all (Eq. 1 as the paper writes it)
    w0 = syn.standard_ffn(D, H, dtype, 81, DEV, sparsity=0.5)
    w1 = syn.standard_ffn(D, H, dtype, 82, DEV, sparsity=0.95)
    cases = [(w0, w0["b_g"], x[0], "relu"), (w1, w1["b_g"], x[1], "sqrelu"), (w1, None, x[2], "rsplus")]
    y_static = torch.empty(D, dtype=torch.float32, device=DEV)          # caller-owned output
    refs = [run_oracle(xt, {"W_g": w["W_g"]}, b, w["W_up"], w["W_down"], act) for w, b, xt, act in cases]
    m.sparse_ffn_forward_static(x[0], w0["W_g"], w0["b_g"], w0["W_up"], w0["W_down"], "relu", y_static)  # set-up call
    torch.cuda.synchronize()
    got = torch.empty((len(cases), D), dtype=torch.float32, device=DEV)   # allocated before the measurement
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(DEV)[0]
    for i, (w, b, xt, act) in enumerate(cases):
        m.sparse_ffn_forward_static(xt, w["W_g"], b, w["W_up"], w["W_down"], act, y_static)
        got[i].copy_(y_static)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info(DEV)[0] >= free_before, "device memory in use grew across the calls"
    for (w, b, xt, act), ref, y in zip(cases, refs, got):
        assert_y_close(y, ref["y"], rel_l2=REL_L2, max_abs=MAX_ABS, what=f"static entry vs oracle ({act})")
        assert y.abs().max() > 0
        want = ffn.sparse_ffn_forward(xt, {"W_g": w["W_g"]}, b, w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert_y_close(y, want.double().cpu().numpy(), rel_l2=REL_L2, max_abs=MAX_ABS,
                       what=f"static entry vs handle entry ({act})")
        assert_active_set(ffn.last_active(), ref, what=f"handle entry ({act})")
    # shapes beyond the built-in scratch are refused with a status, not served
    big = torch.empty((8, 8200), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(m.SFFNError) as e:
        m.sparse_ffn_forward_static(big[0], big, None, big, big, "relu",
                                    torch.empty(8200, dtype=torch.float32, device=DEV))
    assert e.value.code == 2
