"""The allocation-free entry point, checked on a GPU against the handle-based one.

Some callers cannot allocate device memory when they need an FFN (all of HBM already belongs to the
application's own pool, or an allocation's device-wide synchronisation is not acceptable where they
run).  For them the library carries its scratch inside its own device image.  This file is collected
last on purpose: a run that stops at the first failure has then already run every other test.
"""
import pytest
import torch

import synthetic_inputs as syn
from parity import MAX_ABS, REL_L2, assert_y_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_static_scratch_entry_matches_handle_entry_twice_in_a_row():
    import paper_2609_31975_b200 as m

    D, H = 1024, 3001
    ffn = m.SparseFFN(D, H, torch.bfloat16, B_max=1, device=DEV)
    x = syn.tokens(2, D, torch.bfloat16, 81, DEV)
    # first call: about half the neurons fire; second call: far fewer, other weights -- anything the
    # first call left in the shared scratch (a longer index list, other gate values) must not leak
    cases = [(syn.standard_ffn(D, H, torch.bfloat16, 81, DEV, sparsity=0.5), x[0], "relu"),
             (syn.standard_ffn(D, H, torch.bfloat16, 82, DEV, sparsity=0.95), x[1], "sqrelu")]
    y_static = torch.empty(D, dtype=torch.float32, device=DEV)          # caller-owned output
    for w, xt, act in cases:
        m.sparse_ffn_forward_static(xt, w["W_g"], w["b_g"], w["W_up"], w["W_down"], act, y_static)
        torch.cuda.synchronize()
        got = y_static.clone()
        want = ffn.sparse_ffn_forward(xt, {"W_g": w["W_g"]}, w["b_g"], w["W_up"], w["W_down"], act)
        torch.cuda.synchronize()
        assert_y_close(got, want.double().cpu().numpy(), rel_l2=REL_L2, max_abs=MAX_ABS,
                       what=f"static entry vs handle entry ({act})")
        assert got.abs().max() > 0
    # shapes beyond the built-in scratch are refused with a status, not served
    big = torch.empty((8, 8200), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(m.SFFNError) as e:
        m.sparse_ffn_forward_static(big[0], big, None, big, big, "relu",
                                    torch.empty(8200, dtype=torch.float32, device=DEV))
    assert e.value.code == 2
