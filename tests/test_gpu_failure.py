"""The device-side failure path, exercised without ever hanging or faulting the GPU: a test hook makes one wait
run out on purpose (a CTA that never reports in, a copy that is never issued) with the wait budget cut to a
millisecond.  The kernels must come back by themselves, record SFFN_ERR_TIMEOUT, leave y alone, release what they
hold (shared memory, TMEM), and the library must compute correctly again afterwards."""
import pytest
import torch

import synthetic_inputs as syn
from parity import assert_y_close, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SHORT = 2_000_000        # cycles: about a millisecond


@pytest.fixture()
def mod():
    import paper_2609_31975_b200 as m
    m.load_library()
    yield m
    for knob, value in (("wait_cycles", 0), ("skip_arrival_cta", -1), ("drop_stage", -1), ("tensor_gate", -1)):
        m.test_set_knob(knob, value)


@pytest.mark.parametrize("D,H,dtype,tensor_gate", [
    (1024, 2049, torch.bfloat16, 1),   # tensor-core gate kernel: tagged partials, the summing CTAs' reads run out
    (1024, 2049, torch.bfloat16, 0),   # CUDA-core gate kernel: the arrival count never completes
    (512, 1000, torch.float32, 0),
])
def test_single_token_call_times_out_reports_and_recovers(mod, D, H, dtype, tensor_gate):
    w = syn.standard_ffn(D, H, dtype, 11, DEV, sparsity=0.8)
    gate = {"W_g": w["W_g"]}
    x = syn.tokens(2, D, dtype, 11, DEV)
    ref = [run_oracle(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu") for t in range(2)]
    ffn = mod.SparseFFN(D, H, dtype, B_max=1)
    mod.test_set_knob("tensor_gate", tensor_gate)
    y = torch.full((D,), 7.0, dtype=torch.float32, device=DEV)
    mod.test_set_knob("wait_cycles", SHORT)
    mod.test_set_knob("skip_arrival_cta", 3)
    ffn.sparse_ffn_forward(x[0], gate, w["b_g"], w["W_up"], w["W_down"], "relu", y)
    torch.cuda.synchronize()                               # the kernel came back by itself
    assert ffn.device_status() == 5                        # SFFN_ERR_TIMEOUT
    assert torch.all(y == 7.0)                             # a call that failed does not write y
    mod.test_set_knob("skip_arrival_cta", -1)
    mod.test_set_knob("wait_cycles", 0)
    # the status is sticky until the handle is reset; after that the same handle is good again
    ffn.reset()
    for t in range(2):
        y = ffn.sparse_ffn_forward(x[t], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        torch.cuda.synchronize()
        assert ffn.device_status() == 0
        assert_y_close(y, ref[t]["y"], what=f"after reset, token {t}")
    # and so is a new handle
    other = mod.SparseFFN(D, H, dtype, B_max=1)
    y = other.sparse_ffn_forward(x[1], gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    assert_y_close(y, ref[1]["y"], what="new handle after a timeout")
    assert other.device_status() == 0


def test_batched_tcgen05_gate_times_out_releases_tmem_and_recovers(mod):
    D, H, B = 512, 4000, 8
    w = syn.standard_ffn(D, H, torch.bfloat16, 12, DEV, sparsity=0.9)
    gate = {"W_g": w["W_g"]}
    x = syn.tokens(B, D, torch.bfloat16, 12, DEV)
    ref = run_oracle(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    ffn = mod.SparseFFN(D, H, torch.bfloat16, B_max=B)
    mod.test_set_knob("wait_cycles", SHORT)
    mod.test_set_knob("drop_stage", 1)                     # CTA 0 of the gate GEMM never copies its second stage
    ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
    torch.cuda.synchronize()
    assert ffn.device_status() == 5
    mod.test_set_knob("drop_stage", -1)
    mod.test_set_knob("wait_cycles", 0)
    ffn.reset()
    # every SM's TMEM must be free again: the next calls allocate theirs and compute correctly
    for _ in range(3):
        y = ffn.sparse_ffn_forward(x, gate, w["b_g"], w["W_up"], w["W_down"], "relu")
        torch.cuda.synchronize()
        assert ffn.device_status() == 0
        assert_y_close(y, ref["y"], what="batched call after a timeout")
