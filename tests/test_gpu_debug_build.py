"""The bounds-checked build (-DSFFN_DEBUG) on a GPU: small-shape parity under it, and its index check at work.

The debug library is a second build of the same sources whose kernels check every index that comes out of a list or
a computed row number before it addresses global memory.  A process loads one library, so these tests run child
processes with SFFN_LIBRARY pointing at the debug build."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent


def debug_library():
    from paper_2609_31975_b200.build import build

    return build(debug=True)


def run_child(args, code=None):
    env = dict(os.environ, SFFN_LIBRARY=str(debug_library()))
    cmd = [sys.executable, "-c", code] if code else [sys.executable, "-m", "pytest", *args]
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)


def test_small_shape_parity_under_the_bounds_checked_build():
    # every kernel family at small shapes: CUDA-core path, both single-token kernels, LoPA, batches on mma.sync and
    # tcgen05, int8 rows; a recorded bounds violation would fail the tests' device-status checks
    r = run_child(["tests/test_gpu_parity.py", "tests/test_gpu_int8.py", "-x", "-q", "-m", "gpu", "-k",
                   "config1 or small_shapes or wide_rows or batched_union or batched_lopa or edge_shapes or "
                   "full_and_zero or double_activation or int8"])
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


CHILD = r"""
import sys
sys.path.insert(0, "tests")
import torch
import synthetic_inputs as syn
import paper_2609_31975_b200 as m
from parity import assert_y_close, run_oracle
assert m.lib_path().name == "libsparse_ffn_debug.so", m.lib_path()
D, H = 512, 1000
w = syn.standard_ffn(D, H, torch.bfloat16, 11, "cuda:0", sparsity=0.8)
x = syn.tokens(1, D, torch.bfloat16, 11, "cuda:0")
ffn = m.SparseFFN(D, H, torch.bfloat16, B_max=1)
ffn.set_path("general")
m.test_set_knob("poison_list", 1)
ffn.sparse_ffn_forward(x[0], {"W_g": w["W_g"]}, w["b_g"], w["W_up"], w["W_down"], "relu")
torch.cuda.synchronize()
assert ffn.device_status() == 6, ffn.device_status()      # SFFN_ERR_BOUNDS, and no fault
m.test_set_knob("poison_list", 0)
ffn.reset()
y = ffn.sparse_ffn_forward(x[0], {"W_g": w["W_g"]}, w["b_g"], w["W_up"], w["W_down"], "relu")
torch.cuda.synchronize()
assert ffn.device_status() == 0
ref = run_oracle(x[0], {"W_g": w["W_g"]}, w["b_g"], w["W_up"], w["W_down"], "relu")
assert_y_close(y, ref["y"], what="after the recorded violation")
print("bounds check ok")
"""


def test_an_index_outside_its_array_is_recorded_not_used():
    r = run_child(None, CHILD)
    assert r.returncode == 0 and "bounds check ok" in r.stdout, r.stdout[-2000:] + r.stderr[-3000:]


def test_release_build_refuses_the_poison_hook(mod=None):
    import paper_2609_31975_b200 as m

    if m.lib_path().name != "libsparse_ffn.so":
        pytest.skip("runs against the release library only")
    assert m.load_library().sffn_test_set_knob(10, 1) == 2      # SFFN_ERR_UNSUPPORTED
    assert m.load_library().sffn_test_set_knob(10, 0) == 0
