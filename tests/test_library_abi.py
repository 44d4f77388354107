"""CPU-side checks of the product: the C-ABI library builds, loads and exports every declared entry
point; host helpers agree with the oracle's restatement; the oracle is not reachable from the package."""
import ctypes
import re
from pathlib import Path

import numpy as np

import oracle

ROOT = Path(__file__).resolve().parent.parent


def declared_functions():
    text = (ROOT / "include" / "sparse_ffn.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(?:int|const char\*)\s+(\w+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2609_31975_b200 import build

    lib = ctypes.CDLL(str(build.build()))
    names = declared_functions()
    assert {"sparse_ffn_forward", "dense_ffn_forward", "sffn_create", "sffn_workspace_bytes",
            "sparse_ffn_forward_host", "sffn_last_active"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in sparse_ffn.h but not exported"


def test_host_side_validation_without_a_gpu():
    import paper_2609_31975_b200 as m

    lib = m.load_library()
    need = ctypes.c_size_t(0)
    assert lib.sffn_workspace_bytes(4096, 14336, 1024, 64, 1, ctypes.byref(need)) == 0
    assert need.value > 64 * 14336 * 4
    assert lib.sffn_workspace_bytes(4100, 14336, 0, 1, 1, ctypes.byref(need)) == 2      # 8200-byte rows
    assert lib.sffn_workspace_bytes(0, 14336, 0, 1, 1, ctypes.byref(need)) == 1
    assert lib.sffn_workspace_bytes(4096, 14336, 0, 1, 7, ctypes.byref(need)) == 1      # bad dtype
    assert lib.sffn_create(None, 4096, 14336, 0, 1, 1, None, 0) == 1
    h = ctypes.c_void_p()
    assert lib.sffn_create(ctypes.byref(h), 4096, 14336, 0, 1, 1, None, 0) == 3         # no workspace
    assert lib.sffn_status_string(5) == b"device-side bounded wait ran out"
    assert lib.sparse_ffn_forward(None, None, 1, None, None, None, None, 0, None, None) == 1
    assert lib.sffn_set_up_activation(None, 0) == 1                                      # no handle
    buf = (ctypes.c_float * 8)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    assert lib.sffn_residual_cast(None, p, 1.0, p, 8, 0, None) == 1                      # null y
    assert lib.sffn_residual_cast(p, p, 1.0, p, 6, 0, None) == 1                         # n not a multiple of 4
    assert lib.sffn_residual_cast(p, p, 1.0, p, 8, 5, None) == 1                         # bad dtype
    assert lib.sffn_residual_cast(p, ctypes.c_void_p(p.value + 4), 1.0, p, 4, 0, None) == 2   # misaligned
    assert lib.sffn_last_cuda_error() == b"cudaSuccess"


def test_product_index_generators_match_the_oracle_restatement():
    import paper_2609_31975_b200 as m

    for H, D in ((12, 6), (14336, 4096), (28672, 8192), (10240, 3840), (1531, 512)):
        np.testing.assert_array_equal(m.g_diagonal(H, D).numpy(), oracle.g_diagonal(H, D))
        np.testing.assert_array_equal(m.g_tiled(H, D).numpy(), oracle.g_tiled(H, D))
    # byte model: standard gate at the decode shape, 10 % of the rows -> 140.9 MB; dense 352.3 MB
    assert abs(m.touched_bytes(4096, 14336, 1434, 2) / 1e6 - 141.0) < 0.2
    assert abs(m.dense_bytes(4096, 14336, 2) / 1e6 - 352.4) < 0.2


def test_product_never_imports_the_oracle():
    for f in (ROOT / "paper_2609_31975_b200").rglob("*"):
        if f.suffix in (".py", ".cu", ".cuh", ".h"):
            assert "oracle" not in f.read_text().lower(), f
