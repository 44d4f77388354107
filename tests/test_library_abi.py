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
    return sorted(set(re.findall(r"\b(?:int|void|const char\*)\s+(\w+)\s*\(", text)))


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


def test_kernel_geometry_invariants_on_the_host():
    """The launch geometry is host code: its invariants can be checked for many shapes without a GPU."""
    import paper_2609_31975_b200 as m

    lib = m.load_library()
    out = (ctypes.c_int * 9)()
    n_ok = 0
    for bf16 in (1, 0):
        esz = 2 if bf16 else 4
        for D in (256, 512, 1024, 2048, 3840, 4096, 5120, 8192, 16384):
            for H in (64, 777, 1024, 10240, 14336, 28672, 53248):
                for lopa, K in ((0, D), (1, 64), (1, 256), (1, 480), (1, 1024)):
                    lib.sffn_test_fused_plan(bf16, D, H, K, lopa, 148, out)
                    ok, nr, gsb, ng, gw, asb, na, cpt, smem = list(out)
                    if not ok:
                        continue
                    n_ok += 1
                    assert smem <= 227 * 1024
                    assert nr >= 1 and nr * K * esz <= gsb and gsb % 128 == 0
                    assert gw >= 2 and gw % 2 == 0 and gw <= (4 if lopa else 8)
                    assert ng % gw == 0 and ng >= gw          # a ring slot always belongs to the same gate warp
                    assert na >= 2 and asb >= 2 * D * esz
                    act_threads = 256 if lopa else 128
                    assert cpt in (1, 2, 4, 8) and cpt * act_threads * (16 // esz) >= D
    assert n_ok > 300                                          # the benchmark shapes and most others are served
    lib.sffn_test_fused_plan(1, 4096, 14336, 4096, 0, 148, out)
    assert list(out)[0] == 1 and list(out)[3] == 16            # the graded shape: 16 gate slots of one 8 KB row
    tr, nt, own = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    for R in (8, 64, 100, 777, 1184, 1200, 14336, 18944, 18945, 28672, 53248, 200000):
        lib.sffn_test_umma_tiling(R, 148, ctypes.byref(tr), ctypes.byref(nt), ctypes.byref(own))
        assert tr.value % 8 == 0 and 8 <= tr.value <= 128
        assert (nt.value - 1) * tr.value < R <= nt.value * tr.value          # the tiles cover the rows exactly
        assert nt.value <= 148 or tr.value == 128                             # one tile per SM until tiles are full
        if own.value:
            assert 4 * nt.value <= 4 * 384                                    # mask words fit the in-kernel scan
    lib.sffn_test_umma_tiling(14336, 148, ctypes.byref(tr), ctypes.byref(nt), ctypes.byref(own))
    assert (tr.value, nt.value, own.value) == (104, 138, 1)


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
