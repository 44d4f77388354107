"""Builds libsparse_ffn.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Every source file is compiled to an object of its own (in parallel, only when it or a header changed) and the
objects are linked into the shared library.  `python -m paper_2609_31975_b200.build --trace` builds a second
library, libsparse_ffn_trace.so, whose single-token kernels write time stamps (see SFFN_KNOB_TRACE_BUFFER);
`--debug` builds libsparse_ffn_debug.so (-DSFFN_DEBUG), whose kernels check the indices they address global memory
with and report SFFN_ERR_BOUNDS in the device status instead of making the access.  Either is selected at run time
with the environment variable SFFN_LIBRARY."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libsparse_ffn.so"
OBJ = PKG / "build"
SOURCES = ["api.cu", "general_kernels.cu", "fused_kernel.cu", "fused_tc_kernel.cu", "static_entry.cu",
           "batched_kernels.cu", "umma_kernels.cu", "cast_kernels.cu"]


def _headers_mtime() -> float:
    deps = list(CSRC.glob("*.cuh")) + list((ROOT / "include").glob("*.h"))
    return max(d.stat().st_mtime for d in deps)


def build(force: bool = False, verbose: bool = False, trace: bool = False, debug: bool = False) -> Path:
    lib = PKG / "libsparse_ffn_trace.so" if trace else PKG / "libsparse_ffn_debug.so" if debug else LIB
    newest = max(_headers_mtime(), max((CSRC / s).stat().st_mtime for s in SOURCES))
    if not force and lib.exists() and lib.stat().st_mtime >= newest:
        return lib
    objdir = OBJ / ("trace" if trace else "debug" if debug else "plain")
    objdir.mkdir(parents=True, exist_ok=True)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-I", str(ROOT / "include"), "-I", str(CSRC)]
    if trace:
        flags += ["-DSFFN_TRACE"]
    if debug:
        flags += ["-DSFFN_DEBUG"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    hdr = _headers_mtime()
    todo = []
    for s in SOURCES:
        src, obj = CSRC / s, objdir / (s + ".o")
        if force or not obj.exists() or obj.stat().st_mtime < max(src.stat().st_mtime, hdr):
            todo.append((src, obj))

    def compile_one(job):
        src, obj = job
        tmp = obj.with_suffix(f".{os.getpid()}.tmp")
        r = subprocess.run([nvcc, *flags, "-c", str(src), "-o", str(tmp)], capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src.name}:\n{r.stdout}\n{r.stderr}")
        os.replace(tmp, obj)
        return r.stderr

    if todo:
        with ThreadPoolExecutor(max_workers=min(8, len(todo))) as pool:
            for log in pool.map(compile_one, todo):
                if verbose and log:
                    print(log, file=sys.stderr)
    objs = [objdir / (s + ".o") for s in SOURCES]
    if todo or not lib.exists() or any(o.stat().st_mtime > lib.stat().st_mtime for o in objs):
        tmp = lib.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run([nvcc, "-shared", "-o", str(tmp), *map(str, objs)], check=True)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, trace="--trace" in sys.argv, debug="--debug" in sys.argv))
