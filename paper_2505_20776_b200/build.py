"""Compiles the CUDA sources into the in-tree shared libraries (sm_100a only).

libspecext.so is the product.  libspecext_testing.so is the same code compiled with -DSPECEXT_TESTING
plus the CUDA-core cross-check kernel and a few test hooks (csrc/testing.h); only the tests load it.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_PATH = os.path.join(HERE, "libspecext.so")
TESTING_LIB_PATH = os.path.join(HERE, "libspecext_testing.so")
SOURCES = ["api.cu", "attn_tc2.cu", "attn_tc.cu", "prefill_tc2.cu", "merge.cu", "retrieval.cu"]
TESTING_SOURCES = SOURCES + ["attn_simt.cu", "testing.cu"]


def nvcc_path() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "specext.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def needs_build() -> bool:
    return _stale(LIB_PATH)


def _compile(lib: str, sources, defines, verbose: bool) -> str:
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "static", "-o", lib] + list(defines)
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in sources]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(lib)}")
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """Builds libspecext.so next to this file and returns its path."""
    if not force and not needs_build():
        return LIB_PATH
    return _compile(LIB_PATH, SOURCES, [], verbose)


def build_testing(force: bool = False, verbose: bool = False) -> str:
    """Builds the test library (cross-check kernel and test hooks) and returns its path."""
    if not force and not _stale(TESTING_LIB_PATH):
        return TESTING_LIB_PATH
    return _compile(TESTING_LIB_PATH, TESTING_SOURCES, ["-DSPECEXT_TESTING"], verbose)


def build_all(force: bool = False, verbose: bool = False) -> None:
    """Both libraries, compiled side by side."""
    with ThreadPoolExecutor(2) as ex:
        a = ex.submit(build, force, verbose)
        b = ex.submit(build_testing, force, verbose)
        a.result()
        b.result()


if __name__ == "__main__":
    build_all(force=True, verbose="-v" in sys.argv)
    print(LIB_PATH)
    print(TESTING_LIB_PATH)
