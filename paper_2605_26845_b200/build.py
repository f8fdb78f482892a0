"""Build libmoesched.so (CUDA kernels + C ABI) for sm_100a with nvcc, in-tree."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SOURCES = ["api.cu", "mw_kernel.cu", "mw_team_kernel.cu", "bvn_kernel.cu", "bvn_team_kernel.cu", "bvn_real_kernel.cu", "eval_kernel.cu", "eval_team_kernel.cu", "order_kernel.cu", "bvn_static.cu", "probe.cu", "a2a_kernel.cu", "sinkhorn_kernel.cu"]
HEADERS = [os.path.join(CSRC, "common.cuh"), os.path.join(CSRC, "team.cuh"), os.path.join(HERE, "..", "include", "moesched.h")]
LIB = os.path.join(HERE, "libmoesched.so")
LIB_CHECKED = os.path.join(HERE, "libmoesched_checked.so")   # the same sources with -DMOESCHED_CHECKED


def _stale(lib) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile every source to an object file (in parallel, one nvcc per file) and link the library.
    checked=True builds the variant whose kernels range-check their data-dependent indices."""
    lib = LIB_CHECKED if checked else LIB
    if not (force or _stale(lib)):
        return lib
    from concurrent.futures import ThreadPoolExecutor
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(HERE, "_build_checked" if checked else "_build")
    os.makedirs(objdir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]
    if checked:
        flags += ["-DMOESCHED_CHECKED"]
    if verbose:
        flags += ["-Xptxas", "-v"]

    def compile_one(src):
        obj = os.path.join(objdir, os.path.splitext(src)[0] + ".o")
        subprocess.run([nvcc, *flags, "-c", os.path.join(CSRC, src), "-o", obj], check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objects = list(pool.map(compile_one, SOURCES))
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static", "-o", lib,
                    *objects], check=True)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
