"""Build the CUDA library (sm_100a only) next to this file: libatomo_b200.so.

Each source is compiled to an object of its own (in parallel, rebuilt only when it or a header is newer) under
``csrc/build/`` and the objects are linked into the shared library."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(CSRC, "build")
LIB = os.path.join(HERE, "libatomo_b200.so")
SOURCES = ["atomo_api.cu", "atomo_entrywise.cu", "atomo_spectral.cu", "atomo_eig.cu", "atomo_tc.cu", "atomo_static.cu",
           "atomo_average.cu", "atomo_tridiag.cu", "atomo_tridiag_big.cu", "atomo_peaks.cu"]
HEADERS = ["atomo_common.cuh", "atomo_kernels.cuh", "atomo_twisted.cuh"]


def _header_time() -> float:
    deps = [os.path.join(CSRC, f) for f in HEADERS] + [os.path.join(ROOT, "include", "atomo.h")]
    return max(os.path.getmtime(d) for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    ht = _header_time()
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]

    def compile_one(src: str):
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src.replace(".cu", ".o"))
        if not force and os.path.exists(o) and os.path.getmtime(o) > max(os.path.getmtime(s), ht):
            return o, False
        subprocess.check_call([nvcc] + flags + ["-c", s, "-o", o])
        return o, True

    with ThreadPoolExecutor(max_workers=min(8, len(SOURCES))) as ex:
        results = list(ex.map(compile_one, SOURCES))
    objs = [o for o, _ in results]
    if force or any(changed for _, changed in results) or not os.path.exists(LIB):
        subprocess.check_call([nvcc, "-shared", "-o", LIB] + objs)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
