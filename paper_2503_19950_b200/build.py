"""Build the CUDA library (sm_100a only) in-tree: paper_2503_19950_b200/liblogquant.so."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "liblogquant.so")
LIB_BOUNDS = os.path.join(_HERE, "liblogquant_bounds.so")  # the same library with the index checks compiled in
SOURCES = ["lq_api.cu", "lq_store_kernels.cu", "lq_decode_scalar.cu", "lq_decode_mma.cu", "lq_decode_umma.cu", "lq_decode_static.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "--expt-relaxed-constexpr", "--threads", "0"]


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_HERE, "..", "include", "lq.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, bounds: bool = False) -> str:
    """bounds=True builds liblogquant_bounds.so: -DLQ_DEBUG_BOUNDS, every index that comes from the host's bookkeeping
    is checked in the kernels (a failing check sets bit 2 of the status word and skips the access).  Point the
    binding at it with the environment variable LOGQUANT_LIBRARY."""
    lib = LIB_BOUNDS if bounds else LIB
    if force or _stale(lib):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-DLQ_DEBUG_BOUNDS"] if bounds else []) + (["-Xptxas", "-v"] if verbose else []) + \
              [os.path.join(CSRC, s) for s in SOURCES] + ["-o", lib + ".tmp"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode:
            raise RuntimeError("nvcc failed")
        os.replace(lib + ".tmp", lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, bounds="--bounds" in sys.argv))
