"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess
import sys

_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_DIR, "csrc")
LIB = os.environ.get("AAAC_B200_LIB") or os.path.join(_DIR, "libaaac_b200.so")
SOURCES = ["api.cu", "act_stats.cu", "scales.cu", "init.cu", "fit.cu", "pack.cu", "dequant.cu", "prescale.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "--fmad=true", "-prec-div=true", "-prec-sqrt=true", "-ftz=false"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    if os.environ.get("AAAC_B200_LIB"):
        return False                      # a library named explicitly is used as it is
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(os.path.dirname(_DIR), "include", "aaac.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + os.environ.get("AAAC_NVCC_EXTRA", "").split() + (["-Xptxas", "-v"] if verbose else []) + \
              [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB]
        subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
