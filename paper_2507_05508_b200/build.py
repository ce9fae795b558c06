"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libmlmc.so")
SOURCES = ["api.cu", "topk_select.cu", "topk_emit.cu", "bitwise.cu", "floatbits.cu", "rtn.cu", "stopk_sort.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC", "--fmad=true", "-Xptxas", "-v",
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_HERE, "..", "include", f) for f in ("mlmc.h", "mlmc_instr.h")]
    return any(os.path.getmtime(f) > t for f in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libmlmc.so next to this file and return its path."""
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + [os.path.join(CSRC, f) for f in SOURCES] + ["-o", LIB]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:  # noqa
            print(res.stdout)
            print(res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed")
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
