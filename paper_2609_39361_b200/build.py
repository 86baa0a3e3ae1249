"""Build the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
SRC = os.path.join(_HERE, "csrc", "lamp_attn.cu")
LIB = os.path.join(_HERE, "liblamp_attn.so")
DEPS = [SRC] + [os.path.join(_HERE, "csrc", f) for f in ("lamp_common.cuh", "lamp_fwd_sm100.cuh", "sm100_ptx.cuh")] + [
    os.path.join(ROOT, "include", "lamp_attn.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",            # no implicit multiply-add contraction anywhere on the decision path
    "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"),
]


def build(force: bool = False, verbose: bool = False) -> str:
    deps = [d for d in DEPS if os.path.exists(d)]
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in deps):
        return LIB
    extra = ["-DLAMP_PHASE_TIMERS=" + os.environ["LAMP_PHASE_TIMERS"]] if os.environ.get("LAMP_PHASE_TIMERS") else []
    cmd = ["nvcc"] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + [SRC, "-o", LIB]
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
