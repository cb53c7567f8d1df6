"""Builds libhilberta.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhilberta.so")
SOURCES = ["plan.cu", "schedule.cu", "permute.cu", "attn_fp32.cu", "attn_fp32_bwd.cu", "attn_bf16_sm100.cu", "attn_bf16_pair_sm100.cu", "attn_bf16_solo_sm100.cu", "attn_bwd_sm100.cu"]
HEADERS = ["common.cuh", "sm100_ptx.cuh", "attn_softmax_math.cuh"]


def _newest_source() -> float:
    files = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "hilberta.h")]
    return max(os.path.getmtime(f) for f in files if os.path.exists(f))


def build_library(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
