"""Builds the CUDA library in-tree:  python -m paper_2410_03960_b200.build

One nvcc invocation compiles every .cu under csrc/ for sm_100a into libswiftkv.so next to this file.
nvcc cross-compiles without a GPU, so this also runs on a CPU-only machine.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libswiftkv.so")
SOURCES = ["api.cu", "elementwise.cu", "gemm_simt.cu", "gemm_tc.cu", "attention_simple.cu", "attention_tc.cu", "tail.cu", "tail_noalloc.cu", "kv_fp8.cu", "simscore.cu", "distill.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--use_fast_math",
              "-Xcompiler", "-fPIC", "-shared", "-Xptxas", "-v"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "swiftkv.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed building libswiftkv.so")
    # register / spill / shared-memory report of ptxas: scratch output, kept out of the source tree
    log_dir = os.environ.get("SWIFTKV_BUILD_LOG_DIR", os.path.join(HERE, "..", "gpurun_out"))
    try:
        os.makedirs(log_dir, exist_ok=True)
        with open(os.path.join(log_dir, "build_ptxas.log"), "w") as f:
            f.write(proc.stdout + proc.stderr)
    except OSError:
        pass
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
