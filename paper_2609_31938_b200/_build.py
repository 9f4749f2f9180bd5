"""In-tree build of the CUDA library (nvcc, sm_100a only)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.environ.get("CCV3D_LIB") or os.path.join(HERE, "libccv3d.so")   # (CCV3D_LIB: another build of the library, for diagnosis)
SOURCES = ["ccv3d_api.cu"]
DEPS = ["ccv3d_api.cu", "ccv3d_simt.cuh", "ccv3d_tc.cuh", "ccv3d_tc_layout.cuh", "ccv3d_tc_ptx.cuh", "ccv3d_tc_conv.cuh",
        "ccv3d_tc_pointwise.cuh", "ccv3d_host_common.cuh", "ccv3d_host_tc.cuh", "ccv3d_host_ring.cuh",
        os.path.join("..", "..", "include", "ccv3d.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libccv3d.so next to this file; returns its path."""
    if force or stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
              ["-o", LIB + ".tmp"] + [os.path.join(CSRC, s) for s in SOURCES]
        subprocess.run(cmd, check=True)
        os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
