"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = os.path.join(HERE, "csrc", "gac.cu")
HDR = os.path.join(ROOT, "include", "gac.h")
KERNELS = os.path.join(HERE, "csrc", "gac_kernels.cuh")
LIB = os.path.join(HERE, "libgac_b200.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-ldl"]


def build(force: bool = False, verbose: bool = False) -> str:
    newest = max(os.path.getmtime(SRC), os.path.getmtime(HDR), os.path.getmtime(KERNELS))
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= newest:
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-I", os.path.join(ROOT, "include"), "-o", LIB, SRC]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed: " + " ".join(cmd))
    return LIB


PROBE_SRC = os.path.join(HERE, "csrc", "stream_probe.cu")
PROBE = os.path.join(HERE, "stream_probe")


def build_probe(force: bool = False) -> str:
    """Builds the stand-alone HBM stream-pattern probe (an executable, not part of the library)."""
    if not force and os.path.exists(PROBE) and os.path.getmtime(PROBE) >= os.path.getmtime(PROBE_SRC):
        return PROBE
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-o", PROBE, PROBE_SRC]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
        raise RuntimeError("nvcc failed: " + " ".join(cmd))
    return PROBE


if __name__ == "__main__":
    if len(sys.argv) > 1 and sys.argv[1] == "probe":
        print(build_probe(force=True))
    else:
        print(build(force=True, verbose=True))
