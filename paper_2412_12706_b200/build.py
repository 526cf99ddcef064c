"""Builds the CUDA library in-tree: ``paper_2412_12706_b200/libqp.so`` (sm_100a only)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libqp.so")
LIB_CHECKED = os.path.join(HERE, "libqp_checked.so")   # the same sources with -DQP_CHECKED (device-side range checks)

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--shared", "-Xptxas", "-v"]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB) or not os.path.exists(LIB_CHECKED):
        return True
    t = min(os.path.getmtime(LIB), os.path.getmtime(LIB_CHECKED))
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        [os.path.join(os.path.dirname(HERE), "include", "qp.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = os.environ.get("QP_NVCC_EXTRA", "").split()
    cmds = [[nvcc] + NVCC_FLAGS + extra + ["-o", LIB] + sources(),
            [nvcc] + NVCC_FLAGS + extra + ["-DQP_CHECKED", "-o", LIB_CHECKED] + sources()]
    procs = [subprocess.Popen(c, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for c in cmds]
    for p, target in zip(procs, (LIB, LIB_CHECKED)):
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed building {os.path.basename(target)}")
    return LIB


if __name__ == "__main__":
    build(force=True, verbose=True)
    print(LIB)
