"""Build the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "liblossy_b200.so")
CHECK_LIB_PATH = os.path.join(PKG_DIR, "liblossy_b200_check.so")   # the debug build: -DLOSSY_DEVCHECK (index checks in the kernels)
SOURCES = ["lossy_api.cu", "lossy_noalloc.cu"]
HEADERS = ["lossy_device.cuh", "lossy_kernels.cuh", "lossy_tma.cuh", "lossy_gather.cuh", "lossy_phase_tma.cuh", os.path.join("..", "..", "include", "lossy.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false",                      # every fp32 operation of the contract is rounded on its own
    "-Xcompiler", "-fPIC", "-shared",
]


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile liblossy_b200.so and its debug twin liblossy_b200_check.so next to this file (the two nvcc runs side by
    side); returns the path of the normal library."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    jobs = []
    for lib, extra in ((LIB_PATH, []), (CHECK_LIB_PATH, ["-DLOSSY_DEVCHECK=1"])):
        if not force and not _stale(lib):
            continue
        cmd = [nvcc, *NVCC_FLAGS, *extra, *(["-Xptxas", "-v"] if verbose and not extra else []), "-o", lib + ".tmp",
               *[os.path.join(CSRC, s) for s in SOURCES]]
        jobs.append((lib, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)))
    failed = []
    for lib, proc in jobs:
        out, err = proc.communicate()
        if verbose:
            sys.stderr.write(err)
        if proc.returncode != 0:
            failed.append(os.path.basename(lib) + ":\n" + out + err)
        else:
            os.replace(lib + ".tmp", lib)
    if failed:
        raise RuntimeError("nvcc failed:\n" + "\n".join(failed))
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
