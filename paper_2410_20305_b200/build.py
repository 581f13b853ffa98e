"""Builds libpsa.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpsa.so")
LIB_DEBUG = os.path.join(HERE, "libpsa_debug.so")   # the same sources with -DPSA_DEBUG_BOUNDS (checked global indices)
SOURCES = ["psa_plan.cpp", "psa_host_helpers.cpp", "psa_api.cu", "psa_fwd.cu", "psa_bwd.cu", "psa_bwd_static.cu", "psa_selftest.cu",
           "dpo_logp.cu", "dpo_loss.cu", "psa_rope.cu"]


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "psa.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds libpsa.so, or with debug=True libpsa_debug.so: the same code with every index that a thread
    forms itself checked against its tensor (an out-of-range one sets PSA_DEVSTAT_OUT_OF_BOUNDS and is skipped)."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib] + [os.path.join(CSRC, s) for s in SOURCES]
    if debug:
        cmd += ["-DPSA_DEBUG_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building " + os.path.basename(lib))
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build(force=True, debug=True))
