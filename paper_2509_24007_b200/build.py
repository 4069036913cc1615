"""Builds libsdlm.so (the C-ABI library with the sm_100a kernels) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsdlm.so")
LIB_TIMELINE = os.path.join(HERE, "libsdlm_timeline.so")   # the same library with in-kernel wall-clock marks (--timeline)
SOURCES = ["sdlm_api.cu", "sdlm_attn.cu", "sdlm_causal.cu", "sdlm_lmhead.cu", "sdlm_layer.cu"]
HEADERS = ["sdlm_internal.h", "sdlm_ptx.cuh", os.path.join("..", "..", "include", "sdlm.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, timeline: bool = False) -> str:
    """Compile every CUDA source for sm_100a into one shared library; returns its path.  timeline=True
    builds a second library, libsdlm_timeline.so, whose attention kernel leaves wall-clock marks that
    bench.py --timeline reads (a measuring aid; the product library is unchanged)."""
    if timeline:
        out = LIB_TIMELINE
    else:
        out = LIB
        if not force and not needs_build():
            return LIB
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-o", out] + (["-DSDLM_TIMELINE"] if timeline else []) + \
          [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas"); cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        sys.stderr.write(res.stderr)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, timeline="--timeline" in sys.argv))
