"""Builds the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "librpa_b200.so")
# the bounds-checked build (-DRPA_DEBUG): every page id, token row and ring stage is checked before
# the access and the first violation is recorded in the device status word
LIB_DEBUG = os.path.join(PKG, "librpa_b200_debug.so")
SOURCES = ["rpa_api.cu", "rpa_row_kernel.cu", "rpa_row_kernel_fp8.cu", "rpa_tile_kernel.cu", "rpa_tile1_kernel.cu", "rpa_tile2_kernel.cu", "rpa_static.cu", "rpa_plan_kernel.cu", "rpa_planner.cc"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--use_fast_math",
              "-Xcompiler", "-fPIC,-Wall,-Wno-unknown-pragmas", "-Xptxas", "-v"]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    built = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(PKG, "..", "include", "rpa.h")]
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile ``csrc/*`` into ``librpa_b200.so`` next to this file; returns its path.  ``debug``
    builds the bounds-checked variant ``librpa_b200_debug.so`` instead (same sources, -DRPA_DEBUG)."""
    lib = LIB_DEBUG if debug else LIB
    if not (force or _stale(lib)):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(PKG, "build_debug" if debug else "build", os.path.splitext(src)[0] + ".o")
        os.makedirs(os.path.dirname(obj), exist_ok=True)
        cmd = [nvcc, *NVCC_FLAGS, *(["-DRPA_DEBUG"] if debug else []), "-c", os.path.join(CSRC, src), "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True, debug="--debug" in sys.argv))
