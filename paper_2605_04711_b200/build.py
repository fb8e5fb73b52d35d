"""Build the CUDA library in-tree: ``python -m paper_2605_04711_b200.build``.

Compiles every source under ``csrc/`` for sm_100a with nvcc and links
``libbaoc.so`` next to this file.  Works without a GPU (cross-compilation).
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libbaoc.so")
LIB_CHECKED = os.path.join(HERE, "libbaoc_checked.so")     # the same sources with -DBAOC_CHECKED (see csrc/baoc_check.cuh)
SOURCES = ["baoc_host.cpp", "baoc_partition.cpp", "baoc_api.cu", "baoc_stats.cu", "baoc_finalize.cu", "baoc_step.cu", "baoc_noalloc.cu",
           "baoc_convert.cu"]
HEADERS = [os.path.join(ROOT, "include", "baoc.h"), os.path.join(CSRC, "baoc_internal.h"),
           os.path.join(CSRC, "baoc_device.cuh"), os.path.join(CSRC, "baoc_check.cuh")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """checked: build libbaoc_checked.so, the variant whose kernels validate every tile and range before touching memory."""
    lib = LIB_CHECKED if checked else LIB
    if not force and not needs_build(lib):
        return lib
    nvcc = _nvcc()
    bdir = os.path.join(HERE, "_build", "checked" if checked else "plain")
    os.makedirs(bdir, exist_ok=True)
    common = ["-std=c++17", "-O3", "-Wno-deprecated-gpu-targets", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
              "-Xcompiler", "-fPIC,-ffp-contract=off,-Wall"] + (["-DBAOC_CHECKED"] if checked else [])
    cuda_flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo"]
    if verbose:
        cuda_flags += ["-Xptxas", "-v"]
    objs = []
    for src in SOURCES:
        obj = os.path.join(bdir, src + ".o")
        cmd = [nvcc] + common + (cuda_flags if src.endswith(".cu") else []) + \
              ["-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
        objs.append(obj)
    subprocess.run([nvcc, "-shared", "-Wno-deprecated-gpu-targets", "-o", lib] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"], check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
