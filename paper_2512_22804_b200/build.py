"""Builds ``libmor_b200.so`` (the C-ABI library with the sm_100a kernels) in-tree with nvcc.

Run as ``python -m paper_2512_22804_b200.build``.  nvcc cross-compiles, so no GPU is needed.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmor_b200.so")
SOURCES = ["mor_api.cu", "mor_kernels.cu", "mor_static.cu", "mor_main.cu", "mor_main_tensor.cu", "mor_main_row128.cu",
           "mor_main_blk128.cu", "mor_main_blk64.cu", "mor_main_col128.cu", "mor_main_channel.cu", "mor_main_dual.cu", "mor_main_colch.cu"]
OBJ_DIR = os.path.join(HERE, "_build")


def nvcc_path() -> str:
    p = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(p):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return p


def _deps():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "mor.h")]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in _deps())


def build(force: bool = False, verbose: bool = False, lib: str = LIB, extra_flags=(), obj_dir=None) -> str:
    """Compile every source file to an object (side by side: the main kernel's instantiations are spread over
    several files for that purpose) and link the shared library."""
    if not force and lib == LIB and not needs_build():
        return lib
    from concurrent.futures import ThreadPoolExecutor

    obj_dir = obj_dir or (OBJ_DIR if lib == LIB else lib + ".obj")
    os.makedirs(obj_dir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "--ftz=false", "--prec-div=true", "--prec-sqrt=true", "-Xfatbin", "-compress-all",
             "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    flags += list(extra_flags)
    if verbose:
        flags += ["-Xptxas", "-v"]
    newest = max(os.path.getmtime(d) for d in _deps() if d.endswith((".h", ".cuh")))

    def compile_one(src: str) -> str:
        obj = os.path.join(obj_dir, src[:-3] + ".o")
        path = os.path.join(CSRC, src)
        if force or verbose or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(path), newest):
            subprocess.run([nvcc_path(), *flags, "-c", path, "-o", obj], check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 4)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    subprocess.run([nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", *objs, "-o", lib], check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
