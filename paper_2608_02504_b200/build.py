"""Builds the C-ABI CUDA library in-tree: ``python -m paper_2608_02504_b200.build``.

Every ``.cu`` file is compiled to an object of its own (in parallel) and the objects are linked
into ``libtra_b200.so`` next to this file.  ``-DTRA_DEBUG`` builds (``build(debug=True)``) go to
``libtra_b200_debug.so``: the same sources with every global index checked on the device.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtra_b200.so")
LIB_DEBUG = os.path.join(HERE, "libtra_b200_debug.so")
SOURCES = ["tra_plan.cu", "tra_radius.cu", "tra_mask.cu", "tra_attn.cu", "tra_attn_d128_b128.cu",
           "tra_attn_d64_b64.cu", "tra_attn_d64_b128.cu", "tra_attn_d128_b64.cu", "tra_host.cu"] + \
          [f"tra_attn_d{d}_any{bn}.cu" for d in (128, 64) for bn in (48, 64, 80, 96, 112, 128)]


def _headers():
    return sorted(glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h"))) + \
        [os.path.join(ROOT, "include", "tra.h")]


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    objdir = os.path.join(HERE, "build", "debug" if debug else "release")
    srcs = [os.path.join(CSRC, s) for s in SOURCES]
    hdr_time = max(os.path.getmtime(h) for h in _headers())
    if not force and os.path.exists(lib) and all(os.path.getmtime(lib) >= os.path.getmtime(d) for d in srcs) \
            and os.path.getmtime(lib) >= hdr_time:
        return lib
    os.makedirs(objdir, exist_ok=True)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if debug:
        flags.append("-DTRA_DEBUG")
    if verbose:
        flags += ["-Xptxas", "-v"]

    def compile_one(src):
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr_time):
            subprocess.check_call([nvcc] + flags + ["-c", src, "-o", obj])
        return obj

    with ThreadPoolExecutor(max_workers=min(len(srcs), os.cpu_count() or 4)) as pool:
        objs = list(pool.map(compile_one, srcs))
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "--shared", "-o", tmp] + objs)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
