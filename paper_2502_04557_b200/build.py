"""Builds libsprinter.so (the CUDA kernels and their C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libsprinter.so")
SOURCES = ["api.cu", "host_api.cu", "sd_row_stats.cu", "draw.cu", "verifier_simt.cu", "verifier_tensor.cu", "no_alloc.cu", "simulate.cu", "sd_shard.cu", "sd_shard_api.cu", "verifier_fit.cu"]
HEADERS = ["common.cuh", "launch.h", "verifier_common.cuh", "vocab_common.cuh", "draw_common.cuh", "host_util.h"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(ROOT, "include", "sprinter.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles every source that is newer than its object file (all of them after a header
    change), several at a time, and links the objects into the shared library."""
    if not force and not stale():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    obj_dir = os.path.join(PKG, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
             "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    headers = [os.path.join(CSRC, f) for f in HEADERS] + [os.path.join(ROOT, "include", "sprinter.h")]
    newest_header = max(os.path.getmtime(h) for h in headers)

    def compile_one(name):
        src = os.path.join(CSRC, name)
        obj = os.path.join(obj_dir, name[:-3] + ".o")
        if (not force and not verbose and os.path.exists(obj)
                and os.path.getmtime(obj) > max(os.path.getmtime(src), newest_header)):
            return obj
        subprocess.check_call([_nvcc(), *flags, "-c", src, "-o", obj])
        return obj

    with ThreadPoolExecutor(min(len(SOURCES), os.cpu_count() or 4)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.check_call([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objs])
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
