"""Streaming ceilings of the two HBM-bound loops, measured by two stand-alone CUDA programs.

    python -m paper_2502_04557_b200.stream_probes

builds csrc/probes/read_probe.cu and csrc/probes/stats_probe.cu beside the library (nvcc, sm_100a)
and runs them on the current GPU: about 7 GB of device memory, a few seconds.  A development
aid: the tables under profiles/ that split a kernel's distance from the bare loop into parts
come from these programs.  Nothing in the library calls them.
"""
from __future__ import annotations

import os
import subprocess
import sys

from . import build as _build

PROBES = ["read_probe", "stats_probe"]
SRC = os.path.join(_build.CSRC, "probes")
OUT = os.path.join(_build.PKG, "_build")


def build() -> list[str]:
    os.makedirs(OUT, exist_ok=True)
    exes = []
    for name in PROBES:
        exe = os.path.join(OUT, name)
        src = os.path.join(SRC, name + ".cu")
        if not os.path.exists(exe) or os.path.getmtime(exe) < os.path.getmtime(src):
            subprocess.check_call([_build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo",
                                   "-std=c++17", "--extended-lambda", "-I", _build.CSRC, "-I",
                                   os.path.join(_build.ROOT, "include"), "-o", exe, src])
        exes.append(exe)
    return exes


def main() -> int:
    rc = 0
    for exe in build():
        print("==", os.path.basename(exe), flush=True)
        rc |= subprocess.call([exe])
    return rc


if __name__ == "__main__":
    sys.exit(main())
