"""Where the time inside the latency-bound kernels goes: SM-clock stamps of their phases.

    python -m paper_2502_04557_b200.phase_stamps

builds a second copy of the library with the stamps compiled in (-DSPR_VERIFIER_STAMPS
-DSPR_DRAW_STAMPS -> libsprinter_stamps.so beside the library; the normal build has none of it),
runs the tensor-core verifier and the draw kernel on the workload shapes and prints, per phase,
the median / min / max over the CTAs of one launch in microseconds since the CTA started
(SM clocks at 1965 MHz).  A development aid: the numbers quoted under profiles/ come from it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import sys

import numpy as np
import torch

from . import build as _build

STAMP_LIB = os.path.join(_build.PKG, "libsprinter_stamps.so")
MHZ = 1965.0


def build_stamped() -> str:
    cmd = [_build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17", "-shared",
           "-Xcompiler", "-fPIC", "-DSPR_VERIFIER_STAMPS", "-DSPR_DRAW_STAMPS", "-I",
           os.path.join(_build.ROOT, "include"), "-I", _build.CSRC, "-o", STAMP_LIB]
    subprocess.check_call(cmd + [os.path.join(_build.CSRC, f) for f in _build.SOURCES])
    return STAMP_LIB


def _report(tag, st, names):
    ok = st[:, 0] > 0
    rel = (st - st[:, :1]) / MHZ
    print(f"{tag}  (CTAs stamped: {int(ok.sum())})")
    for i, nm in enumerate(names):
        col = rel[ok & (st[:, i] > 0), i]
        if len(col):
            print(f"   {nm:34s} median {np.median(col):7.2f}  min {col.min():7.2f}  max {col.max():7.2f} us  (n={len(col)})")


VERIFIER = ["entry", "set-up done", "first copies issued", "first stage arrived (MMA issuer)", "all MMAs issued",
            "accumulator complete (epilogue)", "cluster hand-shake passed", "columns exchanged", "partial z done",
            "TMEM released", "tile finished"]
DRAW = ["entry", "after griddepcontrol.wait", "live lists built", "warp 0: first run streamed", "warp 0: ticket taken",
        "a draw finished", "warp 0: exit"]


def main():
    if "--no-build" not in sys.argv:
        build_stamped()
    _build.LIB = STAMP_LIB
    _build.stale = lambda: False
    import paper_2502_04557_b200 as spr
    from paper_2502_04557_b200 import binding as bd

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    L = spr.lib()
    for fn in (L.spr_debug_verifier_stamps, L.spr_debug_draw_stamps):
        fn.restype = ctypes.c_int
        fn.argtypes = [ctypes.c_void_p]

    def verifier(tag, M, K, d, h, **shape):
        H = torch.randn((M // K, K, d), device=dev).to(torch.bfloat16)
        W1 = (torch.randn((h, d), device=dev) / d ** 0.5).to(torch.bfloat16)
        b1 = torch.randn(h, device=dev) / d ** 0.5
        W2 = (torch.randn(h, device=dev) / h ** 0.5).to(torch.bfloat16)
        b2 = torch.zeros(1, device=dev)
        ws = spr.Workspace(spr.workspace_bytes(0, M // K, K, 1, d, h, spr.BF16), device=dev)
        def call():
            if shape:
                bd.sprinter_verify_shaped(H, W1, b1, W2, b2, 0.5, ws, **shape)
            else:
                spr.sprinter_verify(H, W1, b1, W2, b2, 0.5, ws)
        buf = np.zeros((512, 64), dtype=np.int64)
        for _ in range(4):
            call()
        torch.cuda.synchronize()
        assert L.spr_debug_verifier_stamps(buf.ctypes.data) == 0      # reads and clears
        call()
        torch.cuda.synchronize()
        assert L.spr_debug_verifier_stamps(buf.ctypes.data) == 0
        _report(f"verifier {tag}: M={M} K={K} d={d} h={h} {shape or 'library shape'}", buf.astype(np.float64), VERIFIER)

    def draw(tag, fn):
        buf = np.zeros((1024, 8), dtype=np.int64)
        for _ in range(4):
            fn()
        torch.cuda.synchronize()
        assert L.spr_debug_draw_stamps(buf.ctypes.data) == 0      # reads and clears
        fn()
        torch.cuda.synchronize()
        assert L.spr_debug_draw_stamps(buf.ctypes.data) == 0
        _report(f"draw {tag}", buf.astype(np.float64), DRAW)

    verifier("llama3", 4096, 16, 2048, 512)
    verifier("llama3, CTA pairs", 4096, 16, 2048, 512, bm=256, bn=128, splits=1, cluster_n=1)
    verifier("sequential B=8", 8, 1, 4096, 1024)
    verifier("sequential B=64", 64, 1, 4096, 1024)
    verifier("sequential B=1024", 1024, 1, 4096, 1024)
    verifier("gpt2", 256, 8, 768, 256)

    for name, B in (("llama3", None), ("sequential", 8), ("sequential", 1024)):
        wl = spr.workloads.make(name, dev, B=B)
        ws = spr.Workspace.for_problem(wl.B, wl.K, wl.V, wl.cfg.d, wl.cfg.h, spr.BF16, device=dev)
        _, _, fr = spr.sprinter_verify(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, 0.5, ws)
        draw(f"replacement draws, {name} B={wl.B}: {int((fr < wl.K).sum())} live of {wl.B}",
             lambda: spr.replace_sample(wl.p_logits, wl.V, wl.u_replace, ws, first_reject=fr, K=wl.K, seq_stride=wl.Kp))
        draw(f"correction draws behind the row statistics, {name} B={wl.B}",
             lambda: spr.sd_verify(wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, ws))


if __name__ == "__main__":
    main()
