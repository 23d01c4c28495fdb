#!/usr/bin/env python
"""Throughput of the verification-and-replacement hot path on synthetic inputs.

One step = one pass of the whole path over one batch: sprinter_verify (verifier scores,
threshold, first-rejection scan) -> replace_sample gated by first_reject (replacement tokens),
issued as the fused sprinter_step call, and sd_verify (exact speculative-decoding verification
of the same draft tokens); one after the other on one stream, or side by side on two
(--streams 2).  The
metric is draft tokens taken through that step per second, summed over all GPUs (each rank
verifies its own batch: weak scaling, no data-path collective).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama3] [--impl reference]

Prints one JSON line on rank 0.
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of one sd_row_stats_kernel launch, from the ncu
# capture summarised under profiles/; reported only while the kernel source is unchanged.
NCU_TRAFFIC = {
    "sources": ("sd_row_stats.cu", "vocab_common.cuh", "common.cuh"),
    "sha256": "92f757294d7190decb7184a5f36af6e55a97fcbc066b770e53c7166cfdb6104c",
    # (394,077,184 read + 3,215,360 written) / 768 tokens in the B = 48 capture (the smallest batch that
    # takes the same kernel variant as the full launch); traffic grows in proportion to the tokens, so a
    # full launch is this times B*K
    "bytes_per_unit": 517308,   # DRAM bytes per verified token at V = 128256, bf16
}


def kernel_sources_sha():
    h = hashlib.sha256()
    for name in NCU_TRAFFIC["sources"]:
        with open(os.path.join(ROOT, "paper_2502_04557_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="llama3")
    ap.add_argument("--batch", type=int, default=None, help="sequences per GPU (default: the configuration's)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--threshold", type=float, default=0.5)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rotate", type=int, default=1,
                    help="1: rotate small workloads through copies that together exceed L2 four times; 0: reuse "
                         "one copy (L2-warm numbers)")
    ap.add_argument("--graph", default="auto", choices=["auto", "0", "1"],
                    help="1: the timed steps are replays of CUDA graphs of the step (no host launch cost between "
                         "kernels); auto: only when a step takes the GPU less time than the host needs to issue it")
    ap.add_argument("--stage-every", type=int, default=8,
                    help="the row-statistics launch is bracketed by CUDA events in every n-th timed step (the event "
                         "records sit between two launches and keep the second from starting early)")
    ap.add_argument("--streams", type=int, default=1, choices=[1, 2],
                    help="1: sd_verify then sprinter_step on one stream; 2: the two calls of a step on two streams")
    ap.add_argument("--shard", default="batch", choices=["batch", "vocab"],
                    help="how --gpus N ranks split the work: every rank its own batch (default), or every "
                         "rank V/N columns of the same logits (sd_verify only, NCCL exchanges between the passes)")
    ap.add_argument("--vocab-shards", type=int, default=8,
                    help="also time the four passes of the vocabulary-sharded sd_verify on one of this many "
                         "column shards (0 = skip)")
    ap.add_argument("--fit-samples", type=int, default=1 << 20,
                    help="hidden states in the timed verifier_train_step call")
    ap.add_argument("--simulator-runs", type=int, default=0,
                    help="also time sprinter_simulate on this many runs (r=5, eta_TP=0.9, eta_FP=0.5)")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peak():
    """Dense bf16 TFLOP/s of a kernel timed alone (the burst figure)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


# sm__pipe_tensor_cycles_active of verifier_tcgen05_kernel from the ncu capture summarised under
# profiles/ (a counter that only a profiler gives); reported while the kernel source is unchanged
NCU_VERIFIER = {
    "sources": ("verifier_tensor.cu", "verifier_common.cuh"),
    "sha256": "05f682cd9270bb251daa1c243f73ac4a3d85c05fe772cea7c27af85fb4de9c86",
    # full-size llama3 launch (128 x 128 tiles, grid (1, 4, 32)): 29.3 % of the pipe's peak while
    # active, 19.5 % of elapsed
    "tensor_pipe_pct_while_active": 29.3,
    "profile": "profiles/draw_kernel_and_verifier_llama3.md",
}


def sources_sha(names):
    h = hashlib.sha256()
    for name in names:
        with open(os.path.join(ROOT, "paper_2502_04557_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs.  Reads NVML from a
    thread of this process every few milliseconds (read-only queries), so that even a timed
    region of a few milliseconds gets samples; nvidia-smi in a loop is the fallback."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period = index, period_s
        self.samples = []          # (wall time, sm MHz, max sm MHz, set of reasons)
        self.proc = self.thread = None
        self.source = None
        self._stop = threading.Event()

    def _physical_index(self):
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "").strip()
        if vis:
            ids = [v.strip() for v in vis.split(",") if v.strip()]
            if self.index < len(ids) and ids[self.index].isdigit():
                return int(ids[self.index])
        return self.index

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self._physical_index())
            mx = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            bits = (("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown),
                    ("hw_thermal_slowdown", nv.nvmlClocksEventReasonHwThermalSlowdown),
                    ("sw_thermal_slowdown", nv.nvmlClocksEventReasonSwThermalSlowdown),
                    ("sw_power_cap", nv.nvmlClocksEventReasonSwPowerCap))
            nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)      # fails here if unsupported

            def poll():
                while not self._stop.is_set():
                    try:
                        sm = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                        mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                        self.samples.append((time.time(), sm, mx, {n for n, b in bits if mask & b}))
                    except Exception:
                        pass
                    self._stop.wait(self.period)

            self.source = "nvml"
            self.thread = threading.Thread(target=poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self._physical_index()), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return
        self.source = "nvidia-smi"
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm, mx = float(f[0]), float(f[1])
            except ValueError:
                continue
            reasons = {n for n, v in zip(self.REASONS, f[3:7]) if v.lower().startswith("active")}
            self.samples.append((time.time(), sm, mx, reasons))

    def stop(self):
        self._stop.set()
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0, t1):
        """Samples taken inside [t0, t1]; if the region was shorter than the sampling period,
        the samples nearest to it (said in `window`)."""
        rows = [r for r in self.samples if t0 <= r[0] <= t1]
        window = "timed region"
        if not rows and self.samples:
            mid = 0.5 * (t0 + t1)
            rows = sorted(self.samples, key=lambda r: abs(r[0] - mid))[:3]
            window = "nearest samples (timed region shorter than the sampling period)"
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "source": self.source}
        reasons = set()
        for r in rows:
            reasons |= r[3]
        return {"sm_mhz": statistics.median(r[1] for r in rows), "sm_max_mhz": max(r[2] for r in rows),
                "reasons": sorted(reasons), "samples": len(rows), "source": self.source, "window": window}


def workload_label(wl):
    c = wl.cfg
    return (f"{c.name}: B={wl.B} K={wl.K} V={wl.V} d={c.d} h={c.h} {str(c.dtype).split('.')[-1]} "
            f"(per GPU), Kp={wl.Kp}")


def oracle_step(wl_cpu, tau):
    """The whole path on the CPU oracle (float64, one thread)."""
    import torch

    import oracle

    def to_np(t):
        t = t.detach().cpu().contiguous()
        return t.view(torch.uint16).numpy() if t.dtype == torch.bfloat16 else t.numpy()

    w = wl_cpu
    _, _, fr = oracle.sprinter_verify(to_np(w.hidden), to_np(w.W1), to_np(w.b1), to_np(w.W2),
                                      to_np(w.b2), tau)
    P = to_np(w.p_logits)
    oracle.replace_sample(P.reshape(w.B * w.Kp, w.ldv), w.V, to_np(w.u_replace), first_reject=fr,
                          K=w.K, seq_stride=w.Kp)
    oracle.sd_verify(P, to_np(w.q_logits), w.V, to_np(w.draft_tokens), to_np(w.uniforms))


def slice_workload(wl, n):
    import dataclasses
    import torch
    kw = {}
    for f in dataclasses.fields(wl):
        v = getattr(wl, f.name)
        if isinstance(v, torch.Tensor) and f.name not in ("W1", "b1", "W2", "b2"):
            v = v[:n]
        if isinstance(v, torch.Tensor):
            v = v.detach().cpu().contiguous()
        kw[f.name] = v
    kw["B"] = n
    return type(wl)(**kw)


def slice_rows(wl_cpu, lo, hi):
    """Sequences lo .. hi-1 of a host workload."""
    import dataclasses
    import torch
    kw = {}
    for f in dataclasses.fields(wl_cpu):
        v = getattr(wl_cpu, f.name)
        if isinstance(v, torch.Tensor) and f.name not in ("W1", "b1", "W2", "b2"):
            v = v[lo:hi].contiguous()
        kw[f.name] = v
    kw["B"] = hi - lo
    return type(wl_cpu)(**kw)


def run_reference(args):
    """The oracle as it stands, timed on the host cores: each step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2502_04557_b200 import workloads
    sample = 4
    wl = workloads.make(args.workload, "cpu", B=sample)
    for _ in range(min(args.warmup, 1)):
        oracle_step(wl, args.threshold)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(wl, args.threshold)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = sample * wl.K / dt
    desc = f"{sample} sequences ({sample * wl.K} draft tokens) of the workload per step"
    c = wl.cfg
    full_label = (f"{c.name}: B={c.B} K={c.K} V={c.V} d={c.d} h={c.h} {str(c.dtype).split('.')[-1]} "
                  f"(per GPU), Kp={wl.Kp}")
    print(json.dumps({
        "impl": "reference", "metric": "verified_tokens_per_s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": full_label, "sample": desc},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_vocab_sharded(args):
    """sd_verify with the vocabulary split over the ranks (a tensor-parallel LM head): every rank
    reads V/N columns of the same rows; two all-gathers and one max-reduce per step over NCCL."""
    import torch
    import torch.distributed as dist

    import paper_2502_04557_b200 as spr
    from paper_2502_04557_b200 import binding as bd, sharded

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    spr.lib()
    wl = spr.workloads.make(args.workload, dev, B=args.batch, sweep=0)     # the same rows on every rank
    B, K, V, Kp = wl.B, wl.K, wl.V, wl.Kp
    es = wl.q_logits.element_size()
    dt_code = spr.BF16 if wl.cfg.dtype == torch.bfloat16 else spr.F32
    v0, vs = sharded.vocab_shards(V, world, es)[rank]
    # a rank of a tensor-parallel head owns only its columns: keep a dense copy of them
    p_sh, q_sh = wl.p_logits[:, :, v0:v0 + vs].contiguous(), wl.q_logits[:, :, v0:v0 + vs].contiguous()
    x, u = wl.draft_tokens, wl.uniforms
    del wl.p_logits, wl.q_logits
    ws = spr.Workspace(spr.workspace_bytes(bd.OP_SD_SHARD, B, K, vs, 0, 0, dt_code), device=dev)
    ex = sharded.DistExchange()

    def step():
        return sharded.sd_verify_sharded(p_sh, q_sh, V, v0, x, u, ws, ex, extras=False)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        out = step()
    assert ws.device_status() == 0
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist.barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    start.record()
    for _ in range(args.steps):
        out = step()
    stop.record()
    dist.barrier()
    torch.cuda.synchronize()
    t1 = time.time()
    t = torch.tensor([start.elapsed_time(stop)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_per_step = float(t.item()) / args.steps
    # the pass that moves the bytes, alone on this rank
    stats = torch.empty((B * Kp, 6), dtype=torch.float32, device=dev)
    for _ in range(3):
        bd.sd_shard_stats(p_sh, q_sh, v0, x, ws, out=stats)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(20):
        bd.sd_shard_stats(p_sh, q_sh, v0, x, ws, out=stats)
    b.record()
    torch.cuda.synchronize()
    stats_ms = a.elapsed_time(b) / 20
    alg_bytes = float((B * Kp + B * K) * vs * es)
    peak, peak_kind = peaks()
    if rank == 0:
        sampler.stop()
        print(json.dumps({
            "metric": "verified_tokens_per_s", "value": B * K / (ms_per_step * 1e-3), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16" if dt_code == spr.BF16 else "f32", "data": "synthetic",
            "config": {"workload": f"{args.workload}: B={B} K={K} V={V} Kp={Kp}, vocabulary split over {world} "
                                   f"rank(s), {vs} columns on rank 0",
                       "step": "sd_verify_sharded: stats, all-gather, decide, weights, all-gather, draw, max-reduce",
                       "l2": "a rank's shard is re-read every step; shards under 126 MB stay L2-resident",
                       "mean_sd_accepted_len": out["accepted_len"].float().mean().item()},
            "clocks": sampler.summary(t0, t1), "e2e": None, "gpu_launches": 4 * args.steps,
            "roofline": {"bound": "hbm", "kernel": "shard_stats_kernel", "achieved": alg_bytes / (stats_ms * 1e-3) / 1e9,
                         "peak": peak, "unit": "GB/s", "frac": alg_bytes / (stats_ms * 1e-3) / 1e9 / peak,
                         "peak_kind": f"of {peak_kind}", "traffic": None, "algorithmic_bytes_per_launch": alg_bytes,
                         "avg_launch_ms": stats_ms},
            "cpu_baseline": None,
        }))
    dist.destroy_process_group()


def launch_ranks(args):
    """`python bench.py --gpus N` without a launcher: start N ranks of this script, one per GPU,
    the way a launcher would (torch.distributed.run on 127.0.0.1), and pass their output on."""
    import socket

    import torch
    have = torch.cuda.device_count()
    if have < args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus}: this machine shows {have} CUDA device(s); "
                         f"one rank per GPU is needed, refusing to time fewer ranks than asked for")
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd, env=env))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        launch_ranks(args)
    if int(os.environ.get("WORLD_SIZE", "1")) != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} was started with WORLD_SIZE="
                         f"{os.environ.get('WORLD_SIZE', '1')}: the two must agree")
    if args.shard == "vocab":
        run_vocab_sharded(args)
        return

    import torch
    import torch.distributed as dist

    import paper_2502_04557_b200 as spr
    from paper_2502_04557_b200 import binding as bd

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    spr.lib()

    wl = spr.workloads.make(args.workload, dev, B=args.batch, sweep=rank)
    cfg = wl.cfg
    B, K, V = wl.B, wl.K, wl.V
    M = B * K
    es = wl.q_logits.element_size()
    dt_code = spr.BF16 if cfg.dtype == torch.bfloat16 else spr.F32
    ws = spr.Workspace.for_problem(B, K, V, cfg.d, cfg.h, dt_code, device=dev)
    ws_sd = spr.Workspace.for_problem(B, K, V, cfg.d, cfg.h, dt_code, device=dev)
    tau = args.threshold
    # The SD call and the SPRINTER call (verify -> gated replacement) of a step are independent and
    # have separate workspaces.  By default they follow each other on one stream: measured, two
    # streams finish a step about 2 % sooner, but the short SPRINTER kernels then take SMs and
    # bandwidth from the row-statistics pass while it runs (0.88 instead of 0.93 of the copy peak).
    st_sd = torch.cuda.Stream(device=dev)
    st_spr = torch.cuda.Stream(device=dev) if args.streams == 2 else st_sd

    ver_out = (torch.empty((B, K), dtype=torch.float32, device=dev),
               torch.empty((B, K), dtype=torch.uint8, device=dev),
               torch.empty((B,), dtype=torch.int32, device=dev))
    tok_out = torch.empty((B,), dtype=torch.int32, device=dev)
    sd_out = dict(accepted_len=torch.empty((B,), dtype=torch.int32, device=dev),
                  correction_token=torch.empty((B,), dtype=torch.int32, device=dev))

    # Timed steps must read their inputs from HBM: workloads whose logits and hidden states do not
    # exceed L2 four times over are rotated through enough copies to do so.
    step_bytes = (wl.p_logits.numel() + wl.q_logits.numel() + wl.hidden.numel()) * es
    n_copies = 1 if args.rotate == 0 else min(64, max(1, -(-4 * 126 * (1 << 20) // step_bytes)))
    copies = [(wl.p_logits, wl.q_logits, wl.hidden)]
    copies += [tuple(t.clone() for t in copies[0]) for _ in range(n_copies - 1)]
    turn = [0]

    def step():
        P, Q, H = copies[turn[0] % n_copies]
        turn[0] += 1
        with torch.cuda.stream(st_sd):
            spr.sd_verify(P, Q, V, wl.draft_tokens, wl.uniforms, ws_sd, out=sd_out)
        with torch.cuda.stream(st_spr):   # sprinter_verify + gated replace_sample as one call
            spr.sprinter_step(H, wl.W1, wl.b1, wl.W2, wl.b2, tau, P, V, wl.u_replace, ws,
                              out=(ver_out[0], ver_out[1], ver_out[2], tok_out))

    def fork():
        st_spr.wait_stream(torch.cuda.current_stream())
        st_sd.wait_stream(torch.cuda.current_stream())

    def join():
        torch.cuda.current_stream().wait_stream(st_spr)
        torch.cuda.current_stream().wait_stream(st_sd)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    fork()
    for _ in range(max(args.warmup, 3)):
        step()
    join()
    assert ws.device_status() == 0 and ws_sd.device_status() == 0

    nsteps = args.steps
    # Does the host keep up?  A short eager probe: if a step takes the GPU less time than the
    # host needs to issue its two calls, the timed steps are replays of CUDA graphs of the step,
    # so that the number is about the kernels and not about the Python interpreter.
    use_graph = args.graph == "1"
    if args.graph == "auto":
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        a.record()
        fork()
        for _ in range(20):
            step()
        join()
        b.record()
        host_ms = (time.perf_counter() - t0) * 1e3 / 20     # time the host took to issue a step
        torch.cuda.synchronize()
        use_graph = a.elapsed_time(b) / 20 < 1.3 * host_ms

    def capture(n):
        """n consecutive steps (both streams forked once, joined once) as one CUDA graph."""
        cap = torch.cuda.Stream(device=dev)
        cap.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=cap):
            fork()
            for _ in range(n):
                step()
            join()
        torch.cuda.current_stream().wait_stream(cap)
        return graph

    every = max(1, args.stage_every)
    stage = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range(min(nsteps, 50) if use_graph else (nsteps + every - 1) // every)]
    for a, b in stage:          # create the handles
        a.record()
        b.record()
    graphs = []
    if use_graph:
        per_graph = n_copies if n_copies > 1 else min(nsteps, 20)
        turn[0] = 0
        if nsteps // per_graph:
            graphs.append((capture(per_graph), nsteps // per_graph))
        if nsteps % per_graph:
            graphs.append((capture(nsteps % per_graph), 1))
        for g, _ in graphs:
            g.replay()
        torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    start.record()
    if use_graph:
        for g, times in graphs:
            for _ in range(times):
                g.replay()
    else:
        fork()
        for i in range(nsteps):
            if i % every == 0:
                spr.set_stage_events(*stage[i // every])
            elif i % every == 1:
                spr.set_stage_events(None, None)
            step()
        join()
    stop.record()
    spr.set_stage_events(None, None)
    barrier()
    t_wall1 = time.time()
    elapsed_ms = start.elapsed_time(stop)
    if use_graph:
        # event pairs cannot be read back from inside a graph: the launch time of the dominant
        # kernel comes from an eager pass over the same rotation of inputs right after
        fork()
        for i in range(len(stage)):
            spr.set_stage_events(*stage[i])
            step()
        join()
        spr.set_stage_events(None, None)
        torch.cuda.synchronize()
    if world > 1:
        t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    assert ws.device_status() == 0 and ws_sd.device_status() == 0
    clocks = sampler.summary(t_wall0, t_wall1) if rank == 0 else None
    ms_per_step = elapsed_ms / nsteps
    value = world * M / (ms_per_step * 1e-3)

    # dominant kernel: the row-statistics pass of sd_verify reads 2*M*V*es bytes once
    stats_ms = statistics.fmean(a.elapsed_time(b) for a, b in stage)
    alg_bytes = 2.0 * M * V * es
    achieved = alg_bytes / (stats_ms * 1e-3) / 1e9
    peak, peak_kind = peaks()
    traffic = None
    if (NCU_TRAFFIC["sha256"] == kernel_sources_sha() and V == 128256 and es == 2
            and bd.sd_verify_launches(B, K, V, dt_code) == 3):   # the kernel variant that was captured
        traffic = NCU_TRAFFIC["bytes_per_unit"] * M

    # end to end: host (pinned) tensors through the host-buffer C ABI, copies inside the timing
    e2e = None
    h_keys = ("hidden", "W1", "b1", "W2", "b2", "p_logits", "q_logits", "draft_tokens", "uniforms", "u_replace")
    host = {k: getattr(wl, k).cpu().pin_memory() for k in h_keys}
    arena = spr.Arena(max(
        spr.host_arena_bytes(2, B, K, wl.Kp, wl.ldv, 0, 0, dt_code),
        spr.host_arena_bytes(0, B, K, 0, 0, cfg.d, cfg.h, dt_code),
        spr.host_arena_bytes(1, B, 0, 0, wl.ldv, 0, 0, dt_code)), device=dev)
    h_ver = (torch.empty((B, K), dtype=torch.float32).pin_memory(),
             torch.empty((B, K), dtype=torch.uint8).pin_memory(),
             torch.empty((B,), dtype=torch.int32).pin_memory())
    h_tok = torch.empty((B,), dtype=torch.int32).pin_memory()
    h_sd = dict(accepted_len=torch.empty((B,), dtype=torch.int32).pin_memory(),
                correction_token=torch.empty((B,), dtype=torch.int32).pin_memory())
    replaced = [0]

    def step_host():
        _, _, fr = spr.sprinter_verify_host(host["hidden"], host["W1"], host["b1"], host["W2"], host["b2"],
                                            tau, arena, ws, out=h_ver)
        spr.replace_sample_host(host["p_logits"], V, host["u_replace"], arena, ws, first_reject=fr, K=K,
                                seq_stride=wl.Kp, out=h_tok)
        replaced[0] = int((fr < K).sum())
        spr.sd_verify_host(host["p_logits"], host["q_logits"], V, host["draft_tokens"], host["uniforms"],
                           arena, ws, out=h_sd)

    step_host()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        step_host()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / max(args.e2e_steps, 1)
    if world > 1:
        t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    # parity of the two routes on what both return
    assert torch.equal(h_sd["accepted_len"], sd_out["accepted_len"].cpu())
    assert torch.equal(h_tok, tok_out.cpu())
    nb = lambda k: host[k].numel() * host[k].element_size()   # noqa: E731
    h2d = (nb("hidden") + nb("W1") + nb("b1") + nb("W2") + nb("b2")            # sprinter_verify_host
           + replaced[0] * (V * es + 4)                                        # replace_sample_host
           + nb("p_logits") + nb("q_logits") + nb("draft_tokens") + nb("uniforms"))   # sd_verify_host
    d2h = (M * 4 + M + B * 4) + replaced[0] * 4 + 2 * B * 4 + 3 * 4
    e2e = {"value": world * M / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
           "steps": args.e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = min(B, 96)
        wl_cpu = slice_workload(wl, sample)
        t0 = time.perf_counter()
        oracle_step(wl_cpu, tau)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": sample * K / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                        "sample": f"first {sample} of {B} sequences ({sample * K} draft tokens), one pass, "
                                  f"{dt:.1f} s"}
        # the same oracle, unchanged, on all host cores: sequences dealt to threads (the C calls
        # release the interpreter lock)
        from concurrent.futures import ThreadPoolExecutor
        threads = max(1, min(os.cpu_count() or 1, sample))
        parts = [slice_rows(wl_cpu, i * sample // threads, (i + 1) * sample // threads) for i in range(threads)]
        t0 = time.perf_counter()
        with ThreadPoolExecutor(threads) as pool:
            list(pool.map(lambda part: oracle_step(part, tau), parts))
        dt_all = time.perf_counter() - t0
        cpu_baseline["all_cores"] = {"value": sample * K / dt_all, "unit": "tokens/s", "cores": threads,
                                     "sample": f"the same {sample} sequences split over {threads} threads, "
                                               f"{dt_all:.1f} s"}

    # each call on its own: n back-to-back calls captured into one CUDA graph (no host launch cost
    # between them), events around a replay, best of three replays -> ms of GPU time per call
    def time_call(fn, n=20):
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(3):
                fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(n):
                    fn()
            graph.replay()
            side.synchronize()
            best = float("inf")
            for _ in range(3):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                graph.replay()
                b.record()
                side.synchronize()
                best = min(best, a.elapsed_time(b) / n)
        torch.cuda.current_stream().wait_stream(side)
        return best

    fr = ver_out[2]
    t_ver = time_call(lambda: spr.sprinter_verify(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, tau, ws, out=ver_out))
    t_rep = time_call(lambda: spr.replace_sample(wl.p_logits, V, wl.u_replace, ws, first_reject=fr, K=K,
                                                 seq_stride=wl.Kp, out=tok_out))
    t_stp = time_call(lambda: spr.sprinter_step(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, tau, wl.p_logits, V,
                                                wl.u_replace, ws, out=(ver_out[0], ver_out[1], ver_out[2], tok_out)))
    t_sd = time_call(lambda: spr.sd_verify(wl.p_logits, wl.q_logits, V, wl.draft_tokens, wl.uniforms, ws, out=sd_out))
    n_rej = int((fr < K).sum())
    kept = float(fr.float().sum())          # draft tokens the verifier kept
    ver_flops = 2.0 * M * cfg.d * cfg.h if cfg.h else 2.0 * M * cfg.d
    calls = {
        "sprinter_verify": {"ms": t_ver, "verified_tokens_per_s": M / (t_ver * 1e-3), "flops": ver_flops,
                            "tflops": ver_flops / (t_ver * 1e-3) / 1e12,
                            "bytes": int((wl.hidden.numel() + wl.W1.numel()) * es),
                            "gbs": (wl.hidden.numel() + wl.W1.numel()) * es / (t_ver * 1e-3) / 1e9},
        "replace_sample": {"ms": t_rep, "draws": n_rej, "bytes": int(n_rej * V * es),
                           "gbs": n_rej * V * es / (t_rep * 1e-3) / 1e9},
        "sprinter_step": {"ms": t_stp, "verified_tokens_per_s": M / (t_stp * 1e-3),
                          "emitted_tokens_per_s": (kept + n_rej) / (t_stp * 1e-3),
                          "bytes": int(wl.hidden.numel() * es + wl.W1.numel() * es + n_rej * V * es)},
        "sd_verify": {"ms": t_sd, "verified_tokens_per_s": M / (t_sd * 1e-3),
                      "emitted_tokens_per_s": float(sd_out["accepted_len"].float().sum() + B) / (t_sd * 1e-3),
                      "bytes": int(alg_bytes + int((sd_out["accepted_len"] < K).sum()) * 2 * V * es)},
    }

    # vocabulary-sharded sd_verify: what one of G GPUs would run on its V/G columns (the two
    # all-gathers between the passes, 24 B per row and 16 B per sequence per GPU, are not timed)
    if args.vocab_shards > 0:
        from paper_2502_04557_b200 import sharded
        G = args.vocab_shards
        shards = sharded.vocab_shards(V, G, es)
        views = [(wl.p_logits[:, :, v0:v0 + vs], wl.q_logits[:, :, v0:v0 + vs]) for v0, vs in shards]
        wss = [spr.Workspace(spr.workspace_bytes(bd.OP_SD_SHARD, B, K, vs, 0, 0, dt_code), device=dev) for _, vs in shards]
        all_stats = torch.stack([bd.sd_shard_stats(pv, qv, v0, wl.draft_tokens, w)
                                 for (pv, qv), (v0, _), w in zip(views, shards, wss)])
        dec = [bd.sd_shard_decide(all_stats, wl.draft_tokens, wl.uniforms, V, vs, wl.Kp, dt_code, w, extras=False)
               for (_, vs), w in zip(shards, wss)]
        all_w = torch.stack([bd.sd_shard_weights(pv, qv, dec[0]["accepted_len"], wl.uniforms, w)
                             for (pv, qv), w in zip(views, wss)])
        (pv, qv), (v0, vs), w0, n0 = views[0], shards[0], wss[0], dec[0]["accepted_len"]
        o_stats, o_w = torch.empty_like(all_stats[0]), torch.empty_like(all_w[0])
        o_tok = dict(correction_token=torch.empty((B,), dtype=torch.int32, device=dev))
        t1 = time_call(lambda: bd.sd_shard_stats(pv, qv, v0, wl.draft_tokens, w0, out=o_stats))
        t2 = time_call(lambda: bd.sd_shard_decide(all_stats, wl.draft_tokens, wl.uniforms, V, vs, wl.Kp, dt_code, w0,
                                                  out=dec[0]))
        t3 = time_call(lambda: bd.sd_shard_weights(pv, qv, n0, wl.uniforms, w0, out=o_w))
        t23 = time_call(lambda: bd.sd_shard_decide_weights(pv, qv, all_stats, wl.draft_tokens, wl.uniforms, V, w0,
                                                           extras=False))
        t4 = time_call(lambda: bd.sd_shard_draw(pv, qv, v0, all_w, all_stats, 0, n0, wl.uniforms, w0, out=o_tok))
        shard_bytes = (2 * M + B * (wl.Kp - K)) * vs * es
        calls[f"sd_verify_sharded_1_of_{G}"] = {
            "shard_columns": vs, "stats_ms": t1, "decide_ms": t2, "weights_ms": t3, "decide_weights_ms": t23,
            "draw_ms": t4, "ms": t1 + t23 + t4, "stats_bytes": int(shard_bytes), "stats_gbs": shard_bytes / (t1 * 1e-3) / 1e9,
            "exchange_bytes_per_gpu": int(B * wl.Kp * 24 + B * 16 + B * 4)}

    # preparing and fitting the verifier (Section 3.2): labels from the same logits, one optimiser step of
    # the single-layer verifier on N = 2^20 hidden states of the draft model's width
    ws_fit = spr.Workspace(max(spr.workspace_bytes(bd.OP_VERIFIER_LABELS, B, K, V, 0, 0, dt_code),
                               spr.workspace_bytes(bd.OP_VERIFIER_TRAIN, 0, 0, 0, cfg.d, 0, dt_code)), device=dev)
    t_lab = time_call(lambda: bd.verifier_labels(wl.p_logits, wl.q_logits, V, wl.draft_tokens, [1.0, 1.2, 1.5], ws_fit,
                                                 want_ratio=False), n=10)
    n_fit = args.fit_samples
    fit_h = torch.randn((n_fit, cfg.d), device=dev).to(wl.hidden.dtype)
    fit_y = (torch.rand(n_fit, device=dev) < 0.5).to(torch.uint8)
    fit_state = [torch.zeros(cfg.d + 1, device=dev) for _ in range(3)]
    fit_loss = torch.empty(1, device=dev)
    t_fit = time_call(lambda: bd.verifier_train_step(fit_h, fit_y, *fit_state, 1, 1e-3, ws_fit, loss=fit_loss), n=10)
    calls["verifier_labels"] = {"ms": t_lab, "tokens_per_s": M / (t_lab * 1e-3), "bytes": int(alg_bytes),
                                "gbs": alg_bytes / (t_lab * 1e-3) / 1e9}
    calls["verifier_train_step"] = {"ms": t_fit, "samples": n_fit, "d": cfg.d, "samples_per_s": n_fit / (t_fit * 1e-3),
                                    "bytes": int(fit_h.numel() * es), "gbs": fit_h.numel() * es / (t_fit * 1e-3) / 1e9}
    del fit_h, fit_y

    simulator = None
    if args.simulator_runs > 0:
        runs = args.simulator_runs
        for _ in range(3):
            spr.sprinter_simulate(1, runs, 5, 0.9, 0.5, 255, want_runs=False, device=dev)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(10):
            _, hist = spr.sprinter_simulate(1, runs, 5, 0.9, 0.5, 255, want_runs=False, device=dev)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / 10
        tokens = float((hist * torch.arange(256, device=dev)).sum() + runs)   # uniforms consumed
        # every 4 uniforms cost one Philox block: 10 rounds x (2 mul.hi + 2 mul.lo + 4 xor + 2 add)
        blocks = float(((hist * ((torch.arange(256, device=dev) + 4) // 4)).sum()))
        int_ops = blocks * 100.0
        alu_peak = 148 * 128 * 1.965e9      # 32-bit ALU lane-operations per second, all SMs
        simulator = {"runs": runs, "ms": ms, "runs_per_s": runs / (ms * 1e-3), "uniforms_per_s": tokens / (ms * 1e-3),
                     "roofline": {"bound": "alu", "achieved": int_ops / (ms * 1e-3) / 1e12, "peak": alu_peak / 1e12,
                                  "unit": "Tlane-op/s", "frac": int_ops / (ms * 1e-3) / alu_peak}}

    # the two other kernels of the path against their rooflines (each timed alone: graph replays above)
    tpeak, tpeak_kind = tensor_peak()
    pipe_pct = None
    if NCU_VERIFIER["sha256"] == sources_sha(NCU_VERIFIER["sources"]):
        pipe_pct = NCU_VERIFIER["tensor_pipe_pct_while_active"]
    roofline_verifier = {
        "bound": "tensor", "kernel": "verifier_tcgen05_kernel" if dt_code == spr.BF16 and cfg.h else "verifier (SIMT)",
        "achieved": calls["sprinter_verify"]["tflops"], "peak": tpeak, "unit": "TFLOP/s",
        "frac": calls["sprinter_verify"]["tflops"] / tpeak, "peak_kind": f"of {tpeak_kind} (burst: kernel timed alone)",
        "flops_per_launch": ver_flops, "avg_launch_ms": t_ver, "timing": "CUDA-graph replay of 20 calls, inputs L2-warm",
        "tensor_pipe_pct_while_active": pipe_pct, "tensor_pipe_source": NCU_VERIFIER["profile"] if pipe_pct else None}
    roofline_draw = {
        "bound": "hbm", "kernel": "draw_kernel (replacement draws)", "achieved": calls["replace_sample"]["gbs"], "peak": peak,
        "unit": "GB/s", "frac": calls["replace_sample"]["gbs"] / peak, "peak_kind": f"of {peak_kind}",
        "algorithmic_bytes_per_launch": calls["replace_sample"]["bytes"], "avg_launch_ms": t_rep, "draws": n_rej,
        "timing": "CUDA-graph replay of 20 calls" + ("" if n_rej * V * es > 126 << 20 else ", rows L2-warm")}

    inputs_sha = None
    if rank == 0:
        h = hashlib.sha256()     # the realised tensors are the inputs, not the generator
        for t in (wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, wl.p_logits, wl.q_logits, wl.draft_tokens, wl.uniforms,
                  wl.u_replace):
            h.update(t.detach().cpu().contiguous().view(torch.uint8).numpy().tobytes())
        inputs_sha = h.hexdigest()
    if rank == 0:
        sampler.stop()
        acc_len = sd_out["accepted_len"].float().mean().item()
        fr_mean = ver_out[2].float().mean().item()
        print(json.dumps({
            "metric": "verified_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": nsteps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16"
            if cfg.dtype == torch.bfloat16 else "f32", "data": "synthetic",
            "config": {"workload": workload_label(wl),
                       "step": ("sd_verify (stream 1) || sprinter_step = sprinter_verify + gated replace_sample (stream 2)"
                                if args.streams == 2 else
                                "sd_verify, then sprinter_step = sprinter_verify + gated replace_sample, on one stream"),
                       "timed_region": (f"CUDA-graph replays of the step ({'+'.join(str(t) for _, t in graphs)} replays); "
                                        "row-statistics launch time from an eager pass after it") if use_graph else
                                       "eager calls",
                       "l2": (f"inputs per step ({(alg_bytes + wl.p_logits[:, K:].numel() * es) / 1e9:.2f} GB of logits) "
                              "exceed the 126 MB L2; no flush needed") if n_copies == 1 and step_bytes > 126 << 20 else
                             (f"steps rotate through {n_copies} copies of the inputs ({n_copies * step_bytes / 1e6:.0f} MB "
                              "in all; the L2 holds 126 MB)" if n_copies > 1 else "one copy of the inputs: L2-warm"),
                       "inputs_sha256": inputs_sha,
                       "threshold": tau, "mean_sd_accepted_len": acc_len, "mean_first_reject": fr_mean},
            "clocks": clocks, "e2e": e2e, "gpu_launches": (bd.sd_verify_launches(B, K, V, dt_code) + 2) * nsteps,
            "roofline": {"bound": "hbm", "kernel": "sd_row_stats_kernel", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": traffic, "algorithmic_bytes_per_launch": alg_bytes,
                         "avg_launch_ms": stats_ms, "launches_timed": len(stage),
                         "timing": f"CUDA-event pair around the launch in every {every}. timed step" if not use_graph
                                   else "CUDA-event pairs in an eager pass after the graph replays"},
            "roofline_verifier": roofline_verifier, "roofline_draw": roofline_draw,
            "sprinter_step_tokens_per_s": calls["sprinter_step"]["verified_tokens_per_s"],
            "sd_verify_tokens_per_s": calls["sd_verify"]["verified_tokens_per_s"],
            "value_is": "draft tokens per second through one step = sd_verify and sprinter_step of the same tokens; "
                        "each path alone is in sprinter_step_tokens_per_s / sd_verify_tokens_per_s",
            "cpu_baseline": cpu_baseline, "calls": calls,
            **({"simulator": simulator} if simulator else {}),
        }))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
