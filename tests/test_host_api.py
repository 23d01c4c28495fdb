"""CPU-side checks: the C-ABI library loads and exports what include/sprinter.h declares,
rejects bad arguments before touching a device, and the workload generator is seeded."""
import ctypes
import os
import re

import pytest
import torch

import paper_2502_04557_b200 as spr
from paper_2502_04557_b200 import binding, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"^\s*(?:const\s+)?(?:int|size_t|char\s*\*|void)\s*\*?\s*(\w+)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    L = spr.lib()
    names = declared_functions()
    assert {"sprinter_verify", "replace_sample", "sd_verify", "spr_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/ but not exported"
    assert set(binding.EXPORTS) <= set(names)
    assert L.spr_version() >= 100
    # launches per sd_verify call: the finish grid exists only behind several waves of four-step CTAs
    assert L.spr_sd_verify_launches(256, 16, 128256, 1) == 3
    assert L.spr_sd_verify_launches(4, 4, 1000, 1) == 2
    assert L.spr_sd_verify_launches(128, 8, 32000, 1) == 2      # one segment per row: nothing to merge
    assert L.spr_sd_verify_launches(0, 4, 1000, 1) == 0


def test_workspace_bytes():
    wb = spr.workspace_bytes
    assert wb(binding.OP_SD_VERIFY, 256, 16, 128256, 1, 0, spr.BF16) > 0
    assert wb(binding.OP_SD_VERIFY, 256, 0, 128256, 1, 0, spr.BF16) == 0
    assert wb(binding.OP_SD_VERIFY, 256, 16, 128256, 1, 0, 7) == 0
    assert wb(9, 1, 1, 1, 1, 1, 0) == 0
    a = wb(binding.OP_REPLACE_SAMPLE, 10, 0, 1000, 0, 0, spr.F32)
    b = wb(binding.OP_REPLACE_SAMPLE, 1000, 0, 1000, 0, 0, spr.F32)
    assert 0 < a < b and a % 256 == 0
    assert wb(binding.OP_SPRINTER_VERIFY, 32, 8, 0, 768, 256, spr.BF16) > 0
    # K = 1: one 64-bit word per token in the ticket zone, which is a quarter of the workspace
    assert wb(binding.OP_SPRINTER_VERIFY, 4096, 1, 0, 4096, 1024, spr.BF16) >= 256 + 4 * 8 * 4096
    assert wb(binding.OP_SPRINTER_STEP, 4096, 1, 128256, 4096, 1024, spr.BF16) >= 256 + 4 * 8 * 4096


def test_argument_validation_happens_on_the_host():
    L = spr.lib()
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    p = ctypes.c_void_p(addr)           # a non-null, aligned stand-in: never dereferenced
    odd = ctypes.c_void_p(addr + 1)
    # null tensors
    assert L.sd_verify(None, p, 8, p, p, 1, 1, 1, 8, 0, p, p, None, None, None, None, p, 4096, None) == 1
    # ldv < V, Kp not in {K, K+1}, bad dtype
    assert L.sd_verify(p, p, 4, p, p, 1, 1, 1, 8, 0, p, p, None, None, None, None, p, 4096, None) == 1
    assert L.sd_verify(p, p, 8, p, p, 1, 1, 3, 8, 0, p, p, None, None, None, None, p, 4096, None) == 1
    assert L.sd_verify(p, p, 8, p, p, 1, 1, 1, 8, 5, p, p, None, None, None, None, p, 4096, None) == 2
    # misaligned pointer, workspace too small / missing
    assert L.sd_verify(odd, p, 8, p, p, 1, 1, 1, 8, 0, p, p, None, None, None, None, p, 4096, None) == 1
    assert L.sd_verify(p, p, 8, p, p, 1, 1, 1, 8, 0, p, p, None, None, None, None, p, 16, None) == 3
    assert L.sd_verify(p, p, 8, p, p, 1, 1, 1, 8, 0, p, p, None, None, None, None, None, 4096, None) == 3
    assert L.replace_sample(p, 8, 0, 1, None, None, 0, 1, 1, p, 0, p, p, 4096, None) == 1
    assert L.replace_sample(p, 8, 8, 1, None, p, 0, 1, 1, p, 0, p, p, 4096, None) == 1      # gate needs K > 0
    assert L.replace_sample(p, 8, 8, 1, None, None, 0, 1, 1, p, 0, p, p, 8, None) == 3
    assert L.sprinter_verify(p, p, None, None, p, 0.5, 1, 1, 8, 4, 0, 0, None, p, p, p, 4096, None) == 1
    assert L.sprinter_verify(p, p, p, p, p, 0.5, 1, 0, 8, 4, 0, 0, None, p, p, p, 4096, None) == 1
    # empty problems are fine and touch nothing
    assert L.sd_verify(None, None, 8, None, None, 0, 1, 1, 8, 0, None, None, None, None, None, None, None, 0, None) == 0
    assert L.replace_sample(None, 8, 8, 0, None, None, 0, 1, 0, None, 0, None, None, 0, None) == 0
    assert L.sprinter_verify(p, p, p, p, p, 0.5, 1, 1, 8, 4, 0, 9, None, p, p, p, 4096, None) == 2
    assert L.spr_status_string(6).decode().startswith("draft token")


def test_binding_rejects_host_tensors():
    with pytest.raises(ValueError):
        binding._dev(torch.zeros(4), name="x")
    with pytest.raises(TypeError):
        binding._dt(torch.zeros(4, dtype=torch.float16))


def test_binding_checks_row_selectors_before_any_launch():
    """rows / first_reject are read by the kernel as n 32-bit integers: int64 tensors (torch's
    default integer type) and selectors shorter than the number of draws are refused."""
    good = torch.zeros(5, dtype=torch.int32)
    with pytest.raises(TypeError):
        binding._selectors(torch.zeros(5, dtype=torch.int64), None, 5)
    with pytest.raises(TypeError):
        binding._selectors(None, torch.zeros(5, dtype=torch.int64), 5)
    with pytest.raises(ValueError, match="one entry per draw"):
        binding._selectors(torch.zeros(4, dtype=torch.int32), None, 5)
    with pytest.raises(ValueError, match="one entry per draw"):
        binding._selectors(None, torch.zeros(3, dtype=torch.int32), 5)
    with pytest.raises(ValueError, match="CUDA"):      # right type and length, but a host tensor
        binding._selectors(good, None, 5)
    binding._selectors(None, None, 5)
    # both wrappers go through the same check before they touch the library
    import inspect
    for fn in (binding.replace_sample, binding.replace_sample_static):
        assert "_selectors(rows, first_reject, n)" in inspect.getsource(fn)


def test_workloads_are_seeded_and_shaped():
    a = workloads.make("tiny", "cpu")
    b = workloads.make("tiny", "cpu")
    c = workloads.make("tiny", "cpu", sweep=1)
    assert torch.equal(a.q_logits, b.q_logits) and torch.equal(a.uniforms, b.uniforms)
    assert not torch.equal(a.q_logits, c.q_logits)
    assert a.hidden.shape == (1, 4, 256) and a.p_logits.shape == (1, 5, 1000)
    assert a.draft_tokens.dtype == torch.int32 and a.hidden.dtype == torch.float32
    assert float(a.uniforms.min()) >= 0 and float(a.uniforms.max()) < 1
    s = workloads.make("sequential", "cpu", B=2, bonus_row=False)
    assert s.hidden.shape == (2, 1, 4096) and s.W1.shape == (1024, 4096)
    assert s.p_logits.shape == (2, 1, 128256) and s.q_logits.dtype == torch.bfloat16
    g = workloads.make("gpt2", "cpu", B=2, ldv=50264)
    assert g.q_logits.shape == (2, 8, 50264) and float(g.q_logits[0, 0, 50257]) == 60.0
    assert int(g.draft_tokens.max()) < 50257
    # target/draft correlation of the llama3-style law
    cfg = workloads.CONFIGS["llama3"]
    assert abs(cfg.rho ** 2 * cfg.q_std ** 2 + cfg.noise_std ** 2 - 9.0) < 1e-9


def test_shard_batch_partitions():
    for B in (1, 7, 256, 1000):
        for world in (1, 2, 3, 8):
            spans = [workloads.shard_batch(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and sum(n for _, n in spans) == B
            for (f0, n0), (f1, _) in zip(spans, spans[1:]):
                assert f0 + n0 == f1
            assert max(n for _, n in spans) - min(n for _, n in spans) <= 1


def test_argument_validation_of_the_later_entry_points():
    """Shards, labels and the training step: sizes and pointers are checked on the host, before any
    device call (the pointers here are never dereferenced)."""
    L = spr.lib()
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    p = ctypes.c_void_p(addr)
    lam = (ctypes.c_float * 3)(1.0, 1.2, 1.5)
    lamp = ctypes.cast(lam, ctypes.c_void_p)
    # shard statistics: null tensor, negative offset, Kp not in {K, K+1}, workspace too small
    assert L.sd_shard_stats(None, p, 8, 8, 0, p, 1, 1, 1, 0, p, p, 1 << 20, None) == 1
    assert L.sd_shard_stats(p, p, 8, 8, -1, p, 1, 1, 1, 0, p, p, 1 << 20, None) == 1
    assert L.sd_shard_stats(p, p, 8, 8, 0, p, 1, 1, 3, 0, p, p, 1 << 20, None) == 1
    assert L.sd_shard_stats(p, p, 8, 8, 0, p, 1, 1, 1, 0, p, p, 16, None) == 3
    assert L.sd_shard_stats(p, p, 8, 8, 0, p, 0, 1, 1, 0, p, p, 16, None) == 0          # empty batch
    # decision: no shards, too many shards
    assert L.sd_shard_decide(p, 0, p, p, 1, 1, 1, 8, 8, 0, p, None, None, None, p, 1 << 20, None) == 1
    assert L.sd_shard_decide(p, 5000, p, p, 1, 1, 1, 8, 8, 0, p, None, None, None, p, 1 << 20, None) == 1
    # draw: rank outside [0, G)
    assert L.sd_shard_draw(p, p, 8, 8, 0, p, p, 2, 2, p, p, 1, 1, 1, 0, p, None, p, 1 << 20, None) == 1
    # labels: no thresholds, too many, null output
    assert L.verifier_labels(p, p, 8, p, 1, 1, 1, 8, 0, lamp, 0, p, None, p, 1 << 20, None) == 1
    assert L.verifier_labels(p, p, 8, p, 1, 1, 1, 8, 0, lamp, 9, p, None, p, 1 << 20, None) == 1
    assert L.verifier_labels(p, p, 8, p, 1, 1, 1, 8, 0, lamp, 3, None, None, p, 1 << 20, None) == 1
    assert L.verifier_labels(p, p, 8, p, 1, 1, 1, 8, 7, lamp, 3, p, None, p, 1 << 20, None) == 2
    # training step: step 0, beta out of range, width not a whole number of vectors / too wide
    f = ctypes.c_float
    assert L.verifier_train_step(p, p, 4, 8, 1, p, p, p, 0, f(.01), f(.9), f(.999), f(1e-8), None, p, 1 << 20, None) == 1
    assert L.verifier_train_step(p, p, 4, 8, 1, p, p, p, 1, f(.01), f(1.0), f(.999), f(1e-8), None, p, 1 << 20, None) == 1
    assert L.verifier_train_step(p, p, 4, 12, 1, p, p, p, 1, f(.01), f(.9), f(.999), f(1e-8), None, p, 1 << 20, None) == 2
    assert L.verifier_train_step(p, p, 4, 8192, 1, p, p, p, 1, f(.01), f(.9), f(.999), f(1e-8), None, p, 1 << 26, None) == 2
    assert L.verifier_train_step(p, p, 0, 8, 1, p, p, p, 1, f(.01), f(.9), f(.999), f(1e-8), None, p, 1 << 20, None) == 0
    assert L.verifier_train_step(p, p, 4, 8, 1, p, p, p, 1, f(.01), f(.9), f(.999), f(1e-8), None, p, 16, None) == 3
    wb = spr.workspace_bytes
    assert wb(binding.OP_SD_SHARD, 4, 2, 1000, 0, 0, spr.BF16) > 0 and wb(binding.OP_SD_SHARD, 4, 0, 1000, 0, 0, spr.BF16) == 0
    assert wb(binding.OP_VERIFIER_LABELS, 4, 2, 1000, 0, 0, spr.BF16) > 0
    assert wb(binding.OP_VERIFIER_TRAIN, 0, 0, 0, 768, 0, spr.BF16) >= 592 * 770 * 4


def test_argument_validation_of_the_host_buffer_static_and_simulator_calls():
    L = spr.lib()
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    p = ctypes.c_void_p(addr)
    f = ctypes.c_float
    # host-buffer variants: bad dtype, bad sizes, arena too small
    assert L.sd_verify_host(p, p, 8, p, p, 1, 1, 1, 8, 9, p, p, None, None, None, None, p, 1 << 20, p, 1 << 20, None) == 2
    assert L.sd_verify_host(p, p, 4, p, p, 1, 1, 1, 8, 0, p, p, None, None, None, None, p, 1 << 20, p, 1 << 20, None) == 1
    assert L.sd_verify_host(p, p, 8, p, p, 1, 1, 1, 8, 0, p, p, None, None, None, None, p, 16, p, 1 << 20, None) == 3
    assert L.sprinter_verify_host(p, p, p, p, p, f(.5), 1, 0, 8, 4, 0, 0, None, p, p, p, 1 << 20, p, 1 << 20, None) == 1
    assert L.replace_sample_host(p, 8, 0, 1, None, None, 0, 1, 1, p, 0, p, p, 1 << 20, p, 1 << 20, None) == 1
    assert L.spr_host_arena_bytes(2, 4, 2, 3, 1000, 0, 0, 1) > 2 * 4 * 2 * 1000 * 2
    assert L.spr_host_arena_bytes(2, 4, 2, 3, 1000, 0, 0, 5) == 0
    # the call without a workspace: too many draws, too long rows, bad sizes
    assert L.replace_sample_static(p, 8, 8, 2000, None, None, 0, 1, 2000, p, 0, p, None) == 3
    assert L.replace_sample_static(p, 8, 0, 1, None, None, 0, 1, 1, p, 0, p, None) == 1
    assert L.replace_sample_static(None, 8, 8, 0, None, None, 0, 1, 0, None, 0, None, None) == 0
    # simulator: nothing to write to, rates outside [0, 1], negative counts
    u64 = ctypes.c_uint64
    assert L.sprinter_simulate(u64(1), 0, 10, 5, f(.9), f(.5), 16, None, None, None) == 1
    assert L.sprinter_simulate(u64(1), 0, 10, 5, f(1.5), f(.5), 16, p, None, None) == 1
    assert L.sprinter_simulate(u64(1), 0, -1, 5, f(.9), f(.5), 16, p, None, None) == 1
    # the fused step: same checks as its two halves
    assert L.sprinter_step(p, p, p, p, p, f(.5), 1, 1, 8, 4, p, 4, 8, 1, p, 0, 0, None, p, p, p, p, 1 << 20, None) == 1   # ldv < V
    assert L.sprinter_step(p, p, p, p, p, f(.5), 1, 1, 8, 4, p, 8, 8, 1, p, 0, 0, None, p, p, p, p, 16, None) == 3


def test_binding_constants_match_the_header():
    text = open(os.path.join(ROOT, "include", "sprinter.h")).read()
    enum = dict((k, int(v)) for k, v in re.findall(r"\b(SPR_[A-Z0-9_]+)\s*=\s*(\d+)", text))
    assert enum["SPR_F32"] == binding.F32 and enum["SPR_BF16"] == binding.BF16
    for name in ("SPRINTER_VERIFY", "REPLACE_SAMPLE", "SD_VERIFY", "SPRINTER_STEP", "SD_SHARD", "VERIFIER_LABELS",
                 "VERIFIER_TRAIN"):
        assert enum["SPR_OP_" + name] == getattr(binding, "OP_" + name), name
    assert (enum["SPR_VERIFIER_AUTO"], enum["SPR_VERIFIER_SIMT"], enum["SPR_VERIFIER_TENSOR"]) == \
        (binding.PATH_AUTO, binding.PATH_SIMT, binding.PATH_TENSOR)
    L = spr.lib()
    for code in range(8):                      # every status has a text
        assert len(L.spr_status_string(code).decode()) >= 2


def test_bench_refuses_to_time_fewer_ranks_than_asked_for():
    """`bench.py --gpus N` without a launcher starts N ranks itself, one per GPU; on a machine with
    fewer GPUs it must stop with a clear message instead of timing one rank and printing n_gpus 1."""
    import subprocess
    import sys
    have = torch.cuda.device_count()
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(have + 2), "--steps", "1"],
                       capture_output=True, text=True, timeout=300,
                       env={k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")})
    assert r.returncode != 0
    assert "refusing to time fewer ranks" in (r.stderr + r.stdout)
    # a launcher whose world size disagrees with --gpus is refused as well
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode != 0 and "must agree" in (r.stderr + r.stdout)


def test_stream_probes_compile():
    """The two stand-alone measurement programs build for sm_100a (no GPU needed to compile)."""
    from paper_2502_04557_b200 import stream_probes
    for exe in stream_probes.build():
        assert os.path.exists(exe) and os.access(exe, os.X_OK)
