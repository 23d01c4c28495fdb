"""Multi-rank host logic on CPU (gloo, world size 2): sequences are independent, so each rank
verifies its own contiguous shard of the batch with no data-path exchange; gathering the
per-rank results reproduces the unsharded result, and the step time is the max over ranks."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    from helpers import to_np
    from paper_2502_04557_b200 import workloads

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B = 5
    wl = workloads.make("tiny", "cpu", B=B)          # same seed on every rank: same batch
    first, count = workloads.shard_batch(B, rank, world)
    sl = slice(first, first + count)
    ref = oracle.sd_verify(to_np(wl.p_logits[sl]), to_np(wl.q_logits[sl]), wl.V,
                           to_np(wl.draft_tokens[sl]), to_np(wl.uniforms[sl]))
    mine = torch.full((B,), -7, dtype=torch.int32)
    mine[sl] = torch.from_numpy(ref["accepted_len"])
    gathered = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    merged = torch.stack(gathered).max(0).values     # every index is owned by exactly one rank
    t = torch.tensor([10.0 + rank], dtype=torch.float64)   # stand-in for this rank's elapsed ms
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        full = oracle.sd_verify(to_np(wl.p_logits), to_np(wl.q_logits), wl.V, to_np(wl.draft_tokens),
                                to_np(wl.uniforms))
        np.save(os.path.join(out_dir, "ok.npy"),
                np.array([int(np.array_equal(merged.numpy(), full["accepted_len"])),
                          int(t.item() == 10.0 + world - 1)]))
    dist.barrier()
    dist.destroy_process_group()


def test_batch_sharding_world_size_2(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    ok = np.load(tmp_path / "ok.npy")
    assert ok.tolist() == [1, 1]
