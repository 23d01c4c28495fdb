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


# ---------------------------------------------------------------- vocabulary shards
def test_vocab_shards_tile_the_vocabulary():
    sys.path.insert(0, ROOT)
    from paper_2502_04557_b200.sharded import vocab_shards
    for V, G, es in [(128256, 8, 2), (50257, 4, 2), (50257, 3, 4), (32000, 2, 2), (17, 2, 2), (64, 8, 2), (5, 1, 4)]:
        shards = vocab_shards(V, G, es)
        assert len(shards) == G and shards[0][0] == 0
        assert all(vs > 0 for _, vs in shards)
        assert all(shards[g][0] + shards[g][1] == shards[g + 1][0] for g in range(G - 1))
        assert shards[-1][0] + shards[-1][1] == V
        assert all((v0 * es) % 16 == 0 for v0, _ in shards)
        assert max(vs for _, vs in shards) - min(vs for _, vs in shards) <= 2 * (16 // es)
    import pytest
    with pytest.raises(ValueError):
        vocab_shards(8, 2, 2)   # one 16-byte unit cannot feed two shards


class _NumpyPasses:
    """float64 numpy stand-ins for the four library passes, written from the record formats in
    include/sprinter.h, so that the exchange protocol of sd_verify_sharded can run under gloo
    on a machine without a GPU."""

    def __init__(self):
        self.rowstats = None

    @staticmethod
    def _f(t):
        return t.double().numpy()

    def stats(self, p_shard, q_shard, v0, draft_tokens, ws, out=None):
        P, Q = self._f(p_shard), self._f(q_shard)
        B, Kp, Vs = P.shape
        K = Q.shape[1]
        rec = np.full((B * Kp, 6), -np.inf)
        rec[:, [1, 3]] = 0.0
        for b in range(B):
            for k in range(Kp):
                r = b * Kp + k
                m = P[b, k].max()
                rec[r, 0], rec[r, 1] = m, np.exp(P[b, k] - m).sum()
                if k < K:
                    m = Q[b, k].max()
                    rec[r, 2], rec[r, 3] = m, np.exp(Q[b, k] - m).sum()
                    x = int(draft_tokens[b, k]) - v0
                    if 0 <= x < Vs:
                        rec[r, 4], rec[r, 5] = P[b, k, x], Q[b, k, x]
        return torch.from_numpy(rec.astype(np.float32))

    def decide(self, all_stats, draft_tokens, uniforms, V, Vs, Kp, dt, ws, extras=True, out=None):
        S = self._f(all_stats)
        B, K = draft_tokens.shape
        M = S[:, :, [0, 2]].max(0)
        lnZ = np.log((S[:, :, [1, 3]] * np.exp(S[:, :, [0, 2]] - M)).sum(0))
        self.rowstats = np.concatenate([M[:, :1], lnZ[:, :1], M[:, 1:], lnZ[:, 1:]], 1)
        lx = S[:, :, 4:6].max(0)
        accept = np.zeros((B, K), np.uint8)
        n = np.full((B,), K, np.int32)
        for b in range(B):
            for k in range(K):
                r = b * Kp + k
                ratio = np.exp((lx[r, 0] - M[r, 0] - lnZ[r, 0]) - (lx[r, 1] - M[r, 1] - lnZ[r, 1]))
                accept[b, k] = float(uniforms[b, k]) <= min(1.0, ratio)
            rej = np.flatnonzero(accept[b] == 0)
            if rej.size:
                n[b] = rej[0]
        return dict(accepted_len=torch.from_numpy(n), accept=torch.from_numpy(accept))

    def _weights_of(self, P, Q, b, nb, K, Kp):
        if nb < K:
            rs = self.rowstats[b * Kp + nb]
            return 0.0, np.maximum(0.0, np.exp(P[b, nb] - rs[0] - rs[1]) - np.exp(Q[b, nb] - rs[2] - rs[3]))
        m = P[b, K].max()
        return m, np.exp(P[b, K] - m)

    def weights(self, p_shard, q_shard, accepted_len, uniforms, ws, out=None):
        P, Q = self._f(p_shard), self._f(q_shard)
        B, Kp, _ = P.shape
        K = Q.shape[1]
        w = np.zeros((B, 2))
        for b in range(B):
            nb = int(accepted_len[b])
            if nb < K or Kp == K + 1:
                m, e = self._weights_of(P, Q, b, nb, K, Kp)
                w[b] = (m, e.sum())
        return torch.from_numpy(w)

    def draw(self, p_shard, q_shard, v0, all_weights, all_stats, rank, accepted_len, uniforms, ws, extras=True,
             out=None):
        P, Q = self._f(p_shard), self._f(q_shard)
        W = all_weights.numpy()
        B, Kp, _ = P.shape
        K = Q.shape[1]
        tok = np.full((B,), -1, np.int32)
        for b in range(B):
            nb = int(accepted_len[b])
            if not (nb < K or Kp == K + 1):
                continue
            ref = W[:, b, 0].max()
            shard_w = W[:, b, 1] * np.exp(W[:, b, 0] - ref)
            target = float(uniforms[b, K]) * shard_w.sum()
            cum = np.cumsum(shard_w)
            owner = int(np.argmax(cum > target))
            if owner != rank:
                continue
            m, e = self._weights_of(P, Q, b, nb, K, Kp)
            inside = (target - (cum[owner] - shard_w[owner])) * np.exp(ref - m)
            tok[b] = v0 + int(np.argmax(np.cumsum(e) > inside))
        return dict(correction_token=torch.from_numpy(tok))


def _rank_main_vocab(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    from helpers import enforce_margins, to_np
    from paper_2502_04557_b200 import binding, sharded, workloads

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ex = sharded.DistExchange()
    assert (ex.rank, ex.world) == (rank, world)
    # layout of the collectives: block g of the gathered tensor is rank g's
    got = ex.all_gather(torch.full((3, 2), float(rank)))
    assert got.shape == (world, 3, 2) and all((got[g] == g).all() for g in range(world))
    assert ex.all_reduce_max(torch.tensor([rank, -1], dtype=torch.int32)).tolist() == [world - 1, -1]

    wl = workloads.make("tiny", "cpu", B=6)          # same seed on every rank: same rows
    enforce_margins(wl)
    passes = _NumpyPasses()
    binding.sd_shard_stats, binding.sd_shard_decide = passes.stats, passes.decide
    binding.sd_shard_weights, binding.sd_shard_draw = passes.weights, passes.draw
    v0, Vs = sharded.vocab_shards(wl.V, world, wl.p_logits.element_size())[rank]
    out = sharded.sd_verify_sharded(wl.p_logits[:, :, v0:v0 + Vs], wl.q_logits[:, :, v0:v0 + Vs], wl.V, v0,
                                    wl.draft_tokens, wl.uniforms, None, ex, fused=False)
    full = oracle.sd_verify(to_np(wl.p_logits), to_np(wl.q_logits), wl.V, to_np(wl.draft_tokens),
                            to_np(wl.uniforms))
    ok = [int(np.array_equal(out[k].numpy(), full[k])) for k in ("accept", "accepted_len", "correction_token")]
    np.save(os.path.join(out_dir, f"vocab{rank}.npy"), np.array(ok))
    dist.barrier()
    dist.destroy_process_group()


def test_vocab_sharding_protocol_world_size_2(tmp_path):
    world = 2
    mp.spawn(_rank_main_vocab, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        assert np.load(tmp_path / f"vocab{rank}.npy").tolist() == [1, 1, 1]
