"""GPU parity of the tensor-core verifier over its launch shapes (tile sizes, CTAs sharing a
tile along d, finish inside a cluster or through the workspace), each forced through the
test hook of the C ABI and compared with the float64 oracle; and the bounded waits of that
kernel made to run out."""
import numpy as np
import pytest
import torch

import oracle
from helpers import MARGIN, assert_close_rel, to_np

pytestmark = pytest.mark.gpu

TIMEOUT = 5   # SPR_ERR_TIMEOUT


@pytest.fixture(scope="module")
def spr():
    import paper_2502_04557_b200 as s
    s.lib()
    return s


def eq(t, want, what):
    got = t.detach().cpu().numpy()
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{what}: {len(bad)} mismatches, first at {bad[0].tolist()}"


def problem(B, K, d, h, tau=0.5):
    """bf16 MLP verifier inputs with every score at least MARGIN away from tau, and the oracle's outputs."""
    g = torch.Generator().manual_seed(B * 7 + K * 3 + d + h)
    H = torch.randn((B, K, d), generator=g).to(torch.bfloat16)
    W1 = (torch.randn((h, d), generator=g) / d ** 0.5).to(torch.bfloat16)
    b1 = torch.randn(h, generator=g) / d ** 0.5
    W2 = (torch.randn(h, generator=g) / h ** 0.5 * 3).to(torch.bfloat16)
    b2 = torch.tensor([0.1])
    for _ in range(20):
        ref = oracle.sprinter_verify(to_np(H), to_np(W1), to_np(b1), to_np(W2), to_np(b2), tau)
        near = np.argwhere(np.abs(ref[0] - tau) < MARGIN)
        if not len(near):
            break
        for b, k in near:
            H[b, k] = torch.randn(d, generator=g).to(torch.bfloat16)
    return (H.cuda(), W1.cuda(), b1.cuda(), W2.cuda(), b2.cuda(), tau), ref


# (B, K, d, h), then (bm, bn, splits, cluster_n): cluster_n = -1 puts all CTAs of a token tile
# into one cluster (finish out of shared memory), 1 finishes through the workspace
SHAPES = [
    # the sequential configuration's verifier at small batch: 8 CTAs share every tile
    ((5, 1, 4096, 1024), (64, 128, 8, 1)),
    ((5, 1, 4096, 1024), (64, 64, 8, 1)),
    ((64, 1, 4096, 1024), (64, 128, 8, 1)),
    ((64, 1, 4096, 1024), (64, 128, 4, 1)),
    ((64, 1, 4096, 1024), (64, 64, 4, 1)),
    ((70, 1, 4096, 1024), (128, 128, 2, 1)),
    ((1, 1, 4096, 1024), (64, 128, 8, 1)),
    # one slice of hidden units: the CTAs of a tile are its splits of d
    ((40, 8, 256, 96), (128, 128, 4, -1)),
    ((40, 8, 256, 96), (128, 128, 1, -1)),
    ((40, 8, 256, 96), (64, 128, 2, 1)),
    ((40, 8, 256, 96), (64, 64, 2, -1)),
    ((40, 8, 256, 96), (64, 64, 4, -1)),
    # several slices per cluster, with and without a split of d
    ((100, 16, 2048, 512), (128, 128, 1, -1)),
    ((100, 16, 2048, 512), (128, 128, 2, -1)),
    ((100, 16, 2048, 512), (128, 128, 2, 1)),
    ((100, 16, 2048, 512), (64, 64, 1, -1)),
    ((100, 16, 2048, 512), (128, 64, 4, 1)),
    ((100, 16, 2048, 512), (64, 128, 8, 1)),
    # sequences longer than a tile / cut by tile boundaries; ragged d, h and M
    ((20, 33, 64, 16), (64, 64, 1, -1)),
    ((3, 200, 128, 16), (64, 64, 2, -1)),
    ((3, 200, 128, 16), (128, 64, 2, 1)),
    ((130, 3, 136, 20), (64, 64, 2, -1)),
    ((130, 3, 136, 20), (128, 64, 1, 1)),
    ((32, 8, 768, 256), (64, 64, 2, -1)),
    ((32, 8, 768, 256), (128, 128, 4, -1)),
    # bm = 256: two CTAs share a 256 x 128 tile (each stages half of the W1 tile)
    ((100, 16, 2048, 512), (256, 128, 1, -1)),
    ((100, 16, 2048, 512), (256, 128, 1, 1)),
    ((36, 8, 256, 96), (256, 128, 1, -1)),       # three token tiles: the last pair's second tile is empty
    ((130, 3, 136, 20), (256, 128, 1, 1)),
    ((20, 33, 64, 16), (256, 128, 1, -1)),       # sequences cut by tile boundaries
    ((300, 1, 4096, 1024), (256, 128, 1, 1)),    # eight slices: tickets
]


@pytest.mark.parametrize("dims,shape", SHAPES, ids=[f"{d}-{s}".replace(" ", "") for d, s in SHAPES])
def test_verifier_tensor_forced_shape(spr, dims, shape):
    B, K, d, h = dims
    bm, bn, splits, cluster_n = shape
    args, (s_ref, a_ref, fr_ref) = problem(B, K, d, h)
    ws = spr.Workspace(spr.workspace_bytes(0, B, K, 1, d, h, spr.BF16))
    out = spr.binding.sprinter_verify_shaped(*args, ws, bm=bm, bn=bn, splits=splits, cluster_n=cluster_n)
    assert ws.device_status() == 0
    eq(out[1], a_ref, "accept")
    eq(out[2], fr_ref, "first_reject")
    assert_close_rel(out[0], s_ref, 1e-3, "scores")
    # same workspace again: counters were left clean, results are reproducible bit for bit
    out2 = spr.binding.sprinter_verify_shaped(*args, ws, bm=bm, bn=bn, splits=splits, cluster_n=cluster_n)
    assert ws.device_status() == 0
    assert torch.equal(out[0], out2[0]) and torch.equal(out[1], out2[1]) and torch.equal(out[2], out2[2])
    # and the shape the library picks for itself
    out3 = spr.sprinter_verify(*args, ws, path=spr.PATH_TENSOR)
    assert ws.device_status() == 0
    eq(out3[1], a_ref, "accept (library's shape)")
    eq(out3[2], fr_ref, "first_reject (library's shape)")


def test_forced_shape_that_does_not_fit_is_refused(spr):
    args, _ = problem(4, 2, 64, 16)
    ws = spr.Workspace(spr.workspace_bytes(0, 4, 2, 1, 64, 16, spr.BF16))
    # d = 64 is a single block of the k-loop: nothing to split
    for kw in (dict(bm=96), dict(splits=3), dict(splits=2), dict(bm=64, bn=64, splits=16)):
        with pytest.raises(spr.SprinterError) as e:
            spr.binding.sprinter_verify_shaped(*args, ws, **kw)
        assert e.value.status == 2


@pytest.mark.parametrize("dims,shape", [((8, 4, 256, 64), (64, 64, 1, -1)),      # one CTA per tile
                                        ((8, 4, 256, 64), (64, 64, 2, -1)),      # cluster of 2 along d
                                        ((40, 8, 512, 256), (128, 128, 2, -1)),  # cluster 2 x 2
                                        ((40, 8, 512, 256), (64, 64, 4, 1)),     # split of d, tickets
                                        ((40, 8, 512, 256), (128, 64, 1, 1)),    # tickets only
                                        ((70, 1, 512, 256), (64, 64, 4, 1)),     # K = 1: per-token atomic finish
                                        ((70, 1, 512, 256), (64, 128, 1, 1)),
                                        ((40, 8, 512, 256), (256, 128, 1, -1)),  # CTA pairs, finish in the cluster
                                        ((40, 8, 512, 256), (256, 128, 1, 1))],  # CTA pairs, tickets
                         ids=["single", "split2", "cluster2x2", "split4-tickets", "tickets", "k1-split4", "k1",
                              "pairs", "pairs-tickets"])
def test_bounded_wait_runs_out_and_the_workspace_survives(spr, dims, shape):
    """Nothing feeds the kernel's pipeline (test flag): every CTA's first wait expires after a
    few thousand polls, the launch ends by itself, reports SPR_ERR_TIMEOUT and marks its outputs;
    a normal call on the same workspace right after is exact."""
    B, K, d, h = dims
    bm, bn, splits, cluster_n = shape
    args, (s_ref, a_ref, fr_ref) = problem(B, K, d, h)
    ws = spr.Workspace(spr.workspace_bytes(0, B, K, 1, d, h, spr.BF16))
    kw = dict(bm=bm, bn=bn, splits=splits, cluster_n=cluster_n)
    spr.binding.sprinter_verify_shaped(*args, ws, **kw)                      # warm: module load, attributes
    assert ws.device_status() == 0
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    scores, accept, fr = spr.binding.sprinter_verify_shaped(*args, ws, flags=1, spin_limit=4000, **kw)
    b.record()
    assert ws.device_status() == TIMEOUT
    assert ws.device_status() == 0                                            # reading the status clears it
    assert (fr == -1).all() and (accept == 0).all() and (scores == -1).all()
    assert a.elapsed_time(b) < 50.0, "the failing launch must end quickly"
    scores, accept, fr = spr.binding.sprinter_verify_shaped(*args, ws, **kw)
    assert ws.device_status() == 0
    eq(accept, a_ref, "accept")
    eq(fr, fr_ref, "first_reject")
    assert_close_rel(scores, s_ref, 1e-3, "scores")
