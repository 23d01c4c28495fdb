"""Vocabulary-sharded sd_verify against the float64 oracle of the unsharded definition.

One GPU stands in for G ranks: every rank is a host thread with its own stream, workspace
and column slice of the logits, and the collectives are host-side rendezvous (each thread
synchronises its stream, then a barrier).  No kernel waits on another kernel."""
import threading

import numpy as np
import pytest
import torch

import oracle
from helpers import MARGIN, RTOL, assert_close_rel, assert_mass_close, enforce_margins, oracle_sd, to_device, to_np
from test_gpu_parity import _clear_sd, _rand_problem, eq

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def spr():
    import paper_2502_04557_b200 as s
    s.lib()
    return s


class ThreadExchange:
    """all_gather / all_reduce_max between G host threads."""

    def __init__(self, shared, rank):
        self.shared, self.rank, self.world = shared, rank, shared["G"]

    def _meet(self):
        self.shared["barrier"].wait(timeout=120)

    def all_gather(self, t):
        torch.cuda.current_stream().synchronize()
        self.shared["slots"][self.rank] = t
        self._meet()
        out = torch.stack(self.shared["slots"]).contiguous()
        torch.cuda.current_stream().synchronize()
        self._meet()   # nobody overwrites a slot that is still being read
        return out

    def all_reduce_max(self, t):
        t.copy_(self.all_gather(t.clone()).amax(dim=0))
        return t


def run_sharded(spr, p, q, V, x, u, G, shards=None, extras=True, fused=True):
    """p [B,Kp,ldv], q [B,K,ldv], x, u on the GPU; returns the result dict of every rank."""
    from paper_2502_04557_b200 import sharded
    shards = shards or sharded.vocab_shards(V, G, p.element_size())
    B, Kp, _ = p.shape
    K = q.shape[1]
    shared = dict(G=G, barrier=threading.Barrier(G), slots=[None] * G)
    results, errors = [None] * G, []
    torch.cuda.synchronize()

    def rank_main(g):
        try:
            v0, Vs = shards[g]
            with torch.cuda.stream(torch.cuda.Stream()):
                ws = spr.Workspace(spr.workspace_bytes(spr.binding.OP_SD_SHARD, B, K, Vs, 0, 0, spr.binding._dt(p)))
                results[g] = sharded.sd_verify_sharded(p[:, :, v0:v0 + Vs], q[:, :, v0:v0 + Vs], V, v0, x, u, ws,
                                                       ThreadExchange(shared, g), extras=extras, fused=fused)
                results[g]["status"] = ws.device_status()
        except BaseException as e:   # noqa: BLE001 - release the other threads, then re-raise in the test
            errors.append(e)
            shared["barrier"].abort()

    threads = [threading.Thread(target=rank_main, args=(g,)) for g in range(G)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    if errors:
        raise errors[0]
    return results


def check_against(ref, results, dtype, status=0):
    for g, out in enumerate(results):
        assert out["status"] == status, f"rank {g}"
        eq(out["accept"], ref["accept"], f"rank {g} accept")
        eq(out["accepted_len"], ref["accepted_len"], f"rank {g} accepted_len")
        eq(out["correction_token"], ref["correction_token"], f"rank {g} correction_token")
        assert_close_rel(out["p_tok"], ref["p_tok"], RTOL[dtype], "p_tok")
        assert_close_rel(out["q_tok"], ref["q_tok"], RTOL[dtype], "q_tok")
        assert_mass_close(out["residual_mass"], ref["residual_mass"], RTOL[dtype])


@pytest.mark.parametrize("G", [1, 2, 3, 8])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("B,K,V,ldv,Kp", [
    (3, 1, 64, None, 2), (5, 2, 200, None, 3), (4, 3, 1000, None, 3), (2, 33, 129, 131, 34),
    (3, 4, 8191, None, 5), (2, 2, 8193, 8200, 2), (2, 5, 16385, None, 6), (1, 40, 50257, None, 40),
])
def test_sharded_ragged_shapes(spr, dtype, B, K, V, ldv, Kp, G):
    p, q, x, u = _rand_problem(B, K, V, dtype, seed=G + B * 1000 + K * 10 + V, ldv=ldv, Kp=Kp)
    ref = _clear_sd(p, q, V, x, u)
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G)
    check_against(ref, results, dtype)
    if G == 3:      # the decision and the weights as separate launches give the same bits
        split = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G, fused=False)
        for k in ("accept", "accepted_len", "correction_token", "p_tok", "q_tok", "residual_mass"):
            assert torch.equal(split[0][k], results[0][k]), k


@pytest.mark.parametrize("name,B,G", [("gpt2", 6, 4), ("llama2", 8, 2), ("llama3", 4, 8), ("sequential", 16, 8)])
def test_sharded_configs(spr, name, B, G):
    wl_cpu = spr.workloads.make(name, "cpu", B=B, bonus_row=(name != "sequential"))
    enforce_margins(wl_cpu)
    wl = to_device(wl_cpu)
    ref = oracle_sd(wl_cpu)
    results = run_sharded(spr, wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, G)
    check_against(ref, results, wl.q_logits.dtype)
    # and the same decisions as the single-GPU call
    ws = spr.Workspace(spr.workspace_bytes(2, wl.B, wl.K, wl.V, 1, 0, spr.binding._dt(wl.p_logits)))
    one = spr.sd_verify(wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, ws)
    for k in ("accept", "accepted_len", "correction_token"):
        assert torch.equal(one[k], results[0][k]), k


def test_sharded_uneven_and_misaligned_shards(spr):
    B, K, V = 3, 4, 5003
    p, q, x, u = _rand_problem(B, K, V, torch.bfloat16, seed=77)
    shards = [(0, 1), (1, 2048), (2049, 7), (2056, 2947)]   # widths 1 .. thousands, odd offsets
    assert sum(s[1] for s in shards) == V
    for b in range(B):          # draft tokens on both sides of every boundary
        for k in range(K):
            v0 = shards[(b * K + k) % 4][0]
            x[b, k] = max(0, v0 - (k % 2))
    ref = _clear_sd(p, q, V, x, u)
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), 4, shards=shards)
    check_against(ref, results, torch.bfloat16)


def test_sharded_disjoint_supports_and_all_accepted(spr):
    g = torch.Generator().manual_seed(8)
    B, K, V, G = 4, 3, 5000, 4
    ninf = float("-inf")
    u = torch.rand((B, K + 1), generator=g).clamp_(min=1e-3, max=0.999)
    # disjoint supports: three of the four p shards carry no mass at all
    p = torch.full((B, K + 1, V), ninf); p[..., :100] = torch.randn((B, K + 1, 100), generator=g)
    q = torch.full((B, K, V), ninf); q[..., 100:] = torch.randn((B, K, V - 100), generator=g)
    x = torch.randint(100, V, (B, K), generator=g, dtype=torch.int32)
    ref = oracle.sd_verify(to_np(p), to_np(q), V, to_np(x), to_np(u))
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G)
    for out in results:
        assert out["status"] == 0
        assert (out["accept"] == 0).all() and (out["accepted_len"] == 0).all()
        assert torch.allclose(out["residual_mass"], torch.ones(B, device="cuda"), rtol=1e-5)
        for b in range(B):
            m, t = oracle.residual_draw_margin(to_np(p)[b, 0], to_np(q)[b, 0], float(u[b, K]))
            if m > 1e-5:
                assert int(out["correction_token"][b]) == t == ref["correction_token"][b]
    # p == q: everything accepted, bonus token from p at position K
    q = (torch.randn((B, K, V), generator=g) * 2).to(torch.bfloat16)
    p = torch.cat([q, q[:, :1]], 1).contiguous()
    x = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    ref = oracle.sd_verify(to_np(p), to_np(q), V, to_np(x), to_np(u))
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G)
    for out in results:
        assert (out["accept"] == 1).all() and (out["accepted_len"] == K).all()
        assert (out["residual_mass"] == 0).all()
        for b in range(B):
            m, t = oracle.softmax_draw_margin(to_np(p)[b, K], float(u[b, K]))
            if m > 1e-5:
                assert int(out["correction_token"][b]) == t == ref["correction_token"][b]
    # no bonus row: nothing to draw
    results = run_sharded(spr, p[:, :K].contiguous().cuda(), q.cuda(), V, x.cuda(), u.cuda(), G)
    for out in results:
        assert (out["accepted_len"] == K).all() and (out["correction_token"] == -1).all()


def test_sharded_bad_token_and_empty_batch(spr):
    B, K, V, G = 3, 4, 3000, 3
    p, q, x, u = _rand_problem(B, K, V, torch.float32, seed=5)
    x[1, 2] = V   # outside the whole vocabulary
    ref = _clear_sd(p, q, V, x.clamp(max=V - 1), u)
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G)
    for out in results:
        assert out["status"] == 6   # SPR_ERR_BAD_TOKEN
        assert int(out["accepted_len"][1]) == -1 and int(out["correction_token"][1]) == -1
        assert (out["accept"][1] == 0).all()
        for b in (0, 2):
            assert int(out["accepted_len"][b]) == ref["accepted_len"][b]
            assert int(out["correction_token"][b]) == ref["correction_token"][b]
    # empty batch: every pass returns without touching a pointer
    e = torch.empty
    ws = spr.Workspace(256)
    st = spr.binding.sd_shard_stats(e((0, K + 1, 8), device="cuda"), e((0, K, 8), device="cuda"), 0,
                                    e((0, K), dtype=torch.int32, device="cuda"), ws)
    assert st.shape == (0, 6)


@pytest.mark.parametrize("rows", ["uniform", "random"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_residual_of_vanishing_mass(spr, dtype, rows):
    """p equals q except for a slightly lower logit at the draft token, which has probability of
    order 1/V: the token is rejected (ratio 0.998 against u = 0.9995) and Eq. 1's residual is
    q_i * (Z_q/Z_p - 1) on every other token, with a total mass of a few 1e-8 - far below what a
    difference of two float32 probabilities resolves.  With uniform rows the row sums are exact
    and the ratio form of the weights recovers the residual itself; with random rows the
    normalisers differ by less than their own rounding, and the kernels then either still see
    a positive ratio (weights proportional to q) or none (the guard for an undefined Eq. 1:
    draw from p).  All of these are the same distribution to 1e-8, so the token must be the
    oracle's in every case, on the single-GPU call and on the sharded one."""
    B, K, V, G = 3, 2, 50257, 4
    g = torch.Generator().manual_seed(31)
    if rows == "uniform":
        q = torch.zeros((B, K, V), dtype=dtype)
    else:
        q = (torch.randn((B, K, V), generator=g) * 2).to(dtype)
    p = torch.cat([q, q[:, :1]], 1).clone()
    x = torch.tensor([[7, 100], [25000, 3], [V - 1, 0]], dtype=torch.int32)
    u = torch.tensor([[0.9995, 0.5, 0.31], [0.9995, 0.5, 0.77], [0.9995, 0.5, 0.123]], dtype=torch.float32)
    for b in range(B):
        q[b, 0, int(x[b, 0])] = 0.0
        p[b, 0, int(x[b, 0])] = -2e-3
    P, Q = to_np(p), to_np(q)
    floor = 8e-6 if rows == "uniform" else 1e-5      # a uniform row's bins are 2e-5 wide
    for b in range(B):
        for _ in range(200):
            m, t = oracle.residual_draw_margin(P[b, 0], Q[b, 0], float(u[b, K]))
            m2, t2 = oracle.softmax_draw_margin(P[b, 0], float(u[b, K]))
            if m >= floor and (rows == "uniform" or (m2 >= floor and t2 == t)):
                break
            u[b, K] = torch.rand((), generator=g)
        assert m >= floor
    ref = oracle.sd_verify(P, Q, V, to_np(x), to_np(u))
    assert (ref["accepted_len"] == 0).all() and (ref["residual_mass"] < 1e-6).all()
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)))
    one = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G)
    for out in [one] + results:
        eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
        eq(out["correction_token"], ref["correction_token"], "correction_token")
        rm = out["residual_mass"].cpu().numpy()
        assert (np.abs(rm - ref["residual_mass"]) < 1e-6).all()
        if rows == "uniform":            # exact row sums: the mass itself comes out to a few per cent
            assert (np.abs(rm / ref["residual_mass"] - 1.0) < 0.05).all()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_residual_far_below_the_resolution_of_the_probabilities(spr, dtype):
    """p equals q except for a logit lowered by 1/32 at a draft token of probability ~4e-4: the
    token is rejected, and Eq. 1's residual (total mass ~1e-5) is q_i * (Z_q/Z_p - 1) on every
    other token - a relative difference of 1e-5, of which a difference of two float32
    probabilities keeps one or two digits.  The ratio form of the weights keeps the residual
    proportional to q, so both the single-GPU call and the sharded one pick the oracle's token."""
    B, K, V, G = 6, 2, 50257, 4
    g = torch.Generator().manual_seed(4242)
    q = (torch.randn((B, K, V), generator=g) * 2).to(dtype)
    p = torch.cat([q, (torch.randn((B, 1, V), generator=g) * 2).to(dtype)], 1).clone()
    x = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    u = torch.rand((B, K + 1), generator=g)
    for b in range(B):
        q[b, 0, int(x[b, 0])] = 5.0
        p[b, 0, int(x[b, 0])] = 4.96875           # representable in bfloat16
        u[b, 0] = 0.99                            # above the ratio ~0.969: rejected at position 0
    P, Q = to_np(p), to_np(q)
    for b in range(B):
        for _ in range(50):
            m, t = oracle.residual_draw_margin(P[b, 0], Q[b, 0], float(u[b, K]))
            if m >= MARGIN:
                break
            u[b, K] = torch.rand((), generator=g)
        assert m >= MARGIN and t != int(x[b, 0])
    ref = oracle.sd_verify(P, Q, V, to_np(x), to_np(u))
    assert (ref["accepted_len"] == 0).all() and (ref["residual_mass"] < 3e-5).all() and (ref["residual_mass"] > 3e-6).all()
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)))
    one = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G)
    for out in [one] + results:
        eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
        eq(out["correction_token"], ref["correction_token"], "correction_token")
        # the mass itself is a difference of two row normalisers kept in float32: absolute 1e-6
        assert np.abs(out["residual_mass"].cpu().numpy() - ref["residual_mass"]).max() < 1e-6


def test_sharded_llama3_full_size_sampled(spr):
    """The benchmark's workload (B=256, K=16, V=128256) cut into 8 column shards: the oracle on a
    sample of sequences, and agreement with the single-GPU call on everything."""
    wl = spr.workloads.make("llama3", "cuda")
    K, V = wl.K, wl.V
    results = run_sharded(spr, wl.p_logits, wl.q_logits, V, wl.draft_tokens, wl.uniforms, 8)
    for out in results[1:]:                                   # every rank reports the same
        for k in ("accept", "accepted_len", "correction_token", "p_tok", "q_tok", "residual_mass"):
            assert torch.equal(out[k], results[0][k]), k
    out = results[0]
    assert out["status"] == 0
    seqs = [0, 1, 37, 100, 128, 254, 255]
    idx = torch.tensor(seqs, device="cuda")
    P, Q = to_np(wl.p_logits[idx]), to_np(wl.q_logits[idx])
    X, U = to_np(wl.draft_tokens[idx]), to_np(wl.uniforms[idx])
    ref = oracle.sd_verify(P, Q, V, X, U)
    clear = np.abs(U[:, :K].astype(np.float64) - ref["p_tok"] / ref["q_tok"]) >= MARGIN
    assert clear.mean() > 0.99
    assert np.array_equal(out["accept"][idx].cpu().numpy()[clear], ref["accept"][clear])
    assert_close_rel(out["p_tok"][idx], ref["p_tok"], 1e-3, "p_tok")
    assert_close_rel(out["q_tok"][idx], ref["q_tok"], 1e-3, "q_tok")
    n_tok = 0
    for j, b in enumerate(seqs):
        if not clear[j].all():
            continue
        nb = int(ref["accepted_len"][j])
        assert int(out["accepted_len"][b]) == nb
        u = float(U[j, K])
        if nb < K:
            m, t = oracle.residual_draw_margin(P[j, nb, :V], Q[j, nb, :V], u)
            assert abs(float(out["residual_mass"][b]) / ref["residual_mass"][j] - 1.0) <= 1e-3
        else:
            m, t = oracle.softmax_draw_margin(P[j, K, :V], u)
        if m >= 1e-6:
            assert int(out["correction_token"][b]) == t
            n_tok += 1
    assert n_tok >= len(seqs) // 2
    # the single-GPU call on the same tensors: different summation order, same decisions up to
    # the rare tie inside the margin
    ws = spr.Workspace(spr.workspace_bytes(2, wl.B, K, V, 1, 0, spr.BF16))
    one = spr.sd_verify(wl.p_logits, wl.q_logits, V, wl.draft_tokens, wl.uniforms, ws)
    assert (one["accept"] == out["accept"]).float().mean() > 0.999
    assert (one["correction_token"] == out["correction_token"]).float().mean() > 0.98
    assert torch.allclose(one["p_tok"], out["p_tok"], rtol=1e-4, atol=1e-30)
