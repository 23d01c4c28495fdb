"""Seeded random shapes, strides and base alignments for the vocabulary calls, each checked
against the float64 oracle: batch and position counts, vocabulary sizes around the vector, step
and segment boundaries, padded rows, and logits that start 0-7 elements past a 16-byte
boundary."""
import numpy as np
import pytest
import torch

import oracle
from helpers import MARGIN, RTOL, assert_close_rel, assert_mass_close, to_np
from oracle import training
from test_gpu_parity import _clear_sd, eq

pytestmark = pytest.mark.gpu

EDGES = [1, 2, 7, 8, 9, 511, 512, 513, 1023, 1024, 1025, 4095, 4096, 4097, 8191, 8192, 8193, 16384, 16385,
         32767, 32768, 32769, 33000]


@pytest.fixture(scope="module")
def spr():
    import paper_2502_04557_b200 as s
    s.lib()
    return s


def draw_case(seed):
    r = np.random.default_rng(seed)
    dtype = [torch.float32, torch.bfloat16][int(r.integers(2))]
    V = int(r.choice(EDGES)) if r.random() < 0.7 else int(r.integers(1, 20000))
    K = int(r.choice([1, 1, 2, 3, 5, 8, 17, 33]))
    B = int(r.integers(1, max(2, 48 // K)))
    Kp = K + int(r.integers(2))
    ldv = V + int(r.choice([0, 0, 1, 3, 8, 13]))
    off_p, off_q = int(r.integers(8)), int(r.integers(8))
    return dtype, B, K, Kp, V, ldv, off_p, off_q


def offset_tensor(t, off):
    """The same values in device memory that starts `off` elements past an aligned address."""
    buf = torch.empty(t.numel() + off + 8, dtype=t.dtype, device="cuda")
    view = buf[off:off + t.numel()].view(t.shape)
    view.copy_(t)
    assert view.is_contiguous() and view.data_ptr() == buf.data_ptr() + off * t.element_size()
    return view


def make_problem(seed, dtype, B, K, Kp, V, ldv):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((B, K, ldv), generator=g) * 2.0
    p = torch.cat([q, torch.randn((B, Kp - K, ldv), generator=g) * 2.0], 1) + 0.7 * torch.randn((B, Kp, ldv), generator=g)
    if ldv > V:                       # padding columns must never be read as logits
        p[..., V:] = 60.0
        q[..., V:] = 60.0
    x = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    u = torch.rand((B, K + 1), generator=g)
    return p.to(dtype).contiguous(), q.to(dtype).contiguous(), x, u


@pytest.mark.parametrize("seed", range(60))
def test_sd_verify_random_case(spr, seed):
    dtype, B, K, Kp, V, ldv, off_p, off_q = draw_case(1000 + seed)
    p, q, x, u = make_problem(seed, dtype, B, K, Kp, V, ldv)
    ref = _clear_sd(p, q, V, x, u)
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)))
    out = spr.sd_verify(offset_tensor(p, off_p), offset_tensor(q, off_q), V, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 0
    eq(out["accept"], ref["accept"], "accept")
    eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
    eq(out["correction_token"], ref["correction_token"], "correction_token")
    assert_close_rel(out["p_tok"], ref["p_tok"], RTOL[dtype], "p_tok")
    assert_close_rel(out["q_tok"], ref["q_tok"], RTOL[dtype], "q_tok")
    assert_mass_close(out["residual_mass"], ref["residual_mass"], RTOL[dtype])


@pytest.mark.parametrize("seed", range(40))
def test_replace_sample_random_case(spr, seed):
    dtype, B, K, Kp, V, ldv, off_p, _ = draw_case(2000 + seed)
    p, _, _, _ = make_problem(seed, dtype, B, K, Kp, V, ldv)
    r = np.random.default_rng(seed)
    R = B * Kp
    n = int(r.integers(1, 2 * R + 1))
    rows = torch.from_numpy(r.integers(0, R, n).astype(np.int32))
    u = torch.from_numpy(r.random(n).astype(np.float32))
    P = to_np(p).reshape(R, ldv)
    want = np.empty(n, np.int64)
    for i in range(n):                               # keep the uniform away from the edges of its bin
        for _ in range(50):
            m, t = oracle.softmax_draw_margin(P[int(rows[i]), :V], float(u[i]))
            if m >= min(MARGIN, 0.1 / V):
                break
            u[i] = float(r.random())
        want[i] = t
    ws = spr.Workspace(spr.workspace_bytes(1, n, 1, V, 1, 0, spr.binding._dt(p)))
    tokens = spr.replace_sample(offset_tensor(p, off_p), V, u.cuda(), ws, rows=rows.cuda())
    assert ws.device_status() == 0
    eq(tokens, want.astype(np.int32), "tokens")


@pytest.mark.parametrize("seed", range(30))
def test_sharded_and_labels_random_case(spr, seed):
    from test_gpu_sharded import check_against, run_sharded
    dtype, B, K, Kp, V, ldv, _, _ = draw_case(3000 + seed)
    p, q, x, u = make_problem(seed, dtype, B, K, Kp, V, ldv)
    ref = _clear_sd(p, q, V, x, u)
    r = np.random.default_rng(seed)
    G = int(r.integers(1, min(V, 6) + 1))
    cuts = sorted(r.choice(np.arange(1, V), size=G - 1, replace=False).tolist()) if G > 1 else []
    bounds = [0] + cuts + [V]
    shards = [(bounds[g], bounds[g + 1] - bounds[g]) for g in range(G)]     # arbitrary, unaligned cuts
    results = run_sharded(spr, p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), G, shards=shards)
    check_against(ref, results, dtype)
    lambdas = [1.0, 1.2, 1.5]
    ws = spr.Workspace(spr.workspace_bytes(spr.binding.OP_VERIFIER_LABELS, B, K, V, 0, 0, spr.binding._dt(p)))
    labels, ratio = spr.binding.verifier_labels(p.cuda(), q.cuda(), V, x.cuda(), lambdas, ws)
    assert ws.device_status() == 0
    want_labels, want_ratio = training.verifier_labels(to_np(p), to_np(q), V, to_np(x), lambdas)
    assert np.all(np.abs(ratio.cpu().double().numpy() / want_ratio - 1.0) <= RTOL[dtype])
    got = labels.cpu().numpy()
    for i, lam in enumerate(lambdas):
        clear = np.abs(want_ratio / lam - 1.0) > 1e-4
        assert np.array_equal(got[i][clear], want_labels[i][clear])


@pytest.mark.parametrize("seed", range(50))
def test_sprinter_verify_random_case(spr, seed):
    """Random verifier shapes through the automatic kernel choice (tensor-core kernel where its
    shape and alignment rules hold, SIMT kernels elsewhere), hidden states and weights at random
    element offsets from an aligned address."""
    r = np.random.default_rng(4000 + seed)
    g = torch.Generator().manual_seed(seed)
    dtype = [torch.float32, torch.bfloat16, torch.bfloat16][int(r.integers(3))]
    d = int(r.choice([8, 37, 64, 100, 128, 136, 256, 768, 1000, 1024, 2048]))
    h = int(r.choice([0, 0, 1, 3, 16, 20, 64, 96, 128, 256]))
    K = int(r.choice([1, 2, 4, 8, 16, 33]))
    B = int(r.integers(1, max(2, 300 // K)))
    tau = float(r.choice([0.5, 0.5, 0.3, 0.7]))
    H = torch.randn((B, K, d), generator=g).to(dtype)
    if h:
        W1 = (torch.randn((h, d), generator=g) / d ** 0.5).to(dtype)
        b1 = torch.randn(h, generator=g) / d ** 0.5
        W2 = (torch.randn(h, generator=g) / h ** 0.5 * 3).to(dtype)
    else:
        W1 = (torch.randn(d, generator=g) / d ** 0.5 * 2).to(dtype)
        b1 = W2 = None
    b2 = torch.tensor([float(r.normal() * 0.2)])
    npo = lambda t: None if t is None else to_np(t)   # noqa: E731
    for _ in range(20):
        s_ref, a_ref, fr_ref = oracle.sprinter_verify(to_np(H), to_np(W1), npo(b1), npo(W2), to_np(b2), tau)
        near = np.argwhere(np.abs(s_ref - float(np.float32(tau))) < MARGIN)
        if not len(near):
            break
        for b, k in near:
            H[b, k] = torch.randn(d, generator=g).to(dtype)
    aligned = r.random() < 0.5            # half of the cases keep 16-byte alignment (tensor-core path eligible)
    off = (lambda: 0) if aligned else (lambda: int(r.integers(8)))
    ws = spr.Workspace(spr.workspace_bytes(0, B, K, 1, d, h, spr.binding._dt(H)))
    cu = lambda t: None if t is None else t.cuda()   # noqa: E731
    scores, accept, fr = spr.sprinter_verify(offset_tensor(H, off()), offset_tensor(W1, off()), cu(b1),
                                             None if W2 is None else offset_tensor(W2, off()), cu(b2), tau, ws)
    assert ws.device_status() == 0
    eq(accept, a_ref, "accept")
    eq(fr, fr_ref, "first_reject")
    assert_close_rel(scores, s_ref, RTOL[dtype], "scores")


def test_many_short_rows(spr):
    """Row counts far above the CTA slots of the GPU (and a grid of 10^5 CTAs): short rows, so the
    oracle still finishes in seconds."""
    B, K, V = 50000, 2, 40
    g = torch.Generator().manual_seed(77)
    q = torch.randn((B, K, V), generator=g) * 2.0
    p = torch.cat([q, torch.randn((B, 1, V), generator=g) * 2.0], 1) + 0.7 * torch.randn((B, K + 1, V), generator=g)
    x = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    u = torch.rand((B, K + 1), generator=g)
    ref = oracle.sd_verify(to_np(p), to_np(q), V, to_np(x), to_np(u))
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.F32))
    out = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 0
    ratio = ref["p_tok"] / ref["q_tok"]
    clear = np.abs(u[:, :K].numpy().astype(np.float64) - ratio) >= MARGIN
    assert clear.mean() > 0.999
    got = out["accept"].cpu().numpy()
    assert np.array_equal(got[clear], ref["accept"][clear])
    seq_clear = clear.all(axis=1)
    assert np.array_equal(out["accepted_len"].cpu().numpy()[seq_clear], ref["accepted_len"][seq_clear])
    tok = out["correction_token"].cpu().numpy()
    agree = (tok == ref["correction_token"])[seq_clear].mean()       # draws are not redrawn here: ties are rare
    assert agree > 0.999 and ((tok >= 0) & (tok < V)).all()
    assert_close_rel(out["p_tok"], ref["p_tok"], RTOL[torch.float32], "p_tok")
    # as many replacement draws, each from its own row
    rows = torch.arange(B, dtype=torch.int32) * (K + 1)
    ur = torch.rand(B, generator=g)
    ws2 = spr.Workspace(spr.workspace_bytes(1, B, 1, V, 1, 0, spr.F32))
    tokens = spr.replace_sample(p.cuda(), V, ur.cuda(), ws2, rows=rows.cuda()).cpu().numpy()
    want = oracle.replace_sample(to_np(p).reshape(B * (K + 1), V), V, ur.numpy(), rows=rows.numpy())
    assert (tokens == want).mean() > 0.999 and ws2.device_status() == 0
