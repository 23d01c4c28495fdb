"""GPU parity: the CUDA library (through its C ABI) against the float64 oracle, element by
element on the same seeded inputs.  Decisions, indices and token ids must be bit-exact;
scores and probabilities within 1e-3 (bf16 inputs) / 1e-5 (fp32 inputs) relative."""
import numpy as np
import pytest
import torch

import oracle
from helpers import (MARGIN, RTOL, assert_close_rel, assert_mass_close, enforce_margins, enforce_margins_parallel,
                     oracle_sd, oracle_step_parallel, oracle_verify, to_device, to_np)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def spr():
    import paper_2502_04557_b200 as s
    s.lib()
    return s


def eq(t: torch.Tensor, want: np.ndarray, what: str):
    got = t.detach().cpu().numpy()
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{what}: {len(bad)} mismatches, first at {bad[0].tolist()}: " \
                          f"got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}"


def check_sd(spr, wl_cpu, wl, ws):
    out = spr.sd_verify(wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, ws)
    assert ws.device_status() == 0
    ref = oracle_sd(wl_cpu)
    eq(out["accept"], ref["accept"], "sd accept")
    eq(out["accepted_len"], ref["accepted_len"], "sd accepted_len")
    eq(out["correction_token"], ref["correction_token"], "sd correction_token")
    rtol = RTOL[wl.q_logits.dtype]
    assert_close_rel(out["p_tok"], ref["p_tok"], rtol, "p_tok")
    assert_close_rel(out["q_tok"], ref["q_tok"], rtol, "q_tok")
    assert_close_rel(out["residual_mass"], ref["residual_mass"], rtol, "residual_mass")
    return out, ref


def check_sprinter_step(spr, wl_cpu, wl, ws, tau, path=0):
    scores, accept, fr = spr.sprinter_verify(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, tau, ws, path=path)
    tokens = spr.replace_sample(wl.p_logits, wl.V, wl.u_replace, ws, first_reject=fr, K=wl.K,
                                seq_stride=wl.Kp)
    assert ws.device_status() == 0
    s_ref, a_ref, fr_ref = oracle_verify(wl_cpu, tau)
    eq(accept, a_ref, "verifier accept")
    eq(fr, fr_ref, "first_reject")
    assert_close_rel(scores, s_ref, RTOL[wl.hidden.dtype], "scores")
    P = to_np(wl_cpu.p_logits).reshape(wl.B * wl.Kp, wl.ldv)
    t_ref = oracle.replace_sample(P, wl.V, to_np(wl_cpu.u_replace), first_reject=fr_ref, K=wl.K,
                                  seq_stride=wl.Kp)
    eq(tokens, t_ref, "replacement tokens")
    return fr_ref, t_ref


CASES = [
    ("tiny", {}, (0.5,)),
    ("gpt2", {}, (0.5,)),
    ("gpt2", {"ldv": 50264, "bonus_row": False}, (0.5,)),
    ("llama2", {}, (0.3, 0.5, 0.7)),
]


@pytest.mark.parametrize("name,kw,taus", CASES, ids=["tiny", "gpt2", "gpt2-padded-nobonus", "llama2"])
def test_config_parity(spr, name, kw, taus):
    wl_cpu = spr.workloads.make(name, "cpu", **kw)
    enforce_margins(wl_cpu, thresholds=taus)
    wl = to_device(wl_cpu)
    cfg = wl.cfg
    ws = spr.Workspace.for_problem(wl.B, wl.K, wl.V, cfg.d, cfg.h, spr.binding._dt(wl.hidden))
    out, ref = check_sd(spr, wl_cpu, wl, ws)
    # the synthetic pairs are built to give a realistic acceptance rate
    if name != "tiny":
        assert 0.2 < ref["accept"].mean() < 0.98
        assert (ref["accepted_len"] < wl.K).any()
    for tau in taus:
        fr_ref, t_ref = check_sprinter_step(spr, wl_cpu, wl, ws, tau)
    # same workspace, second round: results must be bit-identical (deterministic, self-cleaning)
    out2 = spr.sd_verify(wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, ws)
    for k in out:
        assert torch.equal(out[k], out2[k]), k


@pytest.mark.parametrize("B", [1, 8, 64])
def test_sequential_mode_parity(spr, B):
    wl_cpu = spr.workloads.make("sequential", "cpu", B=B, bonus_row=False)
    if B <= 8:   # the sweep forces at least one rejection at tiny batches
        s, _, _ = oracle_verify(wl_cpu, 0.5)
        if (s >= 0.5).all():
            wl_cpu.b2 -= 4.0
    enforce_margins(wl_cpu)
    wl = to_device(wl_cpu)
    ws = spr.Workspace.for_problem(B, 1, wl.V, wl.cfg.d, wl.cfg.h, spr.BF16)
    fr_ref, t_ref = check_sprinter_step(spr, wl_cpu, wl, ws, 0.5)
    assert (fr_ref == 0).any()
    if B == 64:
        assert 0.05 < (fr_ref == 0).mean() < 0.45      # "roughly 20 % rejected"
    # SD on identical inputs (K = 1: also the keep-or-resample rule on a rejected token)
    check_sd(spr, wl_cpu, wl, ws)


def _sampled_rows_check(spr, wl, seqs, tau=0.5):
    """Full-size run on the device, oracle on a sample of sequences copied to the host."""
    cfg = wl.cfg
    ws = spr.Workspace.for_problem(wl.B, wl.K, wl.V, cfg.d, cfg.h, spr.BF16)
    out = spr.sd_verify(wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, ws)
    scores, accept, fr = spr.sprinter_verify(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, tau, ws)
    tokens = spr.replace_sample(wl.p_logits, wl.V, wl.u_replace, ws, first_reject=fr, K=wl.K,
                                seq_stride=wl.Kp)
    assert ws.device_status() == 0
    K, V = wl.K, wl.V
    idx = torch.tensor(seqs, device=wl.hidden.device)
    P = to_np(wl.p_logits[idx])
    Q = to_np(wl.q_logits[idx])
    X = to_np(wl.draft_tokens[idx])
    U = to_np(wl.uniforms[idx])
    ref = oracle.sd_verify(P, Q, V, X, U)
    ratio = ref["p_tok"] / ref["q_tok"]
    got_acc = out["accept"][idx].cpu().numpy()
    clear = np.abs(U[:, :K].astype(np.float64) - ratio) >= MARGIN
    assert clear.mean() > 0.99
    assert np.array_equal(got_acc[clear], ref["accept"][clear])
    assert_close_rel(out["p_tok"][idx], ref["p_tok"], 1e-3, "p_tok")
    assert_close_rel(out["q_tok"][idx], ref["q_tok"], 1e-3, "q_tok")
    s_ref, a_ref, fr_ref = oracle.sprinter_verify(to_np(wl.hidden[idx]), to_np(wl.W1), to_np(wl.b1),
                                                  to_np(wl.W2), to_np(wl.b2), tau)
    s_clear = np.abs(s_ref - tau) >= MARGIN
    assert np.array_equal(accept[idx].cpu().numpy()[s_clear], a_ref[s_clear])
    assert_close_rel(scores[idx], s_ref, 1e-3, "scores")
    n_tok = 0
    for j, b in enumerate(seqs):
        seq_clear = clear[j].all() and s_clear[j].all()
        if not seq_clear:
            continue
        assert int(out["accepted_len"][b]) == int(ref["accepted_len"][j])
        assert int(fr[b]) == int(fr_ref[j])
        nb = int(ref["accepted_len"][j])
        u = float(U[j, K])
        if nb < K:
            m, t = oracle.residual_draw_margin(P[j, nb, :V], Q[j, nb, :V], u)
            assert abs(float(out["residual_mass"][b]) - ref["residual_mass"][j]) <= 1e-3 * ref["residual_mass"][j]
        elif wl.Kp == K + 1:
            m, t = oracle.softmax_draw_margin(P[j, K, :V], u)
        else:
            m, t = 1.0, -1
        if m >= 1e-6:
            assert int(out["correction_token"][b]) == t
            n_tok += 1
        if fr_ref[j] < K:
            m, t = oracle.softmax_draw_margin(P[j, fr_ref[j], :V], float(wl.u_replace[b]))
            if m >= 1e-6:
                assert int(tokens[b]) == t
                n_tok += 1
        else:
            assert int(tokens[b]) == -1
    assert n_tok >= len(seqs) // 2
    return out, fr, tokens


def test_llama3_full_size_sampled(spr):
    wl = spr.workloads.make("llama3", "cuda")
    out, fr, tokens = _sampled_rows_check(spr, wl, [0, 1, 37, 100, 128, 254, 255])
    # properties that hold at any size
    acc = out["accept"].cpu().numpy()
    n = out["accepted_len"].cpu().numpy()
    for b in range(wl.B):
        assert n[b] == next((k for k in range(wl.K) if acc[b, k] == 0), wl.K)
    tok = out["correction_token"].cpu().numpy()
    assert ((tok >= 0) & (tok < wl.V)).all()
    rm = out["residual_mass"].cpu().numpy()
    assert ((rm > 0) & (rm < 1))[n < wl.K].all() and (rm[n == wl.K] == 0).all()
    t = tokens.cpu().numpy()
    frn = fr.cpu().numpy()
    assert ((t >= 0) == (frn < wl.K)).all() and (t < wl.V).all()
    # the launch configuration the benchmark times: sd_verify on one stream, the fused
    # sprinter_step on another, separate workspaces; must give the same bits
    cfg = wl.cfg
    ws1 = spr.Workspace.for_problem(wl.B, wl.K, wl.V, cfg.d, cfg.h, spr.BF16)
    ws2 = spr.Workspace.for_problem(wl.B, wl.K, wl.V, cfg.d, cfg.h, spr.BF16)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(2):
        with torch.cuda.stream(s1):
            out2 = spr.sd_verify(wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, ws1)
        with torch.cuda.stream(s2):
            _, acc2, fr2, tok2 = spr.sprinter_step(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, 0.5, wl.p_logits,
                                                   wl.V, wl.u_replace, ws2)
    torch.cuda.synchronize()
    for k in out:
        assert torch.equal(out[k], out2[k]), k
    assert torch.equal(fr, fr2) and torch.equal(tokens, tok2)


def test_sequential_1024_sampled(spr):
    wl = spr.workloads.make("sequential", "cuda", B=1024, bonus_row=False)
    out, fr, tokens = _sampled_rows_check(spr, wl, list(range(0, 1024, 64)) + [1023])
    rej = (fr.cpu().numpy() == 0).mean()
    assert 0.1 < rej < 0.3


FULL_SIZE = [("llama3", 256, True), ("sequential", 256, True), ("sequential", 1024, False)]


@pytest.mark.parametrize("name,B,bonus", FULL_SIZE, ids=["llama3", "sequential-256", "sequential-1024"])
def test_full_size_parity_every_sequence(spr, name, B, bonus):
    """The configurations the throughput is quoted on, at full size: inputs drawn on the device,
    cleared of ties on the host with the oracle (all host cores), then EVERY accept bit, accepted
    length, first-rejection index, correction token and replacement token compared with the
    oracle, in the launch configuration the benchmark times (sd_verify on one stream, the fused
    sprinter_step on another, separate workspaces)."""
    tau = 0.5
    wl = spr.workloads.make(name, "cuda", B=B, bonus_row=bonus)
    wl_cpu = to_device(wl, "cpu")
    redraws = enforce_margins_parallel(wl_cpu, thresholds=(tau,))
    for k in ("hidden", "uniforms", "u_replace"):     # what the redraws may have touched
        getattr(wl, k).copy_(getattr(wl_cpu, k))
    # accept tests and scores are redrawn rarely (about 2e-4 per decision); draw uniforms often,
    # since a token whose bin is narrower than two margins can never be selected
    print(f"{name} B={B}: {redraws} redraws for {wl.B * wl.K} tokens, {2 * wl.B} draws")
    assert redraws < 20 * wl.B
    cfg = wl.cfg
    ws1 = spr.Workspace.for_problem(wl.B, wl.K, wl.V, cfg.d, cfg.h, spr.BF16)
    ws2 = spr.Workspace.for_problem(wl.B, wl.K, wl.V, cfg.d, cfg.h, spr.BF16)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s1):
        out = spr.sd_verify(wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, wl.uniforms, ws1)
    with torch.cuda.stream(s2):
        scores, accept, fr, tokens = spr.sprinter_step(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, tau,
                                                       wl.p_logits, wl.V, wl.u_replace, ws2)
    torch.cuda.synchronize()
    assert ws1.device_status() == 0 and ws2.device_status() == 0
    ref, s_ref, a_ref, fr_ref, t_ref = oracle_step_parallel(wl_cpu, tau)
    eq(out["accept"], ref["accept"], "sd accept")
    eq(out["accepted_len"], ref["accepted_len"], "sd accepted_len")
    eq(out["correction_token"], ref["correction_token"], "sd correction_token")
    assert_close_rel(out["p_tok"], ref["p_tok"], 1e-3, "p_tok")
    assert_close_rel(out["q_tok"], ref["q_tok"], 1e-3, "q_tok")
    assert_close_rel(out["residual_mass"], ref["residual_mass"], 1e-3, "residual_mass")
    eq(accept, a_ref, "verifier accept")
    eq(fr, fr_ref, "first_reject")
    eq(tokens, t_ref, "replacement tokens")
    assert_close_rel(scores, s_ref, 1e-3, "scores")
    # the separate calls give the same bits as the fused one
    s3, a3, fr3 = spr.sprinter_verify(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, tau, ws2)
    t3 = spr.replace_sample(wl.p_logits, wl.V, wl.u_replace, ws2, first_reject=fr3, K=wl.K, seq_stride=wl.Kp)
    assert torch.equal(a3, accept) and torch.equal(fr3, fr) and torch.equal(t3, tokens)
    if name == "sequential":
        assert 0.1 < (fr_ref == 0).mean() < 0.3       # "roughly 20 % rejected"
    else:
        assert (ref["accepted_len"] < wl.K).mean() > 0.9 and (fr_ref < wl.K).any()


# ---------------------------------------------------------------------------- edge cases


def _rand_problem(B, K, V, dtype, seed, ldv=None, Kp=None, scale=2.0):
    g = torch.Generator().manual_seed(seed)
    ldv = ldv or V
    Kp = Kp or K + 1
    q = torch.randn((B, K, ldv), generator=g) * scale
    p = torch.cat([q, torch.randn((B, Kp - K, ldv), generator=g) * scale], 1) + 0.7 * torch.randn((B, Kp, ldv), generator=g)
    q, p = q.to(dtype), p.to(dtype)
    x = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    u = torch.rand((B, K + 1), generator=g)
    return p.contiguous(), q.contiguous(), x, u


def _clear_sd(p, q, V, x, u):
    """Redraw uniforms near a boundary (small ad-hoc problems)."""
    g = torch.Generator().manual_seed(99)
    B, K = x.shape
    for _ in range(100):
        ref = oracle.sd_verify(to_np(p), to_np(q), V, to_np(x), to_np(u))
        ratio = ref["p_tok"] / ref["q_tok"]
        dirty = False
        near = np.abs(u[:, :K].numpy().astype(np.float64) - ratio) < MARGIN
        for b, k in np.argwhere(near):
            u[b, k] = torch.rand((), generator=g)
            dirty = True
        if dirty:
            continue
        P, Q = to_np(p), to_np(q)
        for b in range(B):
            nb = int(ref["accepted_len"][b])
            if nb < K:
                m, _ = oracle.residual_draw_margin(P[b, nb, :V], Q[b, nb, :V], float(u[b, K]))
            elif p.shape[1] == K + 1:
                m, _ = oracle.softmax_draw_margin(P[b, K, :V], float(u[b, K]))
            else:
                m = 1.0
            if m < min(MARGIN, 0.1 / V):
                u[b, K] = torch.rand((), generator=g)
                dirty = True
        if not dirty:
            return ref
    raise AssertionError("margins not cleared")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("B,K,V,ldv,Kp", [
    (3, 1, 1, None, 2), (5, 2, 7, None, 3), (4, 3, 1000, None, 3), (2, 33, 129, 131, 34),
    (3, 4, 8191, None, 5), (2, 2, 8193, 8200, 2), (2, 5, 16385, None, 6), (1, 40, 50257, None, 40),
])
def test_sd_ragged_shapes(spr, dtype, B, K, V, ldv, Kp):
    p, q, x, u = _rand_problem(B, K, V, dtype, seed=B * 1000 + K * 10 + V, ldv=ldv, Kp=Kp)
    ref = _clear_sd(p, q, V, x, u)
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)))
    out = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 0
    eq(out["accept"], ref["accept"], "accept")
    eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
    eq(out["correction_token"], ref["correction_token"], "correction_token")
    assert_close_rel(out["p_tok"], ref["p_tok"], RTOL[dtype], "p_tok")
    assert_mass_close(out["residual_mass"], ref["residual_mass"], RTOL[dtype])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_replace_sample_rows_gate_and_misaligned_rows(spr, dtype):
    g = torch.Generator().manual_seed(5)
    R, V, ldv = 37, 12345, 12347          # odd row stride: rows start at every 2/4-byte offset
    tl = (torch.randn((R, ldv), generator=g) * 3).to(dtype)
    tl[:, V:] = 90.0
    n = 29
    rows = torch.randint(0, R - 3, (n,), generator=g, dtype=torch.int32)
    fr = torch.randint(0, 4, (n,), generator=g, dtype=torch.int32)      # gate K = 3
    u = torch.rand((n,), generator=g)
    T = to_np(tl)
    for i in range(n):
        if fr[i] < 3:
            for _ in range(50):
                m, _ = oracle.softmax_draw_margin(T[int(rows[i]) + int(fr[i]), :V], float(u[i]))
                if m >= 1e-5:
                    break
                u[i] = torch.rand((), generator=g)
    ws = spr.Workspace(spr.workspace_bytes(1, n, 1, V, 1, 0, spr.binding._dt(tl)))
    got = spr.replace_sample(tl.cuda(), V, u.cuda(), ws, rows=rows.cuda(), first_reject=fr.cuda(), K=3)
    want = oracle.replace_sample(T, V, u.numpy(), rows=rows.numpy(), first_reject=fr.numpy(), K=3)
    assert ws.device_status() == 0
    eq(got, want, "tokens")
    assert (want[fr.numpy() >= 3] == -1).all() and (want[fr.numpy() < 3] >= 0).all()
    # an offset base pointer (tensor view starting 1 element in) must work too
    flat = tl.cuda().flatten()
    view = flat[1:1 + (R - 1) * ldv].view(R - 1, ldv)
    got2 = spr.replace_sample(view, V, u.cuda(), ws, rows=rows.cuda(), first_reject=fr.cuda(), K=3)
    T2 = to_np(tl).reshape(-1)[1:1 + (R - 1) * ldv].reshape(R - 1, ldv)
    for i in range(n):
        if fr[i] < 3:
            m, t = oracle.softmax_draw_margin(T2[int(rows[i]) + int(fr[i]), :V], float(u[i]))
            if m >= 1e-5:
                assert int(got2[i]) == t
        else:
            assert int(got2[i]) == -1


def test_replace_sample_special_rows(spr):
    V = 9000
    ninf = float("-inf")
    rows = torch.full((6, V), ninf)
    rows[0, 4321] = 0.0                       # one-hot: always 4321
    rows[1, 10] = 0.0; rows[1, 8999] = 1.0    # noqa: E702  two tokens far apart (different chunks)
    rows[2] = 1.75                            # uniform: floor(u V)
    rows[3, :] = torch.randn(V) * 2; rows[3, 77] += 50.0    # noqa: E702 dominant logit
    rows[4, 8999] = -3.0                      # only the last token
    rows[5, 0] = 2.0                          # only the first token
    u = torch.tensor([0.999, 0.2, 0.5001, 0.7, 0.0, 0.99999], dtype=torch.float32)
    for dtype in (torch.float32, torch.bfloat16):
        tl = rows.to(dtype).cuda()
        ws = spr.Workspace(spr.workspace_bytes(1, 6, 1, V, 1, 0, spr.binding._dt(tl)))
        got = spr.replace_sample(tl, V, u.cuda(), ws).cpu().numpy()
        want = oracle.replace_sample(to_np(tl), V, u.numpy())
        assert got.tolist() == want.tolist() == [4321, 10, 4500, 77, 8999, 0]
        # u = 0 picks the first token with positive weight
        got0 = spr.replace_sample(tl, V, torch.zeros(6, device="cuda"), ws).cpu().numpy()
        assert got0[0] == 4321 and got0[1] == 10 and got0[2] == 0 and got0[4] == 8999


def test_sd_equal_and_disjoint_distributions(spr):
    g = torch.Generator().manual_seed(8)
    B, K, V = 4, 3, 5000
    q = (torch.randn((B, K, V), generator=g) * 2).to(torch.bfloat16)
    p = torch.cat([q, q[:, :1]], 1).contiguous()
    x = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    u = torch.rand((B, K + 1), generator=g).clamp_(max=0.999)
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.BF16))
    out = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    assert (out["accept"] == 1).all() and (out["accepted_len"] == K).all()
    assert (out["residual_mass"] == 0).all()
    ref = oracle.sd_verify(to_np(p), to_np(q), V, to_np(x), to_np(u))
    for b in range(B):
        m, t = oracle.softmax_draw_margin(to_np(p)[b, K], float(u[b, K]))
        if m > 1e-5:
            assert int(out["correction_token"][b]) == t == ref["correction_token"][b]
    # disjoint supports: everything rejected, correction token from p's support
    ninf = float("-inf")
    p2 = torch.full((B, K, V), ninf); p2[..., :100] = torch.randn((B, K, 100), generator=g)
    q2 = torch.full((B, K, V), ninf); q2[..., 100:] = torch.randn((B, K, V - 100), generator=g)
    x2 = torch.randint(100, V, (B, K), generator=g, dtype=torch.int32)
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.F32))
    out = spr.sd_verify(p2.cuda(), q2.cuda(), V, x2.cuda(), u.clamp(min=1e-3).cuda(), ws)
    assert (out["accept"] == 0).all() and (out["accepted_len"] == 0).all()
    assert ((out["correction_token"] >= 0) & (out["correction_token"] < 100)).all()
    assert torch.allclose(out["residual_mass"], torch.ones(B, device="cuda"), rtol=1e-5)
    assert ws.device_status() == 0


def _small_mass_problem(dtype, V):
    """B single-position sequences (no bonus row) whose target row is the draft row plus noise of
    growing size, each with the draft token the target likes least and a uniform that rejects it."""
    g = torch.Generator().manual_seed(V + (1 if dtype == torch.float32 else 2))
    eps = [1e-4, 1e-3, 0.01, 0.03, 0.05, 0.1, 0.3, 1.0] if dtype == torch.float32 else \
          [0.005, 0.01, 0.02, 0.03, 0.05, 0.1, 0.3, 1.0]
    B, K = 2 * len(eps), 1
    q = torch.randn((B, K, V), generator=g) * 2
    p = q + torch.tensor(eps).repeat(2).view(B, 1, 1) * torch.randn((B, K, V), generator=g)
    p, q = p.to(dtype).contiguous(), q.to(dtype).contiguous()
    x = torch.zeros((B, K), dtype=torch.int32)
    for b in range(B):
        ratio = torch.softmax(p[b, 0].double(), 0) / torch.softmax(q[b, 0].double(), 0)
        x[b, 0] = int(torch.argmin(ratio))
    u = torch.rand((B, K + 1), generator=g)
    u[:, 0] = 0.9999
    return p, q, x, u, _clear_sd(p, q, V, x, u)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("V", [3000, 128256])
def test_sd_correction_draw_over_residual_masses(spr, dtype, V):
    """Correction draws whose residual mass sum max(0, p - q) runs from 1e-4 to 0.5: the kernel forms
    the weights as plain differences where the mass is large and switches to the ratio form below
    0.02; both sides of that switch must give the oracle's token."""
    p, q, x, u, ref = _small_mass_problem(dtype, V)
    masses = ref["residual_mass"][ref["accepted_len"] == 0]
    assert masses.min() < 0.01 and masses.max() > 0.1 and ((masses > 0.02) & (masses < 0.2)).any()
    B, K = x.shape
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)))
    out = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 0
    eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
    eq(out["correction_token"], ref["correction_token"], "correction_token")
    assert_mass_close(out["residual_mass"], ref["residual_mass"], RTOL[dtype])


@pytest.mark.parametrize("dtype,B,K,V,ldv", [(torch.float32, 37, 33, 20000, 20001), (torch.bfloat16, 74, 16, 33000, None),
                                             (torch.bfloat16, 40, 30, 40001, 40003)], ids=["f32", "bf16", "bf16-odd"])
def test_sd_many_waves_of_short_rows(spr, dtype, B, K, V, ldv):
    """More than four waves of statistics CTAs with two segments per row: the launch shape in which
    the merge, the accept test and the scan run in their own grid.  Rows at every alignment
    (odd leading dimension), more than 32 positions per sequence, and - after the clean
    comparison - sequences with an invalid draft token."""
    assert spr.binding.sd_verify_launches(B, K, V, spr.binding._dt(torch.empty(0, dtype=dtype))) == 3
    p, q, x, u = _rand_problem(B, K, V, dtype, seed=B + K + V, ldv=ldv)
    ref = _clear_sd(p, q, V, x, u)
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)))
    pg, qg, ug = p.cuda(), q.cuda(), u.cuda()
    out = spr.sd_verify(pg, qg, V, x.cuda(), ug, ws)
    assert ws.device_status() == 0
    eq(out["accept"], ref["accept"], "accept")
    eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
    eq(out["correction_token"], ref["correction_token"], "correction_token")
    assert_close_rel(out["p_tok"], ref["p_tok"], RTOL[dtype], "p_tok")
    assert_close_rel(out["q_tok"], ref["q_tok"], RTOL[dtype], "q_tok")
    assert_mass_close(out["residual_mass"], ref["residual_mass"], RTOL[dtype])
    bad = {1: (0, -1), 5: (K - 1, V), B - 1: (K // 2, V + 7)}
    for b, (k, tok) in bad.items():
        x[b, k] = tok
    out = spr.sd_verify(pg, qg, V, x.cuda(), ug, ws)
    assert ws.device_status() == 6          # SPR_ERR_BAD_TOKEN
    ref2, rc = oracle.sd_verify(to_np(p), to_np(q), V, to_np(x), to_np(u), return_status=True)
    assert rc == oracle.ERR_TOKEN
    eq(out["accepted_len"], ref2["accepted_len"], "accepted_len with invalid tokens")
    eq(out["correction_token"], ref2["correction_token"], "correction_token with invalid tokens")
    for b in bad:
        assert int(out["accepted_len"][b]) == -1 and int(out["accept"][b].sum()) == 0
    clean = [b for b in range(B) if b not in bad]
    eq(out["accept"][clean], ref["accept"][clean], "accept of the clean sequences")


def test_device_detected_errors(spr):
    p, q, x, u = _rand_problem(3, 2, 300, torch.float32, seed=3)
    x[1, 1] = 300
    ws = spr.Workspace(spr.workspace_bytes(2, 3, 2, 300, 1, 0, spr.F32))
    out = spr.sd_verify(p.cuda(), q.cuda(), 300, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 6          # SPR_ERR_BAD_TOKEN, then cleared
    assert ws.device_status() == 0
    ref, rc = oracle.sd_verify(to_np(p), to_np(q), 300, to_np(x), to_np(u), return_status=True)
    assert rc == oracle.ERR_TOKEN
    assert out["accepted_len"].cpu().tolist()[1] == -1 == ref["accepted_len"][1]
    assert out["correction_token"].cpu().tolist()[1] == -1
    assert out["accept"][1].sum() == 0 and float(out["p_tok"][1, 1]) == -1.0
    for b in (0, 2):
        assert int(out["accepted_len"][b]) == int(ref["accepted_len"][b])
    # row outside the logits tensor
    tl = torch.randn(4, 300).cuda()
    rows = torch.tensor([0, 4, -1, 3], dtype=torch.int32).cuda()
    tok = spr.replace_sample(tl, 300, torch.rand(4).cuda(), ws, rows=rows)
    assert ws.device_status() == 7
    t = tok.cpu().tolist()
    assert t[1] == -1 and t[2] == -1 and t[0] >= 0 and t[3] >= 0
    # a negative first_reject is refused even where row i*seq_stride + first_reject exists
    fr = torch.tensor([1, -1, 0, 2], dtype=torch.int32)
    un = torch.full((4,), 0.37)
    tl8 = torch.randn(8, 300)
    tok = spr.replace_sample(tl8.cuda(), 300, un.cuda(), ws, first_reject=fr.cuda(), K=2, seq_stride=2)
    assert ws.device_status() == 7
    want, rc = oracle.replace_sample(to_np(tl8), 300, un.numpy(), first_reject=fr.numpy(), K=2, seq_stride=2,
                                     return_status=True)
    assert rc == oracle.ERR_ROW and want[1] == -1 and want[3] == -1
    eq(tok, want, "tokens with a negative first_reject")
    # neighbouring sequences may not share rows: seq_stride < K is refused on the host
    with pytest.raises(spr.binding.SprinterError):
        spr.replace_sample(tl8.cuda(), 300, un.cuda(), ws, first_reject=fr.cuda(), K=2, seq_stride=1)
    # the workspace still works afterwards
    x[1, 1] = 0
    out = spr.sd_verify(p.cuda(), q.cuda(), 300, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 0 and int(out["accepted_len"][1]) >= 0


def test_empty_batch_and_all_accepted_gate(spr):
    ws = spr.Workspace(1 << 16)
    p = torch.empty((0, 2, 64), device="cuda")
    q = torch.empty((0, 1, 64), device="cuda")
    out = spr.sd_verify(p, q, 64, torch.empty((0, 1), dtype=torch.int32, device="cuda"),
                        torch.empty((0, 2), device="cuda"), ws)
    assert out["accepted_len"].numel() == 0
    tl = torch.randn(8, 64).cuda()
    fr = torch.full((8,), 1, dtype=torch.int32).cuda()      # K = 1: nothing rejected
    tok = spr.replace_sample(tl, 64, torch.rand(8).cuda(), ws, first_reject=fr, K=1)
    assert (tok == -1).all()
    assert ws.device_status() == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("B,K,d,h", [(1, 4, 256, 64), (3, 5, 37, 11), (2, 1, 8, 3), (7, 33, 100, 20),
                                      (5, 2, 768, 0), (130, 3, 130, 0), (40, 8, 256, 96)])
def test_verifier_simt_shapes(spr, dtype, B, K, d, h):
    g = torch.Generator().manual_seed(B * 100 + K + d + h)
    H = torch.randn((B, K, d), generator=g).to(dtype)
    if h:
        W1 = (torch.randn((h, d), generator=g) / d ** 0.5).to(dtype)
        b1 = torch.randn(h, generator=g) / d ** 0.5
        W2 = (torch.randn(h, generator=g) / h ** 0.5 * 3).to(dtype)
    else:
        W1 = (torch.randn(d, generator=g) / d ** 0.5 * 2).to(dtype)
        b1 = W2 = None
    b2 = torch.tensor([0.1])
    tau = 0.5
    for _ in range(20):
        s_ref, a_ref, fr_ref = oracle.sprinter_verify(to_np(H), to_np(W1), None if b1 is None else to_np(b1),
                                                      None if W2 is None else to_np(W2), to_np(b2), tau)
        near = np.argwhere(np.abs(s_ref - tau) < MARGIN)
        if not len(near):
            break
        for b, k in near:
            H[b, k] = torch.randn(d, generator=g).to(dtype)
    ws = spr.Workspace(spr.workspace_bytes(0, B, K, 1, d, h, spr.binding._dt(H)))
    cu = lambda t: None if t is None else t.cuda()   # noqa: E731
    scores, accept, fr = spr.sprinter_verify(cu(H), cu(W1), cu(b1), cu(W2), cu(b2), tau, ws,
                                             path=spr.PATH_SIMT)
    eq(accept, a_ref, "accept")
    eq(fr, fr_ref, "first_reject")
    assert_close_rel(scores, s_ref, RTOL[dtype], "scores")
    assert len(set(fr_ref.tolist())) > 1 or B < 3


def test_verifier_threshold_equality(spr):
    # all-zero verifier: score is exactly 1/2; Algorithm 2 keeps the token when score >= tau
    H = torch.randn(2, 4, 64).cuda()
    z = torch.zeros
    ws = spr.Workspace(spr.workspace_bytes(0, 2, 4, 1, 64, 8, spr.F32))
    s, a, fr = spr.sprinter_verify(H, z(8, 64).cuda(), z(8).cuda(), z(8).cuda(), z(1).cuda(), 0.5, ws)
    assert (s == 0.5).all() and (a == 1).all() and (fr == 4).all()
    tau = float(np.nextafter(np.float32(0.5), np.float32(1)))
    s, a, fr = spr.sprinter_verify(H, z(8, 64).cuda(), z(8).cuda(), z(8).cuda(), z(1).cuda(), tau, ws)
    assert (a == 0).all() and (fr == 0).all()


@pytest.mark.parametrize("B,K,d,h", [(4, 8, 64, 16), (40, 8, 256, 96), (130, 3, 136, 20), (32, 8, 768, 256),
                                      (64, 1, 4096, 1024), (100, 16, 2048, 512), (20, 33, 64, 16), (3, 200, 64, 16)])
def test_verifier_tensor_core_path(spr, B, K, d, h):
    """tcgen05 kernel forced (PATH_TENSOR) on shapes with ragged M, h and d tails."""
    g = torch.Generator().manual_seed(B * 7 + K + d + h)
    H = torch.randn((B, K, d), generator=g).to(torch.bfloat16)
    W1 = (torch.randn((h, d), generator=g) / d ** 0.5).to(torch.bfloat16)
    b1 = torch.randn(h, generator=g) / d ** 0.5
    W2 = (torch.randn(h, generator=g) / h ** 0.5 * 3).to(torch.bfloat16)
    b2 = torch.tensor([0.1])
    tau = 0.5
    for _ in range(20):
        s_ref, a_ref, fr_ref = oracle.sprinter_verify(to_np(H), to_np(W1), to_np(b1), to_np(W2), to_np(b2), tau)
        near = np.argwhere(np.abs(s_ref - tau) < MARGIN)
        if not len(near):
            break
        for b, k in near:
            H[b, k] = torch.randn(d, generator=g).to(torch.bfloat16)
    ws = spr.Workspace(spr.workspace_bytes(0, B, K, 1, d, h, spr.BF16))
    args = (H.cuda(), W1.cuda(), b1.cuda(), W2.cuda(), b2.cuda(), tau, ws)
    scores, accept, fr = spr.sprinter_verify(*args, path=spr.PATH_TENSOR)
    assert ws.device_status() == 0
    eq(accept, a_ref, "accept")
    eq(fr, fr_ref, "first_reject")
    assert_close_rel(scores, s_ref, 1e-3, "scores")
    # second call on the same workspace, and agreement with the SIMT kernel
    scores2, accept2, fr2 = spr.sprinter_verify(*args, path=spr.PATH_TENSOR)
    assert torch.equal(scores, scores2) and torch.equal(fr, fr2)
    scores3, accept3, _ = spr.sprinter_verify(*args, path=spr.PATH_SIMT)
    assert torch.equal(accept, accept3)
    assert torch.allclose(scores, scores3, rtol=1e-4, atol=1e-6)


def test_verifier_tensor_path_refuses_unsupported_shapes(spr):
    H = torch.randn(2, 4, 64).cuda()          # fp32
    z = torch.zeros
    ws = spr.Workspace(spr.workspace_bytes(0, 2, 4, 1, 64, 8, spr.F32))
    with pytest.raises(spr.SprinterError) as e:
        spr.sprinter_verify(H, z(8, 64).cuda(), z(8).cuda(), z(8).cuda(), z(1).cuda(), 0.5, ws,
                            path=spr.PATH_TENSOR)
    assert e.value.status == 2


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("gpt2", {"B": 6}), ("gpt2", {"B": 5, "ldv": 50264, "bonus_row": False}),
                                     ("sequential", {"B": 16, "bonus_row": False}), ("llama2", {"B": 40})],
                         ids=["tiny", "gpt2", "gpt2-padded", "sequential16", "llama2"])
def test_sprinter_step_fused_call(spr, name, kw):
    """sprinter_step = sprinter_verify + gated replace_sample in one call: same bits as the two
    calls made separately, and as the oracle."""
    wl_cpu = spr.workloads.make(name, "cpu", **kw)
    enforce_margins(wl_cpu)
    wl = to_device(wl_cpu)
    cfg = wl.cfg
    dtc = spr.binding._dt(wl.hidden)
    ws = spr.Workspace.for_problem(wl.B, wl.K, wl.V, cfg.d, cfg.h, dtc)
    scores, accept, fr, tokens = spr.sprinter_step(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, 0.5, wl.p_logits,
                                                   wl.V, wl.u_replace, ws)
    assert ws.device_status() == 0
    s2, a2, fr2 = spr.sprinter_verify(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, 0.5, ws)
    t2 = spr.replace_sample(wl.p_logits, wl.V, wl.u_replace, ws, first_reject=fr2, K=wl.K, seq_stride=wl.Kp)
    assert torch.equal(scores, s2) and torch.equal(accept, a2) and torch.equal(fr, fr2) and torch.equal(tokens, t2)
    s_ref, a_ref, fr_ref = oracle_verify(wl_cpu, 0.5)
    P = to_np(wl_cpu.p_logits).reshape(wl.B * wl.Kp, wl.ldv)
    t_ref = oracle.replace_sample(P, wl.V, to_np(wl_cpu.u_replace), first_reject=fr_ref, K=wl.K, seq_stride=wl.Kp)
    eq(accept, a_ref, "accept")
    eq(fr, fr_ref, "first_reject")
    eq(tokens, t_ref, "tokens")
    # a second fused call on the same workspace gives the same bits
    again = spr.sprinter_step(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, 0.5, wl.p_logits, wl.V, wl.u_replace, ws)
    assert torch.equal(again[3], tokens) and torch.equal(again[2], fr)


@pytest.mark.parametrize("dtype,V", [(torch.bfloat16, 600_011), (torch.float32, 300_007)], ids=["bf16", "f32"])
def test_very_large_vocabulary(spr, dtype, V):
    """More warp steps per row (586) than the last CTA of a draw caches in shared memory (512)."""
    B, K = 3, 2
    p, q, x, u = _rand_problem(B, K, V, dtype, seed=V, Kp=K + 1, scale=3.0)
    # put most of the mass of one row near the end of the vocabulary so draws land in late steps
    p[0, 0, V - 5000:] += 6.0
    ref = _clear_sd(p, q, V, x, u)
    ws = spr.Workspace(max(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)),
                           spr.workspace_bytes(1, B * (K + 1), 1, V, 1, 0, spr.binding._dt(p))))
    out = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 0
    eq(out["accept"], ref["accept"], "accept")
    eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
    eq(out["correction_token"], ref["correction_token"], "correction_token")
    assert_close_rel(out["p_tok"], ref["p_tok"], RTOL[dtype], "p_tok")
    # plain draws from every target row, uniforms spread over [0, 1)
    rows = p.reshape(B * (K + 1), V)
    g = torch.Generator().manual_seed(1)
    uu = torch.rand(B * (K + 1), generator=g)
    uu[0] = 0.97
    R = to_np(rows)
    for i in range(len(uu)):
        for _ in range(50):
            m, _t = oracle.softmax_draw_margin(R[i, :V], float(uu[i]))
            if m >= 1e-6:
                break
            uu[i] = torch.rand((), generator=g)
    got = spr.replace_sample(rows.cuda(), V, uu.cuda(), ws)
    want = oracle.replace_sample(R, V, uu.numpy())
    eq(got, want, "tokens")
    assert want[0] >= V - 5000


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_sd_rows_with_huge_dynamic_range(spr, dtype):
    """Logits that jump by far more than exp() can hold in fp32 between the start and the rest
    of a row (and rows that start with -inf): the row statistics must stay exact."""
    B, K, V = 4, 2, 70_001
    p, q, x, u = _rand_problem(B, K, V, dtype, seed=77, Kp=K, scale=2.0)
    p[0, 0, :40_000] -= 150.0            # everything the first steps see is e^-150 below the rest
    q[0, 1, :20_000] = float("-inf")     # a masked prefix
    p[1, 0, 5_000:] += 120.0
    q[2, 1, 60_000:] += 200.0
    p[3, 1, :] -= 300.0                  # a uniformly tiny row
    x[0, 0] = 50_000
    x[0, 1] = 30_000
    x[2, 1] = 65_000
    ref = _clear_sd(p, q, V, x, u)
    ws = spr.Workspace(spr.workspace_bytes(2, B, K, V, 1, 0, spr.binding._dt(p)))
    out = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    assert ws.device_status() == 0
    eq(out["accept"], ref["accept"], "accept")
    eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
    eq(out["correction_token"], ref["correction_token"], "correction_token")
    ok = ref["p_tok"] > 1e-30
    got_p = out["p_tok"].cpu().double().numpy()
    assert np.all(np.abs(got_p[ok] - ref["p_tok"][ok]) <= RTOL[dtype] * ref["p_tok"][ok])
    ok = ref["q_tok"] > 1e-30
    got_q = out["q_tok"].cpu().double().numpy()
    assert np.all(np.abs(got_q[ok] - ref["q_tok"][ok]) <= RTOL[dtype] * ref["q_tok"][ok])
    # logits of magnitude ~300 carry an absolute fp32 rounding error of ~2e-5 into the exponent
    assert_close_rel(out["residual_mass"], ref["residual_mass"], max(RTOL[dtype], 1e-4), "residual_mass")


def test_host_buffer_entry_points(spr):
    """The *_host calls (host pointers in, host pointers out) give the same bits as the device calls."""
    wl_cpu = spr.workloads.make("gpt2", "cpu", B=5)
    wl = to_device(wl_cpu)
    cfg = wl.cfg
    B, K, V = wl.B, wl.K, wl.V
    ws = spr.Workspace.for_problem(B, K, V, cfg.d, cfg.h, spr.BF16)
    arena = spr.Arena(max(spr.host_arena_bytes(2, B, K, wl.Kp, wl.ldv, 0, 0, spr.BF16),
                          spr.host_arena_bytes(0, B, K, 0, 0, cfg.d, cfg.h, spr.BF16),
                          spr.host_arena_bytes(1, B, 0, 0, wl.ldv, 0, 0, spr.BF16)))
    pin = lambda t: t.contiguous().pin_memory()   # noqa: E731
    s_h, a_h, fr_h = spr.sprinter_verify_host(pin(wl_cpu.hidden), pin(wl_cpu.W1), pin(wl_cpu.b1), pin(wl_cpu.W2),
                                              pin(wl_cpu.b2), 0.5, arena, ws)
    s_d, a_d, fr_d = spr.sprinter_verify(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, 0.5, ws)
    assert torch.equal(s_h, s_d.cpu()) and torch.equal(a_h, a_d.cpu()) and torch.equal(fr_h, fr_d.cpu())
    t_h = spr.replace_sample_host(pin(wl_cpu.p_logits), V, pin(wl_cpu.u_replace), arena, ws, first_reject=fr_h,
                                  K=K, seq_stride=wl.Kp)
    t_d = spr.replace_sample(wl.p_logits, V, wl.u_replace, ws, first_reject=fr_d, K=K, seq_stride=wl.Kp)
    assert torch.equal(t_h, t_d.cpu())
    o_h = spr.sd_verify_host(pin(wl_cpu.p_logits), pin(wl_cpu.q_logits), V, pin(wl_cpu.draft_tokens),
                             pin(wl_cpu.uniforms), arena, ws, extras=True)
    o_d = spr.sd_verify(wl.p_logits, wl.q_logits, V, wl.draft_tokens, wl.uniforms, ws)
    for k in o_d:
        assert torch.equal(o_h[k], o_d[k].cpu()), k
    # device-detected problems come back as the return status of the host call
    bad = wl_cpu.draft_tokens.clone()
    bad[0, 0] = V
    with pytest.raises(spr.SprinterError) as e:
        spr.sd_verify_host(pin(wl_cpu.p_logits), pin(wl_cpu.q_logits), V, pin(bad), pin(wl_cpu.uniforms), arena, ws)
    assert e.value.status == 6
    rows = torch.tensor([0, 10 ** 6], dtype=torch.int32)
    with pytest.raises(spr.SprinterError) as e:
        spr.replace_sample_host(pin(wl_cpu.p_logits), V, pin(wl_cpu.u_replace[:2]), arena, ws, rows=rows)
    assert e.value.status == 7


def test_calls_replay_from_a_cuda_graph(spr):
    """sd_verify and sprinter_step enqueue only stream work (a clear and kernels, one of them
    launched programmatically behind another): captured once, replayed, same bits; and the
    replay follows the inputs when they change in place."""
    wl_cpu = spr.workloads.make("gpt2", "cpu", B=6)
    wl = to_device(wl_cpu)
    cfg = wl.cfg
    B, K, V = wl.B, wl.K, wl.V
    ws = spr.Workspace.for_problem(B, K, V, cfg.d, cfg.h, spr.BF16)
    out_sd = dict(accepted_len=torch.empty((B,), dtype=torch.int32, device="cuda"),
                  correction_token=torch.empty((B,), dtype=torch.int32, device="cuda"))
    out_st = (torch.empty((B, K), device="cuda"), torch.empty((B, K), dtype=torch.uint8, device="cuda"),
              torch.empty((B,), dtype=torch.int32, device="cuda"), torch.empty((B,), dtype=torch.int32, device="cuda"))

    def step():
        spr.sd_verify(wl.p_logits, wl.q_logits, V, wl.draft_tokens, wl.uniforms, ws, out=out_sd)
        spr.sprinter_step(wl.hidden, wl.W1, wl.b1, wl.W2, wl.b2, 0.5, wl.p_logits, V, wl.u_replace, ws, out=out_st)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                   # first call outside capture (one-time set-up)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    eager = [t.clone() for t in (*out_sd.values(), *out_st)]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for t in (*out_sd.values(), *out_st):
        t.fill_(-3)
    g.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, (*out_sd.values(), *out_st)):
        assert torch.equal(a, b)
    # new uniforms in the same buffers: the replay must follow them
    wl.uniforms.copy_(torch.rand_like(wl.uniforms))
    wl.u_replace.copy_(torch.rand_like(wl.u_replace))
    g.replay()
    torch.cuda.synchronize()
    replayed = [t.clone() for t in (*out_sd.values(), *out_st)]
    step()
    torch.cuda.synchronize()
    for a, b in zip(replayed, (*out_sd.values(), *out_st)):
        assert torch.equal(a, b)
    assert ws.device_status() == 0


# ---------------------------------------------------------------------------- K = 1
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("B,V,ldv", [
    (3, 8, None), (5, 64, 72), (4, 1000, None), (7, 1024, None), (2, 8200, 8208), (3, 16384, None),
    (2, 50264, None), (2, 65536, None), (1, 128256, None), (2, 130048, None),
    (3, 1001, None), (2, 131072, None), (2, 8192, 8195),      # misaligned rows, odd lengths
])
def test_sd_single_position_shapes(spr, dtype, B, V, ldv):
    """One position per sequence and no bonus row: the keep-or-resample rule of Section 3 on a
    single token, over aligned and misaligned rows of many lengths."""
    p, q, x, u = _rand_problem(B, 1, V, dtype, seed=17 + B * 1000 + V, ldv=ldv, Kp=1)
    u[::2, 0] = 0.9 + 0.09 * u[::2, 0]       # mostly rejections in the even sequences
    ref = _clear_sd(p, q, V, x, u)
    ws = spr.Workspace(spr.workspace_bytes(2, B, 1, V, 1, 0, spr.binding._dt(p)))
    for _ in range(2):                       # twice on one workspace
        out = spr.sd_verify(p.cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
        assert ws.device_status() == 0
        eq(out["accept"], ref["accept"], "accept")
        eq(out["accepted_len"], ref["accepted_len"], "accepted_len")
        eq(out["correction_token"], ref["correction_token"], "correction_token")
        assert_close_rel(out["p_tok"], ref["p_tok"], RTOL[dtype], "p_tok")
        assert_close_rel(out["q_tok"], ref["q_tok"], RTOL[dtype], "q_tok")
        assert_mass_close(out["residual_mass"], ref["residual_mass"], RTOL[dtype])


def test_sd_single_position_special_cases(spr):
    g = torch.Generator().manual_seed(21)
    B, V = 6, 5000
    u = torch.rand((B, 2), generator=g).clamp_(min=1e-3, max=0.999)
    ws = spr.Workspace(spr.workspace_bytes(2, B, 1, V, 1, 0, spr.F32))
    # p == q: everything accepted, nothing to draw
    q = torch.randn((B, 1, V), generator=g)
    x = torch.randint(0, V, (B, 1), generator=g, dtype=torch.int32)
    out = spr.sd_verify(q.clone().cuda(), q.cuda(), V, x.cuda(), u.cuda(), ws)
    assert (out["accept"] == 1).all() and (out["accepted_len"] == 1).all()
    assert (out["correction_token"] == -1).all() and (out["residual_mass"] == 0).all()
    # disjoint supports: everything rejected, correction token from p's support, residual mass 1
    ninf = float("-inf")
    p2 = torch.full((B, 1, V), ninf); p2[..., 4000:4100] = torch.randn((B, 1, 100), generator=g)
    q2 = torch.full((B, 1, V), ninf); q2[..., :4000] = torch.randn((B, 1, 4000), generator=g)
    x2 = torch.randint(0, 4000, (B, 1), generator=g, dtype=torch.int32)
    out = spr.sd_verify(p2.cuda(), q2.cuda(), V, x2.cuda(), u.cuda(), ws)
    assert (out["accept"] == 0).all() and (out["accepted_len"] == 0).all()
    assert ((out["correction_token"] >= 4000) & (out["correction_token"] < 4100)).all()
    assert torch.allclose(out["residual_mass"], torch.ones(B, device="cuda"), rtol=1e-5)
    for b in range(B):
        m, t = oracle.residual_draw_margin(to_np(p2)[b, 0], to_np(q2)[b, 0], float(u[b, 1]))
        if m > 1e-5:
            assert int(out["correction_token"][b]) == t
    # a draft token outside the vocabulary
    x3 = x.clone(); x3[2, 0] = V; x3[4, 0] = -1
    p3 = q + 0.7 * torch.randn((B, 1, V), generator=g)
    ref = _clear_sd(p3, q, V, x3.clamp(0, V - 1), u)
    out = spr.sd_verify(p3.cuda(), q.cuda(), V, x3.cuda(), u.cuda(), ws)
    assert ws.device_status() == 6
    for b in range(B):
        if b in (2, 4):
            assert int(out["accepted_len"][b]) == -1 and int(out["correction_token"][b]) == -1
            assert int(out["accept"][b, 0]) == 0 and float(out["p_tok"][b, 0]) == -1.0
        else:
            assert int(out["accepted_len"][b]) == ref["accepted_len"][b]
            assert int(out["correction_token"][b]) == ref["correction_token"][b]
