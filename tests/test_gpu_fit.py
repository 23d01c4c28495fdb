"""verifier_labels and verifier_train_step (Section 3.2) against the float64 oracle."""
import numpy as np
import pytest
import torch

from helpers import RTOL, to_np
from oracle import training
from test_gpu_parity import _rand_problem

pytestmark = pytest.mark.gpu

LAMBDAS = [1.0, 1.2, 1.5]          # the thresholds the paper trains with
LABEL_MARGIN = 1e-4                # labels are compared where |ratio / lambda - 1| exceeds this


@pytest.fixture(scope="module")
def spr():
    import paper_2502_04557_b200 as s
    s.lib()
    return s


def bd(spr):
    return spr.binding


def check_labels(spr, p, q, V, x, lambdas, dtype):
    B, K = x.shape
    ws = spr.Workspace(spr.workspace_bytes(bd(spr).OP_VERIFIER_LABELS, B, K, V, 0, 0, bd(spr)._dt(p)))
    labels, ratio = bd(spr).verifier_labels(p.cuda(), q.cuda(), V, x.cuda(), lambdas, ws)
    status = ws.device_status()
    want_labels, want_ratio = training.verifier_labels(to_np(p), to_np(q), V, to_np(x), lambdas)
    got_ratio = ratio.cpu().double().numpy()
    finite = np.isfinite(want_ratio) & (want_ratio > 0)
    assert np.array_equal(np.isfinite(got_ratio), np.isfinite(want_ratio))
    assert np.all(np.abs(got_ratio[finite] / want_ratio[finite] - 1.0) <= RTOL[dtype])
    assert np.array_equal(got_ratio[want_ratio < 0], want_ratio[want_ratio < 0])      # invalid tokens: -1
    got = labels.cpu().numpy()
    skipped = 0
    for i, lam in enumerate(lambdas):
        clear = ~finite | (np.abs(want_ratio / float(np.float32(lam)) - 1.0) > LABEL_MARGIN)
        skipped += int((~clear).sum())
        assert np.array_equal(got[i][clear], want_labels[i][clear]), f"lambda {lam}"
    assert skipped <= max(1, x.numel() // 50)
    return status, want_labels


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("B,K,V,ldv,Kp", [
    (3, 1, 2, None, 2), (5, 2, 7, None, 2), (4, 3, 1000, None, 4), (2, 33, 129, 131, 34),
    (3, 4, 8191, None, 4), (2, 2, 8193, 8200, 3), (2, 5, 32769, None, 6), (1, 40, 50257, None, 40),
    (38, 33, 33001, 33003, 34),      # more than four waves of two-segment rows: records written by the finish grid
])
def test_labels_ragged_shapes(spr, dtype, B, K, V, ldv, Kp):
    p, q, x, _ = _rand_problem(B, K, V, dtype, seed=3 + B * 1000 + K * 10 + V, ldv=ldv, Kp=Kp)
    status, want = check_labels(spr, p, q, V, x, LAMBDAS, dtype)
    assert status == 0
    if V > 100:
        assert 0 < want.sum() < want.size


@pytest.mark.parametrize("name,B", [("tiny", None), ("gpt2", 6), ("llama2", 8), ("llama3", 3)])
def test_labels_on_the_workload_shapes(spr, name, B):
    wl = spr.workloads.make(name, "cpu", B=B)
    status, _ = check_labels(spr, wl.p_logits, wl.q_logits, wl.V, wl.draft_tokens, LAMBDAS + [0.5, 3.0],
                             wl.q_logits.dtype)
    assert status == 0


def test_labels_invalid_token_zero_probability_and_limits(spr):
    B, K, V = 2, 3, 600
    p, q, x, _ = _rand_problem(B, K, V, torch.float32, seed=11)
    x[0, 1] = -1
    x[1, 2] = V
    p[1, 0, int(x[1, 0])] = float("-inf")          # p(x) = 0: ratio +inf, never labelled 1
    status, want = check_labels(spr, p, q, V, x, [1.0, 1e30], torch.float32)
    assert status == 6                                 # SPR_ERR_BAD_TOKEN
    assert want[:, 0, 1].sum() == 0 and want[:, 1, 2].sum() == 0 and want[:, 1, 0].sum() == 0
    ws = spr.Workspace(spr.workspace_bytes(bd(spr).OP_VERIFIER_LABELS, B, K, V, 0, 0, spr.F32))
    with pytest.raises(spr.SprinterError) as e:        # more thresholds than one call takes
        bd(spr).verifier_labels(p.cuda(), q.cuda(), V, x.cuda(), [1.0] * 9, ws)
    assert e.value.status == 1
    empty = bd(spr).verifier_labels(torch.empty((0, K, V), device="cuda"), torch.empty((0, K, V), device="cuda"), V,
                                    torch.empty((0, K), dtype=torch.int32, device="cuda"), [1.0], ws)
    assert empty[0].shape == (1, 0, K)


# ----------------------------------------------------------------------------- training
def teacher_problem(N, d, dtype, seed, noise=0.5):
    g = torch.Generator().manual_seed(seed)
    S = torch.randn((N, d), generator=g).to(dtype)
    w = torch.randn((d,), generator=g) / d ** 0.5
    y = ((S.float() @ w + noise * torch.randn((N,), generator=g)) > 0.1).to(torch.uint8)
    return S, y


def run_steps(spr, S, y, steps, lr, theta0=None, **hyper):
    N, d = S.shape
    ws = spr.Workspace(spr.workspace_bytes(bd(spr).OP_VERIFIER_TRAIN, 0, 0, 0, d, 0, bd(spr)._dt(S)))
    Sg, yg = S.cuda(), y.cuda()
    theta = torch.zeros(d + 1, device="cuda") if theta0 is None else theta0.clone().cuda()
    m, v = torch.zeros(d + 1, device="cuda"), torch.zeros(d + 1, device="cuda")
    hist = []
    for t in range(1, steps + 1):
        loss = bd(spr).verifier_train_step(Sg, yg, theta, m, v, t, lr, ws, **hyper)
        hist.append((float(loss), theta.cpu().double().numpy().copy()))
    return hist, (theta, m, v)


@pytest.mark.parametrize("N,d,dtype", [
    (5000, 768, torch.bfloat16), (1, 768, torch.bfloat16), (7, 64, torch.bfloat16), (20000, 256, torch.bfloat16),
    (3000, 2048, torch.bfloat16), (2000, 4096, torch.bfloat16), (4001, 1000, torch.bfloat16),
    (3000, 100, torch.float32), (1500, 2048, torch.float32), (999, 4, torch.float32),
    # many rows per team of warps: the shared-memory rings go round several times
    (60000, 768, torch.bfloat16), (40000, 1024, torch.bfloat16), (30000, 1536, torch.bfloat16),
    (24000, 2048, torch.bfloat16), (16000, 4096, torch.bfloat16), (12000, 2560, torch.bfloat16),
    (14001, 3072, torch.bfloat16), (70000, 128, torch.bfloat16), (20000, 1024, torch.float32),
    (9000, 2048, torch.float32), (11000, 1240, torch.float32),
    # short rows travel several to a slot: rings that go round, and a last block that is not full
    (70001, 128, torch.bfloat16), (50003, 512, torch.bfloat16), (40002, 200, torch.float32),
], ids=lambda v: str(v).replace("torch.", ""))
def test_train_steps_match_the_oracle(spr, N, d, dtype):
    """fp32 sums on the GPU against float64: the loss agrees to 2e-5 relative, and since an Adam
    step is lr * m_hat / sqrt(v_hat) (of order lr whatever the gradient's size), a relative
    gradient error e moves a parameter by about lr * e per step: bound 1e-3 * lr * t."""
    S, y = teacher_problem(N, d, dtype, seed=N + d)
    lr, steps = 0.02, 12
    hist, _ = run_steps(spr, S, y, steps, lr)
    Sn, yn = to_np(S), y.numpy()
    theta, m, v = np.zeros(d + 1), np.zeros(d + 1), np.zeros(d + 1)
    for t, (loss_gpu, theta_gpu) in enumerate(hist, 1):
        loss, theta, m, v = training.verifier_train_step(Sn, yn, theta, m, v, t, lr)
        assert abs(loss_gpu / loss - 1.0) < 2e-5, f"step {t}: loss {loss_gpu} vs {loss}"
        err = np.abs(theta_gpu - theta).max()
        assert err <= 1e-3 * lr * t, f"step {t}: max parameter error {err:.3e}"
    assert hist[0][0] == pytest.approx(np.log(2.0), rel=1e-6)


def test_train_other_hyperparameters_and_nonzero_start(spr):
    S, y = teacher_problem(2500, 768, torch.bfloat16, seed=5)
    g = torch.Generator().manual_seed(6)
    theta0 = 0.05 * torch.randn(769, generator=g)
    hyper = dict(beta1=0.5, beta2=0.9, eps=1e-6)
    hist, _ = run_steps(spr, S, y, 8, 0.01, theta0=theta0, **hyper)
    theta, m, v = theta0.double().numpy(), np.zeros(769), np.zeros(769)
    for t, (loss_gpu, theta_gpu) in enumerate(hist, 1):
        loss, theta, m, v = training.verifier_train_step(to_np(S), y.numpy(), theta, m, v, t, 0.01, **hyper)
        assert abs(loss_gpu / loss - 1.0) < 2e-5
        assert np.abs(theta_gpu - theta).max() <= 1e-3 * 0.01 * t


def test_train_is_reproducible_and_rejects_unsupported_widths(spr):
    S, y = teacher_problem(6000, 768, torch.bfloat16, seed=9)
    a, sa = run_steps(spr, S, y, 5, 0.02)
    b, sb = run_steps(spr, S, y, 5, 0.02)
    assert [h[0] for h in a] == [h[0] for h in b]
    assert all(torch.equal(x, z) for x, z in zip(sa, sb))
    for d, dtype in [(770, torch.bfloat16), (8192, torch.bfloat16), (4096, torch.float32), (6, torch.float32)]:
        ws = spr.Workspace(spr.workspace_bytes(bd(spr).OP_VERIFIER_TRAIN, 0, 0, 0, d, 0, bd(spr)._dt(torch.empty(0, dtype=dtype))))
        z = torch.zeros(d + 1, device="cuda")
        with pytest.raises(spr.SprinterError) as e:
            bd(spr).verifier_train_step(torch.zeros((4, d), dtype=dtype, device="cuda"),
                                        torch.zeros(4, dtype=torch.uint8, device="cuda"), z, z.clone(), z.clone(), 1,
                                        0.01, ws)
        assert e.value.status == 2


@pytest.mark.parametrize("N,d,dtype", [(5000, 768, torch.bfloat16), (3000, 2048, torch.bfloat16),
                                       (2000, 4096, torch.bfloat16), (9, 64, torch.float32),
                                       (30001, 256, torch.bfloat16)],
                         ids=lambda v: str(v).replace("torch.", ""))
def test_train_bounded_wait_runs_out_and_nothing_is_stepped(spr, N, d, dtype):
    """No row is ever fetched (test flag): every team's first wait expires after a few thousand
    polls, the launch ends by itself, reports SPR_ERR_TIMEOUT and takes no step; the next call on
    the same workspace is a normal step."""
    S, y = teacher_problem(N, d, dtype, seed=21)
    ws = spr.Workspace(spr.workspace_bytes(bd(spr).OP_VERIFIER_TRAIN, 0, 0, 0, d, 0, bd(spr)._dt(S)))
    Sg, yg = S.cuda(), y.cuda()
    g = torch.Generator().manual_seed(22)
    theta = (0.05 * torch.randn(d + 1, generator=g)).cuda()
    m, v = torch.rand(d + 1, generator=g).cuda() * 1e-3, torch.rand(d + 1, generator=g).cuda() * 1e-6
    ref = [x.clone() for x in (theta, m, v)]
    want = [x.clone() for x in ref]
    loss_ok = bd(spr).verifier_train_step(Sg, yg, *want, 3, 0.01, ws)       # warm: module load, attributes
    assert ws.device_status() == 0
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    loss = bd(spr).verifier_train_step(Sg, yg, theta, m, v, 3, 0.01, ws, test_flags=1, spin_limit=4000)
    b.record()
    assert ws.device_status() == 5                                          # SPR_ERR_TIMEOUT
    assert ws.device_status() == 0                                          # reading the status clears it
    assert torch.isnan(loss).all()
    assert all(torch.equal(x, r) for x, r in zip((theta, m, v), ref)), "a failed pass must not take a step"
    assert a.elapsed_time(b) < 50.0, "the failing launch must end quickly"
    loss = bd(spr).verifier_train_step(Sg, yg, theta, m, v, 3, 0.01, ws)
    assert ws.device_status() == 0
    assert torch.equal(loss, loss_ok) and all(torch.equal(x, w) for x, w in zip((theta, m, v), want))


def test_labels_then_training_then_the_verifier_call(spr):
    """The preparation chain on the GPU alone: labels from the two models' logits, a linear
    verifier fitted to hidden states that carry the label, and sprinter_verify using it."""
    wl = spr.workloads.make("gpt2", "cuda", B=64)
    B, K, V, d = wl.B, wl.K, wl.V, wl.hidden.shape[-1]
    ws = spr.Workspace(max(spr.workspace_bytes(bd(spr).OP_VERIFIER_LABELS, B, K, V, 0, 0, spr.BF16),
                           spr.workspace_bytes(bd(spr).OP_VERIFIER_TRAIN, 0, 0, 0, d, 0, spr.BF16),
                           spr.workspace_bytes(0, B, K, V, d, 0, spr.BF16)))
    labels, _ = bd(spr).verifier_labels(wl.p_logits, wl.q_logits, V, wl.draft_tokens, [1.2], ws)
    y = labels[0].reshape(-1).contiguous()
    assert 0.05 < y.float().mean() < 0.95
    g = torch.Generator().manual_seed(1)
    direction = torch.randn(d, generator=g).cuda() / d ** 0.5
    hidden = torch.randn((B * K, d), generator=g).cuda()
    hidden += (y.float() * 2 - 1)[:, None] * 4.0 * direction           # separable along one direction
    hidden = hidden.to(torch.bfloat16).contiguous()
    theta = torch.zeros(d + 1, device="cuda")
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    losses = [float(bd(spr).verifier_train_step(hidden, y, theta, m, v, t, 0.05, ws)) for t in range(1, 101)]
    assert losses[-1] < 0.2 * losses[0]
    scores, accept, _ = spr.sprinter_verify(hidden.view(B, K, d), theta[:d].to(torch.bfloat16).contiguous(), None, None,
                                            theta[d:].contiguous(), 0.5, ws)
    assert ws.device_status() == 0
    assert (accept.reshape(-1) == y).float().mean() > 0.97


def test_labels_llama3_full_size_sampled(spr):
    """The benchmark's workload: the oracle on a sample of sequences, and the link to sd_verify
    (ratio = q(x)/p(x) of its outputs) on all 4096 tokens."""
    wl = spr.workloads.make("llama3", "cuda")
    B, K, V = wl.B, wl.K, wl.V
    ws = spr.Workspace(max(spr.workspace_bytes(bd(spr).OP_VERIFIER_LABELS, B, K, V, 0, 0, spr.BF16),
                           spr.workspace_bytes(2, B, K, V, 1, 0, spr.BF16)))
    labels, ratio = bd(spr).verifier_labels(wl.p_logits, wl.q_logits, V, wl.draft_tokens, LAMBDAS, ws)
    assert ws.device_status() == 0
    seqs = [0, 3, 77, 128, 255]
    idx = torch.tensor(seqs, device="cuda")
    want_labels, want_ratio = training.verifier_labels(to_np(wl.p_logits[idx]), to_np(wl.q_logits[idx]), V,
                                                       to_np(wl.draft_tokens[idx]), LAMBDAS)
    got_ratio = ratio[idx].cpu().double().numpy()
    assert np.all(np.abs(got_ratio / want_ratio - 1.0) <= 1e-3)
    got = labels[:, idx].cpu().numpy()
    for i, lam in enumerate(LAMBDAS):
        clear = np.abs(want_ratio / lam - 1.0) > LABEL_MARGIN
        assert clear.mean() > 0.95 and np.array_equal(got[i][clear], want_labels[i][clear])
    sd = spr.sd_verify(wl.p_logits, wl.q_logits, V, wl.draft_tokens, wl.uniforms, ws)
    assert torch.allclose(ratio, sd["q_tok"] / sd["p_tok"], rtol=1e-4)
    lab = labels.cpu().numpy().astype(int)
    assert np.all(np.diff(lab, axis=0) >= 0)                       # more accepts as lambda grows
    assert np.array_equal(lab[0] == 1, (ratio <= 1.0).cpu().numpy())


def test_train_step_at_the_benchmark_size(spr):
    """N = 2^20 samples of width 2048 (the configuration bench.py times): the first step has a
    closed form - loss ln 2 and a move of lr * g / (|g| + eps) with g = mean((1/2 - y) s) - checked
    against a float64 matrix product; the oracle itself takes one step on a slice that fits."""
    N, d, lr = 1 << 20, 2048, 0.01
    g = torch.Generator(device="cuda").manual_seed(12)
    S = torch.randn((N, d), generator=g, device="cuda").to(torch.bfloat16)
    y = (torch.rand(N, generator=g, device="cuda") < 0.3).to(torch.uint8)
    ws = spr.Workspace(spr.workspace_bytes(bd(spr).OP_VERIFIER_TRAIN, 0, 0, 0, d, 0, spr.BF16))
    theta = torch.zeros(d + 1, device="cuda")
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    loss = bd(spr).verifier_train_step(S, y, theta, m, v, 1, lr, ws)
    assert float(loss) == pytest.approx(np.log(2.0), rel=1e-6)
    r = 0.5 - y.double()
    grad = torch.cat([(r[None, :] @ S.double()).reshape(-1), r.sum()[None]]) / N
    want = -lr * grad / (grad.abs() + 1e-8)
    assert (theta.double() - want).abs().max() <= 1e-3 * lr
    assert torch.allclose(m.double(), 0.1 * grad, rtol=1e-3, atol=1e-9)
    n = 1 << 16                                                     # a slice the oracle handles in seconds
    theta.zero_(); m.zero_(); v.zero_()
    loss = bd(spr).verifier_train_step(S[:n].contiguous(), y[:n].contiguous(), theta, m, v, 1, lr, ws)
    l0, t0, _, _ = training.verifier_train_step(to_np(S[:n]), y[:n].cpu().numpy(), np.zeros(d + 1), np.zeros(d + 1),
                                                np.zeros(d + 1), 1, lr)
    assert abs(float(loss) / l0 - 1.0) < 2e-5 and np.abs(theta.cpu().double().numpy() - t0).max() <= 1e-3 * lr
