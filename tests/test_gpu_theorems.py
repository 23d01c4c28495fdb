"""Statistical check of Theorems 1 and 4 through the CUDA library: with a verifier that errs
i.i.d. (true-positive rate eta_TP, false-positive rate eta_FP), the token SPRINTER emits is
distributed as (1 - eta_FP) p + eta_FP q and the draft token survives with probability
1 - (1 - eta_FP) d_TV(p, q).  Every sampling step runs in the library's kernels: the draft
token is drawn with replace_sample on the draft logits, the keep-or-resample rule is
sd_verify with K = 1; the synthetic verifier is a Bernoulli mask."""
import numpy as np
import pytest
import scipy.special
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("eta_tp,eta_fp", [(1.0, 0.0), (0.9, 0.5), (0.6, 0.25)])
def test_emitted_token_law_and_acceptance_rate(eta_tp, eta_fp):
    import paper_2502_04557_b200 as spr
    g = torch.Generator(device="cuda").manual_seed(31)
    V, n = 48, 1 << 20
    lq = torch.randn(V, generator=g, device="cuda") * 1.5
    lp = lq + torch.randn(V, generator=g, device="cuda") * 0.9
    p = scipy.special.softmax(lp.double().cpu().numpy())
    q = scipy.special.softmax(lq.double().cpu().numpy())
    Q = lq.expand(n, V).contiguous()
    P = lp.expand(n, V).contiguous()
    u = torch.rand((n, 4), generator=g, device="cuda")
    ws = spr.Workspace(max(spr.workspace_bytes(1, n, 1, V, 1, 0, spr.F32), spr.workspace_bytes(2, n, 1, V, 1, 0, spr.F32)))
    # draft token x ~ q
    x = spr.replace_sample(Q, V, u[:, 0].contiguous(), ws)
    assert ws.device_status() == 0
    # ground truth "acceptable" (q(x) <= p(x)) and the verifier's noisy copy of it
    acceptable = torch.from_numpy(q <= p).cuda()[x.long()]
    verifier_accepts = torch.where(acceptable, u[:, 1] < eta_tp, u[:, 1] < eta_fp)
    # target call for the tokens the verifier stopped on: keep w.p. min(1, p/q), else residual
    sd = spr.sd_verify(P.view(n, 1, V), Q.view(n, 1, V), V, x.view(n, 1), u[:, 2:4].contiguous(), ws)
    assert ws.device_status() == 0
    kept_by_target = sd["accepted_len"] == 1
    emitted = torch.where(verifier_accepts | kept_by_target, x, sd["correction_token"])
    hist = torch.bincount(emitted.long(), minlength=V).double().cpu().numpy() / n
    expect = (1 - eta_fp) * p + eta_fp * q                       # Theorem 1
    sigma = np.sqrt(expect * (1 - expect) / n)
    assert np.all(np.abs(hist - expect) <= 5 * sigma + 1e-6)
    # only unacceptable tokens that the verifier also rejects can be replaced (Theorem 4)
    survived = (verifier_accepts | kept_by_target).double().mean().item()
    dtv = 0.5 * np.abs(p - q).sum()
    beta = 1 - (1 - eta_fp) * dtv
    assert abs(survived - beta) <= 5 * np.sqrt(beta * (1 - beta) / n)
    # total-variation statement of Theorem 1
    assert 0.5 * np.abs(expect - p).sum() == pytest.approx(eta_fp * dtv, rel=1e-12)
