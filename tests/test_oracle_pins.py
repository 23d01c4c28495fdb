"""Pins for the float64 oracle: each check ties an oracle function to something fixed by
the paper or by mathematics (closed forms, brute force on tiny inputs, library special
cases, the exactness identity of speculative decoding) rather than to itself."""
import itertools
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sd_worked_examples.txt")


def rng(seed):
    return np.random.default_rng(seed)


def to_bf16_bits(a):
    t = torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16)
    return t.view(torch.uint16).numpy().copy(), t.to(torch.float64).numpy()


# ----------------------------------------------------------------------------- O1 verifier


def np_mlp(H, W1, b1, W2, b2):
    H, W1, W2 = (np.asarray(a, np.float64) for a in (H, W1, W2))
    a = np.maximum(H @ W1.T + np.asarray(b1, np.float64), 0.0)
    z = a @ W2 + float(b2)
    return scipy.special.expit(z)


@pytest.mark.parametrize("B,K,d,h", [(1, 4, 256, 64), (3, 5, 37, 11), (2, 1, 8, 3)])
def test_verifier_equals_numpy_mlp(B, K, d, h):
    r = rng(1)
    H = r.standard_normal((B, K, d)).astype(np.float32)
    W1 = (r.standard_normal((h, d)) / np.sqrt(d)).astype(np.float32)
    b1 = (r.standard_normal(h) / np.sqrt(d)).astype(np.float32)
    W2 = (r.standard_normal(h) / np.sqrt(h)).astype(np.float32)
    b2 = np.float32(0.1)
    s, acc, fr = oracle.sprinter_verify(H, W1, b1, W2, b2, 0.5)
    ref = np_mlp(H, W1, b1, W2, b2)
    np.testing.assert_allclose(s, ref, rtol=1e-12, atol=0)
    assert np.array_equal(acc, (ref >= 0.5).astype(np.uint8))


def test_verifier_single_linear_layer_equals_numpy():
    # the verifier the paper describes: one linear layer and a sigmoid (Section 3.2)
    r = rng(2)
    H = r.standard_normal((4, 3, 768)).astype(np.float32)
    w = (r.standard_normal(768) / np.sqrt(768)).astype(np.float32)
    s, acc, fr = oracle.sprinter_verify(H, w, None, None, np.float32(-0.2), 0.5)
    ref = scipy.special.expit(H.astype(np.float64) @ w.astype(np.float64) + np.float64(np.float32(-0.2)))
    np.testing.assert_allclose(s, ref, rtol=1e-12)


def test_verifier_index_mapping_one_hot():
    # W1[j, i_j] = 1 picks H[m, i_j]; catches a transposed or mis-strided operand
    r = rng(3)
    B, K, d, h = 2, 3, 7, 4
    H = r.standard_normal((B, K, d)).astype(np.float32)
    pick = [5, 0, 6, 2]
    W1 = np.zeros((h, d), np.float32)
    for j, i in enumerate(pick):
        W1[j, i] = 1.0
    b1 = np.array([0.5, -0.25, 0.0, 1.0], np.float32)
    W2 = np.array([1.0, -2.0, 0.5, 0.25], np.float32)
    s, _, _ = oracle.sprinter_verify(H, W1, b1, W2, np.float32(0.125), 0.5)
    for b in range(B):
        for k in range(K):
            z = 0.125
            for j, i in enumerate(pick):
                z += float(W2[j]) * max(0.0, float(H[b, k, i]) + float(b1[j]))
            assert s[b, k] == pytest.approx(1.0 / (1.0 + np.exp(-z)), rel=1e-13)


def test_verifier_zero_weights_and_threshold_equality():
    H = rng(4).standard_normal((2, 4, 16)).astype(np.float32)
    W1 = np.zeros((8, 16), np.float32)
    b1 = np.array([1, -1, 2, -2, 0.5, 0, 0, 0], np.float32)
    W2 = np.arange(8, dtype=np.float32) / 8
    s, acc, fr = oracle.sprinter_verify(H, W1, b1, W2, np.float32(0.25), 0.5)
    z = 0.25 + float(np.sum(W2.astype(np.float64) * np.maximum(b1.astype(np.float64), 0)))
    np.testing.assert_allclose(s, 1 / (1 + np.exp(-z)), rtol=1e-14)
    # all-zero verifier: score is exactly 1/2; Algorithm 2 continues when V >= tau
    s, acc, fr = oracle.sprinter_verify(H, W1, np.zeros(8, np.float32), np.zeros(8, np.float32),
                                        np.float32(0), 0.5)
    assert np.all(s == 0.5) and np.all(acc == 1) and np.all(fr == 4)
    s, acc, fr = oracle.sprinter_verify(H, W1, np.zeros(8, np.float32), np.zeros(8, np.float32),
                                        np.float32(0), np.nextafter(np.float32(0.5), np.float32(1)))
    assert np.all(acc == 0) and np.all(fr == 0)


def test_verifier_sigmoid_symmetry_and_d1():
    H = rng(5).standard_normal((1, 6, 32)).astype(np.float32)
    w = rng(6).standard_normal(32).astype(np.float32)
    s1, _, _ = oracle.sprinter_verify(H, w, None, None, np.float32(0.3), 0.5)
    s2, _, _ = oracle.sprinter_verify(H, -w, None, None, np.float32(-0.3), 0.5)
    np.testing.assert_allclose(s1 + s2, 1.0, rtol=1e-14)
    # d = h = 1 by hand
    s, acc, _ = oracle.sprinter_verify(np.array([[[2.0]]], np.float32), np.array([[3.0]], np.float32),
                                       np.array([-1.0], np.float32), np.array([0.5], np.float32),
                                       np.float32(-2.0), 0.5)
    assert s[0, 0] == pytest.approx(1 / (1 + np.exp(-(0.5 * 5.0 - 2.0))), rel=1e-15)
    assert acc[0, 0] == 1


def test_verifier_monotone_in_threshold():
    r = rng(7)
    H = r.standard_normal((8, 8, 64)).astype(np.float32)
    W1 = (r.standard_normal((16, 64)) / 8).astype(np.float32)
    b1 = np.zeros(16, np.float32)
    W2 = (r.standard_normal(16) / 4).astype(np.float32)
    prev = None
    for tau in (0.1, 0.3, 0.5, 0.7, 0.9):
        s, acc, fr = oracle.sprinter_verify(H, W1, b1, W2, np.float32(0), tau)
        assert np.array_equal(acc, (s >= np.float64(np.float32(tau))).astype(np.uint8))
        if prev is not None:
            assert np.all(acc <= prev[0]) and np.all(fr <= prev[1])
        prev = (acc, fr)


def test_verifier_bf16_inputs_widen_exactly():
    r = rng(8)
    Hb, Hd = to_bf16_bits(r.standard_normal((2, 3, 40)))
    W1b, W1d = to_bf16_bits(r.standard_normal((5, 40)) / 6)
    W2b, W2d = to_bf16_bits(r.standard_normal(5))
    b1 = r.standard_normal(5).astype(np.float32)
    s, _, _ = oracle.sprinter_verify(Hb, W1b, b1, W2b, np.float32(0.05), 0.5)
    np.testing.assert_allclose(s, np_mlp(Hd, W1d, b1, W2d, np.float32(0.05)), rtol=1e-12)


@pytest.mark.parametrize("K", [1, 2, 5, 12])
def test_first_reject_brute_force(K):
    for mask in itertools.product([0, 1], repeat=K):
        expect = next((k for k, a in enumerate(mask) if a == 0), K)
        assert oracle.first_reject(np.array(mask, np.uint8)) == expect


def test_first_reject_inside_verify_matches_accept_bits():
    r = rng(9)
    H = r.standard_normal((64, 6, 16)).astype(np.float32)
    w = r.standard_normal(16).astype(np.float32)
    _, acc, fr = oracle.sprinter_verify(H, w, None, None, np.float32(0.8), 0.5)
    assert len(set(fr.tolist())) > 2
    for b in range(64):
        assert fr[b] == next((k for k in range(6) if acc[b, k] == 0), 6)


# ----------------------------------------------------------------------------- O2 sampling


def test_sample_uniform_logits_is_floor_uV():
    V = 1000
    row = np.full(V, 1.75, np.float32)
    for u in rng(10).random(200):
        assert oracle.sample_softmax_row(row, u) == int(np.floor(u * V))


def test_sample_V1_V2():
    assert oracle.sample_softmax_row(np.array([3.0], np.float32), 0.999) == 0
    l = np.array([0.3, -1.1], np.float64)
    thr = scipy.special.expit(l[0] - l[1])
    for u in np.linspace(0, 0.999, 400):
        if abs(u - thr) < 1e-9:
            continue
        assert oracle.sample_softmax_row(l, u) == (0 if u < thr else 1)


def test_sample_shift_invariance_and_dominant_logit():
    r = rng(11)
    row = r.standard_normal(513) * 2
    us = r.random(64)
    a = [oracle.sample_softmax_row(row, u) for u in us]
    b = [oracle.sample_softmax_row(row + 12.5, u) for u in us]
    assert a == b
    row2 = row.copy()
    row2[77] += 50.0
    assert all(oracle.sample_softmax_row(row2, u) == 77 for u in np.linspace(1e-6, 1 - 1e-6, 50))


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_sample_equals_searchsorted_cumsum(dtype):
    r = rng(12)
    row = (r.standard_normal(4099) * 3).astype(dtype)
    p = scipy.special.softmax(row.astype(np.float64))
    cdf = np.cumsum(p)
    n_checked = 0
    for u in r.random(300):
        j = int(np.searchsorted(cdf, u, side="right"))
        lo = cdf[j - 1] if j else 0.0
        if min(u - lo, cdf[j] - u) < 1e-12:
            continue
        assert oracle.sample_softmax_row(row, u) == j
        n_checked += 1
    assert n_checked > 250


def test_sample_histogram_matches_softmax():
    r = rng(13)
    row = (r.standard_normal(24) * 1.5).astype(np.float32)
    G = 1 << 12
    us = (np.arange(G) + 0.5) / G
    toks = oracle.replace_sample(np.repeat(row[None], G, 0), 24, us.astype(np.float32))
    hist = np.bincount(toks, minlength=24) / G
    assert np.max(np.abs(hist - scipy.special.softmax(row.astype(np.float64)))) <= 1.0 / G + 1e-9


def test_sample_zero_weight_tokens_never_chosen():
    row = np.array([-np.inf, -np.inf, 0.0, -np.inf, 1.0, -np.inf], np.float64)
    assert oracle.sample_softmax_row(row, 0.0) == 2          # u = 0 -> first positive weight
    assert oracle.sample_softmax_row(row, 1.0) == 4          # rounding fallback: last positive
    p2 = 1 / (1 + np.e)
    assert oracle.sample_softmax_row(row, p2 - 1e-9) == 2
    assert oracle.sample_softmax_row(row, p2 + 1e-9) == 4
    assert oracle.inverse_cdf(np.zeros(5), 0.3) == -1


def test_inverse_cdf_brute_force():
    r = rng(14)
    for _ in range(200):
        V = int(r.integers(1, 9))
        w = r.random(V) * (r.random(V) > 0.3)
        if w.sum() == 0:
            continue
        u = r.random()
        c = np.cumsum(w)
        expect = next((j for j in range(V) if c[j] > u * w.sum()), None)
        if expect is None:
            expect = max(j for j in range(V) if w[j] > 0)
        assert oracle.inverse_cdf(w, u) == expect


def test_replace_sample_row_selection_and_gate():
    r = rng(15)
    R, V, ldv, K = 12, 50, 56, 3
    tl = r.standard_normal((R, ldv)).astype(np.float32) * 2
    tl[:, V:] = 80.0  # padding columns must be ignored
    u = r.random(4).astype(np.float32)
    # explicit rows
    rows = np.array([7, 0, 11, 3], np.int32)
    t = oracle.replace_sample(tl, V, u, rows=rows)
    for i in range(4):
        assert t[i] == oracle.sample_softmax_row(tl[rows[i], :V], u[i])
    # gate: sequence i owns rows i*K .. i*K+K-1; first_reject picks the row, K means skip
    fr = np.array([2, 3, 0, 1], np.int32)
    t = oracle.replace_sample(tl, V, u, first_reject=fr, K=K, seq_stride=K)
    assert t[1] == -1
    for i in (0, 2, 3):
        assert t[i] == oracle.sample_softmax_row(tl[i * K + fr[i], :V], u[i])
    # out-of-range row -> -1 and a status
    t, rc = oracle.replace_sample(tl, V, u, rows=np.array([0, 12, -1, 1], np.int32), return_status=True)
    assert rc == oracle.ERR_ROW and t[1] == -1 and t[2] == -1 and t[0] >= 0
    # a negative first_reject is not a position (Algorithm 2's r counts accepted tokens): the
    # draw is refused even though row i*K + first_reject would exist
    fr = np.array([2, -1, 0, 1], np.int32)
    t, rc = oracle.replace_sample(tl, V, u, first_reject=fr, K=K, seq_stride=K, return_status=True)
    assert rc == oracle.ERR_ROW and t[1] == -1
    for i in (0, 2, 3):
        assert t[i] == oracle.sample_softmax_row(tl[i * K + fr[i], :V], u[i])


def test_cdf_margin_by_hand():
    m, t = oracle.cdf_margin(np.array([1.0, 2.0, 1.0]), 0.5)
    assert t == 1 and m == pytest.approx(0.25)
    m, t = oracle.cdf_margin(np.array([1.0, 2.0, 1.0]), 0.8)
    assert t == 2 and m == pytest.approx(0.05)
    row = np.log(np.array([0.2, 0.5, 0.3]))
    m, t = oracle.softmax_draw_margin(row, 0.25)
    assert t == 1 and m == pytest.approx(0.05)


def test_residual_draw_margin_by_hand():
    """Eq. 1 worked by hand; every case fails if the p and q rows are swapped inside the margin
    helper (the swapped residual lives on the other tokens)."""
    # p - q = (0.3, -0.2, -0.1): the residual is all on token 0, whatever u
    p, q = np.log(np.array([0.5, 0.3, 0.2])), np.log(np.array([0.2, 0.5, 0.3]))
    for u in (0.0, 0.1, 0.5, 0.93):
        m, t = oracle.residual_draw_margin(p, q, u)
        assert t == 0 and m == pytest.approx(min(u, 1.0 - u), abs=1e-12)
    # p - q = (-0.4, 0.1, 0.3, 0): residual (0, 1/4, 3/4, 0), bins [0, 1/4) and [1/4, 1)
    p, q = np.log(np.array([0.1, 0.3, 0.4, 0.2])), np.log(np.array([0.5, 0.2, 0.1, 0.2]))
    m, t = oracle.residual_draw_margin(p, q, 0.2)
    assert t == 1 and m == pytest.approx(0.05, abs=1e-12)
    m, t = oracle.residual_draw_margin(p, q, 0.3)
    assert t == 2 and m == pytest.approx(0.05, abs=1e-12)
    m, t = oracle.residual_draw_margin(p, q, 0.9)
    assert t == 2 and m == pytest.approx(0.1, abs=1e-12)
    # shifted logits (unnormalised rows) give the same draw
    m, t = oracle.residual_draw_margin(p + 3.0, q - 2.0, 0.2)
    assert t == 1 and m == pytest.approx(0.05, abs=1e-12)
    # p = q: Eq. 1 is undefined, the draw comes from p itself (bins of p: 0.1, 0.4, 0.8, 1)
    m, t = oracle.residual_draw_margin(p, p.copy(), 0.45)
    assert t == 2 and m == pytest.approx(0.05, abs=1e-12)
    # the token agrees with the correction token of the full check when the draft token is rejected
    out = oracle.sd_verify(p[None, None], q[None, None], 4, np.array([[0]], np.int32),
                           np.array([[0.9, 0.2]], np.float32))
    assert out["accepted_len"][0] == 0 and out["correction_token"][0] == 1


# ----------------------------------------------------------------------------- O3 SD verify


def load_golden():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            p, q, res, beta = [s.strip() for s in line.split(";")]
            out.append((np.array(p.split(), float), np.array(q.split(), float),
                        np.array(res.split(), float), float(beta)))
    return out


@pytest.mark.parametrize("case", load_golden())
def test_golden_worked_examples(case):
    p, q, res, beta = case
    V = len(p)
    lp, lq = np.log(p) + 0.7, np.log(q) - 1.3   # any shift of the logits gives the same softmax
    w, R = oracle.residual_weights(lp, lq)
    np.testing.assert_allclose(w / R, res, atol=1e-14)
    assert R == pytest.approx(1 - beta, abs=1e-14)            # R = d_TV = 1 - beta
    # acceptance probability for x ~ q, integrating the accept set [0, min(1, p/q)] over u
    x = np.arange(V, dtype=np.int32)[:, None]
    P = np.repeat(lp[None, None], V, 0)
    Q = np.repeat(lq[None, None], V, 0)
    u = np.zeros((V, 2), np.float32)
    out = oracle.sd_verify(P, Q, V, x, u)
    acc_prob = np.minimum(1.0, out["p_tok"][:, 0] / out["q_tok"][:, 0])
    np.testing.assert_allclose(out["p_tok"][:, 0], p, rtol=1e-13)
    np.testing.assert_allclose(out["q_tok"][:, 0], q, rtol=1e-13)
    assert float(np.sum(q * acc_prob)) == pytest.approx(beta, abs=1e-13)
    # a rejected draw is replaced only by tokens with p > q, in residual proportions
    G = 1 << 10
    ug = ((np.arange(G) + 0.5) / G).astype(np.float32)
    xr = int(np.argmax(q - p))                                # a token with q > p: can be rejected
    U = np.stack([np.full(G, 0.999999, np.float32), ug], 1)
    out = oracle.sd_verify(np.repeat(lp[None, None], G, 0), np.repeat(lq[None, None], G, 0), V,
                           np.full((G, 1), xr, np.int32), U)
    assert np.all(out["accepted_len"] == 0)
    hist = np.bincount(out["correction_token"], minlength=V) / G
    assert np.max(np.abs(hist - res)) <= 1.0 / G + 1e-9
    assert np.all(p[out["correction_token"]] > q[out["correction_token"]])


def test_sd_accept_threshold_in_u():
    # the accept set in u is [0, min(1, p(x)/q(x))]: just inside accepts, just outside rejects
    r = rng(20)
    V = 6
    lp, lq = r.standard_normal(V), r.standard_normal(V)
    p, q = scipy.special.softmax(lp), scipy.special.softmax(lq)
    seen = set()
    for x in range(V):
        ratio = p[x] / q[x]
        for u in (ratio * (1 - 1e-5), ratio * (1 + 1e-5), 0.0, 0.99999):
            if not 0.0 <= u < 1.0:
                continue
            U = np.array([[u, 0.5]], np.float32)
            expect = 1 if float(U[0, 0]) <= min(1.0, ratio) else 0
            out = oracle.sd_verify(lp[None, None], lq[None, None], V, np.array([[x]], np.int32), U)
            assert out["accept"][0, 0] == expect
            seen.add(expect)
    assert seen == {0, 1}


def test_sd_equal_distributions_accept_everything_and_disjoint_reject():
    r = rng(21)
    V, B, K = 9, 5, 4
    lq = r.standard_normal((B, K, V))
    x = r.integers(0, V, (B, K)).astype(np.int32)
    u = r.random((B, K + 1)).astype(np.float32)
    out = oracle.sd_verify(lq + 3.0, lq, V, x, u)      # p = q (shifted logits)
    assert np.all(out["accept"] == 1) and np.all(out["accepted_len"] == K)
    assert np.all(out["correction_token"] == -1)       # Kp = K: no extra row
    # disjoint supports: p on the first half, q on the second half
    lp = np.where(np.arange(V) < 4, 0.0, -np.inf) + np.zeros((B, K, V))
    lq2 = np.where(np.arange(V) >= 4, 0.0, -np.inf) + np.zeros((B, K, V))
    x2 = r.integers(4, V, (B, K)).astype(np.int32)
    out = oracle.sd_verify(lp, lq2, V, x2, np.maximum(u, 1e-3))
    assert np.all(out["accept"] == 0) and np.all(out["accepted_len"] == 0)
    np.testing.assert_allclose(out["residual_mass"], 1.0, rtol=1e-14)
    assert np.all(out["correction_token"] < 4)


def test_sd_residual_properties_random():
    r = rng(22)
    for V in (2, 5, 33, 257):
        lp, lq = r.standard_normal(V) * 2, r.standard_normal(V) * 2
        p, q = scipy.special.softmax(lp), scipy.special.softmax(lq)
        w, R = oracle.residual_weights(lp, lq)
        dtv = 0.5 * np.sum(np.abs(p - q))
        assert R == pytest.approx(dtv, rel=1e-12)
        assert R == pytest.approx(1 - np.sum(np.minimum(p, q)), rel=1e-12)
        assert np.sum(w / R) == pytest.approx(1.0, rel=1e-13)
        assert np.all((w > 0) == (p > q))
        np.testing.assert_allclose(w, np.maximum(p - q, 0), atol=1e-16)


def _exact_output_distribution(lp, lq):
    """sum_x q(x) [ a(x) 1{y=x} + (1 - a(x)) res(y) ] with every piece read from the oracle."""
    V = len(lp)
    x = np.arange(V, dtype=np.int32)[:, None]
    out = oracle.sd_verify(np.repeat(lp[None, None], V, 0), np.repeat(lq[None, None], V, 0), V, x,
                           np.zeros((V, 2), np.float32))
    a = np.minimum(1.0, out["p_tok"][:, 0] / out["q_tok"][:, 0])
    w, R = oracle.residual_weights(lp, lq)
    qx = out["q_tok"][:, 0]
    return qx * a + np.sum(qx * (1 - a)) * (w / R if R > 0 else 0.0)


@pytest.mark.parametrize("V", [2, 3, 5, 8])
def test_sd_exactness_closed_form(V):
    # SD's output distribution equals the target's (Section 2)
    r = rng(30 + V)
    for _ in range(20):
        lp, lq = r.standard_normal(V) * 1.5, r.standard_normal(V) * 1.5
        np.testing.assert_allclose(_exact_output_distribution(lp, lq), scipy.special.softmax(lp),
                                   atol=1e-12)


@pytest.mark.parametrize("V", [3, 8])
def test_sd_exactness_by_enumeration_over_uniforms(V):
    # every (x, u_accept, u_draw) on a grid goes through oracle_sd_verify; the emitted token
    # (draft token if accepted, correction token otherwise) must be distributed as p
    r = rng(40 + V)
    lp = (r.standard_normal(V) * 1.2).astype(np.float32)
    lq = (r.standard_normal(V) * 1.2).astype(np.float32)
    p = scipy.special.softmax(lp.astype(np.float64))
    q = scipy.special.softmax(lq.astype(np.float64))
    G = 1 << 9
    g = ((np.arange(G) + 0.5) / G).astype(np.float32)
    U = np.stack(np.meshgrid(g, g, indexing="ij"), -1).reshape(-1, 2)
    n = U.shape[0]
    dist = np.zeros(V)
    P = np.repeat(lp[None, None], n, 0)
    Q = np.repeat(lq[None, None], n, 0)
    for x in range(V):
        out = oracle.sd_verify(P, Q, V, np.full((n, 1), x, np.int32), U)
        emitted = np.where(out["accepted_len"] == 1, x, out["correction_token"])
        assert np.all(emitted >= 0)
        dist += q[x] * np.bincount(emitted, minlength=V) / n
    assert np.max(np.abs(dist - p)) <= 2.0 * V / G


@pytest.mark.parametrize("V,K,G", [(3, 2, 64), (2, 3, 32)])
def test_sd_accepted_length_law(V, K, G):
    # independent positions: P(n >= k) = prod_{j<k} beta_j with beta_j = sum_x min(p_j, q_j)
    r = rng(50 + K)
    lp = r.standard_normal((K, V)).astype(np.float32)
    lq = r.standard_normal((K, V)).astype(np.float32)
    p = scipy.special.softmax(lp.astype(np.float64), -1)
    q = scipy.special.softmax(lq.astype(np.float64), -1)
    beta = np.sum(np.minimum(p, q), -1)
    g = ((np.arange(G) + 0.5) / G).astype(np.float32)
    U = np.stack(np.meshgrid(*([g] * K), indexing="ij"), -1).reshape(-1, K)
    U = np.concatenate([U, np.full((U.shape[0], 1), 0.5, np.float32)], 1)
    n = U.shape[0]
    surv = np.zeros(K + 1)
    for xs in itertools.product(range(V), repeat=K):
        wgt = np.prod([q[k, xs[k]] for k in range(K)])
        out = oracle.sd_verify(np.repeat(lp[None], n, 0), np.repeat(lq[None], n, 0), V,
                               np.tile(np.array(xs, np.int32), (n, 1)), U)
        for k in range(K + 1):
            surv[k] += wgt * np.mean(out["accepted_len"] >= k)
    expect = np.concatenate([[1.0], np.cumprod(beta)])
    assert np.max(np.abs(surv - expect)) <= 2.0 * K / G


def test_sd_accepted_len_and_bonus_row():
    r = rng(60)
    B, K, V = 40, 4, 17
    lq = r.standard_normal((B, K, V)).astype(np.float32) * 2
    lp1 = (np.concatenate([lq, r.standard_normal((B, 1, V)).astype(np.float32)], 1)
           + 0.4 * r.standard_normal((B, K + 1, V)).astype(np.float32))
    x = r.integers(0, V, (B, K)).astype(np.int32)
    u = r.random((B, K + 1)).astype(np.float32)
    o1 = oracle.sd_verify(lp1, lq, V, x, u)
    o0 = oracle.sd_verify(np.ascontiguousarray(lp1[:, :K]), lq, V, x, u)
    assert np.array_equal(o1["accept"], o0["accept"])
    assert len(set(o1["accepted_len"].tolist())) >= 3
    for b in range(B):
        n = next((k for k in range(K) if o1["accept"][b, k] == 0), K)
        assert o1["accepted_len"][b] == n == o0["accepted_len"][b]
        ratio = o1["p_tok"][b] / o1["q_tok"][b]
        assert np.array_equal(o1["accept"][b], (u[b, :K].astype(np.float64) <= np.minimum(1, ratio)).astype(np.uint8))
        if n == K:
            assert o0["correction_token"][b] == -1
            assert o1["correction_token"][b] == oracle.sample_softmax_row(lp1[b, K], u[b, K])
        else:
            w, R = oracle.residual_weights(lp1[b, n], lq[b, n])
            assert o1["correction_token"][b] == oracle.inverse_cdf(w, u[b, K]) == o0["correction_token"][b]
            assert o1["residual_mass"][b] == pytest.approx(R)
            assert w[o1["correction_token"][b]] > 0
    assert np.any(o1["accepted_len"] == K)


def test_sd_probabilities_match_scipy_softmax_and_padding_ignored():
    r = rng(61)
    B, K, V, ldv = 3, 2, 11, 16
    lq = r.standard_normal((B, K, ldv)).astype(np.float32)
    lp = r.standard_normal((B, K, ldv)).astype(np.float32)
    lq[..., V:] = 70.0
    lp[..., V:] = -70.0
    x = r.integers(0, V, (B, K)).astype(np.int32)
    u = r.random((B, K + 1)).astype(np.float32)
    out = oracle.sd_verify(lp, lq, V, x, u)
    P = scipy.special.softmax(lp[..., :V].astype(np.float64), -1)
    Q = scipy.special.softmax(lq[..., :V].astype(np.float64), -1)
    for b in range(B):
        for k in range(K):
            assert out["p_tok"][b, k] == pytest.approx(P[b, k, x[b, k]], rel=1e-12)
            assert out["q_tok"][b, k] == pytest.approx(Q[b, k, x[b, k]], rel=1e-12)
    assert np.all(out["correction_token"] < V)


def test_sd_invalid_token_reports_error():
    r = rng(62)
    lq = r.standard_normal((2, 2, 5))
    x = np.array([[1, 5], [0, 4]], np.int32)
    out, rc = oracle.sd_verify(lq, lq, 5, x, r.random((2, 3)).astype(np.float32), return_status=True)
    assert rc == oracle.ERR_TOKEN
    assert out["accepted_len"][0] == -1 and out["correction_token"][0] == -1
    assert out["accepted_len"][1] == 2


def test_sd_k1_is_the_sprinter_keep_or_residual_rule():
    # with a perfect verifier (no false positives) the rejected token is kept w.p. p/q, else
    # replaced from the residual, and the result is distributed as p (Theorem 1 at eta_FP = 0)
    r = rng(63)
    V = 4
    lp, lq = r.standard_normal(V), r.standard_normal(V)
    np.testing.assert_allclose(_exact_output_distribution(lp, lq), scipy.special.softmax(lp), atol=1e-12)


def test_bf16_logits_widen_exactly():
    r = rng(64)
    bits, vals = to_bf16_bits(r.standard_normal(300) * 3)
    assert oracle.softmax_stats(bits) == oracle.softmax_stats(vals)
    for u in r.random(20):
        assert oracle.sample_softmax_row(bits, u) == oracle.sample_softmax_row(vals, u)
    mx, Z = oracle.softmax_stats(vals)
    assert mx == vals.max()
    assert np.log(Z) + mx == pytest.approx(scipy.special.logsumexp(vals), rel=1e-13)
