"""Pins for the verifier-preparation oracle (labels, BCE gradient, Adam): closed forms, finite
differences, the library optimiser, and the link to the exact SD test."""
import numpy as np
import pytest
import torch

import oracle
from oracle import training


def rng(seed):
    return np.random.default_rng(seed)


def bf16_bits(a):
    return torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16).view(torch.uint16).numpy().copy()


# ----------------------------------------------------------------------------- labels
def test_labels_closed_form_two_tokens():
    """p = (1/4, 3/4), q = (3/4, 1/4): q/p is 3 for token 0 and 1/3 for token 1."""
    ln3 = np.log(3.0)
    p = np.array([[[0.0, ln3]] * 2], np.float64)
    q = np.array([[[ln3, 0.0]] * 2], np.float64)
    x = np.array([[0, 1]], np.int32)
    labels, ratio = training.verifier_labels(p, q, 2, x, [1.0, 1.5, 2.99, 3.01, 0.3, 0.34])
    np.testing.assert_allclose(ratio, [[3.0, 1.0 / 3.0]], rtol=1e-14)
    assert labels[:, 0, 0].tolist() == [0, 0, 0, 1, 0, 0]
    assert labels[:, 0, 1].tolist() == [1, 1, 1, 1, 0, 1]


@pytest.mark.parametrize("bits", [False, True], ids=["f32", "bf16"])
def test_labels_lambda_one_is_the_sd_test_that_never_rejects_by_chance(bits):
    """With u = 1 the SD test u <= min(1, p/q) passes exactly when p(x) >= q(x), i.e. when
    q(x)/p(x) <= 1: the ideal verifier rule (Section 3) read off the already pinned SD oracle."""
    r = rng(3)
    B, K, V = 6, 5, 97
    q = (2.0 * r.standard_normal((B, K, V))).astype(np.float32)
    p = (q + 0.8 * r.standard_normal((B, K, V))).astype(np.float32)
    if bits:
        p, q = bf16_bits(p), bf16_bits(q)
    x = r.integers(0, V, (B, K)).astype(np.int32)
    sd = oracle.sd_verify(p, q, V, x, np.ones((B, K + 1), np.float32))
    labels, ratio = training.verifier_labels(p, q, V, x, [1.0])
    assert np.array_equal(labels[0], sd["accept"])
    np.testing.assert_allclose(ratio, sd["q_tok"] / sd["p_tok"], rtol=1e-12)
    assert 0 < labels.sum() < labels.size          # both classes occur


def test_labels_brute_force_monotone_and_invalid_token():
    r = rng(4)
    B, K, V = 3, 4, 11
    p = r.standard_normal((B, K + 1, V))           # a bonus row and row padding must be ignored
    q = np.concatenate([r.standard_normal((B, K, V)), np.full((B, K, 2), 50.0)], 2)
    p = np.concatenate([p, np.full((B, K + 1, 2), 50.0)], 2)
    x = r.integers(0, V, (B, K)).astype(np.int32)
    x[1, 2] = V                                    # outside the vocabulary
    lambdas = [0.5, 1.0, 1.2, 1.5, 4.0]
    labels, ratio = training.verifier_labels(p, q, V, x, lambdas)
    for b in range(B):
        for k in range(K):
            if (b, k) == (1, 2):
                assert ratio[b, k] == -1.0 and labels[:, b, k].sum() == 0
                continue
            pp = np.exp(p[b, k, :V]) / np.exp(p[b, k, :V]).sum()
            qq = np.exp(q[b, k, :V]) / np.exp(q[b, k, :V]).sum()
            want = qq[x[b, k]] / pp[x[b, k]]
            assert abs(ratio[b, k] / want - 1.0) < 1e-12
            assert labels[:, b, k].tolist() == [int(want <= lam) for lam in lambdas]
            assert np.all(np.diff(labels[:, b, k].astype(int)) >= 0)     # more accepts as lambda grows


def test_labels_zero_target_probability():
    p = np.array([[[-np.inf, 0.0, 0.0]]])
    q = np.zeros((1, 1, 3))
    labels, ratio = training.verifier_labels(p, q, 3, np.array([[0]], np.int32), [1.0, 1e30])
    assert np.isinf(ratio[0, 0]) and labels.sum() == 0


# ----------------------------------------------------------------------------- loss, gradient
def test_bce_at_zero_weights_is_ln2_and_gradient_is_mean_residual():
    r = rng(5)
    S = r.standard_normal((40, 7))
    y = r.integers(0, 2, 40)
    loss, grad = training.bce_loss_and_grad(S, y, np.zeros(8))
    assert abs(loss - np.log(2.0)) < 1e-15
    np.testing.assert_allclose(grad[:-1], ((0.5 - y)[:, None] * S).mean(0), rtol=1e-13)
    assert abs(grad[-1] - (0.5 - y).mean()) < 1e-15


def test_bce_matches_its_definition_and_finite_differences():
    r = rng(6)
    N, d = 30, 5
    S = r.standard_normal((N, d))
    y = r.integers(0, 2, N)
    theta = r.standard_normal(d + 1)
    loss, grad = training.bce_loss_and_grad(S, y, theta)
    s = 1.0 / (1.0 + np.exp(-(S @ theta[:-1] + theta[-1])))
    assert abs(loss - -(y * np.log(s) + (1 - y) * np.log(1 - s)).mean()) < 1e-14
    h = 1e-6
    for j in range(d + 1):
        e = np.zeros(d + 1)
        e[j] = h
        fd = (training.bce_loss_and_grad(S, y, theta + e)[0] - training.bce_loss_and_grad(S, y, theta - e)[0]) / (2 * h)
        assert abs(fd - grad[j]) < 1e-8


def test_bce_is_stable_for_large_logits_and_widens_bf16_exactly():
    S = np.array([[1000.0], [-1000.0]])
    loss, grad = training.bce_loss_and_grad(S, np.array([1, 0]), np.array([1.0, 0.0]))
    assert loss == 0.0 and np.all(grad == 0.0)
    loss, _ = training.bce_loss_and_grad(S, np.array([0, 1]), np.array([1.0, 0.0]))
    assert loss == 1000.0
    vals = np.array([[0.5, -1.25, 3.0]], np.float32)
    a = training.bce_loss_and_grad(bf16_bits(vals), np.array([1]), np.array([0.3, -0.2, 0.1, 0.05]))
    b = training.bce_loss_and_grad(vals.astype(np.float64), np.array([1]), np.array([0.3, -0.2, 0.1, 0.05]))
    assert a[0] == b[0] and np.array_equal(a[1], b[1])


# ----------------------------------------------------------------------------- Adam
def test_adam_first_step_closed_form():
    """After one step m_hat = g and v_hat = g^2: theta moves by lr * g / (|g| + eps)."""
    g = np.array([0.3, -2.0, 1e-12, 0.0])
    theta, m, v = training.adam_update(np.ones(4), g, np.zeros(4), np.zeros(4), 1, 0.01, 0.9, 0.999, 1e-8)
    np.testing.assert_allclose(theta, 1.0 - 0.01 * g / (np.abs(g) + 1e-8), rtol=1e-12)
    np.testing.assert_allclose(m, 0.1 * g, rtol=1e-15)
    np.testing.assert_allclose(v, 0.001 * g * g, rtol=1e-12)


def test_adam_without_memory_is_sign_descent():
    theta, m, v = np.zeros(3), np.zeros(3), np.zeros(3)
    for t, g in enumerate([np.array([1.0, -4.0, 0.5]), np.array([-2.0, 3.0, 0.25])], 1):
        new, m, v = training.adam_update(theta, g, m, v, t, 0.1, 0.0, 0.0, 0.0)
        np.testing.assert_allclose(new, theta - 0.1 * np.sign(g), rtol=1e-15, atol=1e-16)
        theta = new


def test_training_steps_match_the_library_optimiser():
    """Twenty steps against torch's Adam and BCE-with-logits in float64 on the CPU."""
    r = rng(7)
    N, d = 64, 9
    S = r.standard_normal((N, d))
    y = (S @ r.standard_normal(d) + 0.3 * r.standard_normal(N) > 0).astype(np.float64)
    lr, b1, b2, eps = (float(np.float32(a)) for a in (0.05, 0.9, 0.999, 1e-8))
    w = torch.zeros(d + 1, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([w], lr=lr, betas=(b1, b2), eps=eps)
    St, yt = torch.from_numpy(S), torch.from_numpy(y)
    theta, m, v = np.zeros(d + 1), np.zeros(d + 1), np.zeros(d + 1)
    for t in range(1, 21):
        opt.zero_grad()
        lt = torch.nn.functional.binary_cross_entropy_with_logits(St @ w[:-1] + w[-1], yt)
        lt.backward()
        opt.step()
        loss, theta, m, v = training.verifier_train_step(S, y, theta, m, v, t, lr, b1, b2, eps)
        assert abs(loss - lt.item()) < 1e-12
        np.testing.assert_allclose(theta, w.detach().numpy(), rtol=1e-9, atol=1e-12)


def test_training_separates_separable_data():
    r = rng(8)
    N, d = 200, 6
    S = r.standard_normal((N, d))
    y = (S @ r.standard_normal(d) > 0).astype(np.uint8)
    theta, m, v = np.zeros(d + 1), np.zeros(d + 1), np.zeros(d + 1)
    losses = []
    for t in range(1, 301):
        loss, theta, m, v = training.verifier_train_step(S, y, theta, m, v, t, 0.05)
        losses.append(loss)
    assert abs(losses[0] - np.log(2)) < 1e-15 and losses[-1] < 0.2 * losses[0]
    assert all(b < a for a, b in zip(losses[:50], losses[1:51]))          # steadily down at the start
    assert np.mean((S @ theta[:-1] + theta[-1] > 0) == y) > 0.98
