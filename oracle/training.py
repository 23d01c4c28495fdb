"""Float64 oracle for preparing and fitting the verifier (Section 3.2).

TEST INFRASTRUCTURE ONLY, like the rest of this package: the CUDA library never imports it
and it imports nothing from the library.

What each function follows:
  verifier_labels      - the training label of a (prefix, draft token) pair: 1 if
                         q(x)/p(x) <= lambda, else 0 (Section 3.2, "Verifier Training
                         Methodology"; lambda = 1 is the ideal verifier rule of Section 3,
                         the appendix on training details varies lambda over 1, 1.2, 1.5).
  bce_loss_and_grad    - mean binary cross-entropy of the verifier sigma(b + w.s) (Section
                         3.2, "Verifier architecture": one linear layer + sigmoid, binary
                         cross-entropy loss) and its gradient.
  adam_update          - one update of the Adam optimiser the same passage names, as its
                         authors define it (Kingma & Ba, Algorithm 1, bias-corrected).
  verifier_train_step  - the two above: one optimiser step on the samples given.

Readings of what the paper leaves open: p and q are softmax(logits) at temperature 1; the
ratio is formed in log space; equality (ratio == lambda) labels 1; a draft token outside
[0, V) gets label 0 and ratio -1; the loss is averaged over the samples of the call (the
batch is whatever the caller passes); beta1, beta2, eps and the learning rate are
arguments; early stopping is the caller's loop over the returned loss.

Pins: tests/test_training_pins.py.
"""
from __future__ import annotations

import numpy as np

from . import softmax_stats


def verifier_labels(p_logits, q_logits, V: int, draft_tokens, lambdas):
    """p_logits [B,Kp,ldv], q_logits [B,K,ldv] (numpy; bf16 as raw uint16), draft_tokens
    [B,K], lambdas: sequence of thresholds.  Returns (labels uint8 [L,B,K], ratio f64 [B,K])
    with ratio = q(x)/p(x)."""
    B, K = draft_tokens.shape
    lambdas = [float(np.float32(lam)) for lam in lambdas]      # thresholds are float32 at the interface
    ratio = np.full((B, K), -1.0)
    labels = np.zeros((len(lambdas), B, K), np.uint8)
    for b in range(B):
        for k in range(K):
            x = int(draft_tokens[b, k])
            if x < 0 or x >= V:
                continue
            prow, qrow = p_logits[b, k, :V], q_logits[b, k, :V]
            mp, zp = softmax_stats(prow)
            mq, zq = softmax_stats(qrow)
            log_p = _widen(prow[x]) - mp - np.log(zp)
            log_q = _widen(qrow[x]) - mq - np.log(zq)
            with np.errstate(over="ignore", invalid="ignore"):
                ratio[b, k] = np.exp(log_q - log_p)
            for i, lam in enumerate(lambdas):
                labels[i, b, k] = 1 if ratio[b, k] <= lam else 0
    return labels, ratio


def _widen(v) -> float:
    """One logit as float64 (bfloat16 arrives as its uint16 bit pattern)."""
    if isinstance(v, np.uint16):
        return float(np.array([int(v) << 16], np.uint32).view(np.float32)[0])
    return float(v)


def widen(a) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def bce_loss_and_grad(hidden, labels, theta):
    """hidden [N,d], labels [N] in {0,1}, theta [d+1] = (w, b).  Returns (loss, grad [d+1]):
    loss = -(1/N) sum_i [y_i ln s_i + (1-y_i) ln(1-s_i)], s_i = sigma(b + w.hidden_i)."""
    S = widen(hidden)
    y = np.asarray(labels, np.float64)
    theta = np.asarray(theta, np.float64)
    N = S.shape[0]
    z = S @ theta[:-1] + theta[-1]
    # -[y ln s + (1-y) ln(1-s)] = ln(1 + e^z) - y z, written without overflow
    loss = float(np.sum(np.maximum(z, 0.0) + np.log1p(np.exp(-np.abs(z))) - y * z) / N)
    with np.errstate(over="ignore"):
        s = 1.0 / (1.0 + np.exp(-z))   # exp overflow gives s = 0, which is the limit
    r = s - y
    grad = np.concatenate([S.T @ r, [np.sum(r)]]) / N
    return loss, grad


def adam_update(theta, grad, m, v, t: int, lr: float, beta1: float, beta2: float, eps: float):
    """Step t (1-based) of Adam.  Returns (theta, m, v) after the step."""
    theta, grad, m, v = (np.asarray(a, np.float64) for a in (theta, grad, m, v))
    m = beta1 * m + (1.0 - beta1) * grad
    v = beta2 * v + (1.0 - beta2) * grad * grad
    m_hat = m / (1.0 - beta1 ** t)
    v_hat = v / (1.0 - beta2 ** t)
    return theta - lr * m_hat / (np.sqrt(v_hat) + eps), m, v


def verifier_train_step(hidden, labels, theta, m, v, t: int, lr: float, beta1: float = 0.9,
                        beta2: float = 0.999, eps: float = 1e-8):
    """One optimiser step.  Returns (loss before the step, theta, m, v)."""
    f32 = lambda a: float(np.float32(a))   # noqa: E731 - hyper-parameters are float32 at the interface
    loss, grad = bce_loss_and_grad(hidden, labels, theta)
    theta, m, v = adam_update(theta, grad, m, v, t, f32(lr), f32(beta1), f32(beta2), f32(eps))
    return loss, theta, m, v
