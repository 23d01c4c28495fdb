"""Pins for the decode-loop simulator of the oracle (i.i.d. verifier, Theorems 2 and 3):
the generator against published known-answer vectors, the simulated law of N against the
closed forms the paper proves, and the degenerate cases."""
import os

import numpy as np
import pytest

import oracle

KAT = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def theorem2_pmf(i, r, tp, fp):
    return tp ** i * (1 - tp) if i < r else tp ** r * fp ** (i - r) * (1 - fp)


def theorem2_mean(r, tp, fp):
    return (tp - tp ** r) / (1 - tp) + tp ** r / (1 - fp)


def theorem3_stop_time(r, tp, fp, td):
    return (1 - tp ** r) * td / (1 - tp) + tp ** r * td / (1 - fp)


def test_philox_known_answers():
    n = 0
    for line in open(KAT):
        if line.startswith("#") or not line.strip():
            continue
        c, k, o = [[int(x, 16) for x in part.split()] for part in line.split(";")]
        got = oracle.philox4x32_10(np.array(c, np.uint32), np.array(k, np.uint32))
        assert got.tolist() == o
        n += 1
    assert n == 3


@pytest.mark.parametrize("r,tp,fp", [(5, 0.9, 0.5), (5, 0.6, 0.2), (1, 0.5, 0.5), (8, 0.95, 0.1), (0, 0.9, 0.3)])
def test_simulated_law_matches_theorem_2(r, tp, fp):
    runs, cap = 400_000, 200
    n, hist = oracle.simulate_runs(2025, runs, r, tp, fp, cap)
    assert hist.sum() == runs and np.array_equal(np.bincount(n, minlength=cap + 1), hist.astype(np.int64))
    tp32, fp32 = float(np.float32(tp)), float(np.float32(fp))
    for i in range(0, 25):
        pmf = theorem2_pmf(i, r, tp32, fp32)
        sigma = np.sqrt(pmf * (1 - pmf) / runs)
        assert abs(hist[i] / runs - pmf) <= 5 * sigma + 1e-7, (i, hist[i] / runs, pmf)
    mean = theorem2_mean(r, tp32, fp32) if r > 0 else fp32 / (1 - fp32)
    assert abs(n.mean() - mean) <= 5 * n.std() / np.sqrt(runs)
    # Theorem 3 with t_d = 0.1: the stopping time is t_d per drafted token, N accepted + 1 rejected
    if r > 0:
        td = 0.1
        assert theorem3_stop_time(r, tp32, fp32, td) == pytest.approx(td * (theorem2_mean(r, tp32, fp32) + 1), rel=1e-12)
        assert abs(td * (n.mean() + 1) - theorem3_stop_time(r, tp32, fp32, td)) <= 5 * td * n.std() / np.sqrt(runs)


def test_figure_value_and_gap():
    # r = 5, eta_TP = 0.9, eta_FP = 0.5 gives E[N] = 4.27608; as eta_TP -> 1 with eta_FP <= 0.5 the
    # verifier accepts at most one unacceptable token on average (the "gap" of the figure)
    assert theorem2_mean(5, 0.9, 0.5) == pytest.approx(4.27608, abs=1e-5)
    n, _ = oracle.simulate_runs(11, 300_000, 5, 1.0, 0.5, 100)
    assert n.min() == 5
    assert abs((n.mean() - 5) - 1.0) <= 5 * n.std() / np.sqrt(len(n))


def test_degenerate_verifiers_and_cap():
    n, hist = oracle.simulate_runs(1, 1000, 5, 1.0, 0.0, 50)       # perfect verifier: exactly r tokens
    assert np.all(n == 5) and hist[5] == 1000
    n, _ = oracle.simulate_runs(1, 1000, 5, 0.0, 0.7, 50)          # rejects the first token
    assert np.all(n == 0)
    n, _ = oracle.simulate_runs(1, 1000, 3, 1.0, 1.0, 17)          # accepts everything: the cap
    assert np.all(n == 17)
    n, _ = oracle.simulate_runs(1, 1000, 3, 0.5, 0.5, 0)
    assert np.all(n == 0)


def test_runs_are_independent_streams():
    a, _ = oracle.simulate_runs(99, 5000, 4, 0.8, 0.3, 40)
    b, _ = oracle.simulate_runs(99, 2000, 4, 0.8, 0.3, 40, first_run=3000)
    assert np.array_equal(a[3000:], b)
    c, _ = oracle.simulate_runs(100, 5000, 4, 0.8, 0.3, 40)
    assert not np.array_equal(a, c)
    # by hand for run 0: uniforms are (word >> 8) * 2^-24 of successive Philox words
    w = oracle.philox4x32_10(np.array([0, 0, 0, 0], np.uint32), np.array([99, 0], np.uint32))
    u = (w >> 8).astype(np.float64) * 2.0 ** -24
    expect = 0
    for k in range(4):
        if u[k] < float(np.float32(0.8 if k < 4 else 0.3)):
            expect += 1
        else:
            break
    if expect < 4:
        assert a[0] == expect
    else:
        assert a[0] >= 4
