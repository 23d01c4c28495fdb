"""GPU parity of sprinter_simulate with the oracle's simulator (same Philox streams: run lengths
must be bit-identical), and the simulated law against Theorems 2 and 3 at full size."""
import numpy as np
import pytest
import torch

import oracle
from test_simulator_pins import theorem2_mean, theorem2_pmf, theorem3_stop_time

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def spr():
    import paper_2502_04557_b200 as s
    s.lib()
    return s


@pytest.mark.parametrize("r,tp,fp,cap,runs,first", [(5, 0.9, 0.5, 64, 100_003, 0), (0, 0.3, 0.8, 7, 4097, 12345),
                                                    (3, 1.0, 0.0, 40, 1000, 0), (12, 0.97, 0.93, 2000, 50_000, 2 ** 33),
                                                    (2, 0.5, 1.0, 33, 777, 5)])
def test_run_lengths_match_oracle(spr, r, tp, fp, cap, runs, first):
    n, hist = spr.sprinter_simulate(4242, runs, r, tp, fp, cap, first_run=first)
    n_ref, h_ref = oracle.simulate_runs(4242, runs, r, tp, fp, cap, first_run=first)
    assert np.array_equal(n.cpu().numpy(), n_ref)
    assert np.array_equal(hist.cpu().numpy(), h_ref.astype(np.int64))
    # histogram-only call, twice: overwritten, not accumulated
    for _ in range(2):
        _, hist2 = spr.sprinter_simulate(4242, runs, r, tp, fp, cap, first_run=first, want_runs=False)
        assert torch.equal(hist, hist2)


def test_full_size_law_matches_theorems(spr):
    runs, r, tp, fp, cap = 1 << 27, 5, 0.9, 0.5, 255
    _, hist = spr.sprinter_simulate(7, runs, r, tp, fp, cap, want_runs=False)
    h = hist.cpu().numpy().astype(np.float64)
    assert h.sum() == runs
    tp32, fp32 = float(np.float32(tp)), float(np.float32(fp))
    for i in range(30):
        pmf = theorem2_pmf(i, r, tp32, fp32)
        assert abs(h[i] / runs - pmf) <= 5 * np.sqrt(pmf * (1 - pmf) / runs) + 2e-8
    mean = float((h * np.arange(cap + 1)).sum() / runs)
    var = float((h * np.arange(cap + 1) ** 2).sum() / runs) - mean ** 2
    assert abs(mean - theorem2_mean(r, tp32, fp32)) <= 5 * np.sqrt(var / runs)
    assert abs(0.1 * (mean + 1) - theorem3_stop_time(r, tp32, fp32, 0.1)) <= 0.5 * np.sqrt(var / runs)
    # sampled runs of the full-size call against the oracle, one by one
    n, _ = spr.sprinter_simulate(7, 4096, r, tp, fp, cap, first_run=runs - 4096)
    n_ref, _ = oracle.simulate_runs(7, 4096, r, tp, fp, cap, first_run=runs - 4096)
    assert np.array_equal(n.cpu().numpy(), n_ref)


def test_simulator_argument_checks(spr):
    L = spr.lib()
    assert L.sprinter_simulate(1, 0, 10, 5, 0.5, 0.5, 8, None, None, None) == 1
    assert L.sprinter_simulate(1, 0, -1, 5, 0.5, 0.5, 8, None, None, None) == 1
    h = torch.zeros(9, dtype=torch.int64, device="cuda")
    assert L.sprinter_simulate(1, 0, 10, 5, 1.5, 0.5, 8, None, h.data_ptr(), None) == 1
    assert L.sprinter_simulate(1, 0, 0, 5, 0.5, 0.5, 8, None, h.data_ptr(), None) == 0
