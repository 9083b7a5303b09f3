"""The paper's own linear simulation design (Section 4.1) run through the C ABI: N = 100,000, p = 500,
Sigma = 0.8^|i-j|, unit signal variance, buffers of 10,000, mini-batches of 1,000, T = 5.

Parity with the oracle on a reduced job, and the statistical behaviour the paper reports for the full one: with a
small alpha T the BMGD estimator is about as accurate as the OLS estimator, and its distance to the OLS estimator
shrinks with alpha T (Theorem 2).
"""
import numpy as np
import pytest
import torch

from paper_2312_08728_b200 import inputs
from paper_2312_08728_b200.inputs import WORKLOADS

from helpers import TOL, buffers_of, gpu_job, oracle_job, rel_l2

pytestmark = pytest.mark.gpu


def test_reduced_job_agrees_with_the_oracle():
    w = WORKLOADS["sim41"].scaled(N=20_000, K=2, T=2, epochs=2, Rc=3)
    bufs = buffers_of(w)
    theta, stats = gpu_job(w, bufs, mode="resident")
    want = oracle_job(w, bufs)
    for c, th in want.items():
        assert rel_l2(theta[c], th) <= TOL[w.dtype], (c, stats)


def test_full_design_is_as_accurate_as_ols_and_closer_to_it_for_smaller_alpha_T():
    base = WORKLOADS["sim41"]
    bufs = buffers_of(base)
    X = torch.cat([x for x, _ in bufs]).to(torch.float64).numpy()
    y = torch.cat([v for _, v in bufs]).to(torch.float64).numpy()
    ols = np.linalg.solve(X.T @ X, X.T @ y)          # Section 3.1: the global OLS estimator
    true = inputs.theta_star(base).numpy()
    mse_ols = float(np.sum((ols - true) ** 2))
    dist = {}
    for lr, passes in ((0.01, 30), (0.002, 100)):    # alpha T = 0.05 and 0.01 at T = 5
        w = base.scaled(lr=lr, epochs=passes, Rc=4)
        theta, _ = gpu_job(w, bufs, mode="resident")
        mse = np.mean([np.sum((theta[c].astype(np.float64) - true) ** 2) for c in range(w.Rc)])
        dist[lr] = np.mean([np.linalg.norm(theta[c].astype(np.float64) - ols) for c in range(w.Rc)])
        assert mse <= 1.5 * mse_ols, (lr, mse, mse_ols)
    assert dist[0.002] < dist[0.01], dist


GRID = sorted(k for k in WORKLOADS if k.startswith("sim41-"))


@pytest.mark.parametrize("name", GRID)
def test_every_setting_of_the_simulation_grid_agrees_with_the_oracle_on_a_reduced_job(name):
    """Section 4.1's settings (T in {1, 5, 10} at fixed alpha T; n in {250, 500, 1000} x K in {2, 5} at two rates), each
    on the first fifth of the sample with two rounds-worth of its own T, two chains: parity with the oracle."""
    full = WORKLOADS[name]
    w = full.scaled(N=20_000, T=min(full.T, 2), epochs=1, Rc=2)
    bufs = buffers_of(w)
    assert len(bufs) == full.K and bufs[0][0].shape[0] == 20_000 // full.K
    theta, stats = gpu_job(w, bufs, mode="resident")
    want = oracle_job(w, bufs)
    for c, th in want.items():
        assert rel_l2(theta[c], th) <= TOL[w.dtype], (name, c, stats)


def test_grid_trends_match_the_papers_reading():
    """The shape of Section 4.1's findings on the full design, five chains each: (1) at a fixed alpha T the accuracy
    does not depend on T (T = 1, plain MGD, against T = 10); (2) with the constant rate 0.005, fewer and larger
    buffers (K = 2) and K = 5 both end near the OLS accuracy after 30 passes."""
    base = WORKLOADS["sim41"]
    bufs10 = buffers_of(base)
    X = torch.cat([x for x, _ in bufs10]).to(torch.float64).numpy()
    y = torch.cat([v for _, v in bufs10]).to(torch.float64).numpy()
    ols = np.linalg.solve(X.T @ X, X.T @ y)
    true = inputs.theta_star(base).numpy()
    mse_ols = float(np.sum((ols - true) ** 2))

    def mse_of(w, bufs):
        theta, _ = gpu_job(w, bufs, mode="resident")
        return float(np.mean([np.sum((theta[c].astype(np.float64) - true) ** 2) for c in range(w.Rc)]))

    m1 = mse_of(WORKLOADS["sim41-T1"].scaled(Rc=5, epochs=60), bufs10)
    m10 = mse_of(WORKLOADS["sim41-T10"].scaled(Rc=5, epochs=60), bufs10)
    assert m1 <= 1.5 * mse_ols and m10 <= 1.5 * mse_ols, (m1, m10, mse_ols)
    assert abs(np.log(m1) - np.log(m10)) < 0.35, (m1, m10)
    for K in (2, 5):
        w = WORKLOADS[f"sim41-K{K}-n1000-a"].scaled(Rc=5)
        m = mse_of(w, buffers_of(w))
        assert m <= 1.6 * mse_ols, (K, m, mse_ols)
