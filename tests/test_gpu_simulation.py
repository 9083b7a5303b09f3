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
