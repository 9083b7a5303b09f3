"""Pins of the oracle's Nesterov and Adam updates and of its cosine learning rate (CPU only).

The buffered variants of Section 4.3 (BNAG, BAdam) differ from their baselines only in where the mini-batches
come from, so the update rules are pinned on their own: against torch.optim fed the same gradients (a library
routine), against closed forms of the first steps, and against an independent numpy loop over the oracle's own
partition.  The learning rate of Section 4.4 is pinned against the values the paper's formula prints.
"""
import numpy as np
import pytest
import torch

import oracle


def problem(N0=400, p=6, seed=0):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((N0, p))
    y = X @ np.ones(p) + rng.standard_normal(N0)
    return X, y


def full_gradient(X, y, th):
    return X.T @ (X @ th - y) / X.shape[0]


@pytest.mark.parametrize("kind", ["nesterov", "adam"])
def test_full_batch_steps_equal_a_library_optimiser_fed_the_same_gradients(kind):
    X, y = problem()
    N0, p = X.shape
    steps, lr = 25, 0.05
    if kind == "nesterov":
        opt = oracle.Optimizer(oracle.OPT_NESTEROV, p, a=0.9)
    else:
        opt = oracle.Optimizer(oracle.OPT_ADAM, p, a=0.9, b=0.999, eps=1e-7)
    th = np.zeros(p)
    # n = N0: one step per round, the mini-batch is the whole buffer whatever the partition
    tr = oracle.run_rounds(oracle.LINEAR, X, y, th, steps, N0, lr, seed=3, trace=True, opt=opt)

    w = torch.zeros(p, dtype=torch.float64, requires_grad=True)
    if kind == "nesterov":
        topt = torch.optim.SGD([w], lr=lr, momentum=0.9, nesterov=True)
    else:
        topt = torch.optim.Adam([w], lr=lr, betas=(0.9, 0.999), eps=1e-7)
    for s in range(steps):
        w.grad = torch.from_numpy(full_gradient(X, y, w.detach().numpy()))
        topt.step()
        assert np.allclose(tr[s], w.detach().numpy(), rtol=1e-11, atol=1e-13), (kind, s)
    assert int(opt.t[0]) == (steps if kind == "adam" else 0)


def test_first_steps_in_closed_form():
    X, y = problem(seed=1)
    N0, p = X.shape
    lr, mu = 0.1, 0.8
    g0 = full_gradient(X, y, np.zeros(p))
    # Nesterov from v = 0: v1 = -lr g0, theta1 = -(1 + mu) lr g0; then one more step written out
    opt = oracle.Optimizer(oracle.OPT_NESTEROV, p, a=mu)
    th = np.zeros(p)
    tr = oracle.run_rounds(oracle.LINEAR, X, y, th, 2, N0, lr, seed=0, trace=True, opt=opt)
    th1 = -(1 + mu) * lr * g0
    assert np.allclose(tr[0], th1, rtol=1e-13)
    g1 = full_gradient(X, y, th1)
    v2 = mu * (-lr * g0) - lr * g1
    assert np.allclose(tr[1], th1 + mu * v2 - lr * g1, rtol=1e-12)
    assert np.allclose(opt.s1, v2, rtol=1e-12)
    # Adam from m = v = 0: the bias corrections give m^ = g, v^ = g^2, so the step is lr g / (|g| + eps)
    eps = 1e-3
    opt = oracle.Optimizer(oracle.OPT_ADAM, p, a=0.9, b=0.99, eps=eps)
    th = np.zeros(p)
    oracle.run_rounds(oracle.LINEAR, X, y, th, 1, N0, lr, seed=0, opt=opt)
    assert np.allclose(th, -lr * g0 / (np.abs(g0) + eps), rtol=1e-12)
    assert np.allclose(opt.s1, 0.1 * g0, rtol=1e-13) and np.allclose(opt.s2, 0.01 * g0 * g0, rtol=1e-13)


def test_zero_momentum_is_plain_gradient_descent():
    X, y = problem(seed=2)
    N0, p = X.shape
    a, b = np.zeros(p), np.zeros(p)
    oracle.run_rounds(oracle.LINEAR, X, y, a, 3, 50, 0.05, seed=5)
    oracle.run_rounds(oracle.LINEAR, X, y, b, 3, 50, 0.05, seed=5, opt=oracle.Optimizer(oracle.OPT_NESTEROV, p, a=0.0))
    assert np.allclose(a, b, rtol=1e-13, atol=1e-15)
    c = np.zeros(p)
    oracle.run_rounds(oracle.LINEAR, X, y, c, 3, 50, 0.05, seed=5, opt=oracle.Optimizer(oracle.OPT_SGD, p))
    assert np.array_equal(a, c)


def test_cosine_rate_takes_the_values_of_section_4_4():
    """alpha_j = 0.025 + 0.025 cos(j pi / J) for j = 1..J with initial value 0.05, again in every pass."""
    X, y = problem(N0=64, p=1, seed=4)
    N0 = 64
    T, M, K = 2, 4, 2   # J = T M K updates per pass
    J = T * M * K
    opt = oracle.Optimizer(oracle.OPT_SGD, 1, sched=oracle.LR_COSINE, period=J)
    th = np.zeros(1)
    rates = []
    for r in range(2):              # two passes
        for k in range(K):          # K buffers (the same rows serve as every buffer here)
            before = th.copy()
            tr = oracle.run_rounds(oracle.LINEAR, X, y, th, T, N0 // M, 0.05, seed=10 + k, trace=True, opt=opt)
            prev = before
            for s in range(T * M):
                idx = oracle.perm(10 + k, 0, s // M, N0)[(s % M) * 16:(s % M + 1) * 16]
                g = X[idx].T @ (X[idx] @ prev - y[idx]) / 16
                rates.append(float((prev - tr[s])[0] / g[0]))
                prev = tr[s]
    want = [0.025 + 0.025 * np.cos(j * np.pi / J) for j in range(1, J + 1)] * 2
    assert np.allclose(rates[:J - 1], want[:J - 1], rtol=1e-9)
    assert abs(rates[J - 1]) < 1e-12            # the last update of a pass has rate 0.025 - 0.025
    assert np.allclose(rates[J:2 * J - 1], want[:J - 1], rtol=1e-9)
    assert int(opt.j_done[0]) == 0


@pytest.mark.parametrize("kind", [oracle.OPT_NESTEROV, oracle.OPT_ADAM])
@pytest.mark.parametrize("loss", [oracle.LINEAR, oracle.LOGISTIC])
def test_mini_batch_chain_equals_an_independent_loop(kind, loss):
    """Ragged mini-batches, two buffers, state carried from call to call: numpy loop over the oracle's partition."""
    rng = np.random.default_rng(7)
    N0, p, n, T, lr = 230, 5, 48, 2, 0.1
    bufs = []
    for k in range(2):
        X = rng.standard_normal((N0, p))
        u = X @ (np.ones(p) / 2)
        y = (rng.random(N0) < 1 / (1 + np.exp(-u))).astype(np.float64) if loss == oracle.LOGISTIC else u + rng.standard_normal(N0)
        bufs.append((X, y))
    a, b, eps = (0.9, 0.999, 1e-7) if kind == oracle.OPT_ADAM else (0.7, 0.0, 0.0)
    opt = oracle.Optimizer(kind, p, a=a, b=b, eps=eps)
    th = np.zeros(p)
    want, s1, s2, t = np.zeros(p), np.zeros(p), np.zeros(p), 0
    for k, (X, y) in enumerate(bufs):
        oracle.run_rounds(loss, X, y, th, T, n, lr, seed=20 + k, opt=opt)
        for r in range(T):
            pi = oracle.perm(20 + k, 0, r, N0)
            for lo in range(0, N0, n):
                idx = pi[lo:lo + n]
                z = X[idx] @ want
                res = (1 / (1 + np.exp(-z)) if loss == oracle.LOGISTIC else z) - y[idx]
                g = X[idx].T @ res / len(idx)
                if kind == oracle.OPT_NESTEROV:
                    s1 = a * s1 - lr * g
                    want = want + a * s1 - lr * g
                else:
                    t += 1
                    s1 = a * s1 + (1 - a) * g
                    s2 = b * s2 + (1 - b) * g * g
                    want = want - lr * (s1 / (1 - a ** t)) / (np.sqrt(s2 / (1 - b ** t)) + eps)
    assert np.allclose(th, want, rtol=1e-10, atol=1e-12)
