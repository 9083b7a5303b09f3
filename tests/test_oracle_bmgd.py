"""Pins for the oracle's computation step against what the paper and the mathematics fix.

Every expected value here is computed by plain numpy written from the formula it cites,
never by the oracle itself: the full-batch closed form and the OLS limit (Section 3.1),
the Gram-matrix recurrence Eq. (3.1)-(3.2), the stable solution below Eq. (3.3), the MGD
special case T = 1, brute force on a four-row buffer, finite differences and the Newton
limit for logistic regression, and the C = 2 softmax/logistic identity.
"""
import itertools

import numpy as np
import pytest

import oracle


def ar_design(rng, rows, p, rho):
    z = rng.standard_normal((rows, p))
    s = np.sqrt(1 - rho * rho)
    for j in range(1, p):
        z[:, j] = rho * z[:, j - 1] + s * z[:, j]
    return z


def linear_data(seed, rows, p, rho=0.5):
    rng = np.random.default_rng(seed)
    X = ar_design(rng, rows, p, rho)
    y = X @ np.ones(p) + rng.standard_normal(rows)
    return X, y


def logistic_data(seed, rows, p):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((rows, p))
    th = rng.standard_normal(p) / np.sqrt(p)
    y = (rng.random(rows) < 1 / (1 + np.exp(-X @ th))).astype(np.float64)
    return X, y


def batches_of(seed, chain, rnd, N0, n):
    pi = oracle.perm(seed, chain, rnd, N0)
    return [pi[m * n:min((m + 1) * n, N0)].astype(np.int64) for m in range(-(-N0 // n))]


# ------------------------------------------------------------------ P1: full batch, closed form, OLS

def test_full_batch_equals_closed_form_gradient_descent():
    """n = N0: the partition does not matter and theta_T = A^T theta_0 + (I - A^T) theta_ols, A = I - alpha Sxx."""
    X, y = linear_data(1, 400, 6)
    N0, p = X.shape
    Sxx, Sxy = X.T @ X / N0, X.T @ y / N0
    ols = np.linalg.solve(Sxx, Sxy)
    lam, V = np.linalg.eigh(Sxx)
    alpha = 0.3
    theta0 = np.linspace(-1, 1, p)
    for T in (1, 7, 40):
        th = theta0.copy()
        oracle.run_rounds(oracle.LINEAR, X, y, th, T, N0, alpha, seed=5)
        AT = V @ np.diag((1 - alpha * lam) ** T) @ V.T
        want = AT @ theta0 + (np.eye(p) - AT) @ ols
        assert np.linalg.norm(th - want) <= 1e-12 * np.linalg.norm(want)


def test_full_batch_converges_to_ols():
    """Section 3.1: the least-squares minimiser is Sxx^{-1} Sxy; full-batch GD reaches it."""
    X, y = linear_data(2, 500, 8)
    ols = np.linalg.lstsq(X, y, rcond=None)[0]
    th = np.zeros(8)
    oracle.run_rounds(oracle.LINEAR, X, y, th, 3000, 500, 0.5, seed=0)
    assert np.linalg.norm(th - ols) <= 1e-10 * np.linalg.norm(ols)


def test_factor_two_reading():
    """One full-batch step from 0 moves theta by +alpha*Sxy (Eq. (3.1)), not 2*alpha*Sxy."""
    X, y = linear_data(3, 50, 4)
    th = np.zeros(4)
    oracle.run_rounds(oracle.LINEAR, X, y, th, 1, 50, 0.1, seed=0)
    assert np.allclose(th, 0.1 * X.T @ y / 50, rtol=1e-13, atol=0)


# ------------------------------------------------------------------ P2: MGD special case

def test_one_round_buffer_equals_minibatch_is_plain_mgd():
    """T = 1 with buffer = mini-batch: BMGD over the buffer sequence is plain MGD (Section 4.1)."""
    X, y = linear_data(4, 600, 5)
    n, alpha = 100, 0.07
    th = np.zeros(5)
    for k in range(6):
        oracle.run_rounds(oracle.LINEAR, X[k * n:(k + 1) * n], y[k * n:(k + 1) * n], th, 1, n, alpha, seed=k)
    want = np.zeros(5)
    for k in range(6):
        Xb, yb = X[k * n:(k + 1) * n], y[k * n:(k + 1) * n]
        want = want - alpha * Xb.T @ (Xb @ want - yb) / n
    assert np.linalg.norm(th - want) <= 1e-13 * np.linalg.norm(want)


# ------------------------------------------------------------------ P3: Gram-matrix recurrence

@pytest.mark.parametrize("N0,n", [(240, 40), (250, 40)])
def test_matches_gram_matrix_recurrence(N0, n):
    """Eq. (3.1): theta <- (I - alpha Sxx^(m)) theta + alpha Sxy^(m), per mini-batch of the oracle's own partition."""
    X, y = linear_data(5, N0, 7)
    alpha, T, seed = 0.05, 3, 77
    th = np.full(7, 0.25)
    tr = oracle.run_rounds(oracle.LINEAR, X, y, th, T, n, alpha, seed=seed, chain=2, trace=True)
    want = np.full(7, 0.25)
    step = 0
    for t in range(T):
        for b in batches_of(seed, 2, t, N0, n):
            Sxx = X[b].T @ X[b] / len(b)
            Sxy = X[b].T @ y[b] / len(b)
            want = (np.eye(7) - alpha * Sxx) @ want + alpha * Sxy
            assert np.linalg.norm(tr[step] - want) <= 1e-12 * np.linalg.norm(want)
            step += 1
    assert step == tr.shape[0]
    assert np.array_equal(tr[-1], th)


def test_buffer_level_affine_map():
    """Eq. (3.2) under a fixed partition: theta_after = A^T theta_before + alpha (I + ... + A^{T-1}) B."""
    N0, n, p, T, alpha = 120, 30, 5, 4, 0.1
    X, y = linear_data(6, N0, p)
    bs = batches_of(9, 0, 0, N0, n)
    A = np.eye(p)
    B = np.zeros(p)
    for b in bs:  # A = Delta^(M) ... Delta^(1); B accumulates with the later Deltas applied
        D = np.eye(p) - alpha * X[b].T @ X[b] / len(b)
        A = D @ A
        B = D @ B + X[b].T @ y[b] / len(b)
    Cmat = np.linalg.matrix_power(A, T)
    Dvec = sum(np.linalg.matrix_power(A, s) for s in range(T)) @ B
    th0 = np.arange(p, dtype=np.float64)
    th = th0.copy()
    oracle.run_rounds(oracle.LINEAR, X, y, th, T, n, alpha, seed=9, fixed_partition=True)
    want = Cmat @ th0 + alpha * Dvec
    assert np.linalg.norm(th - want) <= 1e-12 * np.linalg.norm(want)


# ------------------------------------------------------------------ P4: stable solution

def test_stable_solution_of_the_stacked_system():
    """Fixed partition: end-of-buffer estimates converge to theta* = alpha Omega^{-1} D*, Omega = I - C* (below Eq. (3.3))."""
    K, N0, n, p, T, alpha = 3, 60, 20, 4, 2, 0.2
    X, y = linear_data(7, K * N0, p)
    Cs, Ds = [], []
    for k in range(K):
        Xk, yk = X[k * N0:(k + 1) * N0], y[k * N0:(k + 1) * N0]
        A = np.eye(p); B = np.zeros(p)
        for b in batches_of(100 + k, 0, 0, N0, n):
            D = np.eye(p) - alpha * Xk[b].T @ Xk[b] / len(b)
            A = D @ A
            B = D @ B + Xk[b].T @ yk[b] / len(b)
        Cs.append(np.linalg.matrix_power(A, T))
        Ds.append(sum(np.linalg.matrix_power(A, s) for s in range(T)) @ B)
    Cstar = np.zeros((K * p, K * p))
    for k in range(K):  # block row k reads the estimate of buffer k-1 (cyclically)
        src = (k - 1) % K
        Cstar[k * p:(k + 1) * p, src * p:(src + 1) * p] = Cs[k]
    stable = alpha * np.linalg.solve(np.eye(K * p) - Cstar, np.concatenate(Ds))

    th = np.zeros(p)
    ends = None
    for r in range(400):
        ends = []
        for k in range(K):
            oracle.run_rounds(oracle.LINEAR, X[k * N0:(k + 1) * N0], y[k * N0:(k + 1) * N0], th, T, n, alpha,
                              seed=100 + k, fixed_partition=True)
            ends.append(th.copy())
    got = np.concatenate(ends)
    assert np.linalg.norm(got - stable) <= 1e-10 * np.linalg.norm(stable)


# ------------------------------------------------------------------ P5: Theorem 1 / Theorem 2 trends

def test_contracts_below_and_diverges_above_two_over_lambda1():
    X, y = linear_data(8, 300, 5)
    lam1 = np.linalg.eigvalsh(X.T @ X / 300).max()
    ols = np.linalg.lstsq(X, y, rcond=None)[0]
    good = np.zeros(5); bad = np.zeros(5)
    oracle.run_rounds(oracle.LINEAR, X, y, good, 200, 300, 1.9 / lam1, seed=0)
    oracle.run_rounds(oracle.LINEAR, X, y, bad, 200, 300, 2.1 / lam1, seed=0)
    assert np.linalg.norm(good - ols) < 1e-3
    assert np.linalg.norm(bad - ols) > 1e3


def test_distance_to_ols_grows_with_alpha_T():
    """Theorem 2: the stable solution sits within c*alpha*T of OLS, so halving alpha*T should shrink the gap."""
    K, N0, n, p = 4, 200, 50, 5
    X, y = linear_data(9, K * N0, p)
    ols = np.linalg.lstsq(X, y, rcond=None)[0]
    gaps = []
    for alpha in (0.08, 0.04, 0.02):
        th = np.zeros(p)
        for r in range(600):
            for k in range(K):
                oracle.run_rounds(oracle.LINEAR, X[k * N0:(k + 1) * N0], y[k * N0:(k + 1) * N0], th, 5, n, alpha,
                                  seed=k, fixed_partition=True)
        gaps.append(np.linalg.norm(th - ols))
    assert gaps[0] > gaps[1] > gaps[2]
    assert gaps[2] < 0.45 * gaps[0]


# ------------------------------------------------------------------ P6: tiny-N brute force

def test_tiny_buffer_matches_one_of_the_enumerated_partitions():
    """N0 = 4, n = 2: the oracle's result equals hand enumeration for the ordered partition its shuffle induces,
    and differs from the results of the other partitions."""
    X = np.array([[1.0, 2.0], [0.5, -1.0], [-2.0, 0.25], [3.0, 1.5]])
    y = np.array([1.0, -0.5, 2.0, 0.75])
    alpha = 0.1

    def run(order_per_round):
        th = np.zeros(2)
        for order in order_per_round:
            for pair in (order[:2], order[2:]):
                g = np.zeros(2)
                for i in pair:
                    g += (X[i] @ th - y[i]) * X[i]
                th = th - alpha / 2 * g
        return th

    for seed in range(12):
        th = np.zeros(2)
        oracle.run_rounds(oracle.LINEAR, X, y, th, 2, 2, alpha, seed=seed)
        orders = [tuple(int(v) for v in oracle.perm(seed, 0, t, 4)) for t in range(2)]
        assert np.allclose(th, run(orders), rtol=1e-14, atol=0)
        # the set of all results over ordered partitions contains it; batches are unordered sets
        close = 0
        for o0 in itertools.permutations(range(4)):
            for o1 in itertools.permutations(range(4)):
                if np.allclose(th, run([o0, o1]), rtol=1e-13, atol=0):
                    close += 1
                    assert {frozenset(o0[:2]), frozenset(o0[2:])} == {frozenset(orders[0][:2]), frozenset(orders[0][2:])}
                    assert o0[:2] in (orders[0][:2], orders[0][:2][::-1])
        assert close == 16  # order inside each of the four mini-batches does not matter: 2^4


def test_ragged_last_minibatch_is_averaged_by_its_own_size():
    X, y = linear_data(10, 5, 2)
    th = np.zeros(2)
    oracle.run_rounds(oracle.LINEAR, X, y, th, 1, 2, 0.1, seed=3)
    want = np.zeros(2)
    for b in batches_of(3, 0, 0, 5, 2):
        assert len(b) in (1, 2)
        want = want - 0.1 / len(b) * X[b].T @ (X[b] @ want - y[b])
    assert [len(b) for b in batches_of(3, 0, 0, 5, 2)] == [2, 2, 1]
    assert np.allclose(th, want, rtol=1e-14, atol=0)


# ------------------------------------------------------------------ P7: logistic

def neg_loglik(X, y, th):
    u = X @ th
    return np.mean(np.logaddexp(0, u) - y * u)


def test_logistic_step_is_minus_alpha_times_finite_difference_gradient():
    """Section 3.2.3: the gradient is -mean{(y - sigmoid(x.theta)) x}; checked by central differences of the loss."""
    X, y = logistic_data(11, 80, 5)
    th0 = np.array([0.3, -0.2, 0.1, 0.5, -0.4])
    th = th0.copy()
    oracle.run_rounds(oracle.LOGISTIC, X, y, th, 1, 80, 0.5, seed=1)
    g = np.zeros(5)
    h = 1e-6
    for j in range(5):
        e = np.zeros(5); e[j] = h
        g[j] = (neg_loglik(X, y, th0 + e) - neg_loglik(X, y, th0 - e)) / (2 * h)
    assert np.allclose(th, th0 - 0.5 * g, rtol=0, atol=1e-9)


def test_logistic_full_batch_converges_to_newton_mle():
    X, y = logistic_data(12, 400, 4)
    mle = np.zeros(4)
    for _ in range(50):
        mu = 1 / (1 + np.exp(-X @ mle))
        H = (X * (mu * (1 - mu))[:, None]).T @ X
        mle = mle + np.linalg.solve(H, X.T @ (y - mu))
    th = np.zeros(4)
    oracle.run_rounds(oracle.LOGISTIC, X, y, th, 4000, 400, 1.0, seed=0)
    assert np.linalg.norm(th - mle) <= 1e-9 * max(1.0, np.linalg.norm(mle))


def test_logistic_minibatch_trajectory_against_numpy_loop():
    X, y = logistic_data(13, 130, 6)
    th = np.zeros(6)
    tr = oracle.run_rounds(oracle.LOGISTIC, X, y, th, 2, 32, 0.5, seed=21, chain=1, trace=True)
    want = np.zeros(6)
    s = 0
    for t in range(2):
        for b in batches_of(21, 1, t, 130, 32):
            want = want - 0.5 / len(b) * X[b].T @ (1 / (1 + np.exp(-X[b] @ want)) - y[b])
            assert np.allclose(tr[s], want, rtol=1e-12, atol=1e-15)
            s += 1


def test_logistic_sigmoid_is_stable_for_large_arguments():
    X = np.array([[800.0], [-800.0]])
    y = np.array([1.0, 0.0])
    th = np.array([1.0])
    oracle.run_rounds(oracle.LOGISTIC, X, y, th, 1, 2, 0.1, seed=0)
    assert np.isfinite(th).all() and abs(th[0] - 1.0) < 1e-12


# ------------------------------------------------------------------ P8: softmax

def softmax_loss(X, lab, W):
    Z = X @ W
    Z = Z - Z.max(axis=1, keepdims=True)
    return np.mean(np.log(np.exp(Z).sum(axis=1)) - Z[np.arange(len(lab)), lab])


def test_softmax_step_is_minus_alpha_times_finite_difference_gradient():
    rng = np.random.default_rng(14)
    X = rng.standard_normal((60, 4)); lab = rng.integers(0, 3, 60).astype(np.int32)
    W0 = 0.3 * rng.standard_normal((4, 3))
    W = W0.copy()
    oracle.run_rounds(oracle.SOFTMAX, X, lab, W, 1, 60, 0.2, seed=2, C=3)
    G = np.zeros_like(W0)
    h = 1e-6
    for j in range(4):
        for c in range(3):
            E = np.zeros_like(W0); E[j, c] = h
            G[j, c] = (softmax_loss(X, lab, W0 + E) - softmax_loss(X, lab, W0 - E)) / (2 * h)
    assert np.allclose(W, W0 - 0.2 * G, rtol=0, atol=1e-9)


def test_two_class_softmax_is_logistic_with_doubled_rate():
    """With C = 2, w_1 - w_0 follows the logistic chain run at 2*alpha on the same partition (exact identity)."""
    X, y = logistic_data(15, 150, 5)
    lab = y.astype(np.int32)
    W = np.zeros((5, 2))
    oracle.run_rounds(oracle.SOFTMAX, X, lab, W, 3, 25, 0.1, seed=8, C=2)
    th = np.zeros(5)
    oracle.run_rounds(oracle.LOGISTIC, X, y, th, 3, 25, 0.2, seed=8)
    assert np.linalg.norm((W[:, 1] - W[:, 0]) - th) <= 1e-12 * np.linalg.norm(th)
    assert np.abs(W[:, 1] + W[:, 0]).max() <= 1e-14  # the two columns move symmetrically from zero


def test_softmax_minibatch_trajectory_against_numpy_loop():
    rng = np.random.default_rng(16)
    X = rng.standard_normal((90, 6)); lab = rng.integers(0, 4, 90).astype(np.int32)
    W = np.zeros((6, 4))
    oracle.run_rounds(oracle.SOFTMAX, X, lab, W, 2, 16, 0.3, seed=4, C=4)
    want = np.zeros((6, 4))
    for t in range(2):
        for b in batches_of(4, 0, t, 90, 16):
            Z = X[b] @ want
            P = np.exp(Z - Z.max(axis=1, keepdims=True)); P /= P.sum(axis=1, keepdims=True)
            P[np.arange(len(b)), lab[b]] -= 1
            want = want - 0.3 / len(b) * X[b].T @ P
    assert np.allclose(W, want, rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------ P10 and storage

def test_summation_order_inside_a_minibatch_only_changes_rounding():
    X, y = linear_data(17, 300, 9)
    th = np.zeros(9)
    oracle.run_rounds(oracle.LINEAR, X, y, th, 2, 50, 0.05, seed=6)
    want = np.zeros(9)
    for t in range(2):
        for b in batches_of(6, 0, t, 300, 50):
            b = np.sort(b)
            want = want - 0.05 / len(b) * X[b].T @ (X[b] @ want - y[b])
    assert np.linalg.norm(th - want) <= 1e-13 * np.linalg.norm(want)


def test_stored_fp32_and_bf16_inputs_are_widened_exactly():
    import torch
    X, y = linear_data(18, 64, 8)
    X32 = X.astype(np.float32); y32 = y.astype(np.float32)
    a = np.zeros(8); b = np.zeros(8)
    oracle.run_rounds(oracle.LINEAR, X32, y32, a, 2, 16, 0.05, seed=1)
    oracle.run_rounds(oracle.LINEAR, X32.astype(np.float64), y32.astype(np.float64), b, 2, 16, 0.05, seed=1)
    assert np.array_equal(a, b)
    Xb = torch.from_numpy(X32).to(torch.bfloat16)
    lab = (y > 0).astype(np.int32)
    Wa = np.zeros((8, 2)); Wb = np.zeros((8, 2))
    oracle.run_rounds(oracle.SOFTMAX, Xb, lab, Wa, 1, 16, 0.1, seed=1, C=2)
    oracle.run_rounds(oracle.SOFTMAX, Xb.to(torch.float64).numpy(), lab, Wb, 1, 16, 0.1, seed=1, C=2)
    assert np.array_equal(Wa, Wb)


def test_thread_count_does_not_change_the_result():
    X, y = logistic_data(19, 500, 12)
    a = np.zeros(12); b = np.zeros(12)
    n0 = oracle.num_threads()
    oracle.set_num_threads(1)
    oracle.run_rounds(oracle.LOGISTIC, X, y, a, 2, 64, 0.5, seed=3)
    oracle.set_num_threads(max(2, n0))
    oracle.run_rounds(oracle.LOGISTIC, X, y, b, 2, 64, 0.5, seed=3)
    oracle.set_num_threads(n0)
    assert np.array_equal(a, b)


def test_chains_share_data_but_not_partitions():
    X, y = linear_data(20, 200, 4)
    a = np.zeros(4); b = np.zeros(4); c = np.zeros(4)
    oracle.run_rounds(oracle.LINEAR, X, y, a, 1, 20, 0.1, seed=1, chain=0)
    oracle.run_rounds(oracle.LINEAR, X, y, b, 1, 20, 0.1, seed=1, chain=1)
    oracle.run_rounds(oracle.LINEAR, X, y, c, 1, 20, 0.1, seed=1, chain=1)
    assert not np.allclose(a, b) and np.array_equal(b, c)
