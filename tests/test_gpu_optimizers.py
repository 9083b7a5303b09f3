"""Parity of the buffered Nesterov and Adam updates and of the cosine learning rate with the CPU oracle
(Sections 4.2-4.4 of the paper), through the C ABI.  Tolerances as for the plain update: relative L2 error of
theta at most 1e-10 in fp64 and 1e-4 in fp32.
"""
import numpy as np
import pytest

import oracle
from paper_2312_08728_b200 import binding
from paper_2312_08728_b200.inputs import WORKLOADS, Workload, LOSS_LINEAR, LOSS_LOGISTIC, DTYPE_F32, DTYPE_F64

from helpers import TOL, buffers_of, gpu_job, oracle_job, rel_l2

pytestmark = pytest.mark.gpu

NAG = dict(kind=oracle.OPT_NESTEROV, a=0.9)
ADAM = dict(kind=oracle.OPT_ADAM, a=0.9, b=0.999, eps=1e-7)   # the defaults of Section 4.2's framework


def check(w, opt, mode="resident", **shape):
    bufs = buffers_of(w)
    theta, stats = gpu_job(w, bufs, mode=mode, opt=opt, **shape)
    want = oracle_job(w, bufs, opt=opt)
    for c, th in want.items():
        err = rel_l2(theta[c], th)
        assert err <= TOL[w.dtype], (w.name, opt, c, err, stats)
    return theta, want


def test_constants_agree():
    assert (binding.OPT_SGD, binding.OPT_NESTEROV, binding.OPT_ADAM) == (oracle.OPT_SGD, oracle.OPT_NESTEROV, oracle.OPT_ADAM)
    assert (binding.LR_CONSTANT, binding.LR_COSINE) == (oracle.LR_CONSTANT, oracle.LR_COSINE)


@pytest.mark.parametrize("opt", [NAG, ADAM], ids=["nesterov", "adam"])
def test_fp64_job_with_state_carried_over_buffers_and_passes(opt):
    w = WORKLOADS["cfg1"].scaled(lr=0.01 if opt is NAG else 0.001)
    theta, want = check(w, opt, mode="slots")
    # the rule really ran: the result differs from the plain update's
    plain = oracle_job(w, buffers_of(w))
    assert rel_l2(theta[0], plain[0]) > 1e-3


@pytest.mark.parametrize("opt", [NAG, ADAM], ids=["nesterov", "adam"])
def test_fp32_logistic_across_clusters_with_a_ragged_last_batch(opt):
    w = WORKLOADS["cfg3"].scaled(N=100_000, K=2, T=2, epochs=1, lr=0.05 if opt is NAG else 0.001)
    assert w.N0 % w.n != 0
    check(w, opt)


@pytest.mark.parametrize("opt", [NAG, ADAM], ids=["nesterov", "adam"])
def test_fp32_linear_chains(opt):
    w = WORKLOADS["cfg2"].scaled(N=60_000, K=3, T=2, epochs=2, Rc=8, lr=0.001)
    check(w, opt)


@pytest.mark.parametrize("shape", [dict(cluster_size=1, ctas_per_chain=1), dict(cluster_size=4, ctas_per_chain=4),
                                   dict(cluster_size=1, ctas_per_chain=3), dict(cluster_size=8, ctas_per_chain=24)])
def test_adam_on_every_exchange_path(shape):
    w = Workload("adam-small", LOSS_LOGISTIC, DTYPE_F32, N=6_000, p=40, K=2, n=500, T=2, lr=0.002, epochs=1, seed=3)
    check(w, ADAM, **shape)


def test_cosine_rate_over_two_passes():
    """Section 4.4: alpha_j = lr (1/2 + 1/2 cos(j pi / TMK)), again in every pass; here with the plain update and with
    Nesterov momentum, the count running on from call to call."""
    w = WORKLOADS["cfg1"].scaled(epochs=2)
    M = -(-w.N0 // w.n)
    J = w.T * M * w.K
    for base in (dict(kind=oracle.OPT_SGD), NAG):
        opt = dict(base, sched=oracle.LR_COSINE, period=J)
        theta, want = check(w.scaled(lr=0.02), opt, mode="slots")
    w32 = Workload("cos32", LOSS_LINEAR, DTYPE_F32, N=30_000, p=64, K=3, n=1_000, T=2, lr=0.05, epochs=2, rho=0.5, seed=5)
    check(w32, dict(kind=oracle.OPT_SGD, sched=oracle.LR_COSINE, period=2 * 10 * 3))


def test_wide_rows_and_resetting_the_rule():
    w = Workload("adam-wide", LOSS_LINEAR, DTYPE_F32, N=8_000, p=500, K=2, n=400, T=2, lr=0.001, epochs=1, rho=0.8, seed=8)
    check(w, ADAM)
    # setting the rule again zeroes its state: two identical jobs on one handle give identical results
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS
    s = WORKLOADS["cfg1"].scaled(N=4_000, K=2, epochs=1, lr=0.001)
    bufs = [(x.cuda(), y.cuda()) for x, y in buffers_of(s)]
    out = []
    with Bmgd(s.N, s.p, s.K, loss=s.loss, dtype=s.dtype, flags=FLAG_NO_SLOTS) as h:
        for _ in range(2):
            h.set_theta(np.zeros(s.p))
            h.set_optimizer(binding.OPT_ADAM, 0.9, 0.999, 1e-7)
            for k, (x, y) in enumerate(bufs):
                h.run_rounds_resident(x, y, s.T, s.n, s.lr, 100 + k)
            out.append(h.get_theta())
    assert np.array_equal(out[0], out[1])


def test_bad_rules_are_refused():
    from paper_2312_08728_b200.binding import Bmgd, BmgdError, FLAG_NO_SLOTS
    with Bmgd(1000, 8, 1, flags=FLAG_NO_SLOTS) as h:
        for args in [(7, 0, 0, 0), (binding.OPT_NESTEROV, 1.0, 0, 0), (binding.OPT_ADAM, 0.9, 0.999, 0.0)]:
            with pytest.raises(BmgdError):
                h.set_optimizer(*args)
        with pytest.raises(BmgdError):
            h.set_lr_schedule(binding.LR_COSINE, 0)
