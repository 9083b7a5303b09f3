"""The allocation-free entry point against the handle-based one.

bmgd_run_rounds_noalloc serves callers that cannot allocate device memory at the point where they
call the library (a process with a fixed device-memory budget, a plugin whose host framework owns
the allocator).  Its scratch is a fixed array inside the library, shared by all calls and never
cleared between them by anyone but the call itself, so the check is made on two calls in a row:
the second one starts from whatever the first one left in that array.

This file is collected last on purpose, so that a run that stops at the first failure has already
been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2312_08728_b200 import inputs
from paper_2312_08728_b200.inputs import Workload, LOSS_LINEAR, LOSS_LOGISTIC, DTYPE_F32, DTYPE_F64

import oracle
from helpers import ORACLE_LOSS, TOL, rel_l2

pytestmark = pytest.mark.gpu

JOBS = [
    # p=200, n=4096: default shape spreads one chain over many clusters, so the packet scratch is really used
    Workload("noalloc-logistic", LOSS_LOGISTIC, DTYPE_F32, N=60_000, p=200, K=2, n=4_096, T=2, lr=0.5, epochs=1, seed=11),
    Workload("noalloc-linear-chains", LOSS_LINEAR, DTYPE_F64, N=8_000, p=10, K=2, n=100, T=2, lr=0.05, epochs=1,
             Rc=3, rho=0.5, seed=12),
    # more chains than the GPU has SMs: teams take several chains one after the other inside the launch
    Workload("noalloc-many-chains", LOSS_LINEAR, DTYPE_F32, N=6_000, p=24, K=2, n=500, T=2, lr=0.1, epochs=1,
             Rc=200, rho=0.5, seed=13),
]


@pytest.mark.parametrize("w", JOBS, ids=lambda w: w.name)
def test_noalloc_matches_the_oracle_and_the_handle_path_on_two_calls_in_a_row(w):
    """Two calls in a row, theta carried from the first to the second in the caller's own tensor: after each call
    every chain agrees with the CPU oracle (the independent check) and with the handle-based entry point (same
    kernels, so bit for bit)."""
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS, run_rounds_noalloc
    host = [inputs.make_buffer(w, k) for k in range(2)]
    bufs = [tuple(t.cuda() for t in b) for b in host]
    seeds = [inputs.buffer_seed(w.seed, 0, k, 2) for k in range(2)]

    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, Rc=w.Rc, flags=FLAG_NO_SLOTS) as h:
        handle = []
        for (x, y), s in zip(bufs, seeds):
            h.run_rounds_resident(x, y, w.T, w.n, w.lr, s)
            handle.append(h.get_theta())
        shape = h.get_stats()

    chains = range(w.Rc) if w.Rc <= 8 else [0, 1, w.Rc // 2, w.Rc - 2, w.Rc - 1]
    oracle_theta = {c: np.zeros(w.p) for c in chains}
    theta = torch.zeros(w.Rc, w.p, dtype=w.theta_dtype, device="cuda")
    torch.cuda.synchronize()
    for k, ((x, y), s) in enumerate(zip(bufs, seeds)):
        run_rounds_noalloc(x, y, theta, w.loss, w.dtype, w.T, w.n, w.lr, s)
        got = theta.cpu().numpy()
        for c in chains:
            oracle.run_rounds(ORACLE_LOSS[w.loss], host[k][0], host[k][1], oracle_theta[c], w.T, w.n, w.lr, s, chain=c)
            assert rel_l2(got[c], oracle_theta[c]) <= TOL[w.dtype], (w.name, k, c, shape)
        assert np.array_equal(got, handle[k]), (w.name, k, shape)
    assert np.isfinite(got).all() and np.abs(got).max() > 0


def test_noalloc_at_the_limit_of_its_scratch_then_a_small_job():
    """fp64 with p = BMGD_NOALLOC_MAX_P and a chain spread over several clusters uses the fixed array up to the
    packets of its last predictor; a call with a small p right after it finds that array full of the first call's
    packets beyond the part it clears, and must not be disturbed by them.  Both against the oracle, twice."""
    from paper_2312_08728_b200.binding import NOALLOC_MAX_P, run_rounds_noalloc
    big = Workload("noalloc-limit", LOSS_LINEAR, DTYPE_F64, N=9_000, p=NOALLOC_MAX_P, K=1, n=3_000, T=2, lr=0.002,
                   epochs=1, rho=0.3, seed=14)
    small = Workload("noalloc-after", LOSS_LOGISTIC, DTYPE_F64, N=9_000, p=12, K=1, n=3_000, T=2, lr=0.3, epochs=1, seed=15)
    for rep in range(2):
        for w in (big, small):
            hx, hy = inputs.make_buffer(w, 0)
            x, y = hx.cuda(), hy.cuda()
            theta = torch.zeros(1, w.p, dtype=w.theta_dtype, device="cuda")
            run_rounds_noalloc(x, y, theta, w.loss, w.dtype, w.T, w.n, w.lr, 100 + rep)
            want = np.zeros(w.p)
            oracle.run_rounds(ORACLE_LOSS[w.loss], hx, hy, want, w.T, w.n, w.lr, 100 + rep)
            assert rel_l2(theta.cpu().numpy()[0], want) <= TOL[w.dtype], (w.name, rep)


def test_noalloc_rejects_what_its_fixed_scratch_cannot_hold():
    from paper_2312_08728_b200.binding import BmgdError, ERR_CAPACITY, ERR_UNIMPLEMENTED, NOALLOC_MAX_P, run_rounds_noalloc
    p = NOALLOC_MAX_P + 4
    x = torch.zeros(64, p, device="cuda")
    y = torch.zeros(64, device="cuda")
    theta = torch.zeros(1, p, device="cuda")
    with pytest.raises(BmgdError) as e:
        run_rounds_noalloc(x, y, theta, LOSS_LINEAR, DTYPE_F32, 1, 16, 0.1, 0)
    assert e.value.status == ERR_CAPACITY
    with pytest.raises(BmgdError) as e:
        run_rounds_noalloc(x[:, :8].contiguous(), y, theta[:, :8].contiguous(), 2, DTYPE_F32, 1, 16, 0.1, 0)
    assert e.value.status == ERR_UNIMPLEMENTED
    assert not theta.any()
