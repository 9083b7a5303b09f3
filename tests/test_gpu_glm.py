"""Parity of the fused least-squares / logistic step kernel with the CPU oracle, through the C ABI.

Tolerances are the stated ones: relative L2 error of theta at most 1e-10 in fp64 and 1e-4 in fp32.
"""
import numpy as np
import pytest
import torch

from paper_2312_08728_b200 import inputs
from paper_2312_08728_b200.inputs import WORKLOADS, Workload, LOSS_LINEAR, LOSS_LOGISTIC, DTYPE_F32, DTYPE_F64

from helpers import TOL, buffers_of, gpu_job, oracle_job, rel_l2

pytestmark = pytest.mark.gpu


def check(w, buffers, chains=None, mode="slots", flags=0, **shape):
    theta, stats = gpu_job(w, buffers, mode=mode, flags=flags, **shape)
    want = oracle_job(w, buffers, chains=chains)
    worst = 0.0
    for c, th in want.items():
        err = rel_l2(theta[c], th)
        worst = max(worst, err)
        assert err <= TOL[w.dtype], (w.name, c, err, stats)
    return theta, stats, worst


def test_cfg1_full_job_fp64():
    """Linear fp64, N=10,000, p=10, 5 buffers of 2,000, n=100, T=5, lr=0.05, 2 passes: every step of the job."""
    w = WORKLOADS["cfg1"]
    _, stats, _ = check(w, buffers_of(w))
    assert stats["steps"] == 2 * 5 * 5 * 20
    assert stats["sample_grads"] == 2 * 10_000 * 5


@pytest.mark.parametrize("mode", ["slots", "resident"])
def test_linear_fp32_chains(mode):
    """cfg2's shape scaled down: several tiles per CTA and eight chains sharing the buffer."""
    w = WORKLOADS["cfg2"].scaled(N=60_000, K=3, T=3, epochs=2, Rc=8)
    check(w, buffers_of(w), mode=mode)


def test_logistic_fp32_multi_cluster_ragged():
    """cfg3's shape scaled down: p=200, n=4,096 with a ragged last mini-batch, all clusters on one chain."""
    w = WORKLOADS["cfg3"].scaled(N=100_000, K=2, T=2, epochs=1)
    assert w.N0 % w.n != 0
    _, stats, _ = check(w, buffers_of(w))
    assert stats["ctas_per_chain"] > stats["cluster_size"]  # the cross-cluster exchange ran


def test_linear_fp32_p64_streaming_shape():
    """cfg5's shape scaled down: p=64, n=2,048."""
    w = WORKLOADS["cfg5"].scaled(N=300_000, K=3, T=2)
    check(w, buffers_of(w))


SMALL = Workload("small", LOSS_LOGISTIC, DTYPE_F32, N=6_000, p=40, K=2, n=500, T=2, lr=0.3, epochs=1, seed=3)


@pytest.mark.parametrize("shape", [
    dict(cluster_size=1, ctas_per_chain=1),
    dict(cluster_size=1, ctas_per_chain=4),
    dict(cluster_size=2, ctas_per_chain=2),
    dict(cluster_size=2, ctas_per_chain=12),
    dict(cluster_size=4, ctas_per_chain=4),
    dict(cluster_size=4, ctas_per_chain=40),
    dict(cluster_size=8, ctas_per_chain=8),
    dict(cluster_size=8, ctas_per_chain=64),
    dict(cluster_size=8, ctas_per_chain=8, threads_per_cta=512),
    dict(cluster_size=8, ctas_per_chain=16, pipeline_depth=2),
    dict(cluster_size=8, ctas_per_chain=16, pipeline_depth=3),
    dict(cluster_size=1, ctas_per_chain=1, subpasses_per_stage=1),
    dict(cluster_size=1, ctas_per_chain=1, subpasses_per_stage=4, pipeline_depth=3),
    dict(cluster_size=2, ctas_per_chain=2, subpasses_per_stage=8),
    dict(cluster_size=1, ctas_per_chain=2, subpasses_per_stage=2),
])
def test_launch_shapes_agree_with_the_oracle(shape):
    _, stats, _ = check(SMALL, buffers_of(SMALL), mode="resident", **shape)
    assert stats["cluster_size"] == shape["cluster_size"]
    assert stats["ctas_per_chain"] == shape["ctas_per_chain"]


@pytest.mark.parametrize("shape", [
    dict(cluster_size=1, ctas_per_chain=1, producer_warps=1),
    dict(cluster_size=2, ctas_per_chain=12, producer_warps=2),
    dict(cluster_size=8, ctas_per_chain=8, threads_per_cta=512, producer_warps=3),
    dict(cluster_size=8, ctas_per_chain=8, threads_per_cta=512, producer_warps=1),
    dict(cluster_size=8, ctas_per_chain=16, pipeline_depth=2, subpasses_per_stage=4, producer_warps=2),
    dict(cluster_size=4, ctas_per_chain=4, pipeline_depth=8, subpasses_per_stage=1, producer_warps=1),
    dict(cluster_size=16, ctas_per_chain=32, producer_warps=2),
])
def test_producer_warp_counts_and_ring_depths_agree_with_the_oracle(shape):
    """Rows are fetched by dedicated warps: any number of them, and any ring depth, must give the same theta."""
    check(SMALL, buffers_of(SMALL), mode="resident", **shape)
    w = WORKLOADS["cfg1"].scaled(N=4_000, K=2, epochs=1)
    check(w, buffers_of(w), mode="slots", producer_warps=shape["producer_warps"])


def test_producer_warps_ragged_batches_and_chains():
    w = WORKLOADS["cfg3"].scaled(N=100_000, K=2, T=2, epochs=1)
    check(w, buffers_of(w), producer_warps=1)
    w = WORKLOADS["cfg2"].scaled(N=60_000, K=3, T=2, epochs=1, Rc=8)
    check(w, buffers_of(w), mode="resident", producer_warps=3)
    w = Workload("edge", LOSS_LINEAR, DTYPE_F64, N=257, p=6, K=1, n=3, T=2, lr=0.1, epochs=1, rho=0.5, seed=9)
    check(w, buffers_of(w), mode="resident", producer_warps=1)


@pytest.mark.parametrize("dtype,p", [(DTYPE_F32, 500), (DTYPE_F32, 33), (DTYPE_F64, 130), (DTYPE_F64, 7)])
@pytest.mark.parametrize("shape", [
    dict(cluster_size=1, ctas_per_chain=1),                                      # one producer warp per slot of the default ring
    dict(cluster_size=1, ctas_per_chain=1, pipeline_depth=2, producer_warps=4),  # two warps share a slot's batches
    dict(cluster_size=2, ctas_per_chain=4, pipeline_depth=3, producer_warps=1),  # rounded up to one warp per slot
    dict(cluster_size=4, ctas_per_chain=4, pipeline_depth=2, subpasses_per_stage=1, producer_warps=3),
    dict(cluster_size=2, ctas_per_chain=2, pipeline_depth=4, subpasses_per_stage=4),
    dict(cluster_size=1, ctas_per_chain=2, pipeline_depth=8, subpasses_per_stage=1),  # more slots than the small CTA has warps for
    dict(cluster_size=2, ctas_per_chain=2, pipeline_depth=6, subpasses_per_stage=1, producer_warps=8),
])
def test_rows_not_fetched_by_gathers_have_one_producer_warp_per_ring_slot(dtype, p, shape):
    """Rows wider than 256 values (one bulk copy per row) and rows that are not 16-byte multiples (element-wise copies)
    are fetched by producer warps that each serve one ring slot; ring depths, warps per slot, chains that take turns on
    a team and a ragged last mini-batch must all give the oracle's theta."""
    w = Workload("slots", LOSS_LOGISTIC, dtype, N=2_300, p=p, K=1, n=300, T=2, lr=0.3, epochs=1, Rc=3, seed=200 + p)
    check(w, buffers_of(w), mode="resident", **shape)


def test_cluster_of_sixteen_if_the_device_allows_it():
    from paper_2312_08728_b200.binding import BmgdError
    try:
        check(SMALL, buffers_of(SMALL), mode="resident", cluster_size=16, ctas_per_chain=16)
    except BmgdError as e:  # non-portable cluster size: allowed to be refused, never to be wrong
        assert e.status in (-7, -3), e


@pytest.mark.parametrize("dtype,p", [(DTYPE_F32, 7), (DTYPE_F32, 33), (DTYPE_F64, 5), (DTYPE_F64, 31),
                                     (DTYPE_F32, 4), (DTYPE_F32, 128), (DTYPE_F32, 132), (DTYPE_F32, 260),
                                     (DTYPE_F32, 500), (DTYPE_F32, 1024), (DTYPE_F64, 130), (DTYPE_F64, 512)])
def test_predictor_counts_including_unaligned_rows(dtype, p):
    """Rows that are not 16-byte multiples take the element-wise copy path; every lane/chunk variant is reached."""
    w = Workload("pvar", LOSS_LINEAR, dtype, N=1_500, p=p, K=1, n=128, T=2, lr=0.5 / p, epochs=1, rho=0.3, seed=p)
    check(w, buffers_of(w), mode="resident")


@pytest.mark.parametrize("dtype,p,lanes", [(DTYPE_F32, 40, 4), (DTYPE_F32, 64, 4), (DTYPE_F32, 64, 8), (DTYPE_F32, 100, 4),
                                           (DTYPE_F32, 100, 8), (DTYPE_F32, 112, 0), (DTYPE_F64, 20, 4), (DTYPE_F64, 56, 4),
                                           (DTYPE_F64, 56, 8), (DTYPE_F32, 300, 4)])
def test_lanes_per_row_variants(dtype, p, lanes):
    """Row sizes that have kernels with four and with eight lanes per row give the same theta either way (a row size
    without the asked-for kernel falls back to the default one); chains and a ragged last mini-batch included."""
    w = Workload("lanes", LOSS_LOGISTIC, dtype, N=3_100, p=p, K=1, n=500, T=2, lr=0.3, epochs=1, Rc=3, seed=100 + p)
    check(w, buffers_of(w), mode="resident", lanes_per_row=lanes)
    check(w, buffers_of(w), mode="resident", lanes_per_row=lanes, cluster_size=4, ctas_per_chain=8)


@pytest.mark.parametrize("N0,n", [(1, 1), (7, 1), (7, 7), (7, 100), (33, 32), (1000, 999), (1000, 1000), (257, 3)])
def test_degenerate_sizes(N0, n):
    """One row, one-row mini-batches, a full-batch round, a batch larger than the buffer, a one-row tail."""
    w = Workload("edge", LOSS_LINEAR, DTYPE_F64, N=N0, p=6, K=1, n=n, T=3, lr=0.1, epochs=1, rho=0.5, seed=N0 + n)
    check(w, buffers_of(w), mode="resident")
    check(w, buffers_of(w), mode="resident", cluster_size=4, ctas_per_chain=8)


def test_zero_rounds_is_a_no_op_and_runs_are_bitwise_reproducible():
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS
    w = SMALL
    X, y = [t.cuda() for t in inputs.make_buffer(w, 0)]
    outs = []
    for rep in range(3):
        with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, flags=FLAG_NO_SLOTS) as h:
            h.run_rounds_resident(X, y, 0, w.n, w.lr, 1)
            assert not h.get_theta().any()
            h.run_rounds_resident(X, y, 3, w.n, w.lr, 1)
            outs.append(h.get_theta())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


def test_resume_from_saved_theta():
    """theta handed from call to call equals theta saved, restored into a new handle and continued."""
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS
    w = SMALL
    bufs = [tuple(t.cuda() for t in inputs.make_buffer(w, k)) for k in range(2)]
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, flags=FLAG_NO_SLOTS) as h:
        h.run_rounds_resident(*bufs[0], w.T, w.n, w.lr, 10)
        mid = h.get_theta()
        h.run_rounds_resident(*bufs[1], w.T, w.n, w.lr, 11)
        end = h.get_theta()
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, flags=FLAG_NO_SLOTS) as h2:
        h2.set_theta(mid)
        h2.run_rounds_resident(*bufs[1], w.T, w.n, w.lr, 11)
        assert np.array_equal(h2.get_theta(), end)


def test_fixed_partition_flag():
    from paper_2312_08728_b200.binding import FLAG_FIXED_PARTITION
    w = Workload("fixed", LOSS_LINEAR, DTYPE_F64, N=900, p=8, K=1, n=100, T=4, lr=0.1, epochs=1, rho=0.5, seed=5)
    bufs = buffers_of(w)
    theta, _ = gpu_job(w, bufs, mode="resident", flags=FLAG_FIXED_PARTITION)
    want = oracle_job(w, bufs, fixed_partition=True)[0]
    assert rel_l2(theta[0], want) <= 1e-10
    assert rel_l2(theta[0], oracle_job(w, bufs)[0]) > 1e-8  # and it is not the fresh-partition result


def test_errors_surface_as_codes():
    from paper_2312_08728_b200.binding import Bmgd, BmgdError, ERR_CAPACITY, ERR_STATE, ERR_ARG, ERR_NONFINITE
    w = SMALL.scaled(loss=LOSS_LINEAR)
    X, y = inputs.make_buffer(w, 0)
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype) as h:
        with pytest.raises(BmgdError) as e:
            h.run_rounds(0, 1, 10, 0.1, 0)
        assert e.value.status == ERR_STATE
        big = torch.zeros(w.N0 + 1, w.p), torch.zeros(w.N0 + 1)
        with pytest.raises(BmgdError) as e:
            h.load_buffer(*big)
        assert e.value.status == ERR_CAPACITY
        with pytest.raises(BmgdError) as e:
            h.run_rounds(5, 1, 10, 0.1, 0)
        assert e.value.status == ERR_ARG
        slot = h.load_buffer(X.pin_memory(), y.pin_memory())
        h.run_rounds(slot, 2, w.n, 1e9, 0)  # absurd learning rate: theta blows up
        with pytest.raises(BmgdError) as e:
            h.get_theta()
        assert e.value.status == ERR_NONFINITE


@pytest.mark.parametrize("chains", [[0, 31, 63]])
def test_cfg2_full_buffer_in_the_benchmarked_launch_shape(chains):
    """One full cfg2 buffer (100,000 x 100, n=1,000, T=10) with all 64 chains in one launch, default shape:
    three sampled chains against the oracle."""
    w = WORKLOADS["cfg2"].scaled(N=100_000, K=1, epochs=1)
    bufs = buffers_of(w)
    theta, stats = gpu_job(w, bufs, mode="resident")
    want = oracle_job(w, bufs, chains=chains)
    for c in chains:
        assert rel_l2(theta[c], want[c]) <= 1e-4, (c, stats)
    assert stats["sample_grads"] == 64 * 10 * 100_000
    # chains differ (distinct partitions) but all sit near the least-squares solution
    assert np.abs(theta - 1.0).max() < 0.2 and np.unique(theta[:, 0]).size == 64


def test_cfg3_one_full_buffer_default_shape():
    """One full cfg3 buffer (1,000,000 x 200 logistic, n=4,096, 245 steps per round), two rounds."""
    w = WORKLOADS["cfg3"].scaled(N=1_000_000, K=1, T=2, epochs=1)
    check(w, buffers_of(w), mode="resident")


def test_cfg5_one_full_buffer_default_shape():
    """One full cfg5 buffer (2,500,000 x 64, n=2,048: 1,221 steps per round with a ragged last one), through a slot."""
    w = WORKLOADS["cfg5"].scaled(N=2_500_000, K=1, T=2, epochs=1)
    _, stats, _ = check(w, buffers_of(w), mode="slots")
    assert stats["steps"] == 2 * 1221


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    """Failure detection without a GPU fault: a bounded wait gives up after its budget, the status word carries
    BMGD_ERR_TIMEOUT to the next synchronising call, and the same handle then computes correctly."""
    import time
    from paper_2312_08728_b200.binding import Bmgd, BmgdError, ERR_TIMEOUT, FLAG_NO_SLOTS
    w = SMALL
    bufs = buffers_of(w)
    X, y = [t.cuda() for t in bufs[0]]
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, flags=FLAG_NO_SLOTS) as h:
        t0 = time.perf_counter()
        h.debug_wait_timeout(50.0)
        with pytest.raises(BmgdError) as e:
            h.sync()
        assert e.value.status == ERR_TIMEOUT
        assert 0.04 <= time.perf_counter() - t0 < 5.0
        h.sync()  # reported once, then cleared
        h.run_rounds_resident(X, y, w.T, w.n, w.lr, inputs.buffer_seed(w.seed, 0, 0, w.K))
        theta = h.get_theta()
    want = oracle_job(w.scaled(K=1, N=w.N0), bufs[:1])[0]
    assert rel_l2(theta[0], want) <= 1e-4


@pytest.mark.parametrize("shape", [
    dict(cluster_size=4, ctas_per_chain=4),    # packets inside one cluster
    dict(cluster_size=2, ctas_per_chain=8),    # packets between clusters too
    dict(cluster_size=1, ctas_per_chain=1),    # only the ring's mbarriers to wait on
])
def test_a_step_kernel_wait_that_runs_out_ends_the_launch_and_the_handle_stays_usable(shape):
    """The step kernel's own waits with a budget of a nanosecond: the first wait that does not succeed at its first
    look gives up, every CTA leaves its loops (no copy left in flight, theta not written back), the next
    synchronising call reports BMGD_ERR_TIMEOUT once, and the same handle, given a sane budget, computes correctly.
    A wait that gives up is not a fault: nothing traps, hangs or touches memory out of bounds."""
    from paper_2312_08728_b200.binding import Bmgd, BmgdError, ERR_TIMEOUT, FLAG_NO_SLOTS
    w = SMALL.scaled(T=40)  # 480 steps: were the launch to run on after giving up, it would still end, only later
    bufs = buffers_of(w)
    X, y = [t.cuda() for t in bufs[0]]
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, flags=FLAG_NO_SLOTS, timeout_ms=1e-6, **shape) as h:
        start = np.full((1, w.p), 0.25, dtype=np.float32)
        h.set_theta(start)
        h.run_rounds_resident(X, y, w.T, w.n, w.lr, 5)
        with pytest.raises(BmgdError) as e:
            h.sync()
        assert e.value.status == ERR_TIMEOUT
        h.sync()  # reported once, then cleared
        assert np.array_equal(h.get_theta(), start)  # the abandoned launch did not write theta back
        h.set_timeout(0.0)  # back to the default budget
        h.set_theta(np.zeros((1, w.p), dtype=np.float32))
        h.run_rounds_resident(X, y, 2, w.n, w.lr, inputs.buffer_seed(w.seed, 0, 0, w.K))
        theta = h.get_theta()
    want = oracle_job(w.scaled(K=1, N=w.N0, T=2), bufs[:1])[0]
    assert rel_l2(theta[0], want) <= 1e-4


@pytest.mark.parametrize("opt", [None, "adam"])
@pytest.mark.parametrize("shape", [dict(cluster_size=1), dict(cluster_size=4)])
def test_more_chains_than_resident_teams(shape, opt):
    """Rc = 200 chains on at most 148 SMs: teams take chain after chain inside one launch, the producer warps run
    on across chain boundaries, theta and the update rule's state are reloaded per chain.  Every chain against
    the oracle."""
    import oracle
    w = Workload("many-chains", LOSS_LINEAR, DTYPE_F32, N=6_000, p=24, K=1, n=500, T=2, lr=0.1, epochs=1, Rc=200,
                 rho=0.5, seed=77)
    bufs = buffers_of(w)
    o = None if opt is None else dict(kind=oracle.OPT_ADAM, a=0.9, b=0.999, eps=1e-8)
    if o:
        w = w.scaled(lr=0.01)
    theta, stats = gpu_job(w, bufs, mode="resident", opt=o, **shape)
    assert stats["chains_in_flight"] < w.Rc, stats  # some team really worked on more than one chain
    want = oracle_job(w, bufs, opt=o)
    for c in range(w.Rc):
        assert rel_l2(theta[c], want[c]) <= 1e-4, (c, stats)
    assert np.unique(theta[:, 0]).size == w.Rc


def test_null_rounds_probe_changes_nothing():
    """The latency probe runs the step kernel's waits, exchanges and updates without rows: theta, the update
    rule's state and the step counters stay as they are, and the handle then computes as if it had not run."""
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS, FLAG_TIMING
    import oracle
    w = SMALL
    bufs = buffers_of(w)
    X, y = [t.cuda() for t in bufs[0]]
    for shape in (dict(), dict(cluster_size=2, ctas_per_chain=8)):
        with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, flags=FLAG_NO_SLOTS | FLAG_TIMING, **shape) as h:
            h.set_optimizer(oracle.OPT_NESTEROV, 0.9)
            h.run_rounds_resident(X, y, 1, w.n, w.lr, 3)
            before, s0 = h.get_theta(), h.get_stats()
            h.debug_null_rounds(X.shape[0], 5, w.n)
            after, s1 = h.get_theta(), h.get_stats()
            assert np.array_equal(before, after)
            assert s1["launches"] == s0["launches"] + 1 and s1["steps"] == s0["steps"]
            assert s1["kernel_ms"] > s0["kernel_ms"]
            h.run_rounds_resident(X, y, 1, w.n, w.lr, 4)
            got = h.get_theta()
        with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, flags=FLAG_NO_SLOTS, **shape) as h:
            h.set_optimizer(oracle.OPT_NESTEROV, 0.9)
            h.run_rounds_resident(X, y, 1, w.n, w.lr, 3)
            h.run_rounds_resident(X, y, 1, w.n, w.lr, 4)
            assert np.array_equal(h.get_theta(), got)


def test_algorithm_1_with_a_fresh_partition_of_the_sample_every_pass():
    """All of Algorithm 1: every pass re-partitions the sample into K buffers (host gather into pinned staging
    buffers, two in flight), every round re-partitions the buffer, theta is carried throughout."""
    import oracle
    from paper_2312_08728_b200.binding import Bmgd, PARTITION_CHAIN, gather_buffer
    from helpers import ORACLE_LOSS
    w = Workload("alg1", LOSS_LOGISTIC, DTYPE_F32, N=30_011, p=48, K=4, n=512, T=2, lr=0.3, epochs=3, seed=21)
    X, y = inputs.make_rows(w, 0, w.N)
    part_seed = 4242
    N0 = w.N0
    stage = [(torch.empty(N0, w.p).pin_memory(), torch.empty(N0).pin_memory()) for _ in range(2)]
    copy = torch.cuda.Stream()
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype) as h:
        order = [(e, k) for e in range(w.epochs) for k in range(w.K)]
        def stage_and_load(i):
            e, k = order[i]
            sx, sy = stage[i % 2]
            rows = gather_buffer(X, y, w.K, part_seed, e, k, sx, sy)
            return h.load_buffer(sx[:rows], sy[:rows], stream=copy)
        slot = stage_and_load(0)
        for i, (e, k) in enumerate(order):
            h.run_rounds(slot, w.T, w.n, w.lr, inputs.buffer_seed(w.seed, e, k, w.K))
            if i + 1 < len(order):
                copy.synchronize()  # the staging buffer about to be refilled must have left the host
                slot = stage_and_load(i + 1)
        theta = h.get_theta()[0]
    th = np.zeros(w.p)
    for e in range(w.epochs):
        part = oracle.perm(part_seed, PARTITION_CHAIN, e, w.N).astype(np.int64)
        for k in range(w.K):
            rows = torch.from_numpy(part[k * N0:(k + 1) * N0])
            oracle.run_rounds(ORACLE_LOSS[w.loss], X[rows].contiguous(), y[rows].contiguous(), th, w.T, w.n, w.lr,
                              inputs.buffer_seed(w.seed, e, k, w.K))
    assert rel_l2(theta, th) <= 1e-4
