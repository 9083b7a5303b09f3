"""Parity of the softmax step kernel (bf16 rows, fp32 W) with the CPU oracle, through the C ABI.

Stated tolerance: relative L2 error of W at most 2e-2.  The oracle reads the same bf16 rows widened exactly
and computes in fp64; the kernel rounds W and the residuals to bf16 for its two contractions.
Both contraction paths are checked: tensor cores (default) and CUDA cores (same inputs, same layout).
"""
import dataclasses

import numpy as np
import pytest

from paper_2312_08728_b200.inputs import WORKLOADS, Workload, LOSS_SOFTMAX, DTYPE_BF16

from helpers import TOL, buffers_of, gpu_job, oracle_job, rel_l2

pytestmark = pytest.mark.gpu

CUDA_CORES = 8  # BMGD_FLAG_SOFTMAX_CUDA_CORES


def job(p, C=10, N=2_000, K=1, n=256, T=2, lr=0.1, epochs=1, seed=4):
    return Workload(f"smx-p{p}", LOSS_SOFTMAX, DTYPE_BF16, N=N, p=p, K=K, n=n, T=T, lr=lr, epochs=epochs, C=C, seed=seed)


def check(w, flags, mode="resident", tol=None, **shape):
    bufs = buffers_of(w)
    theta, stats = gpu_job(w, bufs, mode=mode, flags=flags, **shape)
    want = oracle_job(w, bufs)
    err = 0.0
    for c in range(w.Rc):
        e = rel_l2(theta[c], want[c])
        err = max(err, e)
        assert e <= (tol or TOL[w.dtype]), (w.name, c, e, stats)
    return theta[0], stats, err


@pytest.mark.parametrize("p", [128, 192, 384, 1024, 3072])
def test_cuda_core_path_matches_oracle(p):
    """One CTA (p=128, 192), small clusters and the full 16-CTA cluster of the image-shaped workload."""
    check(job(p), CUDA_CORES)


@pytest.mark.parametrize("p", [128, 192, 384, 1024, 2048, 3072])
def test_tensor_core_path_matches_oracle(p):
    _, stats, _ = check(job(p), 0)
    assert stats["cluster_size"] * stats["smem_bytes"] > 0


def test_tensor_and_cuda_core_paths_agree_closely():
    """Same bf16 inputs and fp32 accumulation: the two paths differ only in summation order."""
    w = job(3072, N=1_500, T=1)
    a, _, _ = check(w, 0)
    b, _, _ = check(w, CUDA_CORES)
    assert rel_l2(a, b) <= 1e-3


@pytest.mark.parametrize("N,n,C", [(300, 256, 10), (256, 256, 2), (257, 128, 16), (40, 7, 3), (1, 1, 2)])
def test_ragged_and_small_batches(N, n, C):
    check(job(384, C=C, N=N, n=n, T=3, lr=0.05), 0)


def test_two_class_softmax_follows_logistic_with_doubled_rate():
    """The exact C = 2 identity, on the GPU: w_1 - w_0 of the softmax chain equals the fp32 logistic chain at 2*alpha
    up to the bf16 rounding of the softmax path."""
    import oracle
    from paper_2312_08728_b200 import inputs
    w = job(128, C=2, N=1_000, n=100, T=2, lr=0.05)
    X, lab = inputs.make_buffer(w, 0)
    theta, _ = gpu_job(w, [(X, lab)], mode="resident")
    th = np.zeros(128)
    oracle.run_rounds(oracle.LOGISTIC, X, lab.double(), th, w.T, w.n, 2 * w.lr, inputs.buffer_seed(w.seed, 0, 0, 1))
    assert rel_l2(theta[0][:, 1] - theta[0][:, 0], th) <= 2e-2


def test_slots_path_and_chaining_over_buffers():
    w = job(3072, N=1_200, K=3, n=256, T=2, epochs=2)
    check(w, 0, mode="slots")


def test_cfg4_one_full_buffer():
    """One full buffer of the image-shaped workload: 20,000 x 3,072 bf16, C=10, n=256 (last mini-batch 32 rows), T=4."""
    w = WORKLOADS["cfg4"].scaled(N=20_000, K=1, epochs=1)
    _, stats, err = check(w, 0)
    assert stats["steps"] == 4 * 79


@pytest.mark.parametrize("p", [8, 72, 200, 1000, 2176, 3064])
def test_predictor_counts_that_do_not_fill_the_last_panel(p):
    """Any multiple of eight predictors up to 16 x 192: the columns beyond p in the last CTA's panels are zero columns
    (never read from the buffer, never written to W)."""
    check(job(p, N=1_500, T=2), 0)
    check(job(p, N=600, T=1), CUDA_CORES)


@pytest.mark.parametrize("p,N,n", [(384, 1_500, 300), (1024, 2_100, 512), (3072, 1_300, 1_000), (128, 2_000, 2_000)])
def test_mini_batches_larger_than_one_tile(p, N, n):
    """More than 256 rows per mini-batch: the step takes them in tiles of 256 row slots (the last tile and the last
    mini-batch ragged, one case with a single full-batch step per round), the gradient summed over the tiles before W moves."""
    check(job(p, N=N, n=n, T=2), 0)
    check(job(p, N=N, n=n, T=1), CUDA_CORES)


def test_replicate_chains_one_cluster_per_chain():
    """Four chains with their own W and their own partitions over one buffer, one cluster of CTAs each, in one launch;
    and more chains than clusters fit (a cluster then takes its chains one after the other).  Every chain against
    the oracle."""
    w = dataclasses.replace(job(1024, N=1_500, T=2), Rc=4)
    _, stats, _ = check(w, 0)
    assert stats["chains_in_flight"] == 4 and stats["grid_ctas"] == 4 * stats["cluster_size"]
    w = dataclasses.replace(job(3072, N=700, T=2), Rc=11)   # 16 CTAs per chain: at most 9 clusters on 148 SMs
    _, stats, _ = check(w, 0)
    assert stats["chains_in_flight"] < 11
    w = dataclasses.replace(job(128, N=900, n=100, T=2), Rc=5)  # one CTA per chain
    check(w, 0)


def test_null_rounds_probe_changes_nothing_softmax():
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS, FLAG_TIMING
    w = job(1024, N=1_000, T=1)
    X, y = [t.cuda() for t in buffers_of(w)[0]]
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, C=w.C, flags=FLAG_NO_SLOTS | FLAG_TIMING) as h:
        h.run_rounds_resident(X, y, 1, w.n, w.lr, 3)
        before, s0 = h.get_theta(), h.get_stats()
        h.debug_null_rounds(X.shape[0], 3, w.n)
        after, s1 = h.get_theta(), h.get_stats()
        assert np.array_equal(before, after)
        assert s1["launches"] == s0["launches"] + 1 and s1["steps"] == s0["steps"] and s1["kernel_ms"] > s0["kernel_ms"]


def test_a_softmax_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    """A budget of a nanosecond: the first wait of the softmax kernel that does not succeed at its first look gives up,
    every CTA leaves its loops, frees its tensor memory and returns; W is not written back; then a correct run."""
    from paper_2312_08728_b200.binding import Bmgd, BmgdError, ERR_TIMEOUT, FLAG_NO_SLOTS
    w = job(1024, N=1_000, T=2)
    bufs = buffers_of(w)
    X, y = [t.cuda() for t in bufs[0]]
    with Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, C=w.C, flags=FLAG_NO_SLOTS, timeout_ms=1e-6) as h:
        start = np.full((1, w.p, w.C), 0.125, dtype=np.float32)
        h.set_theta(start)
        h.run_rounds_resident(X, y, 20, w.n, w.lr, 5)
        with pytest.raises(BmgdError) as e:
            h.sync()
        assert e.value.status == ERR_TIMEOUT
        assert np.array_equal(h.get_theta(), start)
        h.set_timeout(0.0)
        h.set_theta(np.zeros((1, w.p, w.C), dtype=np.float32))
        from paper_2312_08728_b200 import inputs
        h.run_rounds_resident(X, y, w.T, w.n, w.lr, inputs.buffer_seed(w.seed, 0, 0, w.K))
        theta = h.get_theta()
    want = oracle_job(w, bufs)[0]
    assert rel_l2(theta[0], want) <= 2e-2


def test_unsupported_shapes_are_refused_not_miscomputed():
    from paper_2312_08728_b200.binding import BmgdError, ERR_UNIMPLEMENTED
    for w in (job(100), job(384, C=17), job(3080)):
        with pytest.raises(BmgdError) as e:
            gpu_job(w, buffers_of(w), mode="resident")
        assert e.value.status == ERR_UNIMPLEMENTED


def test_bitwise_reproducible():
    w = job(1024, N=1_000, T=2)
    bufs = buffers_of(w)
    a, _ = gpu_job(w, bufs, mode="resident")
    b, _ = gpu_job(w, bufs, mode="resident")
    assert np.array_equal(a, b)
