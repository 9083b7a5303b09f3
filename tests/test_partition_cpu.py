"""The per-pass partition of the sample into buffers (Algorithm 1, line 2) and the host-side gather of a buffer.

Pure host code in the library, so these run without a GPU.  The expected partition comes from the oracle's own
shuffle (chain word 0xFFFFFFFF, round word = pass), the expected buffer from numpy fancy indexing.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_08728_b200 import binding

CHAIN = binding.PARTITION_CHAIN


@pytest.mark.parametrize("N", [1, 2, 7, 1000, 1024, 1025, 100_003])
def test_partition_index_equals_the_oracle_shuffle(N):
    for seed, e in [(0, 0), (123456789, 3), (0xFFFFFFFFFFFFFFFF, 17)]:
        want = oracle.perm(seed, CHAIN, e, N)
        js = range(N) if N <= 2000 else np.random.default_rng(N).integers(0, N, 500)
        for j in js:
            assert binding.partition_index(seed, e, N, int(j)) == want[j]


def test_partition_changes_with_the_pass_and_covers_every_row():
    N = 5000
    a = np.array([binding.partition_index(9, 0, N, j) for j in range(N)])
    b = np.array([binding.partition_index(9, 1, N, j) for j in range(N)])
    assert np.array_equal(np.sort(a), np.arange(N)) and np.array_equal(np.sort(b), np.arange(N))
    assert (a == b).sum() < 15


@pytest.mark.parametrize("dtype", [torch.float32, torch.float64, torch.bfloat16])
@pytest.mark.parametrize("threads", [1, 4, 0])
def test_gather_buffer_is_bit_exact(dtype, threads):
    N, p, K = 10_007, 12, 4          # ragged: the last buffer is shorter
    g = torch.Generator().manual_seed(5)
    X = torch.randn(N, p, generator=g).to(dtype)
    y = torch.randn(N, generator=g).to(torch.float64 if dtype == torch.float64 else torch.float32)
    N0 = -(-N // K)
    sx = torch.empty(N0, p, dtype=dtype)
    sy = torch.empty(N0, dtype=y.dtype)
    seen = []
    for k in range(K):
        rows = binding.gather_buffer(X, y, K, seed=77, epoch=2, k=k, stage_x=sx, stage_y=sy, threads=threads)
        want = oracle.perm(77, CHAIN, 2, N)[k * N0:(k + 1) * N0].astype(np.int64)
        assert rows == len(want)
        idx = torch.from_numpy(want)
        assert torch.equal(sx[:rows].view(torch.uint8), X[idx].contiguous().view(torch.uint8))
        assert torch.equal(sy[:rows], y[idx])
        seen.append(want)
    assert np.array_equal(np.sort(np.concatenate(seen)), np.arange(N))


def test_gather_buffer_int_labels_and_argument_errors():
    N, p, K = 300, 64, 3
    X = torch.randn(N, p).to(torch.bfloat16)
    lab = torch.randint(0, 10, (N,), dtype=torch.int32)
    sx = torch.empty(100, p, dtype=torch.bfloat16); sy = torch.empty(100, dtype=torch.int32)
    rows = binding.gather_buffer(X, lab, K, seed=1, epoch=0, k=1, stage_x=sx, stage_y=sy)
    want = torch.from_numpy(oracle.perm(1, CHAIN, 0, N)[100:200].astype(np.int64))
    assert rows == 100 and torch.equal(sy, lab[want])
    with pytest.raises(binding.BmgdError):
        binding.gather_buffer(X, lab, K, seed=1, epoch=0, k=3, stage_x=sx, stage_y=sy)
    with pytest.raises(ValueError):
        binding.gather_buffer(X, lab, K, seed=1, epoch=0, k=0, stage_x=sx[:50], stage_y=sy)
    with pytest.raises(binding.BmgdError):
        binding.partition_index(1, 0, 10, 10)
