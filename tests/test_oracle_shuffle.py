"""Pins for the oracle's shuffle (Algorithm 1, "generate random partition of the buffer").

The paper does not say how the partition is drawn; the build fixes a keyed bijection
(Philox4x32-10 round keys + Feistel network + cycle walking).  These tests pin it to
things other than itself: an independent library Philox, brute-force bijectivity, and
chi-square uniformity of positions and of mini-batch co-membership.
"""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle

_TRITON_PHILOX = r"""
import os, sys, json
os.environ["TRITON_INTERPRET"] = "1"
import torch, triton, triton.language as tl

@triton.jit
def k(out, c0, c1, c2, c3, k0, k1):
    one = tl.arange(0, 1)
    a, b, c, d = tl.philox_impl(tl.full((1,), c0, tl.uint32), tl.full((1,), c1, tl.uint32),
                                tl.full((1,), c2, tl.uint32), tl.full((1,), c3, tl.uint32),
                                tl.full((1,), k0, tl.uint32), tl.full((1,), k1, tl.uint32), 10)
    tl.store(out + one, a); tl.store(out + 1 + one, b)
    tl.store(out + 2 + one, c); tl.store(out + 3 + one, d)

cases = json.loads(sys.argv[1])
res = []
for ctr, key in cases:
    out = torch.zeros(4, dtype=torch.int64)
    k[(1,)](out, *ctr, *key)
    res.append([int(v) & 0xFFFFFFFF for v in out.tolist()])
print("RESULT" + json.dumps(res))
"""


def test_philox_matches_independent_library():
    """Philox4x32-10 (Salmon et al., SC'11) against Triton's own implementation run on the CPU."""
    pytest.importorskip("triton")
    rng = np.random.default_rng(7)
    cases = [([0, 0, 0, 0], [0, 0]),
             ([0xFFFFFFFF] * 4, [0xFFFFFFFF] * 2),
             ([1, 2, 3, 4], [5, 6])]
    for _ in range(5):
        cases.append(([int(v) for v in rng.integers(0, 2**32, 4)], [int(v) for v in rng.integers(0, 2**32, 2)]))
    # the exact counters the shuffle uses: (round, chain, tag, block), key = seed halves
    cases.append(([3, 17, 0x424D4744, 0], [0x9ABCDEF0, 0x12345678]))
    cases.append(([3, 17, 0x424D4744, 1], [0x9ABCDEF0, 0x12345678]))
    p = subprocess.run([sys.executable, "-c", _TRITON_PHILOX, json.dumps(cases)],
                       capture_output=True, text=True, timeout=600,
                       env={**os.environ, "TRITON_INTERPRET": "1"})
    assert p.returncode == 0, p.stderr[-2000:]
    line = [l for l in p.stdout.splitlines() if l.startswith("RESULT")][-1]
    theirs = json.loads(line[len("RESULT"):])
    for (ctr, key), want in zip(cases, theirs):
        assert oracle.philox4x32_10(ctr, key) == want, (ctr, key)


def test_round_keys_are_two_philox_blocks():
    seed = 0x123456789ABCDEF0
    ks = oracle.round_keys(seed, 17, 3)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    assert ks[:4] == oracle.philox4x32_10([3, 17, 0x424D4744, 0], key)
    assert ks[4:] == oracle.philox4x32_10([3, 17, 0x424D4744, 1], key)


def test_philox_round_structure_is_a_bijection_of_the_counter():
    """For a fixed key Philox permutes counters: 2^16 nearby counters give 2^16 distinct blocks."""
    seen = set()
    for c0 in range(256):
        for c2 in range(256):
            seen.add(tuple(oracle.philox4x32_10([c0, 0, c2, 0], [1, 2])))
    assert len(seen) == 65536


@pytest.mark.parametrize("seed", [0, 1, 0xDEADBEEFCAFEF00D])
def test_perm_is_a_bijection_for_every_small_N0(seed):
    for N0 in list(range(1, 300)) + [511, 512, 513, 1000, 2000, 4095, 4096]:
        pi = oracle.perm(seed, 0, 0, N0)
        assert pi.min() == 0 and pi.max() == N0 - 1
        assert np.unique(pi).size == N0, N0


def test_perm_is_a_bijection_all_N0_up_to_4096():
    for N0 in range(300, 4097, 7):
        pi = oracle.perm(42, 1, 2, N0)
        assert np.array_equal(np.sort(pi), np.arange(N0, dtype=np.uint32)), N0


@pytest.mark.parametrize("N0", [2_000, 20_000, 100_000, 1_000_000, 2_500_000])
def test_perm_is_a_bijection_at_workload_sizes(N0):
    pi = oracle.perm(5, 3, 4, N0)
    seen = np.zeros(N0, dtype=np.uint8)
    seen[pi] = 1
    assert int(seen.sum()) == N0


def test_domain_is_the_smallest_near_square_grid_that_holds_the_buffer():
    """a = max(32, ceil(sqrt N0)), c = max(32, ceil(N0 / a)), checked with exact integer arithmetic: the grid holds
    every index, and (beyond the floor of 32 per half) drops fewer than a of its a c values."""
    import math
    sizes = list(range(1, 3000)) + [4095, 4096, 4097, 99_999, 100_000, 100_001, 1_000_000, 2_500_000,
                                    46_340 ** 2, 46_340 ** 2 + 1, 2 ** 31 - 1]
    for N0 in sizes:
        a, c = oracle.domain(N0)
        r = math.isqrt(N0 - 1) + 1 if N0 > 1 else 1      # smallest integer whose square is >= N0
        assert a == max(32, r), N0
        assert c == max(32, -(-N0 // a)), N0
        assert a * c >= N0 and a * c < 2 ** 32
        if N0 >= 1024:
            assert a * c - N0 < a, N0


def test_almost_no_index_walks_the_cycle_at_workload_sizes():
    """With a c barely above N0, the share of indices whose first pass through the network lands at or above N0 is
    about (a c - N0) / (a c): the walk that makes the bijection exact is rare, not the common case."""
    for N0 in (100_000, 1_000_000, 2_500_000):
        a, c = oracle.domain(N0)
        assert (a * c - N0) / (a * c) < 2e-3


def test_perm_index_agrees_with_whole_perm():
    N0 = 777
    ks = oracle.round_keys(9, 2, 5)
    import ctypes
    arr = (ctypes.c_uint32 * 8)(*ks)
    pi = oracle.perm(9, 2, 5, N0)
    for j in [0, 1, 100, 776]:
        assert oracle.lib().orc_perm_index(j, N0, arr) == pi[j]


def test_distinct_round_chain_seed_give_distinct_permutations():
    N0 = 1000
    base = oracle.perm(11, 0, 0, N0)
    for args in [(11, 0, 1), (11, 1, 0), (12, 0, 0), (11 + (1 << 32), 0, 0)]:
        other = oracle.perm(args[0], args[1], args[2], N0)
        # two independent uniform permutations agree in about one position
        assert (other == base).sum() < 12, args
    assert np.array_equal(base, oracle.perm(11, 0, 0, N0))


def _chi2_ok(stat, dof, sigmas=5.0):
    return stat < dof + sigmas * np.sqrt(2.0 * dof)


@pytest.mark.parametrize("N0,seeds", [(5, 100_000), (64, 100_000), (1000, 20_000)])
def test_positions_are_uniform(N0, seeds):
    """Each index j lands on each row i equally often over many seeds (chi-square gate)."""
    cnt = np.zeros((N0, N0), dtype=np.int64)
    ar = np.arange(N0)
    for s in range(seeds):
        pi = oracle.perm(s * 0x9E3779B97F4A7C15 + 1, s & 3, s % 7, N0)
        cnt[ar, pi] += 1
    e = seeds / N0
    stat = ((cnt - e) ** 2 / e).sum()
    assert _chi2_ok(stat, (N0 - 1) ** 2), (stat, (N0 - 1) ** 2)


@pytest.mark.parametrize("N0,n,seeds", [(5, 2, 100_000), (64, 8, 100_000), (1000, 100, 4_000)])
def test_minibatch_comembership_is_uniform(N0, n, seeds):
    """Two rows share a mini-batch with the probability a uniform partition gives."""
    sizes = [min(n, N0 - m * n) for m in range(-(-N0 // n))]
    p_same = sum(b * (b - 1) for b in sizes) / (N0 * (N0 - 1))
    co = np.zeros((N0, N0), dtype=np.int64)
    for s in range(seeds):
        pi = oracle.perm(s + 1000, 0, s % 5, N0)
        batch = np.empty(N0, dtype=np.int64)
        batch[pi] = np.arange(N0) // n
        co += batch[:, None] == batch[None, :]
    iu = np.triu_indices(N0, 1)
    obs = co[iu]
    e = seeds * p_same
    var = seeds * p_same * (1 - p_same)
    stat = ((obs - e) ** 2 / var).sum()
    assert _chi2_ok(stat, obs.size, sigmas=6.0), (stat, obs.size)


def test_every_row_used_once_per_round():
    N0, n = 1003, 100
    pi = oracle.perm(3, 0, 0, N0)
    M = -(-N0 // n)
    rows = np.concatenate([pi[m * n:min((m + 1) * n, N0)] for m in range(M)])
    assert np.array_equal(np.sort(rows), np.arange(N0))
