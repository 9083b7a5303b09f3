"""The device shuffle against the oracle's, word for word (Algorithm 1, partition of the buffer)."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS
    h = Bmgd(1000, 8, 1, flags=FLAG_NO_SLOTS)
    yield h
    h.close()


@pytest.mark.parametrize("N0", [1, 2, 3, 5, 31, 32, 33, 100, 511, 512, 513, 1000, 1023, 1024, 1025, 2000, 4097,
                                20_000, 65_536, 65_537, 100_000, 1_000_000, 2_500_000])
def test_perm_bit_exact(handle, N0):
    for seed, chain, rnd in [(0, 0, 0), (1, 2, 3), (0xFFFFFFFFFFFFFFFF, 63, 19), (0x123456789ABCDEF0, 7, 1)]:
        got = handle.debug_perm(seed, chain, rnd, N0)
        want = oracle.perm(seed, chain, rnd, N0)
        assert np.array_equal(got, want), (N0, seed, chain, rnd)


def test_perm_every_small_N0(handle):
    for N0 in range(1, 260):
        assert np.array_equal(handle.debug_perm(77, 1, 2, N0), oracle.perm(77, 1, 2, N0)), N0


def test_perm_large_is_a_bijection(handle):
    N0 = 10_000_000
    got = handle.debug_perm(9, 0, 4, N0)
    seen = np.zeros(N0, dtype=np.uint8)
    seen[got] = 1
    assert int(seen.sum()) == N0
    idx = np.random.default_rng(0).integers(0, N0, 2000)
    import ctypes
    keys = (ctypes.c_uint32 * 8)(*oracle.round_keys(9, 0, 4))
    for j in idx:
        assert oracle.lib().orc_perm_index(int(j), N0, keys) == got[j]
