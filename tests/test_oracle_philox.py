"""Pins for the oracle's counter-based random stream (CPU only)."""
import ctypes as C
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(x, 16) for x in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = oracle.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == want


def _curand_host():
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so"):
        try:
            return C.CDLL(name)
        except OSError:
            continue
    return None


def test_philox_against_curand_host_generator():
    """An independent implementation (cuRAND's host generator, used as a black
    box, no GPU involved): its first four words for a seed are the block with
    key = seed and a zero counter."""
    cu = _curand_host()
    if cu is None:
        pytest.skip("libcurand not loadable")
    CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161
    for seed in (0, 1, 0xDEADBEEF, 0x0123456789ABCDEF, 2**64 - 1):
        g = C.c_void_p()
        assert cu.curandCreateGeneratorHost(C.byref(g), CURAND_RNG_PSEUDO_PHILOX4_32_10) == 0
        assert cu.curandSetPseudoRandomGeneratorSeed(g, C.c_ulonglong(seed)) == 0
        out = (C.c_uint * 4)()
        assert cu.curandGenerate(g, out, C.c_size_t(4)) == 0
        cu.curandDestroyGenerator(g)
        want = oracle.philox4x32_10([0, 0, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert list(out) == [int(x) for x in want], hex(seed)


def test_philox_is_a_bijection_on_small_counter_sets():
    # distinct counters under one key give distinct blocks; changing any one
    # input word changes the output
    base = oracle.philox4x32_10([5, 6, 7, 8], [9, 10])
    seen = {tuple(base)}
    for i in range(4):
        c = [5, 6, 7, 8]; c[i] ^= 1
        o = tuple(oracle.philox4x32_10(c, [9, 10]))
        assert o not in seen
        seen.add(o)
    for i in range(2):
        k = [9, 10]; k[i] ^= 1
        o = tuple(oracle.philox4x32_10([5, 6, 7, 8], k))
        assert o not in seen
        seen.add(o)


def test_uniform_layout_and_grid():
    # u = (word0 >> 8) * 2^-24 of the block with key = seed and
    # counter = (step lo, step hi, position, tag)
    seed, step, pos, tag = 0x1122334455667788, 0x99AABBCCDDEEFF00, 3, 1
    w = oracle.philox4x32_10([step & 0xFFFFFFFF, step >> 32, pos, tag],
                             [seed & 0xFFFFFFFF, seed >> 32])
    u = oracle.uniform(seed, step, pos, tag)
    assert u == (int(w[0]) >> 8) / 2.0**24
    assert 0.0 <= u < 1.0
    assert np.float32(u) == u            # exactly representable in fp32
    assert (u * 2**24) == int(u * 2**24)


def test_uniform_statistics():
    n = 200_000
    u = np.array([oracle.uniform(7, s, s % 11, s % 2) for s in range(n)])
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * np.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 2e-3
    counts, _ = np.histogram(u, bins=64, range=(0, 1))
    chi2 = ((counts - n / 64) ** 2 / (n / 64)).sum()
    assert chi2 < 63 + 5 * np.sqrt(2 * 63)
    # neighbouring counters are uncorrelated
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.01
