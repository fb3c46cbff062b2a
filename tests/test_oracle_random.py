"""Pins for the oracle's Philox generator, the discrete-Gaussian table and the
three samplers (counter layout and word-to-value maps)."""
import mpmath
import numpy as np

import oracle
from conftest import read_golden


def test_philox_known_answers():
    rows = read_golden("philox4x32_10_kat.txt")
    assert len(rows) == 3
    for row in rows:
        w = [int(x, 16) for x in row.split()]
        got = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in got] == w[6:10]


def test_gauss_table_against_60_digit_recomputation():
    mpmath.mp.dps = 60
    sigma = mpmath.mpf("3.2")
    rho = {x: mpmath.exp(-mpmath.mpf(x * x) / (2 * sigma * sigma)) for x in range(-19, 20)}
    total = sum(rho.values())
    want, cum = [], mpmath.mpf(0)
    for x in range(-19, 19):
        cum += rho[x]
        want.append(int(mpmath.floor(cum / total * mpmath.mpf(2) ** 64)))
    got = [int(v) for v in oracle.gauss_table()]
    assert got == want
    assert all(a < b for a, b in zip(got, got[1:]))


def _words(seed, block, t, client, tag, limb=0):
    key = [seed & 0xffffffff, seed >> 32]
    return [int(x) for x in oracle.philox4x32_10([block, t, client, tag | (limb << 8)], key)]


def test_sampler_coordinates_and_value_maps():
    seed, t, client, N = 0x1234567890abcdef, 7, 3, 64
    table = [int(v) for v in oracle.gauss_table()]
    tern = oracle.sample_ternary(seed, t, client, 4, N)
    gau = oracle.sample_gauss(seed, t, client, 5, N)
    q = 0xffffffffffc0001
    uni = oracle.sample_uniform(seed, t, client, 2, 5, q, N)
    for j in range(N):
        w = _words(seed, j >> 2, t, client, 4)
        assert int(tern[j]) == (w[j & 3] * 3 >> 32) - 1
        w = _words(seed, j >> 1, t, client, 5)
        r = w[2 * (j & 1)] | (w[2 * (j & 1) + 1] << 32)
        assert int(gau[j]) == -19 + sum(r >= th for th in table)
        w = _words(seed, j, t, client, 2, limb=5)
        v = w[0] | (w[1] << 32) | (w[2] << 64) | (w[3] << 96)
        assert int(uni[j]) == v % q
    # distinct tags, clients and ciphertext indices give distinct streams
    assert not np.array_equal(gau, oracle.sample_gauss(seed, t, client, 6, N))
    assert not np.array_equal(gau, oracle.sample_gauss(seed, t + 1, client, 5, N))
    assert not np.array_equal(gau, oracle.sample_gauss(seed, t, client + 1, 5, N))
    assert not np.array_equal(gau, oracle.sample_gauss(seed + (1 << 32), t, client, 5, N))


def test_sampler_statistics():
    N = 1 << 18
    g = oracle.sample_gauss(99, 0, 0, 5, N).astype(np.float64)
    # exact variance of the discrete Gaussian on [-19,19] with sigma 3.2 is 10.24 (to 7 digits)
    assert abs(g.mean()) < 4 * 3.2 / np.sqrt(N)
    assert abs(g.var() - 10.24) < 0.12
    assert abs((g == 0).mean() - 0.124669463) < 0.004
    assert g.min() >= -19 and g.max() <= 19
    u = oracle.sample_ternary(99, 0, 0, 4, N)
    for v in (-1, 0, 1):
        assert abs((u == v).mean() - 1 / 3) < 0.005
    q = 0xfffffdc001
    a = oracle.sample_uniform(99, 0, 0, 2, 1, q, N)
    assert int(a.max()) < q
    assert abs(a.astype(np.float64).mean() / q - 0.5) < 0.005
    hist = np.bincount((a.astype(np.float64) / q * 16).astype(int), minlength=16)[:16]
    chi2 = ((hist - N / 16) ** 2 / (N / 16)).sum()
    assert chi2 < 50   # 15 degrees of freedom
