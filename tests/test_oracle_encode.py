"""Pins for the oracle's CKKS encode/decode: the closed form of the canonical
embedding evaluated with mpmath, the root table recomputed at 50 digits,
round trips and special inputs."""
import mpmath
import numpy as np
import pytest

import oracle
import synthetic_inputs as si


def test_root_table_is_correctly_rounded():
    mpmath.mp.dps = 50
    for N in (8, 64, 8192):
        ctx = oracle.Context(N, [si.PRIMES_SWEEP[0]], 30)
        tw = ctx.twiddle_table()
        M = 2 * N
        step = 1 if N <= 64 else 37
        for t in list(range(0, M, step)) + [M // 8, M // 4, M // 2, 3 * M // 4, M - 1]:
            turn = mpmath.mpf(2 * t) / M          # exact: M is a power of two
            assert tw[t, 0] == float(mpmath.cospi(turn)) + 0.0, (N, t)
            assert tw[t, 1] == float(mpmath.sinpi(turn)) + 0.0, (N, t)
        assert tw[0, 0] == 1.0 and tw[0, 1] == 0.0 and tw[M // 4, 0] == 0.0 and tw[M // 4, 1] == 1.0
        # mirror symmetry is exact
        assert np.array_equal(tw[1:, 0], tw[1:, 0][::-1])
        assert np.array_equal(tw[1:, 1], -tw[1:, 1][::-1])


def closed_form_encode(z, N, log2_delta):
    """m_k = (2 Delta / N) sum_j z_j cos(pi k 5^j / N): inverse of evaluating the real
    polynomial m at the roots zeta^(5^j), zeta = exp(i pi / N), and their conjugates."""
    mpmath.mp.dps = 50
    n = N // 2
    g = [pow(5, j, 2 * N) for j in range(n)]
    out = []
    for k in range(N):
        s = sum(mpmath.mpf(float(z[j])) * mpmath.cos(mpmath.pi * k * g[j] / N) for j in range(n))
        out.append(s * 2 * mpmath.mpf(2) ** log2_delta / N)
    return out


@pytest.mark.parametrize("N", [8, 16, 64, 256])
def test_encode_matches_closed_form(N):
    ctx = oracle.Context(N, [si.PRIMES_SWEEP[0]], 30)
    rng = np.random.default_rng(N)
    z = (rng.standard_normal(N // 2) * 0.02).astype(np.float32)
    m, ov = ctx.encode(z)
    assert not ov
    exact = closed_form_encode(z, N, 30)
    for k in range(N):
        # the fp64 network may round differently only if the exact value is within
        # 1e-6 of a half-integer; the seeds used here avoid that
        frac = abs(exact[k] - mpmath.floor(exact[k]) - mpmath.mpf("0.5"))
        assert frac > 1e-6
        assert int(m[k]) == int(mpmath.nint(exact[k])), (k, m[k], exact[k])


@pytest.mark.parametrize("N", [8, 64])
def test_decode_matches_closed_form(N):
    """z_j = Re( sum_k d_k zeta^(5^j k) ) / Delta"""
    mpmath.mp.dps = 50
    ctx = oracle.Context(N, [si.PRIMES_SWEEP[0]], 30)
    rng = np.random.default_rng(N + 5)
    d = rng.integers(-2**40, 2**40, size=N, dtype=np.int64)
    z = ctx.decode(d)
    for j in range(N // 2):
        g = pow(5, j, 2 * N)
        s = sum(int(d[k]) * mpmath.cos(mpmath.pi * k * g / N) for k in range(N))
        assert abs(float(s / 2**30) - z[j]) < 1e-9 * max(1.0, abs(z[j]))


@pytest.mark.parametrize("N,ld", [(64, 30), (8192, 40), (32768, 45)])
def test_round_trip(N, ld):
    ctx = oracle.Context(N, [si.PRIMES_SWEEP[0]], ld)
    rng = np.random.default_rng(N)
    z = (rng.standard_normal(N // 2) * 0.02).astype(np.float32)
    m, ov = ctx.encode(z)
    assert not ov
    back = ctx.decode(m)
    # rounding each of the N coefficients by at most 1/2 moves a slot by at most N/2 / Delta
    assert np.abs(back - z.astype(np.float64)).max() <= N / 2 / 2.0**ld


def test_special_inputs():
    N, ld = 64, 30
    ctx = oracle.Context(N, [si.PRIMES_SWEEP[0]], ld)
    m, _ = ctx.encode(np.full(N // 2, 0.25, np.float32))       # constant slots -> constant polynomial
    assert int(m[0]) == 2**28 and not m[1:].any()
    m, _ = ctx.encode(np.zeros(N // 2, np.float32))
    assert not m.any()
    z = np.zeros(N // 2, np.float32); z[3] = 1.0               # linearity
    y = np.zeros(N // 2, np.float32); y[10] = -0.5
    mz, my, mzy = ctx.encode(z)[0], ctx.encode(y)[0], ctx.encode(z + y)[0]
    assert np.abs(mz + my - mzy).max() <= 1
    # |coefficients| beyond 2^62 are flagged
    big = oracle.Context(N, [si.PRIMES_SWEEP[0]], 60)
    _, ov = big.encode(np.full(N // 2, 1e6, np.float32))
    assert ov
    _, ov = big.encode(np.full(N // 2, 1.0, np.float32))
    assert not ov
    _, ov = big.encode(np.full(N // 2, np.inf, np.float32))
    assert ov
