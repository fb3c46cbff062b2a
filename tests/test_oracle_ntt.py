"""Pins for the oracle's negacyclic transform: the O(N^2) definition evaluated
with Python integers, the schoolbook product, and the inverse."""
import numpy as np
import pytest

import oracle
import synthetic_inputs as si


def brev(x, bits):
    return int(format(x, "0%db" % bits)[::-1], 2) if bits else 0


def py_schoolbook(a, b, q):
    N = len(a)
    out = [0] * N
    for i in range(N):
        for j in range(N):
            p = int(a[i]) * int(b[j])
            if i + j < N:
                out[i + j] = (out[i + j] + p) % q
            else:
                out[i + j - N] = (out[i + j - N] - p) % q
    return out


@pytest.mark.parametrize("N", [4, 8, 16, 64])
@pytest.mark.parametrize("q", [257, si.PRIMES_SWEEP[0], si.PRIMES_N16384[1]])
def test_forward_matches_definition(N, q):
    ctx = oracle.Context(N, [q], 20)
    psi = ctx.psi(0)
    assert psi == oracle.min_root_2n(q, N) and pow(psi, N, q) == q - 1
    rng = np.random.default_rng(N)
    a = rng.integers(0, q, size=N, dtype=np.uint64)
    got = ctx.ntt_forward(0, a)
    bits = N.bit_length() - 1
    for k in range(N):
        e = 2 * brev(k, bits) + 1
        want = sum(int(a[j]) * pow(psi, e * j, q) for j in range(N)) % q
        assert int(got[k]) == want
    # an impulse at X^1 transforms to the odd powers of psi themselves
    imp = np.zeros(N, np.uint64)
    imp[1] = 1
    assert [int(x) for x in ctx.ntt_forward(0, imp)] == [pow(psi, 2 * brev(k, bits) + 1, q)
                                                         for k in range(N)]


@pytest.mark.parametrize("N,primes", [(8192, si.PRIMES_N8192), (16384, si.PRIMES_N16384),
                                      (32768, si.PRIMES_N32768), (65536, si.PRIMES_SWEEP[:2])])
def test_inverse_of_forward_is_identity(N, primes):
    ctx = oracle.Context(N, primes, 40)
    rng = np.random.default_rng(3)
    for limb, q in enumerate(primes):
        a = rng.integers(0, q, size=N, dtype=np.uint64)
        f = ctx.ntt_forward(limb, a)
        assert not np.array_equal(f, a)
        assert np.array_equal(ctx.ntt_inverse(limb, f), a)
        assert np.array_equal(ctx.ntt_forward(limb, ctx.ntt_inverse(limb, a)), a)


@pytest.mark.parametrize("N", [4, 16, 64])
def test_products_agree_with_python_schoolbook(N):
    for q in (si.PRIMES_N8192[0], si.PRIMES_N8192[1], 257):
        ctx = oracle.Context(N, [q], 20)
        rng = np.random.default_rng(N + 1)
        a = rng.integers(0, q, size=N, dtype=np.uint64)
        b = rng.integers(0, q, size=N, dtype=np.uint64)
        want = py_schoolbook(a, b, q)
        assert [int(x) for x in oracle.negacyclic_mul_schoolbook(N, q, a, b)] == want
        assert [int(x) for x in ctx.negacyclic_mul_ntt(0, a, b)] == want


def test_transform_product_equals_schoolbook_at_larger_size():
    N, q = 1024, si.PRIMES_N16384[0]
    ctx = oracle.Context(N, [q], 40)
    rng = np.random.default_rng(9)
    a = rng.integers(0, q, size=N, dtype=np.uint64)
    b = rng.integers(0, q, size=N, dtype=np.uint64)
    assert np.array_equal(ctx.negacyclic_mul_ntt(0, a, b), oracle.negacyclic_mul_schoolbook(N, q, a, b))
    # X^(N-1) * X = X^N = -1
    x1 = np.zeros(N, np.uint64); x1[1] = 1
    xl = np.zeros(N, np.uint64); xl[N - 1] = 1
    prod = ctx.negacyclic_mul_ntt(0, x1, xl)
    assert int(prod[0]) == q - 1 and not prod[1:].any()
