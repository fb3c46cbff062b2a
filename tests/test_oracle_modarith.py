"""Pins for the oracle's modular arithmetic, prime checks and root search.

Everything here is compared with Python's arbitrary-precision integers or
sympy, never with the oracle itself.
"""
import random

import pytest
import sympy

import oracle
import synthetic_inputs as si


def test_mulmod_powmod_invmod_against_python_ints():
    rnd = random.Random(1)
    for q in list(si.PRIMES_N8192) + list(si.PRIMES_N32768) + [257, 12289]:
        for _ in range(200):
            a, b = rnd.randrange(q), rnd.randrange(q)
            assert oracle.mulmod(a, b, q) == a * b % q
            e = rnd.randrange(1 << 62)
            assert oracle.powmod(a, e, q) == pow(a, e, q)
            if a:
                assert oracle.invmod(a, q) * a % q == 1
        # operands at the edge of the range
        assert oracle.mulmod(q - 1, q - 1, q) == 1
        assert oracle.mulmod(0, q - 1, q) == 0


def test_is_prime_against_sympy():
    rnd = random.Random(2)
    cases = [0, 1, 2, 3, 4, 561, 1105, 1729, 2465, 3215031751, 2**61 - 1, 2**62 - 57,
             (2**31 - 1) * (2**31 - 1), 0xfffffffffffc001, 0xfffffffffffc001 + 2]
    cases += [rnd.randrange(1, 1 << 62) | 1 for _ in range(300)]
    for n in cases:
        assert oracle.is_prime(n) == bool(sympy.isprime(n)), n


def _largest_primes(bits, two_n, count, skip=()):
    """Rule for the parameter sets: largest primes below 2^bits with q = 1 mod 2N."""
    out = []
    q = ((1 << bits) - 1) // two_n * two_n + 1
    while len(out) < count:
        if q < (1 << bits) and sympy.isprime(q) and q not in skip:
            out.append(q)
        q -= two_n
    return out


def test_parameter_sets_follow_the_prime_rule():
    # N = 8192: 60, 40, 60 bits
    p60 = _largest_primes(60, 2 * 8192, 2)
    p40 = _largest_primes(40, 2 * 8192, 1)
    assert si.PRIMES_N8192 == (p60[0], p40[0], p60[1])
    # N = 16384: 60, 40, 40, 60
    p60 = _largest_primes(60, 2 * 16384, 2)
    p40 = _largest_primes(40, 2 * 16384, 2)
    assert si.PRIMES_N16384 == (p60[0], p40[0], p40[1], p60[1])
    # N = 32768: 60, 45 x 4, 60
    p60 = _largest_primes(60, 2 * 32768, 2)
    p45 = _largest_primes(45, 2 * 32768, 4)
    assert si.PRIMES_N32768 == (p60[0], *p45, p60[1])
    # sweep: twelve 60-bit primes = 1 mod 2^17
    assert si.PRIMES_SWEEP == tuple(_largest_primes(60, 1 << 17, 12))


@pytest.mark.parametrize("q,N", [(17, 8), (257, 8), (257, 128), (12289, 64), (12289, 2048),
                                 (65537, 32768)])
def test_min_root_brute_force(q, N):
    roots = [x for x in range(1, q) if pow(x, N, q) == q - 1]
    assert oracle.min_root_2n(q, N) == min(roots)


def test_min_root_large_prime_properties():
    q, N = si.PRIMES_N8192[0], 8192
    psi = oracle.min_root_2n(q, N)
    assert pow(psi, N, q) == q - 1
    # every other primitive 2N-th root is an odd power of psi and none is smaller
    others = [pow(psi, k, q) for k in range(1, 2 * N, 2)]
    assert min(others) == psi
    assert oracle.min_root_2n(q + 2, N) == 0 or (q + 1) % (2 * N) == 0


def test_context_rejects_bad_parameters():
    good = list(si.PRIMES_N8192)
    oracle.Context(8192, good, 40)
    with pytest.raises(ValueError):
        oracle.Context(8192, [good[0], good[0]], 40)          # repeated
    with pytest.raises(ValueError):
        oracle.Context(8192, [good[0] + 2], 40)               # not prime / not 1 mod 2N
    with pytest.raises(ValueError):
        oracle.Context(8190, good, 40)                        # N not a power of two
    with pytest.raises(ValueError):
        oracle.Context(32768, good, 40)                       # q != 1 mod 2N
