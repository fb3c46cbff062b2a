"""Pins for the oracle's key generation, encryption, weighted sum, rescale and
decryption: identities recomputed with Python integers / numpy integer
convolutions, big-integer CRT, and plaintext FedAvg."""
import numpy as np
import pytest

import oracle
import synthetic_inputs as si


def negacyclic_int(a, b):
    """Exact product of small integer polynomials in Z[X]/(X^N+1) (int64 numpy)."""
    N = len(a)
    full = np.convolve(a.astype(np.int64), b.astype(np.int64))
    out = full[:N].copy()
    out[: N - 1] -= full[N:]
    return out


def centred(r, q):
    r = int(r)
    return r - q if r > q // 2 else r


def crt(residues, moduli):
    Q = 1
    for m in moduli:
        Q *= m
    x = 0
    for r, m in zip(residues, moduli):
        Qi = Q // m
        x += int(r) * Qi * pow(Qi, -1, m)
    return x % Q, Q


@pytest.mark.parametrize("N,primes", [(64, si.PRIMES_N8192), (8192, si.PRIMES_N8192)])
def test_public_key_relation(N, primes):
    """pk0 + pk1 s = e (mod q_j), with s, a, e the streams tagged 1, 2, 3."""
    ctx = oracle.Context(N, primes, 40)
    s, pk = ctx.keygen(77)
    assert np.array_equal(s, oracle.sample_ternary(77, 0, 0, 1, N))
    e = oracle.sample_gauss(77, 0, 0, 3, N)
    for j, q in enumerate(primes):
        assert np.array_equal(pk[1, j], oracle.sample_uniform(77, 0, 0, 2, j, q, N))
        sq = np.array([int(v) % q for v in s], np.uint64)
        as_ = oracle.negacyclic_mul_schoolbook(N, q, pk[1, j], sq) if N <= 64 \
            else ctx.negacyclic_mul_ntt(j, pk[1, j], sq)
        got = [centred((int(x) + int(y)) % q, q) for x, y in zip(pk[0, j], as_)]
        assert got == [int(v) for v in e]


@pytest.mark.parametrize("N,primes", [(64, si.PRIMES_N8192), (8192, si.PRIMES_N8192),
                                      (16384, si.PRIMES_N16384)])
def test_decrypt_of_fresh_ciphertext_is_message_plus_known_noise(N, primes):
    """c0 + c1 s = m + (e u + e0 + e1 s) exactly, on every limb."""
    ctx = oracle.Context(N, primes, 40)
    s, pk = ctx.keygen(5)
    rng = np.random.default_rng(N)
    slots = (rng.standard_normal(N // 2) * 0.02).astype(np.float32)
    m, _ = ctx.encode(slots)
    seed, client, t = 6, 2, 9
    ct = ctx.encrypt_one(pk, m, seed, client, t)
    u = oracle.sample_ternary(seed, t, client, 4, N)
    e0 = oracle.sample_gauss(seed, t, client, 5, N)
    e1 = oracle.sample_gauss(seed, t, client, 6, N)
    e = oracle.sample_gauss(5, 0, 0, 3, N)
    noise = negacyclic_int(e, u) + e0 + negacyclic_int(e1, s)
    want = m + noise
    for j, q in enumerate(primes):
        r = ctx.decrypt_limb(s, ct, len(primes), j)
        got = np.array([centred(x, q) for x in r], np.int64)
        assert np.array_equal(got, want), j
    # the noise is small and has the predicted spread sigma^2 (4N/3 + 1)
    var = noise.astype(np.float64).var()
    pred = 3.2**2 * (4 * N / 3 + 1)
    assert 0.6 * pred < var < 1.5 * pred
    # limb-0 decryption entry point gives the same centred integers
    d = ctx.decrypt(s, ct[None], len(primes))
    assert np.array_equal(d[0], want)
    # different client / index / seed change the ciphertext
    assert not np.array_equal(ct, ctx.encrypt_one(pk, m, seed, client + 1, t))
    assert not np.array_equal(ct, ctx.encrypt_one(pk, m, seed, client, t + 1))


def test_weights_are_rounded_products():
    ctx = oracle.Context(64, si.PRIMES_N8192, 40)
    alpha = np.array([0.25, 1 / 3, 0.1, 0.0, 1.0, 5e-324])
    W = ctx.weights(alpha)
    ql = float(si.PRIMES_N8192[-1])
    for a, w in zip(alpha, W):
        assert int(w) == int(round(float(a) * ql))      # Python rounds half to even


def test_weighted_sum_against_python_ints():
    N, primes = 64, si.PRIMES_N8192
    ctx = oracle.Context(N, primes, 40)
    rng = np.random.default_rng(4)
    C, T = 4, 2
    cts = [si.random_residues(10 + i, (T, 2, len(primes), N), primes) for i in range(C)]
    W = rng.integers(0, primes[-1], size=C, dtype=np.uint64)
    acc = ctx.weighted_sum(cts, W)
    for t in range(T):
        for comp in range(2):
            for j, q in enumerate(primes):
                for k in range(0, N, 7):
                    want = sum(int(W[i]) % q * int(cts[i][t, comp, j, k]) for i in range(C)) % q
                    assert int(acc[t, comp, j, k]) == want


def test_rescale_is_exact_rounded_division():
    """out = (X - [X]_{q_last}) / q_last  mod q_j with [.] the centred remainder, and it
    equals round(X / q_last) for the centred representative of X."""
    N, primes = 64, si.PRIMES_N8192
    ctx = oracle.Context(N, primes, 40)
    acc = si.random_residues(3, (1, 2, len(primes), N), primes)
    out = ctx.rescale(acc)
    ql = primes[-1]
    for comp in range(2):
        for k in range(N):
            X, Q = crt([acc[0, comp, j, k] for j in range(3)], primes)
            if X > Q // 2:
                X -= Q
            r = centred(X % ql, ql)
            assert (X - r) % ql == 0
            quo = (X - r) // ql
            # nearest integer to X / ql (no ties: ql is odd)
            assert abs(quo * ql - X) * 2 < ql
            for j in range(2):
                assert int(out[0, comp, j, k]) == quo % primes[j]


def test_limb0_decryption_equals_crt_decryption():
    N, primes = 64, si.PRIMES_N8192
    ctx = oracle.Context(N, primes, 40)
    s, pk = ctx.keygen(8)
    rng = np.random.default_rng(1)
    xs = [(rng.standard_normal(N // 2) * 0.02).astype(np.float32) for _ in range(3)]
    alpha = np.array([0.2, 0.5, 0.3])
    cts = [ctx.encrypt(pk, x, 9, i)[0] for i, x in enumerate(xs)]
    agg = ctx.rescale(ctx.weighted_sum(cts, ctx.weights(alpha)))
    d = ctx.decrypt(s, agg, 2)[0]
    r0 = ctx.decrypt_limb(s, agg[0], 2, 0)
    r1 = ctx.decrypt_limb(s, agg[0], 2, 1)
    for k in range(N):
        X, Q = crt([r0[k], r1[k]], primes[:2])
        if X > Q // 2:
            X -= Q
        assert int(d[k]) == X


@pytest.mark.parametrize("w", [si.scaled(si.TINY, 8192 * 2 + 101, name="tiny-cut"),
                               si.scaled(si.RESNET18, 8192 + 5, clients=4, name="r18-cut")])
def test_homomorphic_weighted_sum_is_plain_fedavg(w):
    ctx = oracle.Context(w.N, w.primes, w.log2_delta)
    s, pk = ctx.keygen(w.key_seed)
    xs = si.client_updates(w)
    alpha = si.client_weights(w)
    assert abs(alpha.sum() - 1) < 1e-12
    cts = []
    for i, x in enumerate(xs):
        sel, rest = ctx.pack(None, w.P, x)
        assert rest is None and sel.size == ctx.num_ct(w.P) * ctx.n
        ct, bad = ctx.encrypt(pk, sel, w.enc_seed, i)
        assert bad == 0
        cts.append(ct)
    agg = ctx.rescale(ctx.weighted_sum(cts, ctx.weights(alpha)))
    assert agg.shape == (ctx.num_ct(w.P), 2, w.L - 1, w.N)
    z = ctx.decode(ctx.decrypt(s, agg, w.L - 1)).reshape(-1)
    got = oracle.unpack(None, w.P, z, None, w.P)
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    err = np.abs(got - want)
    assert err.max() < 1e-6
    # predicted slot error: sigma sqrt((4N/3+1) N/2) sqrt(sum alpha^2) / Delta
    pred = 3.2 * np.sqrt((4 * w.N / 3 + 1) * w.N / 2) * np.sqrt((alpha**2).sum()) / 2.0**w.log2_delta
    assert 0.5 * pred < err.std() < 2.0 * pred
    # padding slots of the last ciphertext decode to (almost) zero
    assert np.abs(z[w.P:]).max() < 1e-6
    # dropping a client and renormalising needs no new keys
    sub = alpha[1:] / alpha[1:].sum()
    agg2 = ctx.rescale(ctx.weighted_sum(cts[1:], ctx.weights(sub)))
    z2 = ctx.decode(ctx.decrypt(s, agg2, w.L - 1)).reshape(-1)[: w.P]
    want2 = sum(a * x.astype(np.float64) for a, x in zip(sub, xs[1:]))
    assert np.abs(z2 - want2).max() < 1e-6


def test_more_scaling_bits_give_a_closer_result():
    """The paper's parameter study: a larger scaling factor brings the decrypted value
    closer to the plaintext one."""
    errs = []
    for ld in (20, 30, 40):
        w = si.Workload("s", 8192, si.PRIMES_N8192, ld, 3, 4096, 0.02, seed=3)
        ctx = oracle.Context(w.N, w.primes, ld)
        out = ctx.round(si.client_updates(w), si.client_weights(w), None, w.P, 1, 2)
        want = sum(a * x.astype(np.float64) for a, x in zip(si.client_weights(w), si.client_updates(w)))
        errs.append(np.abs(out - want).max())
    assert errs[0] > 50 * errs[1] > 50 * 50 * errs[2]
