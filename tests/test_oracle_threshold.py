"""Pins for the oracle's two-party threshold decryption (paper appendix, "Key Management And
Threshold HE"): shares add up to the secret, the merged partial decryptions equal the single-key
decryption plus exactly the two smudging terms, and the decoded result stays close."""
import numpy as np

import oracle
import synthetic_inputs as si


def centred(v, q):
    v = v.astype(object)
    return np.array([int(x) - q if int(x) > q // 2 else int(x) for x in v], dtype=object)


def test_shares_add_up_to_the_secret_and_look_uniform():
    N, primes = 8192, si.PRIMES_N8192
    ctx = oracle.Context(N, primes, 40)
    s, _ = ctx.keygen(3)
    a, b = ctx.threshold_split(s, 77)
    for j, q in enumerate(primes):
        assert np.array_equal(a[j], oracle.sample_uniform(77, 0, 0, 7, j, q, N))
        tot = (a[j].astype(object) + b[j].astype(object)) % q
        want = np.array([int(v) % q for v in s], dtype=object)
        assert np.array_equal(tot, want)
        assert abs(a[j].astype(np.float64).mean() / q - 0.5) < 0.02
    a2, _ = ctx.threshold_split(s, 78)
    assert not np.array_equal(a, a2)


def test_smudging_noise_range_and_coordinates():
    for bits in (0, 8, 20, 40):
        e = oracle.sample_smudge(5, 2, 1, bits, 4096)
        assert e.min() >= -(1 << bits) and e.max() < (1 << bits)
        if bits:
            assert abs(e.astype(np.float64).mean()) < 4 * (1 << bits) / np.sqrt(3 * 4096)
            assert e.astype(np.float64).std() > 0.5 * (1 << bits) / np.sqrt(3)
    # restated from the stream definition over the pinned Philox
    e = oracle.sample_smudge(0x1122334455, 9, 1, 12, 64)
    for j in range(64):
        w = [int(x) for x in oracle.philox4x32_10([j >> 1, 9, 1, 8], [0x22334455, 0x11])]
        r = w[2 * (j & 1)] | (w[2 * (j & 1) + 1] << 32)
        assert int(e[j]) == (r >> (63 - 12)) - (1 << 12)
    assert not np.array_equal(e, oracle.sample_smudge(0x1122334455, 9, 0, 12, 64))


def test_merged_partial_decryptions_equal_decryption_plus_smudging():
    w = si.scaled(si.TINY, 4096 + 50, name="thr")
    ctx = oracle.Context(w.N, w.primes, w.log2_delta)
    s, pk = ctx.keygen(w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    cts = [ctx.encrypt(pk, ctx.pack(None, w.P, x)[0], w.enc_seed, i)[0] for i, x in enumerate(xs)]
    agg = ctx.rescale(ctx.weighted_sum(cts, ctx.weights(alpha)))
    level, bits, seed = w.L - 1, 10, 4242
    shares = ctx.threshold_split(s, 99)
    q0 = w.primes[0]
    single = ctx.decrypt(s, agg, level)
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    for t in range(agg.shape[0]):
        parts = [ctx.partial_decrypt(shares[p], p, agg[t], level, seed, t, bits) for p in range(2)]
        d = ctx.threshold_combine(agg[t], level, parts)
        e = oracle.sample_smudge(seed, t, 0, bits, w.N) + oracle.sample_smudge(seed, t, 1, bits, w.N)
        assert np.array_equal(d, single[t] + e)
        # one part alone reveals nothing close to the message
        alone = ctx.threshold_combine(agg[t], level, parts[:1])
        assert np.abs(alone.astype(np.float64)).mean() > q0 / 8
        z = ctx.decode(d)
        lo, hi = t * w.n, min((t + 1) * w.n, w.P)
        # smudging of 2^10 per coefficient at scale 2^40 costs about 2^10 sqrt(N) / 2^40 per slot
        assert np.abs(z[: hi - lo] - want[lo:hi]).max() < 1e-5
    # without smudging (bits = 0 gives -1 or 0 per party) the result is the plain one up to 2 units
    parts = [ctx.partial_decrypt(shares[p], p, agg[0], level, seed, 0, 0) for p in range(2)]
    d0 = ctx.threshold_combine(agg[0], level, parts)
    assert np.abs(d0 - single[0]).max() <= 2
