"""GPU parity: every step of the CUDA path, called through the C ABI, against the
CPU oracle on the same seeded inputs.  Integer outputs (transforms, keys,
encoded polynomials, ciphertexts, aggregates, masks, packing) must be
bit-exact; decoded fp64 values within 1e-9 of the oracle's decode and within
1e-6 of plaintext FedAvg."""
import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as si
from gpu_common import dev_f32, to_dev_u64, to_host_u64

pytestmark = pytest.mark.gpu

DECODE_TOL = 1e-9     # GPU decode vs oracle decode (same integers in, fp64 transform order differs)
FEDAVG_TOL = 1e-6     # homomorphic result vs plaintext weighted average


@pytest.fixture(scope="module")
def he():
    import paper_2303_10837_b200 as he
    assert torch.cuda.is_available()
    return he


def fresh_noise_bound(N, log2_delta):
    """Bound on the slot error of ONE fresh ciphertext.  The noise polynomial v = e u + e0 + e1 s
    has per-coefficient variance sigma^2 (4N/3 + 1) and a slot's real part sums N coefficients at
    half weight, which gives the standard deviation; but a slot sees e(zeta) u(zeta), a product of
    two near-Gaussian values, so the error is Laplace-tailed, P(|err| > t std) = exp(-sqrt(2) t),
    and the largest of 3e4 slots sits near 7 std.  18 std leaves 1e-11 per slot.  (The 1e-6 bound is
    stated for the weighted aggregate; a single ciphertext on the longest ring at scale 2^40 has a
    standard deviation of 1.6e-7 and exceeds it.)"""
    return 18.0 * 3.2 * np.sqrt((4.0 * N / 3.0 + 1.0) * N / 2.0) / 2.0 ** log2_delta


def contexts(he, N, primes, ld):
    return he.he_ctx_create(N, list(primes), ld), oracle.Context(N, primes, ld)


# --------------------------------------------------------------------------- transforms

@pytest.mark.parametrize("N,L,B", [(8192, 2, 5), (16384, 4, 3), (32768, 2, 3), (65536, 4, 2), (16384, 12, 1)])
def test_ntt_forward_inverse_bit_exact(he, N, L, B):
    primes = si.PRIMES_SWEEP[:L]
    g, o = contexts(he, N, primes, 40)
    a = si.random_residues(N + L, (B, L, N), primes)
    a[0, 0, :] = 0
    a[0, 0, 1] = 1                                   # impulse: output = odd powers of psi
    a[B - 1, L - 1, :] = primes[L - 1] - 1           # all-maximal residues
    d = to_dev_u64(a)
    he.he_ntt_forward(g, d)
    f = to_host_u64(d)
    for b in range(B):
        for j in range(L):
            assert np.array_equal(f[b, j], o.ntt_forward(j, a[b, j])), (b, j)
    he.he_ntt_inverse(g, d)
    assert np.array_equal(to_host_u64(d), a)
    # inverse alone on arbitrary data
    d2 = to_dev_u64(a)
    he.he_ntt_inverse(g, d2)
    i2 = to_host_u64(d2)
    for j in range(L):
        assert np.array_equal(i2[0, j], o.ntt_inverse(j, a[0, j]))


@pytest.mark.parametrize("N,primes", [(8192, si.PRIMES_N8192), (16384, si.PRIMES_N16384),
                                      (32768, si.PRIMES_N32768), (65536, si.PRIMES_SWEEP[:3])])
def test_keygen_bit_exact(he, N, primes):
    g, o = contexts(he, N, primes, 40)
    keys = he.he_keygen(g, 0xABCDEF0123)
    pk, s = he.he_keys_export(g, keys)
    s_o, pk_o = o.keygen(0xABCDEF0123)
    assert np.array_equal(s.cpu().numpy(), s_o)
    assert np.array_equal(to_host_u64(pk), pk_o)


# --------------------------------------------------------------------------- encode / encrypt

def long_ring(name, primes, P, clients=2):
    """N = 65536 (the longest ring of the kernel sweep): the transform is cut into 8 blocks."""
    return si.Workload(name, 65536, tuple(primes), 40, clients, P, 0.01, seed=6, key_seed=61, enc_seed=62)


def workload_cases():
    return [
        si.scaled(si.TINY, 2 * 4096 + 101, name="tiny-ragged"),               # N=8192, 3 cts, ragged tail
        si.scaled(si.RESNET18, 3 * 8192 - 7, clients=3, name="r18-ragged"),    # N=16384, L=4
        si.scaled(si.bert(1.0), 16384 + 33, clients=2, name="bert-ragged"),    # N=32768, L=6, Delta=2^45
        # N=65536: three 60-bit primes (integer limbs), three 45-bit primes (limbs in doubles), mixed
        long_ring("n65536-int", si.PRIMES_SWEEP[:3], 32768 + 77),
        long_ring("n65536-f64", si.PRIMES_SWEEP_45[:3], 2 * 32768 - 5),
        long_ring("n65536-mixed", (si.PRIMES_SWEEP[0], si.PRIMES_SWEEP_45[0], si.PRIMES_SWEEP[1]), 32768 + 1),
    ]


@pytest.mark.parametrize("w", workload_cases(), ids=lambda w: w.name)
def test_encode_bit_exact(he, w):
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    x = si.client_update(w, 0)
    sel_o, _ = o.pack(None, w.P, x)
    sel, _ = he.he_pack(g, None, dev_f32(x))
    assert np.array_equal(sel.cpu().numpy(), sel_o)
    m = he.he_encode(g, sel).cpu().numpy()
    for t in range(w.T):
        m_o, ov = o.encode(sel_o[t * w.n:(t + 1) * w.n])
        assert not ov
        assert np.array_equal(m[t], m_o), t
    assert he.he_ctx_status(g) == he.HE_OK


def test_encode_special_values_and_overflow_flag(he):
    w = si.TINY
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    z = np.zeros(2 * w.n, np.float32)
    z[: w.n] = 0.25                              # constant slots -> constant polynomial
    z[w.n + 5] = -1.5
    m = he.he_encode(g, dev_f32(z)).cpu().numpy()
    assert m[0, 0] == 2**38 and not m[0, 1:].any()
    assert np.array_equal(m[1], o.encode(z[w.n:])[0])
    assert he.he_ctx_status(g) == he.HE_OK
    z[3] = 3e38                                   # |coefficient| >= 2^62: flagged, not trapped
    m = he.he_encode(g, dev_f32(z)).cpu().numpy()
    assert he.he_ctx_status(g) == he.HE_ERR_OVERFLOW
    assert he.he_ctx_status(g) == he.HE_OK        # sticky word is cleared by the read
    m_o, ov = o.encode(z[: w.n])
    assert ov and np.array_equal(m[0], m_o)


@pytest.mark.parametrize("w", workload_cases(), ids=lambda w: w.name)
def test_encrypt_aggregate_decrypt_bit_exact(he, w):
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    s_o, pk_o = o.keygen(w.key_seed)
    xs = si.client_updates(w)
    alpha = si.client_weights(w)
    cts, cts_o = [], []
    for i, x in enumerate(xs):
        sel, _ = he.he_pack(g, None, dev_f32(x))
        ct = he.he_encrypt(g, keys, sel, w.enc_seed, i)
        ct_o, bad = o.encrypt(pk_o, o.pack(None, w.P, x)[0], w.enc_seed, i)
        assert bad == 0
        assert np.array_equal(to_host_u64(ct), ct_o), "ciphertext of client %d" % i
        cts.append(ct)
        cts_o.append(ct_o)
    # chunked encryption uses the absolute ciphertext index
    sel, _ = he.he_pack(g, None, dev_f32(xs[0]))
    part = torch.empty((w.T - 1, 2, w.L, w.N), dtype=torch.int64, device="cuda")
    he.he_encrypt_range(g, keys, sel[w.n:], 1, w.T - 1, w.enc_seed, 0, part)
    assert torch.equal(part, cts[0][1:])
    # server
    agg = he.he_weighted_aggregate(g, cts, alpha)
    agg_o = o.rescale(o.weighted_sum(cts_o, o.weights(alpha)))
    assert np.array_equal(to_host_u64(agg), agg_o)
    # client
    z = he.he_decrypt(g, keys, agg).cpu().numpy()
    z_o = o.decode(o.decrypt(s_o, agg_o, w.L - 1)).reshape(-1)
    assert np.abs(z - z_o).max() <= DECODE_TOL
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(z[: w.P] - want).max() <= FEDAVG_TOL
    out = he.he_unpack(g, None, torch.from_numpy(z).cuda(), None, w.P).cpu().numpy()
    assert np.array_equal(out, z[: w.P])
    # a fresh ciphertext opens to its own message
    z0 = he.he_decrypt_level(g, keys, cts[0], w.L).cpu().numpy()
    assert np.abs(z0[: w.P] - xs[0].astype(np.float64)).max() <= fresh_noise_bound(w.N, w.log2_delta)
    assert he.he_ctx_status(g) == he.HE_OK


@pytest.mark.parametrize("base", [si.TINY, si.RESNET18, si.bert(1.0),
                                  long_ring("n65536-mixed-large", (si.PRIMES_SWEEP[0], si.PRIMES_SWEEP_45[0],
                                                                   si.PRIMES_SWEEP[1]), 32768)],
                         ids=lambda w: w.name)
def test_encrypt_large_messages_bit_exact(he, base):
    """Encoded coefficients above the small primes and close to the large ones: the full
    reduction of m + e0 and every wrap of the final additions, next to a ciphertext of
    ordinary small updates in the same call."""
    w = si.scaled(base, 3 * base.n, clients=1)
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    _, pk_o = o.keygen(w.key_seed)
    rng = np.random.default_rng(77)
    big = 2.0 ** (58.7 - w.log2_delta) * np.sqrt(w.n)  # slot deviation that gives coefficients up to about 2^60.3
    x = np.concatenate([rng.normal(0, 0.01, w.n), rng.normal(0, big, w.n),
                        np.where(rng.random(w.n) < 0.05, rng.normal(0, big, w.n), 0.0)])
    x = x.astype(np.float32)
    m = he.he_encode(g, dev_f32(x)).cpu().numpy()
    assert he.he_ctx_status(g) == he.HE_OK
    assert np.abs(m[0]).max() < min(w.primes) and np.abs(m[2]).max() > min(w.primes)
    assert max(w.primes) < np.abs(m[1]).max() < 2**62
    ct = he.he_encrypt(g, keys, dev_f32(x), w.enc_seed, 0)
    ct_o, bad = o.encrypt(pk_o, x, w.enc_seed, 0)
    assert bad == 0
    assert np.array_equal(to_host_u64(ct), ct_o)


def oracle_ntt_of(o, ct):
    """Every limb polynomial of an oracle ciphertext [T][2][level][N] through the oracle's forward transform."""
    out = np.empty_like(ct)
    for t in range(ct.shape[0]):
        for c in range(2):
            for j in range(ct.shape[2]):
                out[t, c, j] = o.ntt_forward(j, ct[t, c, j])
    return out


@pytest.mark.parametrize("w", workload_cases(), ids=lambda w: w.name)
def test_transform_domain_format_bit_exact(he, w):
    """The alternative wire format: each step equals the transform of the oracle's coefficient-domain
    result, and the decrypted slots are those of the coefficient path."""
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    s_o, pk_o = o.keygen(w.key_seed)
    xs = si.client_updates(w)
    alpha = si.client_weights(w)
    cts, cts_o = [], []
    for i, x in enumerate(xs):
        sel, _ = he.he_pack(g, None, dev_f32(x))
        ct = he.he_encrypt_ntt(g, keys, sel, w.enc_seed, i)
        ct_o, bad = o.encrypt(pk_o, o.pack(None, w.P, x)[0], w.enc_seed, i)
        assert bad == 0
        assert np.array_equal(to_host_u64(ct), oracle_ntt_of(o, ct_o)), "ciphertext of client %d" % i
        # the same bytes as transforming the coefficient-domain ciphertext
        ref = he.he_encrypt(g, keys, sel, w.enc_seed, i)
        he.he_ntt_forward(g, ref.view(-1, w.L, w.N))
        assert torch.equal(ct, ref)
        cts.append(ct)
        cts_o.append(ct_o)
    agg = he.he_weighted_aggregate_ntt(g, cts, alpha)
    agg_o = o.rescale(o.weighted_sum(cts_o, o.weights(alpha)))
    assert np.array_equal(to_host_u64(agg), oracle_ntt_of(o, agg_o))
    z = he.he_decrypt_level_ntt(g, keys, agg, w.L - 1).cpu().numpy()
    z_o = o.decode(o.decrypt(s_o, agg_o, w.L - 1)).reshape(-1)
    assert np.abs(z - z_o).max() <= DECODE_TOL
    z0 = he.he_decrypt_level_ntt(g, keys, cts[0], w.L).cpu().numpy()
    assert np.abs(z0[: w.P] - xs[0].astype(np.float64)).max() <= fresh_noise_bound(w.N, w.log2_delta)
    assert he.he_ctx_status(g) == he.HE_OK


def test_dropout_subset_of_clients(he):
    """Aggregating any subset with renormalised weights needs no new keys."""
    w = si.scaled(si.RESNET18, 8192 + 11, clients=4, name="r18-dropout")
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    cts = [he.he_encrypt(g, keys, he.he_pack(g, None, dev_f32(x))[0], w.enc_seed, i) for i, x in enumerate(xs)]
    keep = [0, 2, 3]
    sub = alpha[keep] / alpha[keep].sum()
    z = he.he_decrypt(g, keys, he.he_weighted_aggregate(g, [cts[i] for i in keep], sub)).cpu().numpy()
    want = sum(a * xs[i].astype(np.float64) for a, i in zip(sub, keep))
    assert np.abs(z[: w.P] - want).max() <= FEDAVG_TOL
    # one client with weight 1 is a plain re-scaling
    z1 = he.he_decrypt(g, keys, he.he_weighted_aggregate(g, [cts[1]], [1.0])).cpu().numpy()
    assert np.abs(z1[: w.P] - xs[1].astype(np.float64)).max() <= FEDAVG_TOL


# --------------------------------------------------------------------------- mask and packing

def test_select_mask_bit_exact(he):
    g, _ = contexts(he, 8192, si.PRIMES_N8192, 40)
    w = si.scaled(si.RESNET50_TOP10, 100_003)
    score = si.sensitivity_scores(w)
    d = dev_f32(score)
    for k in (0, 1, 1000, w.k, 99_999, w.P):
        mask = he.he_select_mask(g, d, k)
        assert mask.k == k
        got = he.he_mask_indices(mask).cpu().numpy().view(np.uint32)
        assert np.array_equal(got, oracle.select_mask(score, k)), k


def test_select_mask_ties_and_special_values(he):
    g, _ = contexts(he, 8192, si.PRIMES_N8192, 40)
    rng = np.random.default_rng(5)
    score = rng.integers(0, 4, size=5000).astype(np.float32)        # heavy ties
    score[17] = np.nan
    score[18] = -1.0
    score[19] = -0.0
    score[20] = np.inf
    d = dev_f32(score)
    for k in (1, 2, 100, 1234, 2500, 4999, 5000):
        got = he.he_mask_indices(he.he_select_mask(g, d, k)).cpu().numpy().view(np.uint32)
        assert np.array_equal(got, oracle.select_mask(score, k)), k
    same = np.full(4097, 0.125, np.float32)
    got = he.he_mask_indices(he.he_select_mask(g, dev_f32(same), 33)).cpu().numpy()
    assert list(got) == list(range(33))


def test_mask_with_forced_ranges(he):
    """Top-k plus whole index ranges (first and last layers)."""
    g, _ = contexts(he, 8192, si.PRIMES_N8192, 40)
    w = si.scaled(si.RESNET50_TOP10, 50_000)
    score = si.sensitivity_scores(w)
    ranges = [(0, 700), (49_000, 50_000)]
    mask = he.he_select_mask_ranges(g, dev_f32(score), w.k, ranges)
    got = he.he_mask_indices(mask).cpu().numpy().view(np.uint32)
    top = oracle.select_mask(score, w.k)
    want = np.union1d(top, np.concatenate([np.arange(a, b) for a, b in ranges])).astype(np.uint32)
    assert np.array_equal(got, want) and mask.k == want.size


def test_pack_unpack_plain_aggregate_bit_exact(he):
    w = si.scaled(si.RESNET50_TOP10, 70_001, clients=4)
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    score = si.sensitivity_scores(w)
    mask = he.he_select_mask(g, dev_f32(score), w.k)
    idx = oracle.select_mask(score, w.k)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    rests = []
    for x in xs:
        sel, rest = he.he_pack(g, mask, dev_f32(x))
        sel_o, rest_o = o.pack(idx, w.k, x)
        assert np.array_equal(sel.cpu().numpy(), sel_o)
        assert np.array_equal(rest.cpu().numpy(), rest_o)
        rests.append(rest)
    avg = he.he_plain_aggregate(g, rests, alpha)
    avg_o = oracle.plain_aggregate([r.cpu().numpy() for r in rests], alpha)
    assert np.array_equal(avg.cpu().numpy(), avg_o)
    z = np.random.default_rng(1).standard_normal(he.he_num_ct(g, w.k) * w.n)
    out = he.he_unpack(g, mask, torch.from_numpy(z).cuda(), avg, w.P).cpu().numpy()
    assert np.array_equal(out, oracle.unpack(idx, w.k, z, avg_o, w.P))


# --------------------------------------------------------------------------- whole rounds

def run_round_gpu(he, g, keys, mask, xs, alpha, w):
    cts, rests = [], []
    for i, x in enumerate(xs):
        sel, rest = he.he_pack(g, mask, dev_f32(x))
        cts.append(he.he_encrypt(g, keys, sel, w.enc_seed, i))
        rests.append(rest)
    z = he.he_decrypt(g, keys, he.he_weighted_aggregate(g, cts, alpha))
    avg = he.he_plain_aggregate(g, rests, alpha) if mask is not None else None
    return he.he_unpack(g, mask, z, avg, w.P).cpu().numpy()


def test_tiny_config_whole_round(he):
    """Config 1 in full: N=8192, 60/40/60-bit primes, 3 clients, 100,000 parameters."""
    w = si.TINY
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    out = run_round_gpu(he, g, keys, None, xs, alpha, w)
    out_o = o.round(xs, alpha, None, w.P, w.key_seed, w.enc_seed)
    assert np.abs(out - out_o).max() <= DECODE_TOL
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(out - want).max() <= FEDAVG_TOL
    # the same through the host-buffer entry point
    host = torch.empty(w.P, dtype=torch.float64)
    he.he_round_host(g, keys, None, [torch.from_numpy(x) for x in xs], alpha, w.enc_seed, host)
    assert np.array_equal(host.numpy(), out)


def test_host_round_in_several_chunks(he):
    """The host-buffer entry point splits a large round into chunks of ciphertext indices (here
    296 + 296 + 8, ragged tail in the last ciphertext) and downloads each chunk's slots while the
    next is computed: same result as the device calls on the whole range, bit for bit, and FedAvg."""
    w = si.scaled(si.TINY, 600 * 4096 - 37, clients=2, name="tiny-600cts")
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    out = run_round_gpu(he, g, keys, None, xs, alpha, w)
    host = torch.full((w.P,), np.nan, dtype=torch.float64).pin_memory()
    he.he_round_host(g, keys, None, [torch.from_numpy(x).pin_memory() for x in xs], alpha, w.enc_seed, host)
    assert np.array_equal(host.numpy(), out)
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(out - want).max() <= FEDAVG_TOL


@pytest.mark.parametrize("P,clients", [(1, 1), (4096, 2), (148 * 4096, 1), (449 * 4096 + 17, 3), (30 * 4096 - 1, 5)])
def test_host_round_sizes(he, P, clients):
    """The host-buffer entry point on one context after the other of several sizes (one slot, exactly
    one ciphertext, exactly one wave, several chunks with a ragged tail, more clients): the same bits
    as the device calls, whatever the chunk schedule."""
    w = si.scaled(si.TINY, P, clients=clients, name="host-%d-%d" % (P, clients))
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    out = run_round_gpu(he, g, keys, None, xs, alpha, w)
    for _ in range(2):                                  # the second call reuses the buffers of the first
        host = torch.full((w.P,), np.nan, dtype=torch.float64).pin_memory()
        he.he_round_host(g, keys, None, [torch.from_numpy(x).pin_memory() for x in xs], alpha, w.enc_seed, host)
        assert np.array_equal(host.numpy(), out)
    assert he.he_ctx_status(g) == he.HE_OK


def test_selective_round_with_mask(he):
    """Config 3 shape at reduced size: top-10 % encrypted, the rest averaged in plaintext."""
    w = si.scaled(si.RESNET50_TOP10, 300_000, clients=4)
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    score = si.sensitivity_scores(w)
    mask = he.he_select_mask(g, dev_f32(score), w.k)
    idx = oracle.select_mask(score, w.k)
    assert np.array_equal(he.he_mask_indices(mask).cpu().numpy().view(np.uint32), idx)
    out = run_round_gpu(he, g, keys, mask, xs, alpha, w)
    out_o = o.round(xs, alpha, idx, w.k, w.key_seed, w.enc_seed)
    comp = np.setdiff1d(np.arange(w.P), idx)
    assert np.array_equal(out[comp], out_o[comp])                   # plaintext part: bit-exact
    assert np.abs(out[idx] - out_o[idx]).max() <= DECODE_TOL
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(out - want).max() <= FEDAVG_TOL
    host = torch.empty(w.P, dtype=torch.float64)
    he.he_round_host(g, keys, mask, [torch.from_numpy(x) for x in xs], alpha, w.enc_seed, host)
    assert np.array_equal(host.numpy(), out)


def test_empty_and_degenerate_inputs(he):
    w = si.TINY
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, 1)
    # P = 1: one slot used, one whole ciphertext
    x = np.array([0.5], np.float32)
    sel, _ = he.he_pack(g, None, dev_f32(x))
    assert sel.numel() == w.n and float(sel[0]) == 0.5 and not sel[1:].any()
    ct = he.he_encrypt(g, keys, sel, 3, 0)
    assert ct.shape == (1, 2, w.L, w.N)
    z = he.he_decrypt(g, keys, he.he_weighted_aggregate(g, [ct], [1.0])).cpu().numpy()
    assert abs(z[0] - 0.5) <= FEDAVG_TOL and np.abs(z[1:]).max() <= FEDAVG_TOL
    # k = 0: nothing is encrypted, everything is averaged in plaintext
    score = dev_f32(np.arange(1000, dtype=np.float32))
    mask = he.he_select_mask(g, score, 0)
    xs = [np.full(1000, 1.0, np.float32), np.full(1000, 3.0, np.float32)]
    sel, rest = he.he_pack(g, mask, dev_f32(xs[0]))
    assert sel.numel() == 0 and rest.numel() == 1000
    out = run_round_gpu(he, g, keys, mask, xs, [0.25, 0.75], si.scaled(w, 1000, clients=2))
    assert np.array_equal(out, np.full(1000, 2.5))
    # invalid arguments come back as error codes
    with pytest.raises(he.HeError) as ei:
        he.he_select_mask(g, score, 1001)
    assert ei.value.code == he.HE_ERR_INVALID_ARG
    with pytest.raises(he.HeError) as ei:
        he.he_weighted_aggregate(g, [ct], [1.5])
    assert ei.value.code == he.HE_ERR_INVALID_ARG
    with pytest.raises(he.HeError) as ei:
        he.he_decrypt_level(g, keys, ct, w.L + 1)
    assert ei.value.code == he.HE_ERR_LEVEL
    other = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    with pytest.raises(he.HeError) as ei:
        he.he_encrypt(other, keys, sel if sel.numel() else dev_f32(np.zeros(w.n, np.float32)), 1, 0)
    assert ei.value.code == he.HE_ERR_INVALID_ARG


def test_unaligned_word_buffers_are_refused(he):
    """Ciphertext-like buffers are moved two words at a time: a pointer at an odd word offset comes
    back as an error from the host-side check, never as a misaligned access on the device."""
    w = si.scaled(si.TINY, 4096, clients=1)
    g, _ = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, 1)
    sel, _ = he.he_pack(g, None, dev_f32(si.client_update(w, 0)))

    def odd(shape):
        count = int(np.prod(shape))
        return torch.zeros(count + 1, dtype=torch.int64, device="cuda")[1:].view(shape)

    ct = he.he_encrypt(g, keys, sel, 1, 0)
    agg = he.he_weighted_aggregate(g, [ct], [1.0])
    ct_odd, agg_odd = odd(ct.shape), odd(agg.shape)
    ct_odd.copy_(ct)
    agg_odd.copy_(agg)
    assert ct_odd.data_ptr() % 16 == 8
    calls = [
        lambda: he.he_encrypt(g, keys, sel, 1, 0, out=ct_odd),
        lambda: he.he_encrypt_ntt(g, keys, sel, 1, 0, out=ct_odd),
        lambda: he.he_weighted_aggregate(g, [ct_odd], [1.0]),
        lambda: he.he_weighted_aggregate(g, [ct], [1.0], out=agg_odd),
        lambda: he.he_decrypt(g, keys, agg_odd),
        lambda: he.he_decrypt_level(g, keys, ct_odd, w.L),
        lambda: he.he_decrypt_noalloc(g, keys, agg_odd, torch.empty(w.n, dtype=torch.float64, device="cuda")),
        lambda: he.he_ntt_forward(g, odd((1, w.L, w.N))),
        lambda: he.he_ntt_inverse(g, odd((1, w.L, w.N))),
    ]
    for call in calls:
        with pytest.raises(he.HeError) as ei:
            call()
        assert ei.value.code == he.HE_ERR_INVALID_ARG
    # the context is as usable as before
    z = he.he_decrypt(g, keys, agg).cpu().numpy()
    assert np.abs(z[: w.P] - si.client_update(w, 0).astype(np.float64)).max() <= FEDAVG_TOL


def test_host_round_refuses_bad_arguments_before_queueing(he):
    """A missing client buffer or a weight outside [0, 1] is an error return with nothing queued,
    and the same context then runs a correct round."""
    import ctypes as C
    w = si.scaled(si.TINY, 3 * 4096 + 5, clients=3)
    g, _ = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    xs_t = [torch.from_numpy(x).pin_memory() for x in xs]
    host = torch.full((w.P,), np.nan, dtype=torch.float64).pin_memory()
    lib = C.CDLL(he.LIB_PATH)
    lib.he_round_host.restype = C.c_int
    lib.he_round_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_size_t,
                                  C.c_uint64, C.c_void_p, C.c_void_p]
    al = (C.c_double * 3)(*[float(a) for a in alpha])
    ptrs = (C.c_void_p * 3)(xs_t[0].data_ptr(), None, xs_t[2].data_ptr())          # client 1 is missing
    before = he.he_launch_count()
    rc = lib.he_round_host(g.handle, keys.handle, None, C.cast(ptrs, C.c_void_p), C.cast(al, C.c_void_p), 3, w.P,
                           w.enc_seed, host.data_ptr(), None)
    assert rc == he.HE_ERR_INVALID_ARG and he.he_launch_count() == before
    assert bool(torch.isnan(host).all())                                             # nothing was written
    with pytest.raises(he.HeError) as ei:
        he.he_round_host(g, keys, None, xs_t, [0.5, 0.7, -0.2], w.enc_seed, host)
    assert ei.value.code == he.HE_ERR_INVALID_ARG and he.he_launch_count() == before
    he.he_round_host(g, keys, None, xs_t, alpha, w.enc_seed, host)
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(host.numpy() - want).max() <= FEDAVG_TOL


@pytest.mark.parametrize("primes,C", [((si.PRIMES_SWEEP[0], si.PRIMES_SWEEP_45[0], si.PRIMES_SWEEP_45[1]), 70),
                                      (si.PRIMES_SWEEP_45[:3], 131), (si.PRIMES_N8192, 37),
                                      ((si.PRIMES_SWEEP_45[0], si.PRIMES_SWEEP[0], si.PRIMES_SWEEP[1]), 5)],
                         ids=["f64-last-70", "all-f64-131", "mixed-37", "int-last-5"])
def test_weighted_aggregate_many_clients_bit_exact(he, primes, C):
    """The server's sum on arbitrary residues (all-maximal ones among them) for client counts beyond
    one unrolled group and beyond the interval at which the sums in doubles are reduced, with the
    dropped prime in either arithmetic; also in two halves."""
    N, T = 8192, 2
    g, o = contexts(he, N, primes, 30)
    rng = np.random.default_rng(77)
    cts_o = []
    for i in range(C):
        ct = si.random_residues(100 + i, (T, 2, len(primes), N), primes)
        if i % 9 == 0:
            for j, q in enumerate(primes):
                ct[0, :, j, : N // 2] = q - 1
        cts_o.append(ct)
    alpha = rng.random(C)
    alpha /= alpha.sum()
    cts = [to_dev_u64(c) for c in cts_o]
    W = o.weights(alpha)
    want = o.rescale(o.weighted_sum(cts_o, W))
    assert np.array_equal(to_host_u64(he.he_weighted_aggregate(g, cts, alpha)), want)
    half = C // 2 + 1
    parts = [he.he_weighted_partial(g, cts[:half], alpha[:half]), he.he_weighted_partial(g, cts[half:], alpha[half:])]
    assert np.array_equal(to_host_u64(parts[0]), o.weighted_sum(cts_o[:half], W[:half]))
    assert np.array_equal(to_host_u64(he.he_rescale_partial_parts(g, parts)), want)


@pytest.mark.parametrize("N,primes,ld", [(8192, si.PRIMES_N8192, 40), (16384, si.PRIMES_N16384, 40),
                                         (32768, si.PRIMES_N32768, 45)],
                         ids=["n8192", "n16384", "n32768"])
def test_client_partition_reproduces_the_whole_aggregate(he, N, primes, ld):
    """The server step in two halves (clients spread over GPUs): the partial weighted sums of
    three groups of clients equal the oracle's, and their word-by-word sum, rescaled, equals both
    the one-call aggregate and the oracle's rescale, bit for bit."""
    w = si.Workload("client-groups", N, primes, ld, 5, 2 * (N // 2) + 11, 0.01, ratio=1.0, seed=31,
                    key_seed=311, enc_seed=312, weights="uniform")
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    cts = [he.he_encrypt(g, keys, he.he_pack(g, None, dev_f32(x))[0], w.enc_seed, i) for i, x in enumerate(xs)]
    cts_o = [to_host_u64(c) for c in cts]                 # ciphertext parity is covered above
    W = o.weights(alpha)
    groups = [(0, 1), (1, 4), (4, 5)]
    parts = []
    for b, e in groups:
        part = he.he_weighted_partial(g, cts[b:e], alpha[b:e])
        assert np.array_equal(to_host_u64(part), o.weighted_sum(cts_o[b:e], W[b:e])), (b, e)
        parts.append(part)
    summed = parts[0] + parts[1] + parts[2]               # 64-bit words, as a reduce-scatter would add them
    agg = he.he_rescale_partial_sum(g, summed, len(parts))
    whole = he.he_weighted_aggregate(g, cts, alpha)
    assert torch.equal(agg, whole)
    assert np.array_equal(to_host_u64(agg), o.rescale(o.weighted_sum(cts_o, W)))
    assert torch.equal(he.he_rescale_partial_parts(g, parts), whole)       # added by the kernel itself
    # a single part is the one-call aggregate as well
    assert torch.equal(he.he_rescale_partial_sum(g, he.he_weighted_partial(g, cts, alpha), 1), whole)
    # seventeen sums of residues of a 60-bit prime could overflow 64 bits
    with pytest.raises(he.HeError) as ei:
        he.he_rescale_partial_sum(g, summed, 17)
    assert ei.value.code == he.HE_ERR_SIZE
    with pytest.raises(he.HeError) as ei:
        he.he_rescale_partial_sum(g, summed, 0)
    assert ei.value.code == he.HE_ERR_INVALID_ARG
    z = he.he_decrypt(g, keys, agg).cpu().numpy()
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(z[: w.P] - want).max() <= FEDAVG_TOL
    assert he.he_ctx_status(g) == he.HE_OK


def test_index_partition_reproduces_the_whole_round(he):
    """The multi-GPU partition (contiguous ciphertext indices and remainder entries per rank, context,
    keys and mask replicated), played by one GPU one rank after the other: the ranks' ciphertexts,
    aggregates, decoded slots and plaintext averages, put side by side, are the single run's, bit for bit."""
    from paper_2303_10837_b200.sharding import shard_range, slot_range
    w = si.Workload("partition", 16384, si.PRIMES_N16384, 40, 3, 7 * 8192 + 123, 0.01, ratio=0.6, seed=9,
                    key_seed=91, enc_seed=92)                      # 5 ciphertexts, the last one ragged
    g, _ = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    xs, alpha = [dev_f32(x) for x in si.client_updates(w)], si.client_weights(w)
    mask = he.he_select_mask(g, dev_f32(si.sensitivity_scores(w)), w.k)
    packed = [he.he_pack(g, mask, x) for x in xs]
    cts = [he.he_encrypt(g, keys, sel, w.enc_seed, i) for i, (sel, _) in enumerate(packed)]
    agg = he.he_weighted_aggregate(g, cts, alpha)
    z = he.he_decrypt(g, keys, agg)
    ravg = he.he_plain_aggregate(g, [rest for _, rest in packed], alpha)
    whole = he.he_unpack(g, mask, z, ravg, w.P)
    world = 3
    z_parts, r_parts = [], []
    for rank in range(world):
        tb, te, sb, se = slot_range(w.T, w.n, w.k, rank, world)
        rb, re = shard_range(w.P - w.k, rank, world)
        mine = []
        for i, (sel, _) in enumerate(packed):
            ct = torch.empty((te - tb, 2, w.L, w.N), dtype=torch.int64, device="cuda")
            he.he_encrypt_range(g, keys, sel[tb * w.n:te * w.n], tb, te - tb, w.enc_seed, i, ct)
            assert torch.equal(ct, cts[i][tb:te])
            mine.append(ct)
        a = he.he_weighted_aggregate(g, mine, alpha)
        assert torch.equal(a, agg[tb:te])
        z_parts.append(he.he_decrypt(g, keys, a)[: se - sb])
        r_parts.append(he.he_plain_aggregate(g, [rest[rb:re] for _, rest in packed], alpha))
    zf = torch.cat(z_parts)
    assert zf.numel() == w.k and torch.equal(zf, z[: w.k])
    assert torch.equal(torch.cat(r_parts), ravg)
    pad = torch.zeros(w.T * w.n - w.k, dtype=torch.float64, device="cuda")
    assert torch.equal(he.he_unpack(g, mask, torch.cat([zf, pad]), torch.cat(r_parts), w.P), whole)


def test_runs_are_deterministic(he):
    """Bit-identical outputs on repeated runs (a race would show up here)."""
    w = si.scaled(si.RESNET18, 5 * 8192, clients=2)
    g, _ = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    sel, _ = he.he_pack(g, None, dev_f32(si.client_update(w, 0)))
    a = he.he_encrypt(g, keys, sel, 5, 1)
    b = he.he_encrypt(g, keys, sel, 5, 1)
    assert torch.equal(a, b)
    c = he.he_encrypt(g, keys, sel, 6, 1)
    assert not torch.equal(a, c)


def test_sensitivity_map_round(he):
    """Stage 2 of Algorithm 1: the clients' sensitivity maps go through the same fully encrypted
    path, the aggregated map is decrypted and the mask is selected from it."""
    w = si.scaled(si.RESNET18, 60_000, clients=3, name="sens-map")
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    s_o, pk_o = o.keygen(w.key_seed)
    rng = np.random.default_rng(17)
    # non-negative, heavy-tailed maps (means of absolute values in the paper)
    maps = [np.abs(rng.standard_cauchy(w.P)).clip(0, 50).astype(np.float32) * np.float32(0.01) for _ in range(w.clients)]
    alpha = si.client_weights(w)
    cts, cts_o = [], []
    for i, s_map in enumerate(maps):
        sel, _ = he.he_pack(g, None, dev_f32(s_map))
        cts.append(he.he_encrypt(g, keys, sel, 99, i))
        cts_o.append(o.encrypt(pk_o, o.pack(None, w.P, s_map)[0], 99, i)[0])
        assert np.array_equal(to_host_u64(cts[-1]), cts_o[-1])
    agg = he.he_weighted_aggregate(g, cts, alpha)
    z = he.he_decrypt(g, keys, agg)[: w.P]
    z_o = o.decode(o.decrypt(s_o, o.rescale(o.weighted_sum(cts_o, o.weights(alpha))), w.L - 1)).reshape(-1)[: w.P]
    assert np.abs(z.cpu().numpy() - z_o).max() <= DECODE_TOL
    want = sum(a * m.astype(np.float64) for a, m in zip(alpha, maps))
    assert np.abs(z.cpu().numpy() - want).max() <= FEDAVG_TOL
    score = z.float().contiguous()
    k = int(round(0.3 * w.P))
    mask = he.he_select_mask(g, score, k)
    got = he.he_mask_indices(mask).cpu().numpy().view(np.uint32)
    assert np.array_equal(got, oracle.select_mask(score.cpu().numpy(), k))
    # the mask agrees with the one a plaintext aggregation would give, except at the noise-level boundary
    plain = oracle.select_mask(want.astype(np.float32), k)
    assert np.intersect1d(got, plain).size >= 0.999 * k


@pytest.mark.parametrize("w", [si.scaled(si.TINY, 4096 + 50, name="thr-tiny"),
                               si.scaled(si.bert(1.0), 16384 + 9, clients=2, name="thr-bert"),
                               long_ring("thr-n65536", (si.PRIMES_SWEEP[0], si.PRIMES_SWEEP_45[0],
                                                        si.PRIMES_SWEEP[1]), 32768 + 3)],
                         ids=lambda w: w.name)
def test_threshold_decryption_bit_exact(he, w):
    """Two-party threshold decryption: partial results bit-exact against the oracle, merged result
    within the decode tolerance, and close to FedAvg up to the smudging noise."""
    g, o = contexts(he, w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    s_o, pk_o = o.keygen(w.key_seed)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    cts = [he.he_encrypt(g, keys, he.he_pack(g, None, dev_f32(x))[0], w.enc_seed, i) for i, x in enumerate(xs)]
    agg = he.he_weighted_aggregate(g, cts, alpha)
    agg_o = to_host_u64(agg)
    level, bits, seed = w.L - 1, 10, 777
    shares = he.he_threshold_split(g, keys, 31)
    shares_o = o.threshold_split(s_o, 31)
    parts = [he.he_partial_decrypt(g, shares[p], p, agg, level, seed, bits) for p in range(2)]
    T = agg.shape[0]
    d_o = np.empty((T, w.N), np.int64)
    for t in range(T):
        po = [o.partial_decrypt(shares_o[p], p, agg_o[t], level, seed, t, bits) for p in range(2)]
        for p in range(2):
            assert np.array_equal(to_host_u64(parts[p][t]), po[p]), (t, p)
        d_o[t] = o.threshold_combine(agg_o[t], level, po)
    z = he.he_threshold_combine(g, agg, level, parts).cpu().numpy()
    assert np.abs(z - o.decode(d_o).reshape(-1)).max() <= DECODE_TOL
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(z[: w.P] - want).max() <= 1e-5           # 2^10 of smudging per coefficient and party
    # shares are not keys: the single-key entry points refuse them
    for bad in (lambda: he.he_decrypt(g, shares[0], agg), lambda: he.he_keys_export(g, shares[0]),
                lambda: he.he_partial_decrypt(g, keys, 0, agg, level, seed, bits)):
        with pytest.raises(he.HeError) as ei:
            bad()
        assert ei.value.code == he.HE_ERR_INVALID_ARG
