"""GPU parity at the full workload sizes, in the launch configuration the benchmark times
(one he_encrypt launch per client over all ciphertexts of the workload; chunks of ciphertext
indices through he_encrypt_range where the ciphertexts of all clients exceed the device).

Extent of the comparison with the oracle:
  * tiny, ResNet-18-sized and ResNet-50-sized workloads: EVERY ciphertext of every client, every
    aggregated ciphertext and every decoded slot (the oracle runs on all host cores, chunk by
    chunk of ciphertext indices, and each chunk is dropped after it was compared);
  * BERT-sized workloads: a seeded sample of ciphertext indices (all of them at 1 %, 256 at 10 %
    and at 100 %), every client, the aggregate and the decoded slots of those indices;
  * on top, at every size: the round equals plaintext FedAvg within 1e-6 on every parameter, the
    mask has the defining order properties, packing is bit-exact.
Integer outputs are compared bit for bit, decoded fp64 values within 1e-9.
"""
import os
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as si
from gpu_common import to_host_u64

pytestmark = pytest.mark.gpu

DECODE_TOL = 1e-9
FEDAVG_TOL = 1e-6

# the oracle's per-ciphertext functions are single-threaded C calls that release the GIL
POOL = ThreadPoolExecutor(max_workers=os.cpu_count() or 4)


@pytest.fixture(scope="module")
def he():
    import paper_2303_10837_b200 as he
    return he


def fedavg(xs_dev, alpha):
    out = torch.zeros(xs_dev[0].numel(), dtype=torch.float64, device="cuda")
    for a, x in zip(alpha, xs_dev):
        out += float(a) * x.double()
    return out


def slots_of(w, idx, x, t):
    """The n slot values of ciphertext index t of one client's update (zero-padded tail)."""
    lo, hi = t * w.n, min((t + 1) * w.n, w.k)
    slots = np.zeros(w.n, np.float32)
    src = np.arange(lo, hi) if idx is None else idx[lo:hi].astype(np.int64)
    slots[: hi - lo] = x[src]
    return slots


def oracle_ciphertexts(o, pk_o, w, idx, x, client, ts):
    """Oracle encryption of the given absolute ciphertext indices: uint64 [len(ts)][2][L][N]."""
    def one(t):
        m, ov = o.encode(slots_of(w, idx, x, t))
        assert not ov
        return o.encrypt_one(pk_o, m, w.enc_seed, client, t)
    return np.stack(list(POOL.map(one, ts)))


def check_indices(w, o, s_o, pk_o, idx, xs, alpha, ts, cts_of, agg_of, z_of):
    """Ciphertexts of every client, the aggregate and the decoded slots of the absolute ciphertext
    indices `ts` against the oracle.  cts_of(i, ts) / agg_of(ts) / z_of(ts) fetch the GPU's values
    (uint64 [len][2][L][N], uint64 [len][2][L-1][N], float64 [len][n])."""
    ts = list(ts)
    mine = []
    for i, x in enumerate(xs):
        want = oracle_ciphertexts(o, pk_o, w, idx, x, i, ts)
        got = cts_of(i, ts)
        assert np.array_equal(got, want), ("ciphertext", i, ts[0], ts[-1])
        mine.append(want)
    agg_o = o.rescale(o.weighted_sum(mine, o.weights(alpha)))
    assert np.array_equal(agg_of(ts), agg_o), ("aggregate", ts[0], ts[-1])
    z_o = o.decode(o.decrypt(s_o, agg_o, w.L - 1))
    assert np.abs(z_of(ts) - z_o).max() <= DECODE_TOL, ("decoded", ts[0], ts[-1])


def run_round(he, g, keys, mask, xs_dev, alpha, w):
    cts, rests = [], []
    for i, x in enumerate(xs_dev):
        sel, rest = he.he_pack(g, mask, x)
        cts.append(he.he_encrypt(g, keys, sel, w.enc_seed, i))
        rests.append(rest)
        del sel
    agg = he.he_weighted_aggregate(g, cts, alpha)
    z = he.he_decrypt(g, keys, agg)
    avg = he.he_plain_aggregate(g, rests, alpha) if mask is not None else None
    return cts, agg, z, he.he_unpack(g, mask, z, avg, w.P)


def check_resident_round(w, o, s_o, pk_o, idx, xs, alpha, cts, agg, z, ts, chunk=64):
    """The indices `ts` of a round whose ciphertexts are all resident on the device."""
    for c0 in range(0, len(ts), chunk):
        part = ts[c0:c0 + chunk]
        sel = torch.as_tensor(part, device="cuda")
        check_indices(w, o, s_o, pk_o, idx, xs, alpha, part,
                      lambda i, _: to_host_u64(cts[i][sel]),
                      lambda _: to_host_u64(agg[sel]),
                      lambda _: z.view(-1, w.n)[sel].cpu().numpy())


def setup(he, w):
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    o = oracle.Context(w.N, w.primes, w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    s_o, pk_o = o.keygen(w.key_seed)
    return g, o, keys, s_o, pk_o


def test_tiny_every_ciphertext(he):
    """100,000 parameters, 3 clients, N = 8192, 60/40/60-bit primes: all 25 ciphertext indices."""
    w = si.TINY
    g, o, keys, s_o, pk_o = setup(he, w)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    xs_dev = [torch.from_numpy(x).cuda() for x in xs]
    cts, agg, z, out = run_round(he, g, keys, None, xs_dev, alpha, w)
    assert float((out - fedavg(xs_dev, alpha)).abs().max()) <= FEDAVG_TOL
    check_resident_round(w, o, s_o, pk_o, None, xs, alpha, cts, agg, z, list(range(w.T)))


def test_resnet18_sized_full_encryption(he):
    """11.7 M parameters, 10 clients, N = 16384, 4 primes: the benchmark's first workload, all
    1429 ciphertext indices of all 10 clients."""
    w = si.RESNET18
    g, o, keys, s_o, pk_o = setup(he, w)
    xs = si.client_updates(w)
    alpha = si.client_weights(w)
    xs_dev = [torch.from_numpy(x).cuda() for x in xs]
    cts, agg, z, out = run_round(he, g, keys, None, xs_dev, alpha, w)
    assert cts[0].shape == (w.T, 2, w.L, w.N) and w.T == 1429
    assert float((out - fedavg(xs_dev, alpha)).abs().max()) <= FEDAVG_TOL
    t0 = time.time()
    check_resident_round(w, o, s_o, pk_o, None, xs, alpha, cts, agg, z, list(range(w.T)))
    print("resnet18-sized: %d ciphertexts x %d clients compared in %.0f s" % (w.T, w.clients, time.time() - t0))
    assert he.he_ctx_status(g) == he.HE_OK


def test_resnet50_sized_top10_percent(he):
    """25.6 M parameters, top 10 % by sensitivity encrypted, the rest averaged in plaintext: all 313
    ciphertext indices of all 10 clients, and the plaintext part bit for bit."""
    w = si.RESNET50_TOP10
    g, o, keys, s_o, pk_o = setup(he, w)
    score = si.sensitivity_scores(w)
    mask = he.he_select_mask(g, torch.from_numpy(score).cuda(), w.k)
    idx = oracle.select_mask(score, w.k)                               # full sort on the host
    assert mask.k == w.k == 2_560_000
    assert np.array_equal(he.he_mask_indices(mask).cpu().numpy().view(np.uint32), idx)
    xs = si.client_updates(w)
    alpha = si.client_weights(w)
    xs_dev = [torch.from_numpy(x).cuda() for x in xs]
    cts, agg, z, out = run_round(he, g, keys, mask, xs_dev, alpha, w)
    want = fedavg(xs_dev, alpha)
    assert float((out - want).abs().max()) <= FEDAVG_TOL
    # packing: the encrypted slots are exactly x[idx], the remainder is exactly the complement
    sel, rest = he.he_pack(g, mask, xs_dev[3])
    assert np.array_equal(sel[: w.k].cpu().numpy(), xs[3][idx])
    comp = np.ones(w.P, bool)
    comp[idx] = False
    assert np.array_equal(rest.cpu().numpy(), xs[3][comp])
    # plaintext positions are bit-exact sums in client order
    ref_plain = np.zeros(int(comp.sum()))
    for a, x in zip(alpha, xs):
        ref_plain = ref_plain + a * x[comp].astype(np.float64)
    out_h = out.cpu().numpy()
    assert np.array_equal(out_h[comp], ref_plain)
    check_resident_round(w, o, s_o, pk_o, idx, xs, alpha, cts, agg, z, list(range(w.T)))
    # the merged model holds the decoded slots at the masked positions
    assert np.array_equal(out_h[idx], z.cpu().numpy()[: w.k])


def mask_properties(score_dev, idx_dev, k):
    """What defines the mask at any size: k indices, ascending, holding the k largest keys, ties
    taken at the lowest indices."""
    P = score_dev.numel()
    key = score_dev.view(torch.int32).clone()
    key[(key < 0) | (key > 0x7f800000)] = 0
    idx = idx_dev.long()
    assert idx.numel() == k
    assert bool((idx[1:] > idx[:-1]).all())
    chosen = torch.zeros(P, dtype=torch.bool, device="cuda")
    chosen[idx] = True
    tau = int(key[chosen].min())
    assert int(key[~chosen].max()) <= tau
    tied = torch.nonzero(key == tau).flatten()
    take = int(chosen[tied].sum())
    assert bool(chosen[tied[:take]].all())                      # the lowest indices among the ties
    assert int((key > tau).sum()) + take == k


def sampled_indices(T, count, seed):
    """`count` ciphertext indices out of T, first and last always among them."""
    if T <= count:
        return list(range(T))
    rng = np.random.default_rng([seed, 33])
    pick = set(rng.choice(np.arange(1, T - 1), size=count - 2, replace=False).tolist())
    return sorted(pick | {0, T - 1})


@pytest.mark.parametrize("ratio", [0.01, 0.10])
def test_bert_sized_selective(he, ratio):
    """110 M parameters, 8 clients, N = 32768, 6 primes, scale 2^45, 1 % and 10 % encrypted."""
    w = si.bert(ratio)
    g, o, keys, s_o, pk_o = setup(he, w)
    score = torch.from_numpy(si.sensitivity_scores(w)).cuda()
    mask = he.he_select_mask(g, score, w.k)
    idx_dev = he.he_mask_indices(mask)
    mask_properties(score, idx_dev, w.k)
    idx = idx_dev.cpu().numpy().view(np.uint32)
    del score
    xs = si.client_updates(w)
    alpha = si.client_weights(w)
    xs_dev = [torch.from_numpy(x).cuda() for x in xs]
    cts, agg, z, out = run_round(he, g, keys, mask, xs_dev, alpha, w)
    assert cts[0].shape == (w.T, 2, w.L, w.N)
    assert float((out - fedavg(xs_dev, alpha)).abs().max()) <= FEDAVG_TOL
    ts = sampled_indices(w.T, 256, 4)                  # all 68 indices at 1 %, 256 of 672 at 10 %
    check_resident_round(w, o, s_o, pk_o, idx, xs, alpha, cts, agg, z, ts, chunk=32)
    assert he.he_ctx_status(g) == he.HE_OK


def test_bert_sized_full_encryption_streamed(he):
    """At 100 % the 8 clients' ciphertexts (169 GB) do not fit: every chunk of ciphertext indices is
    encrypted with he_encrypt_range, aggregated and decrypted, with the chunk size the benchmark
    uses; 256 sampled ciphertext indices (first and last among them) of every client go against
    the oracle, and every parameter against plaintext FedAvg."""
    w = si.bert(1.0)
    assert w.T == 6714
    g, o, keys, s_o, pk_o = setup(he, w)
    alpha = si.client_weights(w)
    xs = si.client_updates(w)
    xs_dev = [torch.from_numpy(x).cuda() for x in xs]
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    ct_bytes = 8 * 2 * w.L * w.N
    Tc = max(n_sm, int(16e9 // (w.clients * ct_bytes)) // n_sm * n_sm)
    cts = [torch.empty((Tc, 2, w.L, w.N), dtype=torch.int64, device="cuda") for _ in range(w.clients)]
    agg = torch.empty((Tc, 2, w.L - 1, w.N), dtype=torch.int64, device="cuda")
    z = torch.empty(w.T * w.n, dtype=torch.float64, device="cuda")
    sels = [he.he_pack(g, None, x)[0] for x in xs_dev]
    ts_all = sampled_indices(w.T, 256, 5)
    t_oracle = 0.0
    for t0 in range(0, w.T, Tc):
        tc = min(Tc, w.T - t0)
        for i in range(w.clients):
            he.he_encrypt_range(g, keys, sels[i][t0 * w.n:(t0 + tc) * w.n], t0, tc, w.enc_seed, i, cts[i][:tc])
        he.he_weighted_aggregate(g, [c[:tc] for c in cts], alpha, out=agg[:tc])
        he.he_decrypt(g, keys, agg[:tc], out=z[t0 * w.n:(t0 + tc) * w.n])
        ts = [t for t in ts_all if t0 <= t < t0 + tc]
        tic = time.time()
        for c0 in range(0, len(ts), 16):
            part = ts[c0:c0 + 16]
            loc = torch.as_tensor([t - t0 for t in part], device="cuda")
            absolute = torch.as_tensor(part, device="cuda")
            check_indices(w, o, s_o, pk_o, None, xs, alpha, part,
                          lambda i, _: to_host_u64(cts[i][loc]),
                          lambda _: to_host_u64(agg[loc]),
                          lambda _: z.view(-1, w.n)[absolute].cpu().numpy())
        t_oracle += time.time() - tic
    print("bert-sized at 100 %%: %d sampled ciphertext indices x %d clients compared in %.0f s"
          % (len(ts_all), w.clients, t_oracle))
    out = he.he_unpack(g, None, z, None, w.P)
    assert float((out - fedavg(xs_dev, alpha)).abs().max()) <= FEDAVG_TOL
    assert he.he_ctx_status(g) == he.HE_OK
