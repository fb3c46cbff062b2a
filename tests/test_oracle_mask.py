"""Pins for the oracle's mask selection, packing, remainder average and the
whole-round entry point."""
import numpy as np
import pytest

import oracle
import synthetic_inputs as si
from conftest import read_golden


def brute_select(score, k):
    bits = score.view(np.uint32).astype(np.int64)
    key = np.where((bits >> 31) == 1, 0, bits)
    key = np.where(key > 0x7f800000, 0, key)
    order = np.lexsort((np.arange(score.size), -key))       # key descending, then index ascending
    return np.sort(order[:k]).astype(np.uint32)


def test_select_against_full_sort():
    rng = np.random.default_rng(0)
    score = np.abs(rng.standard_normal(100_000).astype(np.float32))
    for k in (0, 1, 10_000, 99_999, 100_000):
        got = oracle.select_mask(score, k)
        assert np.array_equal(got, brute_select(score, k))
        assert np.all(np.diff(got.astype(np.int64)) > 0)
    # the selected set holds the largest scores
    got = oracle.select_mask(score, 10_000)
    rest = np.setdiff1d(np.arange(score.size), got)
    assert score[got].min() >= score[rest].max()


def test_select_ties_and_special_values():
    score = np.array([1.0, 2.0, 2.0, 2.0, 0.5, 2.0, np.nan, -3.0, -0.0, 0.0, np.inf, 2.0], np.float32)
    assert list(oracle.select_mask(score, 1)) == [10]                 # +inf is the largest key
    assert list(oracle.select_mask(score, 3)) == [1, 2, 10]           # ties: lower index first
    assert list(oracle.select_mask(score, 5)) == [1, 2, 3, 5, 10]
    assert list(oracle.select_mask(score, 8)) == [0, 1, 2, 3, 4, 5, 10, 11]
    # NaN, negatives, -0 and +0 all have the lowest key: taken last, by index
    assert list(oracle.select_mask(score, 10)) == [0, 1, 2, 3, 4, 5, 6, 7, 10, 11]
    for k in range(score.size + 1):
        assert np.array_equal(oracle.select_mask(score, k), brute_select(score, k))
    same = np.full(1000, 0.125, np.float32)
    assert list(oracle.select_mask(same, 17)) == list(range(17))


def test_packing_counts_follow_the_paper():
    """A vector shorter than the batch size still costs one whole ciphertext."""
    for row in read_golden("paper_facts.txt"):
        params, batch, cts = (int(v) for v in row.split())
        ctx = oracle.Context(2 * batch, si.PRIMES_N8192, 40)
        assert ctx.num_ct(params) == cts
        sel, _ = ctx.pack(None, params, np.ones(params, np.float32))
        assert sel.size == cts * batch and sel[:params].all() and not sel[params:].any()


def test_pack_unpack_round_trip_with_mask():
    ctx = oracle.Context(64, si.PRIMES_N8192, 40)
    rng = np.random.default_rng(2)
    P, k = 1000, 137
    x = rng.standard_normal(P).astype(np.float32)
    idx = oracle.select_mask(np.abs(x), k)
    sel, rest = ctx.pack(idx, k, x)
    T = ctx.num_ct(k)
    assert T == 5 and sel.size == T * 32 and rest.size == P - k
    assert np.array_equal(sel[:k], x[idx]) and not sel[k:].any()
    comp = np.setdiff1d(np.arange(P), idx)
    assert np.array_equal(rest, x[comp])
    back = oracle.unpack(idx, k, sel.astype(np.float64), rest.astype(np.float64), P)
    assert np.array_equal(back, x.astype(np.float64))


def test_plain_aggregate_is_the_ordered_weighted_sum():
    rng = np.random.default_rng(3)
    rests = [rng.standard_normal(501).astype(np.float32) for _ in range(5)]
    alpha = rng.random(5)
    got = oracle.plain_aggregate(rests, alpha)
    want = np.zeros(501)
    for a, r in zip(alpha, rests):
        want = want + a * r.astype(np.float64)
    assert np.array_equal(got, want)


def test_whole_round_equals_the_steps_and_fedavg():
    """Aggregation equation: encrypted part + plaintext part = FedAvg on every index."""
    w = si.Workload("mini", 8192, si.PRIMES_N8192, 40, 3, 30_000, 0.02, ratio=0.3, seed=5)
    ctx = oracle.Context(w.N, w.primes, w.log2_delta)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    idx = oracle.select_mask(si.sensitivity_scores(w), w.k)
    out = ctx.round(xs, alpha, idx, w.k, w.key_seed, w.enc_seed)
    # the same thing step by step
    s, pk = ctx.keygen(w.key_seed)
    cts, rests = [], []
    for i, x in enumerate(xs):
        sel, rest = ctx.pack(idx, w.k, x)
        cts.append(ctx.encrypt(pk, sel, w.enc_seed, i)[0])
        rests.append(rest)
    agg = ctx.rescale(ctx.weighted_sum(cts, ctx.weights(alpha)))
    z = ctx.decode(ctx.decrypt(s, agg, w.L - 1)).reshape(-1)
    step = oracle.unpack(idx, w.k, z, oracle.plain_aggregate(rests, alpha), w.P)
    assert np.array_equal(out, step)
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(out - want).max() < 1e-6
    comp = np.setdiff1d(np.arange(w.P), idx)
    assert np.abs(out[comp] - want[comp]).max() < 1e-15        # plaintext part: exact up to fp64 order
    assert np.abs(out[idx] - want[idx]).max() > 1e-12          # encrypted part carries CKKS noise
    # a sample of ciphertext indices reproduces exactly those positions
    part = ctx.round(xs, alpha, idx, w.k, w.key_seed, w.enc_seed, t_begin=1, t_end=2, do_rest=False)
    sl = idx[ctx.n: 2 * ctx.n]
    assert np.array_equal(part[sl], out[sl])
