"""The multi-GPU partition of one round (contiguous ranges of ciphertext indices and of the
plaintext remainder per rank, replicated context, keys and mask, no collective but the optional
gather of the decoded pieces): the range arithmetic, and two gloo ranks on the CPU with the
oracle as the worker -- the union of the ranks' outputs must equal the single-rank oracle round
bit for bit, ragged last range included."""
import os
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2303_10837_b200.sharding import shard_range, slot_range


@pytest.mark.parametrize("count,world", [(0, 1), (1, 2), (7, 2), (1429, 8), (6714, 4), (313, 3), (5, 8)])
def test_ranges_are_contiguous_disjoint_and_balanced(count, world):
    edges = [shard_range(count, r, world) for r in range(world)]
    assert edges[0][0] == 0 and edges[-1][1] == count
    for (b0, e0), (b1, e1) in zip(edges, edges[1:]):
        assert e0 == b1 and b0 <= e0
    sizes = [e - b for b, e in edges]
    assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_range(count, world, world)


def test_slot_ranges_stop_at_the_last_encrypted_parameter():
    n, k = 4096, 3 * 4096 + 17                      # 4 ciphertexts, the last one holds 17 slots
    T = (k + n - 1) // n
    got = [slot_range(T, n, k, r, 3) for r in range(3)]
    assert got == [(0, 1, 0, 4096), (1, 2, 4096, 8192), (2, 4, 8192, k)]


def _rank_main(rank, world, port, q):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import oracle
    import synthetic_inputs as si
    from paper_2303_10837_b200.sharding import even_edges, gather_pieces, shard_range, slot_edges, slot_range
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # 5 ciphertexts (ragged last one) over 2 ranks: 2 + 3; top 40 % encrypted, the rest in plaintext
    w = si.Workload("shard", 8192, si.PRIMES_N8192, 40, 3, 50_000, 0.02, ratio=0.4, seed=8, key_seed=81, enc_seed=82)
    o = oracle.Context(w.N, w.primes, w.log2_delta)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    idx = oracle.select_mask(si.sensitivity_scores(w), w.k)          # replicated mask
    tb, te, sb, se = slot_range(w.T, w.n, w.k, rank, world)
    # this rank's ciphertext indices through the whole path (no plaintext part)
    piece = o.round(xs, alpha, idx, w.k, w.key_seed, w.enc_seed, t_begin=tb, t_end=te, do_rest=False)
    z_local = torch.from_numpy(piece[idx[sb:se].astype(np.int64)].copy())
    # this rank's range of the compacted plaintext remainder
    rests = [o.pack(idx, w.k, x)[1] for x in xs]
    rb, re = shard_range(w.P - w.k, rank, world)
    r_local = torch.from_numpy(oracle.plain_aggregate([r[rb:re] for r in rests], alpha))
    z = gather_pieces(z_local, slot_edges(w.T, w.n, w.k, world), rank)
    ravg = gather_pieces(r_local, even_edges(w.P - w.k, world), rank)
    merged = oracle.unpack(idx, w.k, np.concatenate([z.numpy(), np.zeros(w.T * w.n - w.k)]), ravg.numpy(), w.P)
    q.put((rank, (tb, te), merged))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_rank_round_bit_for_bit():
    sys.path.insert(0, ROOT)
    import oracle
    import synthetic_inputs as si
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=120) for _ in procs), key=lambda v: v[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [(0, 2), (2, 5)]
    w = si.Workload("shard", 8192, si.PRIMES_N8192, 40, 3, 50_000, 0.02, ratio=0.4, seed=8, key_seed=81, enc_seed=82)
    o = oracle.Context(w.N, w.primes, w.log2_delta)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    idx = oracle.select_mask(si.sensitivity_scores(w), w.k)
    whole = o.round(xs, alpha, idx, w.k, w.key_seed, w.enc_seed)
    for _, _, merged in got:                          # every rank holds the whole model after the gather
        assert np.array_equal(merged, whole)
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(whole - want).max() <= 1e-6
