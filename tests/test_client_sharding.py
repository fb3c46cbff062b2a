"""The client layout of a multi-GPU server (every rank holds the ciphertexts of some clients, forms
their weighted sum without the rescale, one reduce-scatter of 64-bit words sums over the clients
and leaves every rank the ciphertext indices it then rescales and decrypts): two gloo ranks on the
CPU with the oracle as the worker must reproduce the single-rank oracle round bit for bit, with an
uneven split of both the clients (1 + 2) and the ciphertext indices (2 + 3)."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _workload():
    import synthetic_inputs as si
    # 5 ciphertexts (the last one ragged), 3 clients, full encryption
    return si.Workload("clients", 8192, si.PRIMES_N8192, 40, 3, 4 * 4096 + 33, 0.02, ratio=1.0, seed=21,
                       key_seed=211, enc_seed=212)


def _rank_main(rank, world, port, q):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import oracle
    import synthetic_inputs as si
    from paper_2303_10837_b200.sharding import gather_pieces, scatter_sum, shard_range, slot_edges
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = _workload()
    o = oracle.Context(w.N, w.primes, w.log2_delta)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    s, pk = o.keygen(w.key_seed)                                        # replicated keys
    W = o.weights(alpha)                                                # weights of the whole round
    cb, ce = shard_range(w.clients, rank, world)
    cts = [o.encrypt(pk, o.pack(None, w.k, xs[i])[0], w.enc_seed, i)[0] for i in range(cb, ce)]
    partial = o.weighted_sum(cts, W[cb:ce])                             # [T][2][L][N], canonical residues
    mine = scatter_sum(torch.from_numpy(partial.view(np.int64)), rank, world).numpy().view(np.uint64)
    primes = np.array(w.primes, dtype=np.uint64).reshape(1, 1, -1, 1)
    acc = mine % primes                                                 # what he_rescale_partial_sum reduces first
    z = o.decode(o.decrypt(s, o.rescale(acc), w.L - 1)).reshape(-1)
    tb, te = shard_range(w.T, rank, world)
    z = z[: min(w.k, te * w.n) - tb * w.n]                              # the ragged last ciphertext
    whole = gather_pieces(torch.from_numpy(z.copy()), slot_edges(w.T, w.n, w.k, world), rank)
    q.put((rank, (cb, ce), (tb, te), whole.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_with_clients_split_reproduce_the_single_rank_round():
    sys.path.insert(0, ROOT)
    import oracle
    import synthetic_inputs as si
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=120) for _ in procs), key=lambda v: v[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [(0, 1), (1, 3)]                      # clients per rank
    assert [g[2] for g in got] == [(0, 2), (2, 5)]                      # ciphertext indices per rank
    w = _workload()
    o = oracle.Context(w.N, w.primes, w.log2_delta)
    xs, alpha = si.client_updates(w), si.client_weights(w)
    whole = o.round(xs, alpha, None, w.k, w.key_seed, w.enc_seed)
    for _, _, _, merged in got:
        assert np.array_equal(merged, whole)
    want = sum(a * x.astype(np.float64) for a, x in zip(alpha, xs))
    assert np.abs(whole - want).max() <= 1e-6


def test_scatter_sum_pads_unequal_shares():
    """One rank: the identity; the padded layout of the NCCL branch is index arithmetic only."""
    import torch
    from paper_2303_10837_b200.sharding import scatter_sum, shard_range
    x = torch.arange(5 * 6, dtype=torch.int64).reshape(5, 2, 3)
    assert torch.equal(scatter_sum(x, 0, 1), x)
    T, world = 5, 3
    width = -(-T // world)
    rows = [shard_range(T, r, world) for r in range(world)]
    assert all(e - b <= width for b, e in rows) and rows[-1][1] == T
