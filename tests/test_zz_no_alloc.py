"""he_decrypt_noalloc, the entry point for callers that must not allocate device memory (their
HBM is fully handed to their own pool, or they sit in a loop that cannot take cudaMalloc's
device-wide synchronisation): it must give what he_decrypt gives, on repeated calls that share
its fixed work array, and must refuse sizes beyond that array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import synthetic_inputs as si

pytestmark = pytest.mark.gpu

DECODE_TOL = 1e-9     # same tolerance as the decode parity tests


def test_noalloc_decrypt_matches_decrypt_twice_in_a_row():
    import paper_2303_10837_b200 as he
    w = si.scaled(si.RESNET18, 5 * 8192 - 3, clients=3, name="noalloc")
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    alpha = si.client_weights(w)
    aggs = []
    for round_seed in (1, 2):                       # two different aggregates
        cts = []
        for i in range(w.clients):
            x = torch.from_numpy(si.client_update(w, i) * np.float32(round_seed)).cuda()
            sel, _ = he.he_pack(g, None, x)
            cts.append(he.he_encrypt(g, keys, sel, 100 + round_seed, i))
        aggs.append(he.he_weighted_aggregate(g, cts, alpha))
    want = [he.he_decrypt(g, keys, a) for a in aggs]
    outs = [torch.empty_like(wv) for wv in want]
    # the first call on a device is the set-up call: it looks up the array's address, which is
    # also when the CUDA runtime loads the library's device image (array included) if it has
    # not done so yet; from then on the free memory must not move
    he.he_decrypt_noalloc(g, keys, aggs[1], outs[0])
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    stats_before = torch.cuda.memory_stats()
    # back to back on one stream: the second call reuses the array the first one filled
    he.he_decrypt_noalloc(g, keys, aggs[0], outs[0])
    he.he_decrypt_noalloc(g, keys, aggs[1], outs[1])
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                 # nothing was allocated on the device
    # the free-memory figure is device-wide; torch's own allocator must not have moved either
    stats_after = torch.cuda.memory_stats()
    for key in ("num_alloc_retries", "allocation.all.allocated", "segment.all.allocated"):
        assert stats_after.get(key, 0) == stats_before.get(key, 0), key
    for got, ref in zip(outs, want):
        assert float((got - ref).abs().max()) <= DECODE_TOL
    assert float((outs[0] - outs[1]).abs().max()) > 1e-4      # the two results really differ
    # and once more in the other order
    he.he_decrypt_noalloc(g, keys, aggs[0], outs[1])
    torch.cuda.synchronize()
    assert float((outs[1] - want[0]).abs().max()) <= DECODE_TOL
    assert he.he_ctx_status(g) == he.HE_OK


def test_noalloc_decrypt_rejects_what_does_not_fit():
    import paper_2303_10837_b200 as he
    w = si.RESNET18
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, 1)
    T = he.HE_NOALLOC_MAX_WORDS // w.N + 1            # one ciphertext too many
    agg = torch.zeros((T, 2, w.L - 1, w.N), dtype=torch.int64, device="cuda")
    out = torch.empty(T * w.n, dtype=torch.float64, device="cuda")
    with pytest.raises(he.HeError) as ei:
        he.he_decrypt_noalloc(g, keys, agg, out)
    assert ei.value.code == he.HE_ERR_SIZE
    he.he_decrypt_noalloc(g, keys, agg[: T - 1], out)   # the largest size that fits is accepted
    torch.cuda.synchronize()
    b = si.bert(1.0)                                     # N = 32768: decoder would need a second buffer
    gb = he.he_ctx_create(b.N, list(b.primes), b.log2_delta)
    kb = he.he_keygen(gb, 1)
    aggb = torch.zeros((1, 2, b.L - 1, b.N), dtype=torch.int64, device="cuda")
    with pytest.raises(he.HeError) as ei:
        he.he_decrypt_noalloc(gb, kb, aggb, torch.empty(b.n, dtype=torch.float64, device="cuda"))
    assert ei.value.code == he.HE_ERR_SIZE


def test_noalloc_decrypt_smallest_ring_and_its_limit():
    """N = 8192: up to 256 ciphertexts fit the fixed array; 257 are refused, 256 give he_decrypt's result."""
    import paper_2303_10837_b200 as he
    w = si.scaled(si.TINY, 256 * 4096 - 11, clients=2, name="noalloc-8192")
    g = he.he_ctx_create(w.N, list(w.primes), w.log2_delta)
    keys = he.he_keygen(g, w.key_seed)
    alpha = si.client_weights(w)
    cts = [he.he_encrypt(g, keys, he.he_pack(g, None, torch.from_numpy(si.client_update(w, i)).cuda())[0], 5, i)
           for i in range(w.clients)]
    agg = he.he_weighted_aggregate(g, cts, alpha)
    assert agg.shape[0] == 256 == he.HE_NOALLOC_MAX_WORDS // w.N
    want = he.he_decrypt(g, keys, agg)
    out = torch.empty_like(want)
    he.he_decrypt_noalloc(g, keys, agg, out)
    he.he_decrypt_noalloc(g, keys, agg, out)          # again, over the array the first call left behind
    torch.cuda.synchronize()
    assert float((out - want).abs().max()) <= DECODE_TOL
    more = torch.zeros((257, 2, w.L - 1, w.N), dtype=torch.int64, device="cuda")
    with pytest.raises(he.HeError) as ei:
        he.he_decrypt_noalloc(g, keys, more, torch.empty(257 * w.n, dtype=torch.float64, device="cuda"))
    assert ei.value.code == he.HE_ERR_SIZE
    # nothing to do is not an error; a missing buffer is
    empty = torch.zeros((0, 2, w.L - 1, w.N), dtype=torch.int64, device="cuda")
    he.he_decrypt_noalloc(g, keys, empty, torch.empty(0, dtype=torch.float64, device="cuda"))
    import ctypes as C
    lib = C.CDLL(he.LIB_PATH)
    lib.he_decrypt_noalloc.restype = C.c_int
    lib.he_decrypt_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    assert lib.he_decrypt_noalloc(g.handle, keys.handle, None, 1, out.data_ptr(), None) == he.HE_ERR_INVALID_ARG
    assert lib.he_decrypt_noalloc(g.handle, keys.handle, agg.data_ptr(), 1, None, None) == he.HE_ERR_INVALID_ARG
    assert he.he_ctx_status(g) == he.HE_OK
