"""The Python binding refuses buffers of the wrong size on the host, before the C call: the C ABI
takes plain pointers and cannot know a buffer's extent, and a short buffer on the device would be
an out-of-bounds access, not an error.  No GPU is needed: the size checks come before the check
that a tensor lives on the device, so host tensors of the wrong size must raise HeError and host
tensors of the right size must get as far as the device check (TypeError)."""
import pytest
import torch

import paper_2303_10837_b200 as he

N, L = 8192, 3
n = N // 2


@pytest.fixture()
def ctx():
    return he.Ctx(0, N, L, 40)          # handle 0: never passed to the library, never destroyed


def keys(ctx):
    return he.Keys(0, ctx)


def ct(T, level=L):
    return torch.zeros((T, 2, level, N), dtype=torch.int64)


def refused(call):
    with pytest.raises(he.HeError) as ei:
        call()
    assert ei.value.code == he.HE_ERR_INVALID_ARG


def reaches_device_check(call):
    with pytest.raises(TypeError):
        call()


def test_encrypt_sizes(ctx):
    k = keys(ctx)
    refused(lambda: he.he_encrypt(ctx, k, torch.zeros(2 * n - 1), 1, 0))                       # not whole ciphertexts
    refused(lambda: he.he_encrypt(ctx, k, torch.zeros(2 * n), 1, 0, out=ct(1)))                # out too short
    refused(lambda: he.he_encrypt_ntt(ctx, k, torch.zeros(2 * n), 1, 0, out=ct(1)))
    refused(lambda: he.he_encrypt_range(ctx, k, torch.zeros(2 * n), 5, 3, 1, 0, ct(3)))        # sel too short
    refused(lambda: he.he_encrypt_range(ctx, k, torch.zeros(3 * n), 5, 3, 1, 0, ct(2)))        # out too short
    refused(lambda: he.he_encode(ctx, torch.zeros(n + 1)))
    reaches_device_check(lambda: he.he_encrypt_range(ctx, k, torch.zeros(3 * n), 5, 3, 1, 0, ct(3)))


def test_aggregate_sizes(ctx):
    good = [ct(4), ct(4)]
    refused(lambda: he.he_weighted_aggregate(ctx, good, [1.0]))                                 # one weight missing
    refused(lambda: he.he_weighted_aggregate(ctx, [], []))
    refused(lambda: he.he_weighted_aggregate(ctx, [ct(4), ct(3)], [0.5, 0.5]))                  # a shorter client
    refused(lambda: he.he_weighted_aggregate(ctx, [ct(4, L - 1), ct(4, L - 1)], [0.5, 0.5]))    # wrong level
    refused(lambda: he.he_weighted_aggregate(ctx, good, [0.5, 0.5], out=ct(3, L - 1)))          # out too short
    refused(lambda: he.he_weighted_aggregate_ntt(ctx, [ct(4), ct(3)], [0.5, 0.5]))
    refused(lambda: he.he_weighted_partial(ctx, [ct(4), ct(3)], [0.5, 0.5]))                     # a shorter client
    refused(lambda: he.he_weighted_partial(ctx, good, [0.5, 0.5], out=ct(4, L - 1)))              # partial sums keep all limbs
    refused(lambda: he.he_rescale_partial_sum(ctx, ct(4, L - 1), 2))                              # not a sum on all limbs
    refused(lambda: he.he_rescale_partial_sum(ctx, ct(4), 2, out=ct(3, L - 1)))
    refused(lambda: he.he_rescale_partial_parts(ctx, [ct(4), ct(3)]))
    refused(lambda: he.he_rescale_partial_parts(ctx, []))
    reaches_device_check(lambda: he.he_rescale_partial_parts(ctx, [ct(4), ct(4)], out=ct(4, L - 1)))
    reaches_device_check(lambda: he.he_weighted_partial(ctx, good, [0.5, 0.5], out=ct(4)))
    reaches_device_check(lambda: he.he_rescale_partial_sum(ctx, ct(4), 2, out=ct(4, L - 1)))
    refused(lambda: he.he_plain_aggregate(ctx, [torch.zeros(10), torch.zeros(9)], [0.5, 0.5]))
    refused(lambda: he.he_plain_aggregate(ctx, [torch.zeros(10)], [0.5, 0.5]))
    reaches_device_check(lambda: he.he_weighted_aggregate(ctx, good, [0.5, 0.5], out=ct(4, L - 1)))


def test_decrypt_sizes(ctx):
    k = keys(ctx)
    agg = ct(2, L - 1)
    refused(lambda: he.he_decrypt(ctx, k, ct(2, L)))                                             # fresh level given as aggregate
    refused(lambda: he.he_decrypt(ctx, k, agg, out=torch.zeros(2 * n - 1, dtype=torch.float64)))
    refused(lambda: he.he_decrypt_level(ctx, k, agg, L))
    refused(lambda: he.he_decrypt_level_ntt(ctx, k, agg, L - 1, out=torch.zeros(n, dtype=torch.float64)))
    refused(lambda: he.he_decrypt_noalloc(ctx, k, agg, torch.zeros(2 * n - 1, dtype=torch.float64)))
    refused(lambda: he.he_decrypt_noalloc(ctx, k, ct(2, L), torch.zeros(2 * n, dtype=torch.float64)))
    refused(lambda: he.he_partial_decrypt(ctx, k, 0, agg, L, 1, 10))
    parts = [torch.zeros((2, N), dtype=torch.int64), torch.zeros((1, N), dtype=torch.int64)]
    refused(lambda: he.he_threshold_combine(ctx, agg, L - 1, parts))
    reaches_device_check(lambda: he.he_decrypt(ctx, k, agg, out=torch.zeros(2 * n, dtype=torch.float64)))


def test_unpack_pack_and_transform_sizes(ctx):
    mask = he.Mask(0, 100, 30, 0)
    z = torch.zeros(n, dtype=torch.float64)
    rest = torch.zeros(70, dtype=torch.float64)
    refused(lambda: he.he_unpack(ctx, mask, z[:29], rest, 100))                                  # fewer slots than k
    refused(lambda: he.he_unpack(ctx, mask, z, rest[:69], 100))                                  # remainder too short
    refused(lambda: he.he_unpack(ctx, mask, z, None, 100))
    refused(lambda: he.he_unpack(ctx, mask, z, rest, 101))                                       # mask of another size
    refused(lambda: he.he_unpack(ctx, mask, z, rest, 100, out=torch.zeros(99, dtype=torch.float64)))
    refused(lambda: he.he_unpack(ctx, None, z[:99], None, 100))
    refused(lambda: he.he_pack(ctx, mask, torch.zeros(101)))
    refused(lambda: he.he_ntt_forward(ctx, torch.zeros((2, L - 1, N), dtype=torch.int64)))
    refused(lambda: he.he_ntt_inverse(ctx, torch.zeros((2, L, N - 1), dtype=torch.int64)))
    refused(lambda: he.he_round_host(ctx, keys(ctx), None, [torch.zeros(10)], [0.5, 0.5], 1,
                                     torch.zeros(10, dtype=torch.float64)))
    reaches_device_check(lambda: he.he_unpack(ctx, mask, z, rest, 100, out=torch.zeros(100, dtype=torch.float64)))
