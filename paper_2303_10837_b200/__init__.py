"""Python binding of ``libfedhe.so``: the sm_100a CUDA library for the hot path of
FedML-HE secure aggregation (mask selection, CKKS encode + encrypt, weighted
ciphertext aggregation with rescale, decrypt + decode, pack/unpack).

The functions have the names of the C entry points in ``include/fedhe.h`` and do
argument marshalling only: torch owns device memory and streams, every step of
the path runs in the library's kernels.  There is no CPU fallback: importing
this package without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfedhe.so")

HE_MAX_LIMBS = 16
HE_MAX_CLIENTS = 256
HE_OK = 0
HE_ERR_INVALID_ARG, HE_ERR_PARAMS, HE_ERR_ALLOC, HE_ERR_CUDA = -1, -2, -3, -4
HE_ERR_OVERFLOW, HE_ERR_LEVEL, HE_ERR_SIZE = -5, -6, -7


class HeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, he_strerror(code), code))


class he_params(C.Structure):
    _fields_ = [("N", C.c_uint32), ("L", C.c_uint32), ("q", C.c_uint64 * HE_MAX_LIMBS),
                ("log2_delta", C.c_int32)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libfedhe.so is missing: build it with `python paper_2303_10837_b200/build.py` "
            "(there is no fallback path)")
    return C.CDLL(LIB_PATH)


_lib = _load()
_vp, _sz, _u64, _u32 = C.c_void_p, C.c_size_t, C.c_uint64, C.c_uint32

_SIGS = {
    "he_strerror": (C.c_char_p, [C.c_int]),
    "he_launch_count": (_u64, []),
    "he_ctx_create": (C.c_int, [C.POINTER(he_params), C.POINTER(_vp)]),
    "he_ctx_destroy": (C.c_int, [_vp]),
    "he_ctx_status": (C.c_int, [_vp, C.POINTER(C.c_int)]),
    "he_ctx_reserve": (C.c_int, [_vp, _sz]),
    "he_slots": (_sz, [_vp]),
    "he_num_ct": (_sz, [_vp, _sz]),
    "he_ct_words": (_sz, [_vp, _u32]),
    "he_keygen": (C.c_int, [_vp, _u64, C.POINTER(_vp), _vp]),
    "he_keys_destroy": (C.c_int, [_vp]),
    "he_keys_export": (C.c_int, [_vp, _vp, _vp, _vp, _vp]),
    "he_select_mask": (C.c_int, [_vp, _vp, _sz, _sz, C.POINTER(_vp), _vp]),
    "he_select_mask_ranges": (C.c_int, [_vp, _vp, _sz, _sz, _vp, _sz, C.POINTER(_vp), _vp]),
    "he_mask_indices": (C.c_int, [_vp, C.POINTER(_vp), C.POINTER(_sz)]),
    "he_mask_copy_indices": (C.c_int, [_vp, _vp, _vp]),
    "he_mask_destroy": (C.c_int, [_vp]),
    "he_pack": (C.c_int, [_vp, _vp, _vp, _sz, _vp, _vp, _vp]),
    "he_encode": (C.c_int, [_vp, _vp, _sz, _vp, _vp]),
    "he_encrypt": (C.c_int, [_vp, _vp, _vp, _sz, _u64, _u32, _vp, _vp]),
    "he_encrypt_range": (C.c_int, [_vp, _vp, _vp, _sz, _sz, _u64, _u32, _vp, _vp]),
    "he_weighted_aggregate": (C.c_int, [_vp, _vp, _vp, C.c_int, _sz, _vp, _vp]),
    "he_weighted_partial": (C.c_int, [_vp, _vp, _vp, C.c_int, _sz, _vp, _vp]),
    "he_rescale_partial_sum": (C.c_int, [_vp, _vp, _u32, _sz, _vp, _vp]),
    "he_rescale_partial_parts": (C.c_int, [_vp, _vp, C.c_int, _sz, _vp, _vp]),
    "he_encrypt_ntt": (C.c_int, [_vp, _vp, _vp, _sz, _u64, _u32, _vp, _vp]),
    "he_weighted_aggregate_ntt": (C.c_int, [_vp, _vp, _vp, C.c_int, _sz, _vp, _vp]),
    "he_decrypt_level_ntt": (C.c_int, [_vp, _vp, _vp, _u32, _sz, _vp, _vp]),
    "he_plain_aggregate": (C.c_int, [_vp, _vp, _vp, C.c_int, _sz, _vp, _vp]),
    "he_decrypt": (C.c_int, [_vp, _vp, _vp, _sz, _vp, _vp]),
    "he_decrypt_level": (C.c_int, [_vp, _vp, _vp, _u32, _sz, _vp, _vp]),
    "he_decrypt_noalloc": (C.c_int, [_vp, _vp, _vp, _sz, _vp, _vp]),
    "he_threshold_split": (C.c_int, [_vp, _vp, _u64, C.POINTER(_vp), C.POINTER(_vp), _vp]),
    "he_partial_decrypt": (C.c_int, [_vp, _vp, _u32, _vp, _u32, _sz, _u64, _u32, _vp, _vp]),
    "he_threshold_combine": (C.c_int, [_vp, _vp, _u32, _vp, C.c_int, _sz, _vp, _vp]),
    "he_unpack": (C.c_int, [_vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "he_ntt_forward": (C.c_int, [_vp, _vp, _sz, _vp]),
    "he_ntt_inverse": (C.c_int, [_vp, _vp, _sz, _vp]),
    "he_round_host": (C.c_int, [_vp, _vp, _vp, _vp, _vp, C.c_int, _sz, _u64, _vp, _vp]),
}
for _name, (_res, _args) in _SIGS.items():
    _f = getattr(_lib, _name)
    _f.restype = _res
    _f.argtypes = _args

EXPORTS = tuple(_SIGS)


def he_strerror(code: int) -> str:
    return _lib.he_strerror(code).decode()


def he_launch_count() -> int:
    return int(_lib.he_launch_count())


def _check(code: int, where: str) -> None:
    if code != HE_OK:
        raise HeError(code, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype: torch.dtype) -> int:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError("expected a contiguous CUDA tensor of dtype %s" % dtype)
    return t.data_ptr()


# The C ABI takes plain pointers and cannot know how large a buffer is, so this
# layer is where a short buffer is caught: before the call, on the host, as an
# error instead of an out-of-bounds access on the device.
def _sized(t: torch.Tensor, count: int, what: str, exact: bool = False) -> None:
    have = t.numel()
    if have != count if exact else have < count:
        raise HeError(HE_ERR_INVALID_ARG, "%s: %d entries, %s%d needed" % (what, have, "" if exact else "at least ", count))


def _same_len(a, b, what: str) -> None:
    if len(a) != len(b) or len(a) < 1:
        raise HeError(HE_ERR_INVALID_ARG, "%s: %d and %d entries" % (what, len(a), len(b)))


def _whole_cts(ctx: "Ctx", sel: torch.Tensor, what: str) -> int:
    """Number of ciphertexts of a slot buffer, which must hold whole ciphertexts."""
    if sel.numel() % ctx.n:
        raise HeError(HE_ERR_INVALID_ARG, "%s: %d slots is not a multiple of n = %d" % (what, sel.numel(), ctx.n))
    return sel.numel() // ctx.n


def _ct_count(ctx: "Ctx", ct: torch.Tensor, level: int, what: str) -> int:
    """T of a ciphertext tensor [T][2][level][N] (taken from its first extent, checked against its size)."""
    if not 1 <= level <= ctx.L:
        raise HeError(HE_ERR_LEVEL, what)
    T = ct.shape[0] if ct.dim() else 0
    _sized(ct, T * 2 * level * ctx.N, what, exact=True)
    return T


class Ctx:
    """Owner of a ``he_ctx*``."""

    def __init__(self, handle: int, N: int, L: int, log2_delta: int):
        self.handle, self.N, self.L, self.log2_delta = handle, N, L, log2_delta
        self.n = N // 2

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:     # _lib is gone at interpreter exit
            _lib.he_ctx_destroy(self.handle)
            self.handle = None


class Keys:
    def __init__(self, handle: int, ctx: Ctx):
        self.handle, self.ctx = handle, ctx

    def __del__(self):
        if getattr(self, "handle", None) and getattr(self.ctx, "handle", None) and _lib is not None:
            _lib.he_keys_destroy(self.handle)
            self.handle = None


class Mask:
    def __init__(self, handle: int, P: int, k: int, idx_ptr: int):
        self.handle, self.P, self.k, self.idx_ptr = handle, P, k, idx_ptr

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.he_mask_destroy(self.handle)
            self.handle = None


def he_ctx_create(N: int, primes: Sequence[int], log2_delta: int) -> Ctx:
    p = he_params()
    p.N, p.L, p.log2_delta = N, len(primes), log2_delta
    if len(primes) > HE_MAX_LIMBS:
        raise HeError(HE_ERR_PARAMS, "he_ctx_create")
    for j, q in enumerate(primes):
        p.q[j] = q
    h = _vp()
    _check(_lib.he_ctx_create(C.byref(p), C.byref(h)), "he_ctx_create")
    return Ctx(h.value, N, len(primes), log2_delta)


def he_ctx_status(ctx: Ctx) -> int:
    st = C.c_int(0)
    _check(_lib.he_ctx_status(ctx.handle, C.byref(st)), "he_ctx_status")
    return st.value


def he_ctx_reserve(ctx: Ctx, max_k: int) -> None:
    _check(_lib.he_ctx_reserve(ctx.handle, max_k), "he_ctx_reserve")


def he_slots(ctx: Ctx) -> int:
    return int(_lib.he_slots(ctx.handle))


def he_num_ct(ctx: Ctx, k: int) -> int:
    return int(_lib.he_num_ct(ctx.handle, k))


def he_ct_words(ctx: Ctx, level: int) -> int:
    return int(_lib.he_ct_words(ctx.handle, level))


def he_keygen(ctx: Ctx, seed: int) -> Keys:
    h = _vp()
    _check(_lib.he_keygen(ctx.handle, seed, C.byref(h), _stream()), "he_keygen")
    return Keys(h.value, ctx)


def he_keys_export(ctx: Ctx, keys: Keys):
    """(pk uint64-as-int64 [2][L][N], s int8 [N]) on the device."""
    pk = torch.empty((2, ctx.L, ctx.N), dtype=torch.int64, device="cuda")
    s = torch.empty(ctx.N, dtype=torch.int8, device="cuda")
    _check(_lib.he_keys_export(ctx.handle, keys.handle, pk.data_ptr(), s.data_ptr(), _stream()),
           "he_keys_export")
    return pk, s


def _finish_mask(h: _vp, P: int) -> Mask:
    ip, k = _vp(), _sz()
    _check(_lib.he_mask_indices(h.value, C.byref(ip), C.byref(k)), "he_mask_indices")
    return Mask(h.value, P, int(k.value), ip.value or 0)


def he_select_mask(ctx: Ctx, score: torch.Tensor, k: int) -> Mask:
    h = _vp()
    _check(_lib.he_select_mask(ctx.handle, _dev(score, torch.float32), score.numel(), k, C.byref(h),
                               _stream()), "he_select_mask")
    return _finish_mask(h, score.numel())


def he_select_mask_ranges(ctx: Ctx, score: torch.Tensor, k: int, ranges: Sequence[Sequence[int]]) -> Mask:
    flat = (C.c_uint64 * (2 * len(ranges)))(*[int(v) for r in ranges for v in r])
    h = _vp()
    _check(_lib.he_select_mask_ranges(ctx.handle, _dev(score, torch.float32), score.numel(), k,
                                      C.cast(flat, _vp), len(ranges), C.byref(h), _stream()),
           "he_select_mask_ranges")
    return _finish_mask(h, score.numel())


def he_mask_indices(mask: Mask) -> torch.Tensor:
    """Copy of the ascending index list (int32 view of the uint32 values)."""
    out = torch.empty(mask.k, dtype=torch.int32, device="cuda")
    _check(_lib.he_mask_copy_indices(mask.handle, out.data_ptr() if mask.k else None, _stream()),
           "he_mask_copy_indices")
    return out


def he_pack(ctx: Ctx, mask: Optional[Mask], x: torch.Tensor):
    """(sel float32 [T*n], rest float32 [P-k] or None)."""
    P = x.numel()
    if mask is not None and mask.P != P:
        raise HeError(HE_ERR_INVALID_ARG, "he_pack: the mask was built for %d parameters, x has %d" % (mask.P, P))
    k = mask.k if mask is not None else P
    sel = torch.empty(he_num_ct(ctx, k) * ctx.n, dtype=torch.float32, device="cuda")
    rest = torch.empty(P - k, dtype=torch.float32, device="cuda") if mask is not None else None
    _check(_lib.he_pack(ctx.handle, mask.handle if mask else None, _dev(x, torch.float32), P,
                        sel.data_ptr(), rest.data_ptr() if rest is not None else None, _stream()),
           "he_pack")
    return sel, rest


def he_encode(ctx: Ctx, sel: torch.Tensor) -> torch.Tensor:
    T = _whole_cts(ctx, sel, "he_encode sel")
    m = torch.empty((T, ctx.N), dtype=torch.int64, device="cuda")
    _check(_lib.he_encode(ctx.handle, _dev(sel, torch.float32), sel.numel(), m.data_ptr(), _stream()),
           "he_encode")
    return m


def he_encrypt(ctx: Ctx, keys: Keys, sel: torch.Tensor, seed: int, client_id: int,
               out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Fresh ciphertexts uint64-as-int64 [T][2][L][N]."""
    T = _whole_cts(ctx, sel, "he_encrypt sel")
    if out is None:
        out = torch.empty((T, 2, ctx.L, ctx.N), dtype=torch.int64, device="cuda")
    _sized(out, T * 2 * ctx.L * ctx.N, "he_encrypt out")
    _check(_lib.he_encrypt(ctx.handle, keys.handle, _dev(sel, torch.float32), sel.numel(), seed, client_id,
                           _dev(out, torch.int64), _stream()), "he_encrypt")
    return out


def he_encrypt_ntt(ctx: Ctx, keys: Keys, sel: torch.Tensor, seed: int, client_id: int,
                   out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The same ciphertexts in the transform-domain wire format."""
    T = _whole_cts(ctx, sel, "he_encrypt_ntt sel")
    if out is None:
        out = torch.empty((T, 2, ctx.L, ctx.N), dtype=torch.int64, device="cuda")
    _sized(out, T * 2 * ctx.L * ctx.N, "he_encrypt_ntt out")
    _check(_lib.he_encrypt_ntt(ctx.handle, keys.handle, _dev(sel, torch.float32), sel.numel(), seed, client_id,
                               _dev(out, torch.int64), _stream()), "he_encrypt_ntt")
    return out


def he_encrypt_range(ctx: Ctx, keys: Keys, sel: torch.Tensor, t_begin: int, t_count: int, seed: int,
                     client_id: int, out: torch.Tensor) -> torch.Tensor:
    """`sel` holds the slots of ciphertexts t_begin .. t_begin+t_count-1."""
    _sized(sel, t_count * ctx.n, "he_encrypt_range sel")
    _sized(out, t_count * 2 * ctx.L * ctx.N, "he_encrypt_range out")
    _check(_lib.he_encrypt_range(ctx.handle, keys.handle, _dev(sel, torch.float32), t_begin, t_count, seed,
                                 client_id, _dev(out, torch.int64), _stream()), "he_encrypt_range")
    return out


def he_weighted_aggregate(ctx: Ctx, cts: List[torch.Tensor], alpha: Sequence[float],
                          out: Optional[torch.Tensor] = None) -> torch.Tensor:
    _same_len(cts, alpha, "he_weighted_aggregate cts and alpha")
    Cn = len(cts)
    T = _ct_count(ctx, cts[0], ctx.L, "he_weighted_aggregate cts[0]")
    for i, c in enumerate(cts):
        _sized(c, T * 2 * ctx.L * ctx.N, "he_weighted_aggregate cts[%d]" % i, exact=True)
    if out is None:
        out = torch.empty((T, 2, ctx.L - 1, ctx.N), dtype=torch.int64, device="cuda")
    _sized(out, T * 2 * (ctx.L - 1) * ctx.N, "he_weighted_aggregate out")
    ptrs = (_vp * Cn)(*[_dev(c, torch.int64) for c in cts])
    al = (C.c_double * Cn)(*[float(a) for a in alpha])
    _check(_lib.he_weighted_aggregate(ctx.handle, C.cast(ptrs, _vp), C.cast(al, _vp), Cn, T,
                                      _dev(out, torch.int64), _stream()), "he_weighted_aggregate")
    return out


def he_weighted_partial(ctx: Ctx, cts: List[torch.Tensor], alpha: Sequence[float],
                        out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Weighted sum of a subset of the clients on all L limbs, no rescale: int64 [T][2][L][N]."""
    _same_len(cts, alpha, "he_weighted_partial cts and alpha")
    Cn = len(cts)
    T = _ct_count(ctx, cts[0], ctx.L, "he_weighted_partial cts[0]")
    for i, c in enumerate(cts):
        _sized(c, T * 2 * ctx.L * ctx.N, "he_weighted_partial cts[%d]" % i, exact=True)
    if out is None:
        out = torch.empty((T, 2, ctx.L, ctx.N), dtype=torch.int64, device="cuda")
    _sized(out, T * 2 * ctx.L * ctx.N, "he_weighted_partial out")
    ptrs = (_vp * Cn)(*[_dev(c, torch.int64) for c in cts])
    al = (C.c_double * Cn)(*[float(a) for a in alpha])
    _check(_lib.he_weighted_partial(ctx.handle, C.cast(ptrs, _vp), C.cast(al, _vp), Cn, T,
                                    _dev(out, torch.int64), _stream()), "he_weighted_partial")
    return out


def he_rescale_partial_sum(ctx: Ctx, summed: torch.Tensor, parts: int,
                           out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Rescale of the word-by-word sum of `parts` results of he_weighted_partial."""
    T = _ct_count(ctx, summed, ctx.L, "he_rescale_partial_sum summed")
    if out is None:
        out = torch.empty((T, 2, ctx.L - 1, ctx.N), dtype=torch.int64, device="cuda")
    _sized(out, T * 2 * (ctx.L - 1) * ctx.N, "he_rescale_partial_sum out")
    _check(_lib.he_rescale_partial_sum(ctx.handle, _dev(summed, torch.int64), int(parts), T,
                                       _dev(out, torch.int64), _stream()), "he_rescale_partial_sum")
    return out


def he_rescale_partial_parts(ctx: Ctx, parts: List[torch.Tensor], out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Rescale of the sum of several results of he_weighted_partial, added by the kernel itself."""
    if len(parts) < 1:
        raise HeError(HE_ERR_INVALID_ARG, "he_rescale_partial_parts: no parts")
    T = _ct_count(ctx, parts[0], ctx.L, "he_rescale_partial_parts parts[0]")
    for i, p in enumerate(parts):
        _sized(p, T * 2 * ctx.L * ctx.N, "he_rescale_partial_parts parts[%d]" % i, exact=True)
    if out is None:
        out = torch.empty((T, 2, ctx.L - 1, ctx.N), dtype=torch.int64, device="cuda")
    _sized(out, T * 2 * (ctx.L - 1) * ctx.N, "he_rescale_partial_parts out")
    ptrs = (_vp * len(parts))(*[_dev(p, torch.int64) for p in parts])
    _check(_lib.he_rescale_partial_parts(ctx.handle, C.cast(ptrs, _vp), len(parts), T,
                                         _dev(out, torch.int64), _stream()), "he_rescale_partial_parts")
    return out


def he_weighted_aggregate_ntt(ctx: Ctx, cts: List[torch.Tensor], alpha: Sequence[float],
                              out: Optional[torch.Tensor] = None) -> torch.Tensor:
    _same_len(cts, alpha, "he_weighted_aggregate_ntt cts and alpha")
    Cn = len(cts)
    T = _ct_count(ctx, cts[0], ctx.L, "he_weighted_aggregate_ntt cts[0]")
    for i, c in enumerate(cts):
        _sized(c, T * 2 * ctx.L * ctx.N, "he_weighted_aggregate_ntt cts[%d]" % i, exact=True)
    if out is None:
        out = torch.empty((T, 2, ctx.L - 1, ctx.N), dtype=torch.int64, device="cuda")
    _sized(out, T * 2 * (ctx.L - 1) * ctx.N, "he_weighted_aggregate_ntt out")
    ptrs = (_vp * Cn)(*[_dev(c, torch.int64) for c in cts])
    al = (C.c_double * Cn)(*[float(a) for a in alpha])
    _check(_lib.he_weighted_aggregate_ntt(ctx.handle, C.cast(ptrs, _vp), C.cast(al, _vp), Cn, T,
                                          _dev(out, torch.int64), _stream()), "he_weighted_aggregate_ntt")
    return out


def he_plain_aggregate(ctx: Ctx, rests: List[torch.Tensor], alpha: Sequence[float]) -> torch.Tensor:
    _same_len(rests, alpha, "he_plain_aggregate rests and alpha")
    Cn = len(rests)
    n = rests[0].numel()
    for i, r in enumerate(rests):
        _sized(r, n, "he_plain_aggregate rests[%d]" % i, exact=True)
    ptrs = (_vp * Cn)(*[_dev(r, torch.float32) if n else 1 for r in rests])
    al = (C.c_double * Cn)(*[float(a) for a in alpha])
    out = torch.empty(n, dtype=torch.float64, device="cuda")
    _check(_lib.he_plain_aggregate(ctx.handle, C.cast(ptrs, _vp), C.cast(al, _vp), Cn, n, out.data_ptr(),
                                   _stream()), "he_plain_aggregate")
    return out


def he_decrypt(ctx: Ctx, keys: Keys, agg: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    T = _ct_count(ctx, agg, ctx.L - 1, "he_decrypt agg")
    if out is None:
        out = torch.empty(T * ctx.n, dtype=torch.float64, device="cuda")
    _sized(out, T * ctx.n, "he_decrypt out")
    _check(_lib.he_decrypt(ctx.handle, keys.handle, _dev(agg, torch.int64), T, _dev(out, torch.float64),
                           _stream()), "he_decrypt")
    return out


def he_decrypt_level(ctx: Ctx, keys: Keys, ct: torch.Tensor, level: int) -> torch.Tensor:
    T = _ct_count(ctx, ct, level, "he_decrypt_level ct")
    z = torch.empty(T * ctx.n, dtype=torch.float64, device="cuda")
    _check(_lib.he_decrypt_level(ctx.handle, keys.handle, _dev(ct, torch.int64), level, T, z.data_ptr(),
                                 _stream()), "he_decrypt_level")
    return z


def he_decrypt_level_ntt(ctx: Ctx, keys: Keys, ct: torch.Tensor, level: int,
                         out: Optional[torch.Tensor] = None) -> torch.Tensor:
    T = _ct_count(ctx, ct, level, "he_decrypt_level_ntt ct")
    if out is None:
        out = torch.empty(T * ctx.n, dtype=torch.float64, device="cuda")
    _sized(out, T * ctx.n, "he_decrypt_level_ntt out")
    _check(_lib.he_decrypt_level_ntt(ctx.handle, keys.handle, _dev(ct, torch.int64), level, T,
                                     _dev(out, torch.float64), _stream()), "he_decrypt_level_ntt")
    return out


def he_threshold_split(ctx: Ctx, keys: Keys, seed: int):
    """Two additive shares of the secret key (handles accepted by he_partial_decrypt only)."""
    a, b = _vp(), _vp()
    _check(_lib.he_threshold_split(ctx.handle, keys.handle, seed, C.byref(a), C.byref(b), _stream()),
           "he_threshold_split")
    return Keys(a.value, ctx), Keys(b.value, ctx)


def he_partial_decrypt(ctx: Ctx, share: Keys, party: int, ct: torch.Tensor, level: int, seed: int,
                       smudge_bits: int) -> torch.Tensor:
    """Residues mod q_0, uint64-as-int64 [T][N]."""
    T = _ct_count(ctx, ct, level, "he_partial_decrypt ct")
    part = torch.empty((T, ctx.N), dtype=torch.int64, device="cuda")
    _check(_lib.he_partial_decrypt(ctx.handle, share.handle, party, _dev(ct, torch.int64) or None, level, T,
                                   seed, smudge_bits, part.data_ptr() or None, _stream()), "he_partial_decrypt")
    return part


def he_threshold_combine(ctx: Ctx, ct: torch.Tensor, level: int, parts: List[torch.Tensor]) -> torch.Tensor:
    T = _ct_count(ctx, ct, level, "he_threshold_combine ct")
    for i, p in enumerate(parts):
        _sized(p, T * ctx.N, "he_threshold_combine parts[%d]" % i, exact=True)
    ptrs = (_vp * len(parts))(*[_dev(p, torch.int64) for p in parts])
    z = torch.empty(T * ctx.n, dtype=torch.float64, device="cuda")
    _check(_lib.he_threshold_combine(ctx.handle, _dev(ct, torch.int64) or None, level, C.cast(ptrs, _vp),
                                     len(parts), T, z.data_ptr() or None, _stream()), "he_threshold_combine")
    return z


HE_NOALLOC_MAX_WORDS = 1 << 21


def he_decrypt_noalloc(ctx: Ctx, keys: Keys, agg: torch.Tensor, out: torch.Tensor) -> torch.Tensor:
    """he_decrypt without any allocation inside the library: the work buffer is a fixed array
    in the library image, so T * N must not exceed HE_NOALLOC_MAX_WORDS and N must be <= 16384.
    `out` (float64 [T*n]) is supplied by the caller for the same reason."""
    T = _ct_count(ctx, agg, ctx.L - 1, "he_decrypt_noalloc agg")
    _sized(out, T * ctx.n, "he_decrypt_noalloc out")
    _check(_lib.he_decrypt_noalloc(ctx.handle, keys.handle, _dev(agg, torch.int64) or None, T,
                                   _dev(out, torch.float64) or None, _stream()), "he_decrypt_noalloc")
    return out


def he_unpack(ctx: Ctx, mask: Optional[Mask], z: torch.Tensor, rest_avg: Optional[torch.Tensor], P: int,
              out: Optional[torch.Tensor] = None) -> torch.Tensor:
    k = P
    if mask is not None:
        if mask.P != P:
            raise HeError(HE_ERR_INVALID_ARG, "he_unpack: the mask was built for %d parameters, P is %d" % (mask.P, P))
        k = mask.k
        if k < P:
            if rest_avg is None:
                raise HeError(HE_ERR_INVALID_ARG, "he_unpack: rest_avg is missing")
            _sized(rest_avg, P - k, "he_unpack rest_avg")
    _sized(z, k, "he_unpack z")
    if out is None:
        out = torch.empty(P, dtype=torch.float64, device="cuda")
    _sized(out, P, "he_unpack out")
    _check(_lib.he_unpack(ctx.handle, mask.handle if mask else None, _dev(z, torch.float64) or None,
                          _dev(rest_avg, torch.float64) if (rest_avg is not None and rest_avg.numel()) else None,
                          P, _dev(out, torch.float64), _stream()), "he_unpack")
    return out


def he_ntt_forward(ctx: Ctx, polys: torch.Tensor) -> torch.Tensor:
    """In place on uint64-as-int64 [B][L][N]."""
    _sized(polys, (polys.shape[0] if polys.dim() else 0) * ctx.L * ctx.N, "he_ntt_forward polys", exact=True)
    _check(_lib.he_ntt_forward(ctx.handle, _dev(polys, torch.int64), polys.shape[0], _stream()),
           "he_ntt_forward")
    return polys


def he_ntt_inverse(ctx: Ctx, polys: torch.Tensor) -> torch.Tensor:
    _sized(polys, (polys.shape[0] if polys.dim() else 0) * ctx.L * ctx.N, "he_ntt_inverse polys", exact=True)
    _check(_lib.he_ntt_inverse(ctx.handle, _dev(polys, torch.int64), polys.shape[0], _stream()),
           "he_ntt_inverse")
    return polys


def he_round_host(ctx: Ctx, keys: Keys, mask: Optional[Mask], xs: List[torch.Tensor],
                  alpha: Sequence[float], enc_seed: int, out: torch.Tensor) -> torch.Tensor:
    """Whole round with HOST tensors in (float32 [P] each, ideally pinned) and out (float64 [P])."""
    _same_len(xs, alpha, "he_round_host xs and alpha")
    Cn = len(xs)
    P = xs[0].numel()
    if mask is not None and mask.P != P:
        raise HeError(HE_ERR_INVALID_ARG, "he_round_host: the mask was built for %d parameters, xs have %d" % (mask.P, P))
    for x in xs:
        if x.is_cuda or x.dtype != torch.float32 or not x.is_contiguous() or x.numel() != P:
            raise TypeError("xs must be contiguous host float32 tensors of one size")
    if out.is_cuda or out.dtype != torch.float64 or out.numel() != P:
        raise TypeError("out must be a host float64 tensor of P entries")
    ptrs = (_vp * Cn)(*[x.data_ptr() for x in xs])
    al = (C.c_double * Cn)(*[float(a) for a in alpha])
    _check(_lib.he_round_host(ctx.handle, keys.handle, mask.handle if mask else None, C.cast(ptrs, _vp),
                              C.cast(al, _vp), Cn, P, enc_seed, out.data_ptr(), _stream()), "he_round_host")
    return out
