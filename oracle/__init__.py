"""ctypes view of the CPU oracle (``fedhe_oracle.c``).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH: only the tests, the smoke check and
the benchmark's CPU-baseline leg import this package.  It never imports the
CUDA package, and the CUDA package never imports it.

The shared object is built on first import with gcc (``-ffp-contract=off`` so
that every floating-point operation of the encode network is a separate IEEE
operation, ``-fopenmp`` so that independent ciphertext indices can run on all
host cores).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fedhe_oracle.c")
_HDR = os.path.join(_HERE, "fedhe_oracle.h")
_SO = os.path.join(_HERE, "libfedhe_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or stale."""
    stale = (not os.path.exists(_SO)
             or os.path.getmtime(_SO) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _SO + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=gnu11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lquadmath", "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _SO)
    return _SO


_lib = C.CDLL(build())

_u64 = C.c_uint64
_u32 = C.c_uint32
_sz = C.c_size_t
_vp = C.c_void_p


def _sig(name, res, *args):
    f = getattr(_lib, name)
    f.restype = res
    f.argtypes = list(args)
    return f


_mulmod = _sig("orc_mulmod", _u64, _u64, _u64, _u64)
_powmod = _sig("orc_powmod", _u64, _u64, _u64, _u64)
_invmod = _sig("orc_invmod", _u64, _u64, _u64)
_is_prime = _sig("orc_is_prime", C.c_int, _u64)
_min_root = _sig("orc_min_root_2n", _u64, _u64, _u32)
_ctx_create = _sig("orc_ctx_create", _vp, _u32, _u32, _vp, C.c_int)
_ctx_destroy = _sig("orc_ctx_destroy", None, _vp)
_ctx_psi = _sig("orc_ctx_psi", _u64, _vp, _u32)
_tw = _sig("orc_twiddle_table", None, _vp, _vp)
_ntt_f = _sig("orc_ntt_forward", None, _vp, _u32, _vp)
_ntt_i = _sig("orc_ntt_inverse", None, _vp, _u32, _vp)
_mul_ntt = _sig("orc_negacyclic_mul_ntt", None, _vp, _u32, _vp, _vp, _vp)
_mul_sb = _sig("orc_negacyclic_mul_schoolbook", None, _u32, _u64, _vp, _vp, _vp)
_philox = _sig("orc_philox4x32_10", None, _vp, _vp, _vp)
_gauss_table = _sig("orc_gauss_table", None, _vp)
_s_tern = _sig("orc_sample_ternary", None, _u64, _u32, _u32, _u32, _u32, _vp)
_s_gauss = _sig("orc_sample_gauss", None, _u64, _u32, _u32, _u32, _u32, _vp)
_s_unif = _sig("orc_sample_uniform", None, _u64, _u32, _u32, _u32, _u32, _u64, _u32, _vp)
_keygen = _sig("orc_keygen", None, _vp, _u64, _vp, _vp)
_encode = _sig("orc_encode", C.c_int, _vp, _vp, _vp)
_encrypt_one = _sig("orc_encrypt_one", None, _vp, _vp, _vp, _u64, _u32, _u32, _vp)
_encrypt = _sig("orc_encrypt", C.c_int, _vp, _vp, _vp, _sz, _u64, _u32, _vp)
_weights = _sig("orc_weights", None, _vp, _vp, _u32, _vp)
_wsum = _sig("orc_weighted_sum", None, _vp, _vp, _vp, _u32, _sz, _vp)
_rescale = _sig("orc_rescale", None, _vp, _vp, _sz, _vp)
_plain = _sig("orc_plain_aggregate", None, _vp, _vp, _u32, _sz, _vp)
_dec_limb = _sig("orc_decrypt_limb", None, _vp, _vp, _vp, _u32, _u32, _vp)
_decrypt = _sig("orc_decrypt", None, _vp, _vp, _vp, _u32, _sz, _vp)
_decode = _sig("orc_decode", None, _vp, _vp, _vp)
_th_split = _sig("orc_threshold_split", None, _vp, _vp, _u64, _vp, _vp)
_smudge = _sig("orc_sample_smudge", None, _u64, _u32, _u32, _u32, _u32, _vp)
_th_partial = _sig("orc_partial_decrypt", None, _vp, _vp, _u32, _vp, _u32, _u64, _u32, _u32, _vp)
_th_combine = _sig("orc_threshold_combine", None, _vp, _vp, _u32, _vp, _u32, _vp)
_select = _sig("orc_select_mask", None, _vp, _sz, _sz, _vp)
_pack = _sig("orc_pack", None, _vp, _vp, _sz, _vp, _sz, _vp, _vp)
_unpack = _sig("orc_unpack", None, _vp, _sz, _vp, _vp, _sz, _vp)
_round = _sig("orc_round", C.c_int, _vp, _vp, _vp, _u32, _sz, _vp, _sz, _u64, _u64, _sz, _sz,
              C.c_int, _vp)
_nthreads = _sig("orc_num_threads", C.c_int)


def _p(a):
    return a.ctypes.data_as(_vp) if a is not None else None


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _ptr_array(arrs):
    return (_vp * len(arrs))(*[a.ctypes.data for a in arrs])


def mulmod(a, b, q):
    return int(_mulmod(a, b, q))


def powmod(a, e, q):
    return int(_powmod(a, e, q))


def invmod(a, q):
    return int(_invmod(a, q))


def is_prime(q):
    return bool(_is_prime(q))


def min_root_2n(q, N):
    return int(_min_root(q, N))


def philox4x32_10(ctr, key):
    c = _arr(ctr, np.uint32)
    k = _arr(key, np.uint32)
    out = np.empty(4, np.uint32)
    _philox(_p(c), _p(k), _p(out))
    return out


def gauss_table():
    out = np.empty(38, np.uint64)
    _gauss_table(_p(out))
    return out


def sample_ternary(seed, t, client, tag, N):
    out = np.empty(N, np.int8)
    _s_tern(seed, t, client, tag, N, _p(out))
    return out


def sample_gauss(seed, t, client, tag, N):
    out = np.empty(N, np.int8)
    _s_gauss(seed, t, client, tag, N, _p(out))
    return out


def sample_uniform(seed, t, client, tag, limb, q, N):
    out = np.empty(N, np.uint64)
    _s_unif(seed, t, client, tag, limb, q, N, _p(out))
    return out


def sample_smudge(seed, t, party, bits, N):
    out = np.empty(N, np.int64)
    _smudge(seed, t, party, bits, N, _p(out))
    return out


def negacyclic_mul_schoolbook(N, q, a, b):
    a = _arr(a, np.uint64)
    b = _arr(b, np.uint64)
    out = np.empty(N, np.uint64)
    _mul_sb(N, q, _p(a), _p(b), _p(out))
    return out


def select_mask(score, k):
    score = _arr(score, np.float32)
    idx = np.empty(k, np.uint32)
    _select(_p(score), score.size, k, _p(idx))
    return idx


def plain_aggregate(rests, alpha):
    rests = [_arr(r, np.float32) for r in rests]
    alpha = _arr(alpha, np.float64)
    out = np.empty(rests[0].size, np.float64)
    _plain(_ptr_array(rests), _p(alpha), len(rests), rests[0].size, _p(out))
    return out


def unpack(idx, k, z, rest_avg, P):
    z = _arr(z, np.float64)
    out = np.empty(P, np.float64)
    if idx is not None:
        idx = _arr(idx, np.uint32)
        rest_avg = _arr(rest_avg, np.float64)
    _unpack(_p(idx), k, _p(z), _p(rest_avg) if idx is not None else None, P, _p(out))
    return out


def num_threads():
    return int(_nthreads())


class Context:
    """Ring degree N, primes q (all ciphertext limbs), scale 2**log2_delta."""

    def __init__(self, N, q, log2_delta):
        self.N = int(N)
        self.n = self.N // 2
        self.q = [int(x) for x in q]
        self.L = len(self.q)
        self.log2_delta = int(log2_delta)
        qa = np.asarray(self.q, np.uint64)
        self._h = _ctx_create(self.N, self.L, _p(qa), self.log2_delta)
        if not self._h:
            raise ValueError("oracle rejected the parameters")

    def __del__(self):
        if getattr(self, "_h", None):
            _ctx_destroy(self._h)
            self._h = None

    def psi(self, limb):
        return int(_ctx_psi(self._h, limb))

    def twiddle_table(self):
        out = np.empty((2 * self.N, 2), np.float64)
        _tw(self._h, _p(out))
        return out

    def ntt_forward(self, limb, a):
        a = np.array(a, np.uint64, copy=True)
        _ntt_f(self._h, limb, _p(a))
        return a

    def ntt_inverse(self, limb, a):
        a = np.array(a, np.uint64, copy=True)
        _ntt_i(self._h, limb, _p(a))
        return a

    def negacyclic_mul_ntt(self, limb, a, b):
        a = _arr(a, np.uint64)
        b = _arr(b, np.uint64)
        out = np.empty(self.N, np.uint64)
        _mul_ntt(self._h, limb, _p(a), _p(b), _p(out))
        return out

    def keygen(self, seed):
        s = np.empty(self.N, np.int8)
        pk = np.empty((2, self.L, self.N), np.uint64)
        _keygen(self._h, seed, _p(s), _p(pk))
        return s, pk

    def encode(self, slots):
        slots = _arr(slots, np.float32)
        assert slots.size == self.n
        m = np.empty(self.N, np.int64)
        ov = _encode(self._h, _p(slots), _p(m))
        return m, bool(ov)

    def encrypt_one(self, pk, m, seed, client, t):
        pk = _arr(pk, np.uint64)
        m = _arr(m, np.int64)
        ct = np.empty((2, self.L, self.N), np.uint64)
        _encrypt_one(self._h, _p(pk), _p(m), seed, client, t, _p(ct))
        return ct

    def num_ct(self, k):
        return (k + self.n - 1) // self.n

    def encrypt(self, pk, sel, seed, client):
        pk = _arr(pk, np.uint64)
        sel = _arr(sel, np.float32)
        T = sel.size // self.n
        assert T * self.n == sel.size
        ct = np.empty((T, 2, self.L, self.N), np.uint64)
        bad = _encrypt(self._h, _p(pk), _p(sel), T, seed, client, _p(ct))
        return ct, int(bad)

    def weights(self, alpha):
        alpha = _arr(alpha, np.float64)
        W = np.empty(alpha.size, np.uint64)
        _weights(self._h, _p(alpha), alpha.size, _p(W))
        return W

    def weighted_sum(self, cts, W):
        cts = [_arr(c, np.uint64) for c in cts]
        W = _arr(W, np.uint64)
        T = cts[0].shape[0]
        acc = np.empty((T, 2, self.L, self.N), np.uint64)
        _wsum(self._h, _ptr_array(cts), _p(W), len(cts), T, _p(acc))
        return acc

    def rescale(self, acc):
        acc = _arr(acc, np.uint64)
        T = acc.shape[0]
        out = np.empty((T, 2, self.L - 1, self.N), np.uint64)
        _rescale(self._h, _p(acc), T, _p(out))
        return out

    def decrypt_limb(self, s, ct, level, limb):
        s = _arr(s, np.int8)
        ct = _arr(ct, np.uint64)
        out = np.empty(self.N, np.uint64)
        _dec_limb(self._h, _p(s), _p(ct), level, limb, _p(out))
        return out

    def decrypt(self, s, ct, level):
        s = _arr(s, np.int8)
        ct = _arr(ct, np.uint64)
        T = ct.shape[0]
        d = np.empty((T, self.N), np.int64)
        _decrypt(self._h, _p(s), _p(ct), level, T, _p(d))
        return d

    def decode(self, d):
        d = _arr(d, np.int64)
        if d.ndim == 1:
            z = np.empty(self.n, np.float64)
            _decode(self._h, _p(d), _p(z))
            return z
        z = np.empty((d.shape[0], self.n), np.float64)
        for t in range(d.shape[0]):
            _decode(self._h, d[t].ctypes.data_as(_vp), z[t].ctypes.data_as(_vp))
        return z

    def threshold_split(self, s, seed):
        s = _arr(s, np.int8)
        a = np.empty((self.L, self.N), np.uint64)
        b = np.empty((self.L, self.N), np.uint64)
        _th_split(self._h, _p(s), seed, _p(a), _p(b))
        return a, b

    def partial_decrypt(self, share, party, ct, level, seed, t, bits):
        share = _arr(share, np.uint64)
        ct = _arr(ct, np.uint64)
        out = np.empty(self.N, np.uint64)
        _th_partial(self._h, _p(share), party, _p(ct), level, seed, t, bits, _p(out))
        return out

    def threshold_combine(self, ct, level, parts):
        ct = _arr(ct, np.uint64)
        parts = [_arr(x, np.uint64) for x in parts]
        d = np.empty(self.N, np.int64)
        _th_combine(self._h, _p(ct), level, _ptr_array(parts), len(parts), _p(d))
        return d

    def pack(self, idx, k, x):
        x = _arr(x, np.float32)
        T = self.num_ct(k)
        sel = np.empty(T * self.n, np.float32)
        if idx is None:
            _pack(self._h, None, k, _p(x), x.size, _p(sel), None)
            return sel, None
        idx = _arr(idx, np.uint32)
        rest = np.empty(x.size - k, np.float32)
        _pack(self._h, _p(idx), k, _p(x), x.size, _p(sel), _p(rest))
        return sel, rest

    def round(self, xs, alpha, idx, k, key_seed, enc_seed, t_begin=0, t_end=None, do_rest=True,
              out=None):
        """Whole round on ciphertext indices [t_begin, t_end); returns w_glob (fp64)."""
        xs = [_arr(x, np.float32) for x in xs]
        alpha = _arr(alpha, np.float64)
        P = xs[0].size
        if t_end is None:
            t_end = self.num_ct(k)
        if idx is not None:
            idx = _arr(idx, np.uint32)
        if out is None:
            out = np.zeros(P, np.float64)
        rc = _round(self._h, _ptr_array(xs), _p(alpha), len(xs), P, _p(idx), k, key_seed,
                    enc_seed, t_begin, t_end, 1 if do_rest else 0, _p(out))
        if rc != 0:
            raise MemoryError("oracle round failed")
        return out
