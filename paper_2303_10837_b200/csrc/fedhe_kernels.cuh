// Shared by the kernel files of the library: launch bookkeeping, the error
// samplers, small modular helpers, the per-limb choice of arithmetic and the
// outer stages of the long transforms.
#pragma once

#include "fedhe_launch.h"

#include <atomic>
#include <type_traits>

namespace fedhe {

extern std::atomic<uint64_t> g_launches;      // kernels launched by this library (fedhe_transform.cu)

#define FEDHE_LAUNCHED() (g_launches.fetch_add(1), cudaGetLastError())

static inline unsigned blocks_for(size_t count, unsigned per_block) {
    return (unsigned)((count + per_block - 1) / per_block);
}

// ---------------------------------------------------------------------------
// discrete Gaussian, sigma = 3.2 on [-19, 19]: thresholds floor(2^64 Pr[X <= x])
// for x = -19 .. 18; a 64-bit uniform r maps to -19 + #{x : r >= T[x]}
// ---------------------------------------------------------------------------
static __constant__ uint64_t c_gauss_cdf[38] = {
    0x0000000bd798c7acull, 0x00000053f5e234f7ull, 0x000001e24b89625aull, 0x000009adbc7900e1ull,
    0x00002d17ca1e3a82ull, 0x0000bf05ff772ee2ull, 0x0002e06843bbf95dull, 0x000a19062dceb033ull,
    0x00204c0ded173b17ull, 0x005e3163ffc656a8ull, 0x00fab6a7e614dfaeull, 0x0261b16e99bc14f8ull,
    0x054c69348bbc9867ull, 0x0acd276539458231ull, 0x143796b3c337f00bull, 0x22d43df09de40e7aull,
    0x37651d96aa4fb429ull, 0x51a5da2b40f1bff1ull, 0x700ad4bf5a6e80e2ull, 0x8ff52b40a5917f1dull,
    0xae5a25d4bf0e400eull, 0xc89ae26955b04bd6ull, 0xdd2bc20f621bf185ull, 0xebc8694c3cc80ff4ull,
    0xf532d89ac6ba7dceull, 0xfab396cb74436798ull, 0xfd9e4e916643eb07ull, 0xff05495819eb2051ull,
    0xffa1ce9c0039a957ull, 0xffdfb3f212e8c4e8ull, 0xfff5e6f9d2314fccull, 0xfffd1f97bc4406a2ull,
    0xffff40fa0088d11dull, 0xffffd2e835e1c57dull, 0xfffff6524386ff1eull, 0xfffffe1db4769da5ull,
    0xffffffac0a1dcb08ull, 0xfffffff428673853ull};

__device__ __forceinline__ int gauss_from_u64(uint64_t r) {
    int v = -19;
#pragma unroll
    for (int x = 0; x < 38; x++) v += (r >= c_gauss_cdf[x]) ? 1 : 0;
    return v;
}

// The same map through shared-memory tables: the top byte of r selects the
// thresholds that are certainly below r (`base`) and the few that share its
// byte (`nb`, compared one by one).
struct GaussTables {
    uint64_t cdf[38];
    uint8_t base[256];
    uint8_t nb[256];
};

__device__ __forceinline__ void gauss_tables_init(GaussTables &g, uint32_t tid) {
    if (tid < 38) g.cdf[tid] = c_gauss_cdf[tid];
    if (tid < 256) {
        const uint64_t lo = (uint64_t)tid << 56, hi = lo | 0x00ffffffffffffffull;
        int base = 0, nb = 0;
        for (int x = 0; x < 38; x++) {
            const uint64_t t = c_gauss_cdf[x];
            if (t <= lo) base++;
            else if (t <= hi) nb++;
        }
        g.base[tid] = (uint8_t)base;
        g.nb[tid] = (uint8_t)nb;
    }
}

__device__ __forceinline__ int gauss_from_u64(const GaussTables &g, uint64_t r) {
    const uint32_t b = (uint32_t)(r >> 56);
    const int base = g.base[b], nb = g.nb[b];
    int v = base;
    for (int i = 0; i < nb; i++) v += (r >= g.cdf[base + i]) ? 1 : 0;
    return v - 19;
}

__device__ __forceinline__ uint64_t addmod(uint64_t a, uint64_t b, uint64_t q) { return csub(a + b, q); }
__device__ __forceinline__ uint64_t submod(uint64_t a, uint64_t b, uint64_t q) { return a >= b ? a - b : a + q - b; }

// slow exact helpers, used only when keys and key shares are made
static __device__ uint64_t mod_u128(uint64_t hi, uint64_t lo, uint64_t q) {
    uint64_t r = 0;
    for (int i = 63; i >= 0; i--) { r = (r << 1) | ((hi >> i) & 1); r = csub(r, q); }
    for (int i = 63; i >= 0; i--) { r = (r << 1) | ((lo >> i) & 1); r = csub(r, q); }
    return r;
}
static __device__ uint64_t mulmod_slow(uint64_t a, uint64_t b, uint64_t q) {
    return mod_u128(__umul64hi(a, b), a * b, q);
}
static __device__ uint64_t shoup_companion(uint64_t w, uint64_t q) {   // floor(w 2^64 / q), w < q
    uint64_t rem = w, quo = 0;
    for (int i = 0; i < 64; i++) {
        rem <<= 1; quo <<= 1;
        if (rem >= q) { rem -= q; quo |= 1; }
    }
    return quo;
}

// A limb runs in double-precision arithmetic when its prime allows it.
#define FEDHE_FOR_ARITH(lb, CALL)                               \
    if ((lb).fwd_d) { using M_ = ModF64; CALL; }                \
    else { using M_ = ModInt; CALL; }

// the same with the select flavour of the integer arithmetic (kernels bound by the multiply pipe)
#define FEDHE_FOR_ARITH_SEL(lb, CALL)                           \
    if ((lb).fwd_d) { using M_ = ModF64; CALL; }                \
    else { using M_ = ModIntSel; CALL; }

// The A = logN - LOGB outer stages of a long transform on two neighbouring
// columns of the 2^A x B matrix view (x[a], y[a] = row a): forward from
// canonical input, inverse with 1/N folded into stage 0.
template <uint32_t A, class M>
__device__ __forceinline__ void outer_forward(typename M::val (&x)[1u << A], typename M::val (&y)[1u << A],
                                              const NttArgsT<M> &t) {
    constexpr uint32_t rows = 1u << A;
#pragma unroll
    for (uint32_t s = 0; s < A; s++) {
        const uint32_t bit = 1u << (A - 1 - s);
#pragma unroll
        for (uint32_t a = 0; a < rows; a++) {
            if (a & bit) continue;
            const auto w = M::load(t.tw + (1u << s) + (a >> (A - s)));
            t.m.fwd(x[a], x[a | bit], w);
            t.m.fwd(y[a], y[a | bit], w);
        }
    }
}

template <uint32_t A, class M, class T>
__device__ __forceinline__ void outer_inverse(typename M::val (&x)[1u << A], typename M::val (&y)[1u << A],
                                              const NttArgsT<M> &t, const T &ninv, const T &wn) {
    constexpr uint32_t rows = 1u << A;
#pragma unroll
    for (int s = (int)A - 1; s >= 1; s--) {
        const uint32_t bit = 1u << (A - 1 - s);
#pragma unroll
        for (uint32_t a = 0; a < rows; a++) {
            if (a & bit) continue;
            const auto w = M::load(t.tw + (1u << s) + (a >> (A - s)));
            t.m.inv(x[a], x[a | bit], w);
            t.m.inv(y[a], y[a | bit], w);
        }
    }
    constexpr uint32_t bit = 1u << (A - 1);      // stage 0 with 1/N folded in
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        if (a & bit) continue;
        t.m.inv_scaled(x[a], x[a | bit], ninv, wn);
        t.m.inv_scaled(y[a], y[a | bit], ninv, wn);
    }
}

// The outer stages as an elementwise pass over HBM: every thread owns two
// neighbouring columns and reads and writes whole 16-byte words.
// launches kern<A> for the context's A (1, 2 or 3)
#define FEDHE_FOR_A(c, CALL)                 \
    switch ((c).A) {                         \
    case 1: { constexpr uint32_t A_ = 1; CALL; } break; \
    case 2: { constexpr uint32_t A_ = 2; CALL; } break; \
    default: { constexpr uint32_t A_ = 3; CALL; } break; \
    }

// the block (inner) stages of a batch of transforms only (fedhe_transform.cu)
cudaError_t launch_ntt_inner(const CtxDev &c, bool forward, uint64_t *data, size_t npoly, size_t poly_stride,
                             uint32_t limb0, uint32_t nlimbs, cudaStream_t s);

}  // namespace fedhe
