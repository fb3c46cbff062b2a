// CUDA kernels (sm_100a) of the FedML-HE secure-aggregation hot path and their
// launch wrappers.  Nothing here is a dense floating-point contraction, so no
// tensor-core path exists: the transforms are bound by the issue rate of
// integer multiplies (limbs with large primes) and double-precision
// operations (limbs with primes below 2^46), the pointwise passes by HBM
// bandwidth.
#include "fedhe_launch.h"

#include <atomic>
#include <type_traits>

namespace fedhe {

static std::atomic<uint64_t> g_launches{0};
uint64_t launch_count() { return g_launches.load(); }

#define FEDHE_LAUNCHED() (g_launches.fetch_add(1), cudaGetLastError())

static inline unsigned blocks_for(size_t count, unsigned per_block) {
    return (unsigned)((count + per_block - 1) / per_block);
}

// ---------------------------------------------------------------------------
// discrete Gaussian, sigma = 3.2 on [-19, 19]: thresholds floor(2^64 Pr[X <= x])
// for x = -19 .. 18; a 64-bit uniform r maps to -19 + #{x : r >= T[x]}
// ---------------------------------------------------------------------------
__constant__ uint64_t c_gauss_cdf[38] = {
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

// slow exact helpers, used only at key generation
__device__ uint64_t mod_u128(uint64_t hi, uint64_t lo, uint64_t q) {
    uint64_t r = 0;
    for (int i = 63; i >= 0; i--) { r = (r << 1) | ((hi >> i) & 1); r = csub(r, q); }
    for (int i = 63; i >= 0; i--) { r = (r << 1) | ((lo >> i) & 1); r = csub(r, q); }
    return r;
}
__device__ uint64_t mulmod_slow(uint64_t a, uint64_t b, uint64_t q) {
    return mod_u128(__umul64hi(a, b), a * b, q);
}
__device__ uint64_t shoup_companion(uint64_t w, uint64_t q) {   // floor(w 2^64 / q), w < q
    uint64_t rem = w, quo = 0;
    for (int i = 0; i < 64; i++) {
        rem <<= 1; quo <<= 1;
        if (rem >= q) { rem -= q; quo |= 1; }
    }
    return quo;
}

// ===========================================================================
// batched negacyclic NTT
// ===========================================================================

// A limb runs in double-precision arithmetic when its prime allows it.
#define FEDHE_FOR_ARITH(lb, CALL)                               \
    if ((lb).fwd_d) { using M_ = ModF64; CALL; }                \
    else { using M_ = ModInt; CALL; }

// Representations in global memory.  What a caller hands in or gets back is
// canonical residues.  Between the two passes of a long transform the data is
// in the arithmetic's own form (lazy 64-bit integers, or the bits of signed
// doubles): forward, outer pass -> block pass; inverse, block pass -> outer
// pass.  The inverse block pass reads residues below 2q.

// One block of B = 2^LOGB residues (a whole limb for N <= 2^14), transformed
// in place in shared memory; every thread plays V virtual threads per phase
// with E residues in registers at a time.
template <class M, class L, int V, bool FWD, bool SCALED>
__device__ __forceinline__ void ntt_block(const CtxDev &c, const LimbDev &lb, uint64_t *sm, uint64_t *p,
                                          uint32_t blk) {
    using val = typename M::val;
    const uint32_t tid = threadIdx.x;
    const auto a = LimbOf<M>::args(lb, FWD, c.A, blk);
    const M &ar = a.m;
    if constexpr (FWD) {
        const bool piece = c.A > 0;
        smem_ntt_forward<L, V>(
            sm, tid, a, [&](uint32_t i) { return piece ? M::from_bits(p[i]) : ar.from_residue(p[i]); },
            [&](uint32_t i, val u, val v) {
                u64x2 o;
                o.x = ar.canon_wide(u);
                o.y = ar.canon_wide(v);
                *reinterpret_cast<u64x2 *>(p + i) = o;
            });
    } else {
        smem_ntt_inverse<L, V, SCALED>(
            sm, tid, a, LimbOf<M>::ninv(lb), LimbOf<M>::wn(lb),
            [&](uint32_t i) {
                const u64x2 t = *reinterpret_cast<const u64x2 *>(p + i);
                return pair_of<val>{ar.from_residue(t.x), ar.from_residue(t.y)};
            },
            [&](uint32_t i, val v) { p[i] = SCALED ? ar.canon(v) : M::bits(v); });
    }
}

template <class L, int V, bool FWD, bool SCALED>
__global__ void __launch_bounds__(L::NT / V, (L::NT / V) <= 512 ? 2 : 1)
ntt_block_kernel(const __grid_constant__ CtxDev c, uint64_t *data, size_t poly_stride, uint32_t limb0,
                         uint32_t nlimbs) {
    extern __shared__ __align__(16) uint64_t sm[];
    uint32_t b = blockIdx.x;
    const uint32_t blk = b & ((1u << c.A) - 1u);
    b >>= c.A;
    const uint32_t limb = b % nlimbs;
    const size_t poly = b / nlimbs;
    const LimbDev &lb = c.limb[limb0 + limb];
    uint64_t *p = data + poly * poly_stride + (size_t)limb * c.N + ((size_t)blk << L::LOGB);
    FEDHE_FOR_ARITH(lb, (ntt_block<M_, L, V, FWD, SCALED>(c, lb, sm, p, blk)));
}

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
template <class M, bool FWD, uint32_t A>
__device__ __forceinline__ void ntt_outer(const LimbDev &lb, uint64_t *p, uint32_t B) {
    using val = typename M::val;
    constexpr uint32_t rows = 1u << A;
    const auto t = LimbOf<M>::args(lb, FWD, 0, 0);
    val x[rows], y[rows];
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        const u64x2 v = *reinterpret_cast<const u64x2 *>(p + (size_t)a * B);
        x[a] = FWD ? t.m.from_residue(v.x) : M::from_bits(v.x);
        y[a] = FWD ? t.m.from_residue(v.y) : M::from_bits(v.y);
    }
    if constexpr (FWD) outer_forward<A>(x, y, t);
    else outer_inverse<A>(x, y, t, LimbOf<M>::ninv(lb), LimbOf<M>::wn(lb));
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        u64x2 v;
        v.x = FWD ? M::bits(x[a]) : t.m.canon(x[a]);
        v.y = FWD ? M::bits(y[a]) : t.m.canon(y[a]);
        *reinterpret_cast<u64x2 *>(p + (size_t)a * B) = v;
    }
}

template <bool FWD, uint32_t A>
__global__ void __launch_bounds__(256)
ntt_outer_kernel(const __grid_constant__ CtxDev c, uint64_t *data, size_t poly_stride, uint32_t limb0,
                 uint32_t nlimbs, size_t total) {
    size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t B = 1u << c.LOGB, half = B >> 1;
    const uint32_t col = (uint32_t)(g % half) * 2;
    g /= half;
    const uint32_t limb = (uint32_t)(g % nlimbs);
    const size_t poly = g / nlimbs;
    const LimbDev &lb = c.limb[limb0 + limb];
    uint64_t *p = data + poly * poly_stride + (size_t)limb * c.N + col;
    FEDHE_FOR_ARITH(lb, (ntt_outer<M_, FWD, A>(lb, p, B)));
}

// launches kern<A> for the context's A (1, 2 or 3)
#define FEDHE_FOR_A(c, CALL)                 \
    switch ((c).A) {                         \
    case 1: { constexpr uint32_t A_ = 1; CALL; } break; \
    case 2: { constexpr uint32_t A_ = 2; CALL; } break; \
    default: { constexpr uint32_t A_ = 3; CALL; } break; \
    }

template <class L, int V>
static cudaError_t launch_ntt_blocks(const CtxDev &c, bool forward, uint64_t *data, size_t npoly,
                                             size_t poly_stride, uint32_t limb0, uint32_t nlimbs,
                                             cudaStream_t s) {
    const size_t smem = sizeof(uint64_t) << L::LOGB;
    const unsigned grid = (unsigned)((npoly * nlimbs) << c.A);
    cudaError_t e;
    if (forward) {
        auto k = ntt_block_kernel<L, V, true, false>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
        k<<<grid, L::NT / V, smem, s>>>(c, data, poly_stride, limb0, nlimbs);
    } else if (c.A == 0) {
        auto k = ntt_block_kernel<L, V, false, true>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
        k<<<grid, L::NT / V, smem, s>>>(c, data, poly_stride, limb0, nlimbs);
    } else {
        auto k = ntt_block_kernel<L, V, false, false>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
        k<<<grid, L::NT / V, smem, s>>>(c, data, poly_stride, limb0, nlimbs);
    }
    return FEDHE_LAUNCHED();
}

// the block (inner) stages only
static cudaError_t launch_ntt_inner(const CtxDev &c, bool forward, uint64_t *data, size_t npoly,
                                    size_t poly_stride, uint32_t limb0, uint32_t nlimbs, cudaStream_t s) {
    if (c.LOGB == 13) return launch_ntt_blocks<Lay<13, 3>, 2>(c, forward, data, npoly, poly_stride, limb0, nlimbs, s);
    return launch_ntt_blocks<Lay<14, 3>, 2>(c, forward, data, npoly, poly_stride, limb0, nlimbs, s);
}

cudaError_t launch_ntt(const CtxDev &c, bool forward, uint64_t *data, size_t npoly, size_t poly_stride,
                       uint32_t limb0, uint32_t nlimbs, cudaStream_t s) {
    if (npoly == 0 || nlimbs == 0) return cudaSuccess;
    cudaError_t e;
    const size_t outer_threads = npoly * nlimbs * ((size_t)1 << (c.LOGB - 1));
    if (forward && c.A > 0) {
        FEDHE_FOR_A(c, (ntt_outer_kernel<true, A_><<<blocks_for(outer_threads, 256), 256, 0, s>>>(
                           c, data, poly_stride, limb0, nlimbs, outer_threads)));
        if ((e = FEDHE_LAUNCHED())) return e;
    }
    if ((e = launch_ntt_inner(c, forward, data, npoly, poly_stride, limb0, nlimbs, s))) return e;
    if (!forward && c.A > 0) {
        FEDHE_FOR_A(c, (ntt_outer_kernel<false, A_><<<blocks_for(outer_threads, 256), 256, 0, s>>>(
                           c, data, poly_stride, limb0, nlimbs, outer_threads)));
        if ((e = FEDHE_LAUNCHED())) return e;
    }
    return cudaSuccess;
}

// ===========================================================================
// key generation
// ===========================================================================

// tmp[0] = s, tmp[1] = a, tmp[2] = e as residues, each [L][N]
__global__ void __launch_bounds__(256)
keygen_sample_kernel(const __grid_constant__ CtxDev c, uint64_t seed, int8_t *s8, uint64_t *tmp) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= c.N) return;
    u32x4 ws = stream_block(seed, i >> 2, 0, 0, TAG_SK);
    const uint32_t wsel = (i & 3) == 0 ? ws.x : (i & 3) == 1 ? ws.y : (i & 3) == 2 ? ws.z : ws.w;
    const int sv = ternary_from_word(wsel);
    u32x4 we = stream_block(seed, i >> 1, 0, 0, TAG_PK_E);
    const uint64_t r = (i & 1) ? ((uint64_t)we.z | ((uint64_t)we.w << 32)) : ((uint64_t)we.x | ((uint64_t)we.y << 32));
    const int ev = gauss_from_u64(r);
    s8[i] = (int8_t)sv;
    const size_t LN = (size_t)c.L * c.N;
    for (uint32_t j = 0; j < c.L; j++) {
        const uint64_t q = c.limb[j].q;
        u32x4 wa = stream_block(seed, i, 0, 0, TAG_PK_A | (j << 8));
        const uint64_t lo = (uint64_t)wa.x | ((uint64_t)wa.y << 32), hi = (uint64_t)wa.z | ((uint64_t)wa.w << 32);
        tmp[0 * LN + (size_t)j * c.N + i] = small_residue(sv, q);
        tmp[1 * LN + (size_t)j * c.N + i] = mod_u128(hi, lo, q);
        tmp[2 * LN + (size_t)j * c.N + i] = small_residue(ev, q);
    }
}

// transform-domain keys with Shoup companions: pk1^ = a^, pk0^ = e^ - a^ s^
__global__ void __launch_bounds__(256)
keygen_combine_kernel(const __grid_constant__ CtxDev c, const uint64_t *tmp, tw_t *pk0_hat, tw_t *pk1_hat,
                      tw_t *s_hat) {
    const size_t LN = (size_t)c.L * c.N;
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= LN) return;
    const uint64_t q = c.limb[g / c.N].q;
    const uint64_t S = tmp[g], A = tmp[LN + g], E = tmp[2 * LN + g];
    const uint64_t p0 = submod(E, mulmod_slow(A, S, q), q);
    pk0_hat[g] = tw_t{p0, shoup_companion(p0, q)};
    pk1_hat[g] = tw_t{A, shoup_companion(A, q)};
    s_hat[g] = tw_t{S, shoup_companion(S, q)};
}

__global__ void __launch_bounds__(256) extract_values_kernel(const tw_t *src, uint64_t *dst, size_t count) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g < count) dst[g] = src[g].w;
}

cudaError_t launch_keygen_sample(const CtxDev &c, uint64_t seed, int8_t *s8, uint64_t *tmp, cudaStream_t s) {
    keygen_sample_kernel<<<blocks_for(c.N, 256), 256, 0, s>>>(c, seed, s8, tmp);
    return FEDHE_LAUNCHED();
}
cudaError_t launch_keygen_combine(const CtxDev &c, const uint64_t *tmp, tw_t *pk0_hat, tw_t *pk1_hat,
                                  tw_t *s_hat, cudaStream_t s) {
    keygen_combine_kernel<<<blocks_for((size_t)c.L * c.N, 256), 256, 0, s>>>(c, tmp, pk0_hat, pk1_hat, s_hat);
    return FEDHE_LAUNCHED();
}
cudaError_t launch_extract_values(const tw_t *src, uint64_t *dst, size_t count, cudaStream_t s) {
    extract_values_kernel<<<blocks_for(count, 256), 256, 0, s>>>(src, dst, count);
    return FEDHE_LAUNCHED();
}

// ===========================================================================
// CKKS slot transform (fp64).  Encoding must reproduce one fixed radix-2
// network operation by operation (separate IEEE multiply and add, no fused
// multiply-add), because the rounded integers are compared bit for bit.
// ===========================================================================

struct cpx { double re, im; };

__device__ __forceinline__ cpx cadd_rn(cpx a, cpx b) { return cpx{__dadd_rn(a.re, b.re), __dadd_rn(a.im, b.im)}; }
__device__ __forceinline__ cpx csub_rn(cpx a, cpx b) { return cpx{__dsub_rn(a.re, b.re), __dsub_rn(a.im, b.im)}; }
// (a + bi)(c + di) = (ac - bd) + (ad + bc) i, data operand first
__device__ __forceinline__ cpx cmul_rn(cpx x, cpx w) {
    cpx r;
    r.re = __dsub_rn(__dmul_rn(x.re, w.re), __dmul_rn(x.im, w.im));
    r.im = __dadd_rn(__dmul_rn(x.re, w.im), __dmul_rn(x.im, w.re));
    return r;
}
__device__ __forceinline__ cpx load_ftw(const double2 *ftw, uint32_t i) {
    double2 v = __ldg(ftw + i);
    return cpx{v.x, v.y};
}

// decimation-in-frequency stage of the inverse (encoding) network
template <class L, int P, int I>
__device__ __forceinline__ void dif_stage(cpx (&x)[L::E], uint32_t tid, const double2 *ftw) {
    constexpr int s = P * L::LE + I;
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    constexpr int bit = nst - 1 - I;
    constexpr uint32_t half = 1u << (L::LOGB - 1 - s);
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        if (r & (1 << bit)) continue;
        const uint32_t j = L::template idx<P>(tid, r) & (half - 1u);
        cpx w = load_ftw(ftw, half + j);
        w.im = -w.im;
        const cpx U = x[r], V = x[r | (1 << bit)];
        x[r] = cadd_rn(U, V);
        x[r | (1 << bit)] = cmul_rn(csub_rn(U, V), w);
    }
}

// decimation-in-time stage of the forward (decoding) network
template <class L, int P, int I>
__device__ __forceinline__ void dit_stage(cpx (&x)[L::E], uint32_t tid, const double2 *ftw) {
    constexpr int s = P * L::LE + I;
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    constexpr int bit = nst - 1 - I;
    constexpr uint32_t half = 1u << (L::LOGB - 1 - s);
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        if (r & (1 << bit)) continue;
        const uint32_t j = L::template idx<P>(tid, r) & (half - 1u);
        const cpx w = load_ftw(ftw, half + j);
        const cpx U = x[r], V = cmul_rn(x[r | (1 << bit)], w);
        x[r] = cadd_rn(U, V);
        x[r | (1 << bit)] = csub_rn(U, V);
    }
}

template <class L, int P, int I = 0>
__device__ __forceinline__ void dif_phase(cpx (&x)[L::E], uint32_t tid, const double2 *ftw) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    if constexpr (I < nst) {
        dif_stage<L, P, I>(x, tid, ftw);
        dif_phase<L, P, I + 1>(x, tid, ftw);
    }
}
template <class L, int P, int I>
__device__ __forceinline__ void dit_phase_from(cpx (&x)[L::E], uint32_t tid, const double2 *ftw) {
    if constexpr (I >= 0) {
        dit_stage<L, P, I>(x, tid, ftw);
        dit_phase_from<L, P, I - 1>(x, tid, ftw);
    }
}

template <class L, int PF, int PT>
__device__ __forceinline__ void cpx_exchange(cpx (&x)[L::E], cpx *sm, uint32_t tid) {
    __syncthreads();
#pragma unroll
    for (int r = 0; r < L::E; r++) sm[swz(L::template idx<PF>(tid, r))] = x[r];
    __syncthreads();
#pragma unroll
    for (int r = 0; r < L::E; r++) x[r] = sm[swz(L::template idx<PT>(tid, r))];
}

template <class L, int P = 0>
__device__ __forceinline__ void block_dif(cpx (&x)[L::E], cpx *sm, uint32_t tid, const double2 *ftw) {
    dif_phase<L, P>(x, tid, ftw);
    if constexpr (P + 1 < L::NPH) {
        cpx_exchange<L, P, P + 1>(x, sm, tid);
        block_dif<L, P + 1>(x, sm, tid, ftw);
    }
}
template <class L, int P = L::NPH - 1>
__device__ __forceinline__ void block_dit(cpx (&x)[L::E], cpx *sm, uint32_t tid, const double2 *ftw) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    dit_phase_from<L, P, nst - 1>(x, tid, ftw);
    if constexpr (P > 0) {
        cpx_exchange<L, P, P - 1>(x, sm, tid);
        block_dit<L, P - 1>(x, sm, tid, ftw);
    }
}

__device__ __forceinline__ uint32_t bitrev(uint32_t v, int bits) { return __brev(v) >> (32 - bits); }
// index swizzle of the encoder's output staging buffer: bit-reversed writes of
// a warp differ only in high index bits; folding them into the low nibble
// spreads them over the banks (checked exhaustively for both block sizes)
__device__ __forceinline__ uint32_t stage_swz(uint32_t k) { return k ^ (((k >> 8) ^ (k >> 4)) & 15u); }

// Block part of the encoder: the last LOGB stages on one block of 2^LOGB
// slots, the bit-reversal, the scaling by Delta/n and the rounding.
// FROM_CPLX: the block's input comes from the outer stages (n > block).
template <class L, bool FROM_CPLX>
__global__ void __launch_bounds__(L::NT)
encode_block_kernel(const __grid_constant__ CtxDev c, const float *sel, const double2 *cplx, int64_t *m) {
    extern __shared__ __align__(16) unsigned char smraw[];
    cpx *sm = reinterpret_cast<cpx *>(smraw);
    const uint32_t tid = threadIdx.x;
    const uint32_t n = c.N >> 1, logn = c.logN - 1;
    const uint32_t nblk = n >> L::LOGB;
    const uint32_t blk = blockIdx.x % nblk;
    const size_t t = blockIdx.x / nblk;
    const size_t base = t * n + ((size_t)blk << L::LOGB);
    cpx x[L::E];
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        const uint32_t i = L::template idx<0>(tid, r);
        if constexpr (FROM_CPLX) {
            double2 v = cplx[base + i];
            x[r] = cpx{v.x, v.y};
        } else {
            x[r] = cpx{(double)sel[base + i], 0.0};
        }
    }
    block_dif<L>(x, sm, tid, c.ftw);
    // Delta / n is a power of two: one exact multiplication
    const double scale = __longlong_as_double((long long)(1023 + c.log2_delta - (int)logn) << 52);
    const double lim = 4611686018427387904.0;   // 2^62
    int64_t *mt = m + t * c.N;
    bool bad = false;
    // The bit-reversed order would scatter 8-byte writes over the whole
    // polynomial: the rounded integers go through shared memory (real parts
    // in the first half, imaginary parts in the second) and leave in order.
    int64_t *stage = reinterpret_cast<int64_t *>(smraw);
    constexpr uint32_t NB = 1u << L::LOGB;
    __syncthreads();                                   // the exchange buffer is free again
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        const uint32_t kk = bitrev(L::template idx<L::NPH - 1>(tid, r), L::LOGB);
        double re = __dmul_rn(x[r].re, scale), im = __dmul_rn(x[r].im, scale);
        if (!(fabs(re) < lim) || !(fabs(im) < lim)) { bad = true; re = 0.0; im = 0.0; }
        stage[stage_swz(kk)] = __double2ll_rn(re);
        stage[NB + stage_swz(kk)] = __double2ll_rn(im);
    }
    __syncthreads();
    // slot k of the whole transform = (local bit-reversed index, bit-reversed block number)
    const uint32_t A = logn - L::LOGB, rb = A ? bitrev(blk, A) : 0u;
    for (uint32_t kk = tid; kk < NB; kk += L::NT) {
        const uint32_t k = (kk << A) | rb;
        mt[k] = stage[stage_swz(kk)];
        mt[k + n] = stage[NB + stage_swz(kk)];
    }
    if (bad) atomicOr(c.status, 1);
}

// Outer stages of the encoder for n > block: each thread owns one column of
// the (n / block) x block view and does the first log2(n / block) stages.
template <int LOGB>
__global__ void __launch_bounds__(256)
encode_outer_kernel(const __grid_constant__ CtxDev c, const float *sel, double2 *cplx, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t n = c.N >> 1, B = 1u << LOGB;
    const uint32_t A = (c.logN - 1) - LOGB, rows = 1u << A;   // 1 or 2
    const uint32_t col = (uint32_t)(g % B);
    const size_t t = g / B;
    cpx x[4];
    for (uint32_t a = 0; a < rows; a++) x[a] = cpx{(double)sel[t * n + (size_t)a * B + col], 0.0};
    for (uint32_t s = 0; s < A; s++) {
        const uint32_t bit = 1u << (A - 1 - s), half = n >> (s + 1);
        for (uint32_t a = 0; a < rows; a++) {
            if (a & bit) continue;
            const uint32_t j = (a * B + col) & (half - 1u);
            cpx w = load_ftw(c.ftw, half + j);
            w.im = -w.im;
            const cpx U = x[a], V = x[a | bit];
            x[a] = cadd_rn(U, V);
            x[a | bit] = cmul_rn(csub_rn(U, V), w);
        }
    }
    for (uint32_t a = 0; a < rows; a++) cplx[t * n + (size_t)a * B + col] = make_double2(x[a].re, x[a].im);
}

// Block part of the decoder: bit-reversed load of (d_k + i d_{k+n}) / Delta,
// the first LOGB stages.  TO_CPLX: more stages follow in decode_outer_kernel.
template <class L, bool TO_CPLX>
__global__ void __launch_bounds__(L::NT)
decode_block_kernel(const __grid_constant__ CtxDev c, const int64_t *d, double2 *cplx, double *z) {
    extern __shared__ __align__(16) unsigned char smraw[];
    cpx *sm = reinterpret_cast<cpx *>(smraw);
    const uint32_t tid = threadIdx.x;
    const uint32_t n = c.N >> 1, logn = c.logN - 1;
    const uint32_t nblk = n >> L::LOGB;
    const uint32_t blk = blockIdx.x % nblk;
    const size_t t = blockIdx.x / nblk;
    const int64_t *dt = d + t * c.N;
    const double inv_delta = __longlong_as_double((long long)(1023 - c.log2_delta) << 52);
    cpx x[L::E];
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        const uint32_t p = (blk << L::LOGB) | L::template idx<L::NPH - 1>(tid, r);
        const uint32_t k = bitrev(p, logn);
        x[r] = cpx{(double)dt[k] * inv_delta, (double)dt[k + n] * inv_delta};
    }
    block_dit<L>(x, sm, tid, c.ftw);
    const size_t base = t * n + ((size_t)blk << L::LOGB);
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        const uint32_t i = L::template idx<0>(tid, r);
        if constexpr (TO_CPLX) cplx[base + i] = make_double2(x[r].re, x[r].im);
        else z[base + i] = x[r].re;
    }
}

template <int LOGB>
__global__ void __launch_bounds__(256)
decode_outer_kernel(const __grid_constant__ CtxDev c, const double2 *cplx, double *z, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t n = c.N >> 1, B = 1u << LOGB;
    const uint32_t A = (c.logN - 1) - LOGB, rows = 1u << A;
    const uint32_t col = (uint32_t)(g % B);
    const size_t t = g / B;
    cpx x[4];
    for (uint32_t a = 0; a < rows; a++) {
        double2 v = cplx[t * n + (size_t)a * B + col];
        x[a] = cpx{v.x, v.y};
    }
    for (int s = (int)A - 1; s >= 0; s--) {
        const uint32_t bit = 1u << (A - 1 - s), half = n >> (s + 1);
        for (uint32_t a = 0; a < rows; a++) {
            if (a & bit) continue;
            const uint32_t j = (a * B + col) & (half - 1u);
            const cpx w = load_ftw(c.ftw, half + j);
            const cpx U = x[a], V = cmul_rn(x[a | bit], w);
            x[a] = cadd_rn(U, V);
            x[a | bit] = csub_rn(U, V);
        }
    }
    for (uint32_t a = 0; a < rows; a++) z[t * n + (size_t)a * B + col] = x[a].re;
}

template <class L>
static cudaError_t launch_encode_t(const CtxDev &c, const float *sel, size_t T, double2 *cplx, int64_t *m,
                                   cudaStream_t s) {
    const uint32_t n = c.N >> 1;
    const size_t smem = sizeof(cpx) << L::LOGB;
    const unsigned grid = (unsigned)(T * (n >> L::LOGB));
    cudaError_t e;
    if ((n >> L::LOGB) > 1) {
        const size_t total = T << L::LOGB;
        encode_outer_kernel<L::LOGB><<<blocks_for(total, 256), 256, 0, s>>>(c, sel, cplx, total);
        if ((e = FEDHE_LAUNCHED())) return e;
        auto k = encode_block_kernel<L, true>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
        k<<<grid, L::NT, smem, s>>>(c, sel, cplx, m);
    } else {
        auto k = encode_block_kernel<L, false>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
        k<<<grid, L::NT, smem, s>>>(c, sel, cplx, m);
    }
    return FEDHE_LAUNCHED();
}

cudaError_t launch_encode(const CtxDev &c, const float *sel, size_t T, double2 *cplx, int64_t *m,
                          cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    if (c.logN == 13) return launch_encode_t<Lay<12, 4>>(c, sel, T, cplx, m, s);
    return launch_encode_t<Lay<13, 4>>(c, sel, T, cplx, m, s);
}

template <class L>
static cudaError_t launch_decode_t(const CtxDev &c, const int64_t *d, size_t T, double2 *cplx, double *z,
                                   cudaStream_t s) {
    const uint32_t n = c.N >> 1;
    const size_t smem = sizeof(cpx) << L::LOGB;
    const unsigned grid = (unsigned)(T * (n >> L::LOGB));
    cudaError_t e;
    if ((n >> L::LOGB) > 1) {
        auto k = decode_block_kernel<L, true>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
        k<<<grid, L::NT, smem, s>>>(c, d, cplx, z);
        if ((e = FEDHE_LAUNCHED())) return e;
        const size_t total = T << L::LOGB;
        decode_outer_kernel<L::LOGB><<<blocks_for(total, 256), 256, 0, s>>>(c, cplx, z, total);
    } else {
        auto k = decode_block_kernel<L, false>;
        if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
        k<<<grid, L::NT, smem, s>>>(c, d, cplx, z);
    }
    return FEDHE_LAUNCHED();
}

cudaError_t launch_decode(const CtxDev &c, const int64_t *d, size_t T, double2 *cplx, double *z,
                          cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    if (c.logN == 13) return launch_decode_t<Lay<12, 4>>(c, d, T, cplx, z, s);
    return launch_decode_t<Lay<13, 4>>(c, d, T, cplx, z, s);
}

// ===========================================================================
// encryption:  c0 = pk0 u + e0 + m,  c1 = pk1 u + e1   (mod every q_j)
// ===========================================================================

// One (ciphertext, limb) unit of the fused path in the limb's arithmetic.
// u^ pk1^ is parked, in the arithmetic's own form, in the c1 slot it will
// finally occupy while u^ pk0^ stays in shared memory; then two passes over
// one copy of the inverse-transform code: h = 0 gives c0 = pk0 u + e0 + m from
// shared memory, h = 1 reloads the parked product and gives c1 = pk1 u + e1.
template <class M, class L, int V, bool NTT_OUT>
__device__ __forceinline__ void encrypt_unit(const LimbDev &lb, const tw_t *p0, const tw_t *p1, uint64_t *sm,
                                             const int8_t *su, const int8_t *se0, const int64_t *mt,
                                             uint64_t *cbase, size_t cstride) {
    using val = typename M::val;
    constexpr uint32_t B = 1u << L::LOGB;
    const uint32_t tid = threadIdx.x;
    const uint64_t q = lb.q;
    if constexpr (NTT_OUT) {
        // transform-domain output: c0^ = pk0^ u^ + (e0 + m)^, c1^ = pk1^ u^ + e1^.  Three
        // passes over one copy of the forward-transform code: u (both products wait in
        // their final slots), then e0 + m and e1, each added to its product.
        const auto fa = LimbOf<M>::args(lb, true, 0, 0);
        const M &ar = fa.m;
#pragma unroll 1
        for (int h = 0; h < 3; h++) {
            uint64_t *cc = cbase + (h == 2 ? cstride : 0);
            const int8_t *se = se0 + (h == 2 ? B : 0);
            smem_ntt_forward<L, V>(
                sm, tid, fa,
                [&](uint32_t i) {
                    if (h == 0) return ar.small(su[i]);
                    if (h == 2) return ar.small(se[i]);
                    return ar.from_residue(signed_residue(mt[i] + (int64_t)se[i], q, lb.mu));
                },
                [&](uint32_t p, val a, val b) {
                    if (h == 0) {
                        const auto a0 = M::load_key(p0 + p), a1 = M::load_key(p0 + p + 1);
                        const auto b0 = M::load_key(p1 + p), b1 = M::load_key(p1 + p + 1);
                        *reinterpret_cast<u64x2 *>(cbase + p) =
                            u64x2{M::bits(ar.mul_key(a, a0)), M::bits(ar.mul_key(b, a1))};
                        *reinterpret_cast<u64x2 *>(cbase + cstride + p) =
                            u64x2{M::bits(ar.mul_key(a, b0)), M::bits(ar.mul_key(b, b1))};
                    } else {
                        const u64x2 t = *reinterpret_cast<const u64x2 *>(cc + p);
                        *reinterpret_cast<u64x2 *>(cc + p) =
                            u64x2{ar.canon_sum(a, M::from_bits(t.x)), ar.canon_sum(b, M::from_bits(t.y))};
                    }
                });
            __syncthreads();   // last-phase readers are done before the next transform writes
        }
        return;
    }
    {
        uint64_t *c1 = cbase + cstride;
        const auto fa = LimbOf<M>::args(lb, true, 0, 0);
        const M &ar = fa.m;
        smem_ntt_forward<L, V>(
            sm, tid, fa, [&](uint32_t i) { return ar.small(su[i]); },
            [&](uint32_t p, val a, val b) {
                const auto a0 = M::load_key(p1 + p), a1 = M::load_key(p1 + p + 1);
                u64x2 v;
                v.x = M::bits(ar.mul_key(a, a0));
                v.y = M::bits(ar.mul_key(b, a1));
                *reinterpret_cast<u64x2 *>(c1 + p) = v;
                const auto b0 = M::load_key(p0 + p), b1 = M::load_key(p0 + p + 1);
                sm[swz(p)] = M::bits(ar.mul_key(a, b0));
                sm[swz(p + 1)] = M::bits(ar.mul_key(b, b1));
            });
    }
#pragma unroll 1
    for (int h = 0; h < 2; h++) {
        uint64_t *cc = cbase + h * cstride;
        const int8_t *se = se0 + h * B;
        const auto ia = LimbOf<M>::args(lb, false, 0, 0);
        const M &ar = ia.m;
        smem_ntt_inverse<L, V, true>(
            sm, tid, ia, LimbOf<M>::ninv(lb), LimbOf<M>::wn(lb),
            [&](uint32_t p) {
                if (h == 0) return pair_of<val>{M::from_bits(sm[swz(p)]), M::from_bits(sm[swz(p + 1)])};
                const u64x2 t = *reinterpret_cast<const u64x2 *>(cc + p);
                return pair_of<val>{M::from_bits(t.x), M::from_bits(t.y)};
            },
            [&](uint32_t i, val v) {
                // e1 is a small value; e0 + m needs a full reduction
                const uint64_t add = h == 0 ? signed_residue(mt[i] + (int64_t)se[i], q, lb.mu)
                                            : small_residue(se[i], q);
                cc[i] = ar.canon_add(v, add);
            });
        __syncthreads();   // phase-0 readers are done before the next transform writes
    }
}

// Fused path for N <= 2^14 (one block holds a whole limb): a thread block
// draws u, e0, e1 of a ciphertext once into shared memory, then for every
// limb of it transforms u, multiplies by both halves of the public key,
// transforms back and adds the error (and message) terms.  Only the
// ciphertext itself is written to global memory; the second product waits,
// in transform order, in the c1 slot it will finally occupy.
template <class L, int V, bool NTT_OUT>
__global__ void __launch_bounds__(L::NT / V, (L::NT / V) <= 512 ? 2 : 1)
encrypt_fused_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const int64_t *m, uint32_t t0,
                     uint64_t seed, uint32_t client, uint64_t *ct, uint32_t T) {
    extern __shared__ __align__(16) uint64_t sm[];
    constexpr uint32_t B = 1u << L::LOGB, RT = L::NT / V;
    int8_t *su = reinterpret_cast<int8_t *>(sm + B);
    int8_t *se0 = su + B, *se1 = se0 + B;
    const uint32_t tid = threadIdx.x;
    __shared__ GaussTables gt;
    gauss_tables_init(gt, tid);

    // Work units are (ciphertext, limb) pairs in ciphertext-major order, dealt
    // evenly to the blocks of the grid (one block per SM), so that the last
    // wave is as full as the others; a block re-draws u, e0, e1 whenever its
    // range moves on to the next ciphertext.
    const uint64_t units = (uint64_t)T * c.L;
    const uint32_t u_begin = (uint32_t)(units * blockIdx.x / gridDim.x);
    const uint32_t u_end = (uint32_t)(units * (blockIdx.x + 1) / gridDim.x);
    const size_t cstride = (size_t)c.L * B;          // from c0 to c1 of the same limb
    uint32_t sampled = 0xffffffffu;
    for (uint32_t unit = u_begin; unit < u_end; unit++) {
        const uint32_t tl = unit / c.L, j = unit % c.L;   // ciphertext within this call, limb
        if (tl != sampled) {
            sampled = tl;
            const uint32_t t = t0 + tl;                   // stream coordinate
            __syncthreads();                              // tables ready / previous samples no longer read
            for (uint32_t b = tid; b < B / 4; b += RT) {
                u32x4 w = stream_block(seed, b, t, client, TAG_ENC_U);
                char4 v = make_char4((signed char)ternary_from_word(w.x), (signed char)ternary_from_word(w.y),
                                     (signed char)ternary_from_word(w.z), (signed char)ternary_from_word(w.w));
                reinterpret_cast<char4 *>(su)[b] = v;
            }
            for (uint32_t b = tid; b < B / 2; b += RT) {
                u32x4 w0 = stream_block(seed, b, t, client, TAG_ENC_E0);
                u32x4 w1 = stream_block(seed, b, t, client, TAG_ENC_E1);
                char2 a = make_char2((signed char)gauss_from_u64(gt, (uint64_t)w0.x | ((uint64_t)w0.y << 32)),
                                     (signed char)gauss_from_u64(gt, (uint64_t)w0.z | ((uint64_t)w0.w << 32)));
                char2 e = make_char2((signed char)gauss_from_u64(gt, (uint64_t)w1.x | ((uint64_t)w1.y << 32)),
                                     (signed char)gauss_from_u64(gt, (uint64_t)w1.z | ((uint64_t)w1.w << 32)));
                reinterpret_cast<char2 *>(se0)[b] = a;
                reinterpret_cast<char2 *>(se1)[b] = e;
            }
            __syncthreads();
        }
        const LimbDev &lb = c.limb[j];
        uint64_t *cbase = ct + (((size_t)tl * 2 + 0) * c.L + j) * B;
        FEDHE_FOR_ARITH(lb, (encrypt_unit<M_, L, V, NTT_OUT>(lb, k.pk0_hat + (size_t)j * B, k.pk1_hat + (size_t)j * B, sm, su,
                                                    se0, m + (size_t)tl * B, cbase, cstride)));
    }
}

// One (ciphertext, limb) unit of the two-group kernel below (N = 2 * 2^LOGB).
template <class M, class L, int V, bool NTT_OUT>
__device__ __forceinline__ void encrypt_unit2(const LimbDev &lb, const tw_t *pk0, const tw_t *pk1, uint64_t *sm,
                                              const int8_t *su, const int8_t *se0, const int64_t *mt,
                                              uint64_t *cbase, size_t cstride) {
    using val = typename M::val;
    constexpr uint32_t H = 1u << L::LOGB, B = 2 * H;
    constexpr uint32_t GT = L::NT / V, RT = 2 * GT;
    const uint32_t tid = threadIdx.x;
    const uint32_t grp = tid / GT, gt = tid % GT;
    uint64_t *smg = sm + grp * H;                          // this group's half
    const GroupSync gsync = {1 + grp, GT};
    const uint64_t q = lb.q;
    {
        const tw_t *p0 = pk0 + grp * H, *p1 = pk1 + grp * H;
        uint64_t *c1 = cbase + cstride + grp * H;
        const auto fa = LimbOf<M>::args(lb, true, 1, grp);
        const M &ar = fa.m;
        const auto w0 = M::load(fa.tw + 1);                // twiddle of the stage that pairs the halves
        auto src = [&](uint32_t i) {
            // u is ternary: the twiddle product is 0, w or -w
            const int b = su[i + H];
            if constexpr (std::is_same<M, ModF64>::value) {
                return f64_fma(grp == 0 ? (double)b : (double)-b, w0, (double)su[i]);
            } else {
                const uint64_t u = small_residue(su[i], q);
                const uint64_t v = b == 0 ? 0 : (b > 0 ? w0.w : q - w0.w);
                return grp == 0 ? u + v : u - v + ar.q2;
            }
        };
        if constexpr (NTT_OUT) {
            // transform-domain output: three passes over one copy of the forward code: u
            // (both products wait in their final slots), then e0 + m and e1, whose pairing
            // stage costs one product per element, each added to its product
            uint64_t *c0 = cbase + grp * H;
#pragma unroll 1
            for (int h = 0; h < 3; h++) {
                uint64_t *cc = h == 2 ? c1 : c0;
                const int8_t *se = se0 + (h == 2 ? B : 0);
                auto value = [&](uint32_t i) {
                    if (h == 2) return ar.small(se[i]);
                    return ar.from_residue(signed_residue(mt[i] + (int64_t)se[i], q, lb.mu));
                };
                smem_ntt_forward<L, V>(
                    smg, gt, fa,
                    [&](uint32_t i) {
                        if (h == 0) return src(i);
                        const val lo = value(i), hi = value(i + H);
                        if constexpr (std::is_same<M, ModF64>::value) {
                            const double t = ar.mul(hi, w0);
                            return grp == 0 ? f64_add(lo, t) : f64_sub(lo, t);
                        } else {
                            const uint64_t t = shoup_lazy(hi, w0.w, w0.wp, q);
                            return grp == 0 ? lo + t : lo - t + ar.q2;
                        }
                    },
                    [&](uint32_t p, val a, val b) {
                        if (h == 0) {
                            const auto a0 = M::load_key(p0 + p), a1 = M::load_key(p0 + p + 1);
                            const auto b0 = M::load_key(p1 + p), b1 = M::load_key(p1 + p + 1);
                            *reinterpret_cast<u64x2 *>(c0 + p) =
                                u64x2{M::bits(ar.mul_key(a, a0)), M::bits(ar.mul_key(b, a1))};
                            *reinterpret_cast<u64x2 *>(c1 + p) =
                                u64x2{M::bits(ar.mul_key(a, b0)), M::bits(ar.mul_key(b, b1))};
                        } else {
                            const u64x2 t = *reinterpret_cast<const u64x2 *>(cc + p);
                            *reinterpret_cast<u64x2 *>(cc + p) =
                                u64x2{ar.canon_sum(a, M::from_bits(t.x)), ar.canon_sum(b, M::from_bits(t.y))};
                        }
                    },
                    gsync);
                gsync();   // last-phase readers of this half are done before phase 0 writes
            }
            __syncthreads();
            return;
        }
        auto dst = [&](uint32_t p, val a, val b) {
            const auto a0 = M::load_key(p1 + p), a1 = M::load_key(p1 + p + 1);
            u64x2 v;
            v.x = M::bits(ar.mul_key(a, a0));
            v.y = M::bits(ar.mul_key(b, a1));
            *reinterpret_cast<u64x2 *>(c1 + p) = v;      // parked until the second pass
            const auto b0 = M::load_key(p0 + p), b1 = M::load_key(p0 + p + 1);
            smg[swz(p)] = M::bits(ar.mul_key(a, b0));
            smg[swz(p + 1)] = M::bits(ar.mul_key(b, b1));
        };
        smem_ntt_forward<L, V>(smg, gt, fa, src, dst, gsync);
    }
#pragma unroll 1
    for (int h = 0; h < 2; h++) {
        uint64_t *cc = cbase + h * cstride;
        const int8_t *se = se0 + h * B;
        const auto ia = LimbOf<M>::args(lb, false, 1, grp);
        const M &ar = ia.m;
        const auto ninv = LimbOf<M>::ninv(lb), wn = LimbOf<M>::wn(lb);
        auto isrc = [&](uint32_t p) {
            if (h == 0) return pair_of<val>{M::from_bits(smg[swz(p)]), M::from_bits(smg[swz(p + 1)])};
            const u64x2 t = *reinterpret_cast<const u64x2 *>(cc + grp * H + p);
            return pair_of<val>{M::from_bits(t.x), M::from_bits(t.y)};
        };
        auto idst = [&](uint32_t i, val v) { smg[swz(i)] = M::bits(v); };
        smem_ntt_inverse<L, V, false>(smg, gt, ia, ninv, wn, isrc, idst, gsync);
        __syncthreads();
        // last stage across the halves with 1/N folded in, then the error / message terms
        for (uint32_t e = tid; e < H; e += RT) {
            val lo = M::from_bits(sm[swz(e)]), hi = M::from_bits(sm[H + swz(e)]);
            ar.inv_scaled(lo, hi, ninv, wn);
            uint64_t add_lo, add_hi;
            if (h == 0) {
                add_lo = signed_residue(mt[e] + (int64_t)se[e], q, lb.mu);
                add_hi = signed_residue(mt[e + H] + (int64_t)se[e + H], q, lb.mu);
            } else {
                add_lo = small_residue(se[e], q);
                add_hi = small_residue(se[e + H], q);
            }
            cc[e] = ar.canon_add(lo, add_lo);
            cc[e + H] = ar.canon_add(hi, add_hi);
        }
        __syncthreads();
    }
}

// The same for N = 2 * 2^LOGB (N = 2^14 with LOGB = 13): the thread block is
// two groups of threads, each of which transforms one half of the limb as a
// sub-block of the long transform on its own schedule (named barriers), so
// that one group's barrier and memory waits overlap the other's arithmetic.
// The stage that pairs the two halves is done where both are at hand: on the
// way in for the forward transform (u is ternary, so the twiddle product is
// 0, w or q-w, computed by both groups from the shared samples) and by the
// whole block after the two inverse sub-transforms, fused with the epilogue.
template <class L, int V, bool NTT_OUT>
__global__ void __launch_bounds__(2 * L::NT / V, 1)
encrypt_fused2_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const int64_t *m, uint32_t t0,
                      uint64_t seed, uint32_t client, uint64_t *ct, uint32_t T) {
    extern __shared__ __align__(16) uint64_t sm[];
    constexpr uint32_t H = 1u << L::LOGB, B = 2 * H;       // half and whole limb
    constexpr uint32_t GT = L::NT / V, RT = 2 * GT;        // threads per group, per block
    int8_t *su = reinterpret_cast<int8_t *>(sm + B);
    int8_t *se0 = su + B, *se1 = se0 + B;
    const uint32_t tid = threadIdx.x;
    __shared__ GaussTables gt_tab;
    gauss_tables_init(gt_tab, tid);

    const uint64_t units = (uint64_t)T * c.L;
    const uint32_t u_begin = (uint32_t)(units * blockIdx.x / gridDim.x);
    const uint32_t u_end = (uint32_t)(units * (blockIdx.x + 1) / gridDim.x);
    const size_t cstride = (size_t)c.L * B;
    uint32_t sampled = 0xffffffffu;
    for (uint32_t unit = u_begin; unit < u_end; unit++) {
        const uint32_t tl = unit / c.L, j = unit % c.L;
        if (tl != sampled) {
            sampled = tl;
            const uint32_t t = t0 + tl;
            __syncthreads();
            for (uint32_t b = tid; b < B / 4; b += RT) {
                u32x4 w = stream_block(seed, b, t, client, TAG_ENC_U);
                char4 v = make_char4((signed char)ternary_from_word(w.x), (signed char)ternary_from_word(w.y),
                                     (signed char)ternary_from_word(w.z), (signed char)ternary_from_word(w.w));
                reinterpret_cast<char4 *>(su)[b] = v;
            }
            for (uint32_t b = tid; b < B / 2; b += RT) {
                u32x4 w0 = stream_block(seed, b, t, client, TAG_ENC_E0);
                u32x4 w1 = stream_block(seed, b, t, client, TAG_ENC_E1);
                char2 a = make_char2((signed char)gauss_from_u64(gt_tab, (uint64_t)w0.x | ((uint64_t)w0.y << 32)),
                                     (signed char)gauss_from_u64(gt_tab, (uint64_t)w0.z | ((uint64_t)w0.w << 32)));
                char2 e = make_char2((signed char)gauss_from_u64(gt_tab, (uint64_t)w1.x | ((uint64_t)w1.y << 32)),
                                     (signed char)gauss_from_u64(gt_tab, (uint64_t)w1.z | ((uint64_t)w1.w << 32)));
                reinterpret_cast<char2 *>(se0)[b] = a;
                reinterpret_cast<char2 *>(se1)[b] = e;
            }
            __syncthreads();
        }
        const LimbDev &lb = c.limb[j];
        uint64_t *cbase = ct + (((size_t)tl * 2 + 0) * c.L + j) * B;
        FEDHE_FOR_ARITH(lb, (encrypt_unit2<M_, L, V, NTT_OUT>(lb, k.pk0_hat + (size_t)j * B, k.pk1_hat + (size_t)j * B, sm, su,
                                                     se0, m + (size_t)tl * B, cbase, cstride)));
    }
}

// Long rings (N = 2^15, 2^16), where a limb does not fit one SM: the ciphertext
// buffer itself is the only work space and every pass over it does as much as
// it can.  (1) draw u and run the outer forward stages into the c1 slots;
// (2) block transforms of the c1 slots whose last phase writes both products
// u^ pk0^ -> c0 and u^ pk1^ -> c1; (3) inverse block transforms of all slots;
// (4) outer inverse stages fused with the error and message terms.

template <class M, uint32_t A>
__device__ __forceinline__ void enc_outer_sample_limb(const LimbDev &lb, const int (&u)[1u << A][2], uint64_t *p,
                                                      uint32_t B) {
    constexpr uint32_t rows = 1u << A;
    const auto t = LimbOf<M>::args(lb, true, 0, 0);
    typename M::val x[rows], y[rows];
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        x[a] = t.m.small(u[a][0]);
        y[a] = t.m.small(u[a][1]);
    }
    outer_forward<A>(x, y, t);
#pragma unroll
    for (uint32_t a = 0; a < rows; a++)
        *reinterpret_cast<u64x2 *>(p + (size_t)a * B) = u64x2{M::bits(x[a]), M::bits(y[a])};
}

// (1) one thread per pair of neighbouring columns of one ciphertext, all limbs;
// the limbs of ciphertext tl go to dst + tl * ct_stride
template <uint32_t A>
__global__ void __launch_bounds__(256)
enc_outer_sample_kernel(const __grid_constant__ CtxDev c, uint32_t t0, uint64_t seed, uint32_t client,
                        uint64_t *dst, size_t ct_stride, size_t total) {
    size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t B = 1u << c.LOGB, half = B >> 1;
    constexpr uint32_t rows = 1u << A;
    const uint32_t col = (uint32_t)(g % half) * 2;
    const size_t tl = g / half;
    int u[rows][2];
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        const uint32_t i = a * B + col;               // even: both columns share a Philox block
        const u32x4 w = stream_block(seed, i >> 2, t0 + (uint32_t)tl, client, TAG_ENC_U);
        u[a][0] = ternary_from_word((i & 2) ? w.z : w.x);
        u[a][1] = ternary_from_word((i & 2) ? w.w : w.y);
    }
#pragma unroll 1
    for (uint32_t j = 0; j < c.L; j++) {
        const LimbDev &lb = c.limb[j];
        uint64_t *p = dst + tl * ct_stride + (size_t)j * c.N + col;   // limb j of ciphertext tl
        FEDHE_FOR_ARITH(lb, (enc_outer_sample_limb<M_, A>(lb, u, p, B)));
    }
}

// (2) one thread block per (ciphertext, limb, block): forward block transform of
// the c1 slot, products with both halves of the public key on the way out
template <class M, class L, int V, bool ACC>
__device__ __forceinline__ void enc_block_forward(const CtxDev &c, const LimbDev &lb, uint64_t *sm, uint32_t blk,
                                                  const tw_t *p0, const tw_t *p1, const uint64_t *u,
                                                  uint64_t *c0, uint64_t *c1) {
    using val = typename M::val;
    const auto a = LimbOf<M>::args(lb, true, c.A, blk);
    const M &ar = a.m;
    smem_ntt_forward<L, V>(
        sm, threadIdx.x, a, [&](uint32_t i) { return M::from_bits(u[i]); },
        [&](uint32_t p, val x, val y) {
            const auto a0 = M::load_key(p0 + p), a1 = M::load_key(p0 + p + 1);
            const auto b0 = M::load_key(p1 + p), b1 = M::load_key(p1 + p + 1);
            u64x2 v0, v1;
            if constexpr (ACC) {       // the slots hold canonical residues to add to
                v0 = *reinterpret_cast<const u64x2 *>(c0 + p);
                v1 = *reinterpret_cast<const u64x2 *>(c1 + p);
                v0.x = ar.canon_add(ar.mul_key(x, a0), v0.x);
                v0.y = ar.canon_add(ar.mul_key(y, a1), v0.y);
                v1.x = ar.canon_add(ar.mul_key(x, b0), v1.x);
                v1.y = ar.canon_add(ar.mul_key(y, b1), v1.y);
            } else {
                v0.x = ar.to_residue(ar.mul_key(x, a0));
                v0.y = ar.to_residue(ar.mul_key(y, a1));
                v1.x = ar.to_residue(ar.mul_key(x, b0));
                v1.y = ar.to_residue(ar.mul_key(y, b1));
            }
            *reinterpret_cast<u64x2 *>(c0 + p) = v0;
            *reinterpret_cast<u64x2 *>(c1 + p) = v1;
        });
}

// ACC = false: u comes from the c1 slot and the products replace both slots;
// ACC = true: u comes from `ubuf` ([T][L][N]) and the products are added to the slots
template <class L, int V, bool ACC>
__global__ void __launch_bounds__(L::NT / V, (L::NT / V) <= 512 ? 2 : 1)
enc_block_forward_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const uint64_t *ubuf, uint64_t *ct) {
    extern __shared__ __align__(16) uint64_t sm[];
    uint32_t b = blockIdx.x;
    const uint32_t blk = b & ((1u << c.A) - 1u);
    b >>= c.A;
    const uint32_t j = b % c.L;
    const size_t tl = b / c.L;
    const LimbDev &lb = c.limb[j];
    const size_t off = ((size_t)blk << L::LOGB);
    uint64_t *c0 = ct + ((tl * 2 + 0) * c.L + j) * c.N + off;
    uint64_t *c1 = ct + ((tl * 2 + 1) * c.L + j) * c.N + off;
    const uint64_t *u = ACC ? ubuf + (tl * c.L + j) * c.N + off : c1;
    const tw_t *p0 = k.pk0_hat + (size_t)j * c.N + off, *p1 = k.pk1_hat + (size_t)j * c.N + off;
    FEDHE_FOR_ARITH(lb, (enc_block_forward<M_, L, V, ACC>(c, lb, sm, blk, p0, p1, u, c0, c1)));
}

// long rings, transform-domain format: residues of e0 + m into the c0 slots and
// of e1 into the c1 slots; one thread per pair of neighbouring coefficients
__global__ void __launch_bounds__(256)
enc_fill_errors_kernel(const __grid_constant__ CtxDev c, const int64_t *m, uint32_t t0, uint64_t seed,
                       uint32_t client, uint64_t *ct, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t pairs = c.N >> 1;
    const uint32_t b = (uint32_t)(g % pairs), i = 2 * b;   // one Philox block per pair
    const size_t tl = g / pairs;
    const uint32_t t = t0 + (uint32_t)tl;
    const u32x4 w0 = stream_block(seed, b, t, client, TAG_ENC_E0);
    const u32x4 w1 = stream_block(seed, b, t, client, TAG_ENC_E1);
    const longlong2 mm = *reinterpret_cast<const longlong2 *>(m + tl * c.N + i);
    const int64_t ax = mm.x + gauss_from_u64((uint64_t)w0.x | ((uint64_t)w0.y << 32));
    const int64_t ay = mm.y + gauss_from_u64((uint64_t)w0.z | ((uint64_t)w0.w << 32));
    const int ex = gauss_from_u64((uint64_t)w1.x | ((uint64_t)w1.y << 32));
    const int ey = gauss_from_u64((uint64_t)w1.z | ((uint64_t)w1.w << 32));
    for (uint32_t j = 0; j < c.L; j++) {
        const LimbDev &lb = c.limb[j];
        const uint64_t q = lb.q;
        *reinterpret_cast<u64x2 *>(ct + ((tl * 2 + 0) * c.L + j) * c.N + i) =
            u64x2{signed_residue(ax, q, lb.mu), signed_residue(ay, q, lb.mu)};
        *reinterpret_cast<u64x2 *>(ct + ((tl * 2 + 1) * c.L + j) * c.N + i) =
            u64x2{small_residue(ex, q), small_residue(ey, q)};
    }
}

template <class M, uint32_t A>
__device__ __forceinline__ void enc_outer_inverse_add_limb(const LimbDev &lb, uint64_t *p, uint32_t B, bool first,
                                                           const int64_t (&me0)[1u << A][2],
                                                           const int (&e1)[1u << A][2]) {
    constexpr uint32_t rows = 1u << A;
    const uint64_t q = lb.q;
    const auto t = LimbOf<M>::args(lb, false, 0, 0);
    typename M::val x[rows], y[rows];
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        const u64x2 v = *reinterpret_cast<const u64x2 *>(p + (size_t)a * B);
        x[a] = M::from_bits(v.x);
        y[a] = M::from_bits(v.y);
    }
    outer_inverse<A>(x, y, t, LimbOf<M>::ninv(lb), LimbOf<M>::wn(lb));
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        u64x2 o;
        if (first) {
            o.x = t.m.canon_add(x[a], signed_residue(me0[a][0], q, lb.mu));
            o.y = t.m.canon_add(y[a], signed_residue(me0[a][1], q, lb.mu));
        } else {
            o.x = t.m.canon_add(x[a], small_residue(e1[a][0], q));
            o.y = t.m.canon_add(y[a], small_residue(e1[a][1], q));
        }
        *reinterpret_cast<u64x2 *>(p + (size_t)a * B) = o;
    }
}

// (4) one thread per pair of neighbouring columns of one ciphertext: draws the
// errors once, then for every limb finishes both components
template <uint32_t A>
__global__ void __launch_bounds__(256, 2)
enc_outer_inverse_add_kernel(const __grid_constant__ CtxDev c, const int64_t *m, uint32_t t0, uint64_t seed,
                             uint32_t client, uint64_t *ct, size_t total) {
    size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t B = 1u << c.LOGB, half = B >> 1;
    constexpr uint32_t rows = 1u << A;
    const uint32_t col = (uint32_t)(g % half) * 2;
    const size_t tl = g / half;
    const uint32_t t = t0 + (uint32_t)tl;
    int e1[rows][2];
    int64_t me0[rows][2];                              // m + e0
#pragma unroll
    for (uint32_t a = 0; a < rows; a++) {
        const uint32_t i = a * B + col;               // one Philox block per pair of coefficients
        const u32x4 w0 = stream_block(seed, i >> 1, t, client, TAG_ENC_E0);
        const u32x4 w1 = stream_block(seed, i >> 1, t, client, TAG_ENC_E1);
        const longlong2 mm = *reinterpret_cast<const longlong2 *>(m + tl * c.N + i);
        me0[a][0] = mm.x + gauss_from_u64((uint64_t)w0.x | ((uint64_t)w0.y << 32));
        me0[a][1] = mm.y + gauss_from_u64((uint64_t)w0.z | ((uint64_t)w0.w << 32));
        e1[a][0] = gauss_from_u64((uint64_t)w1.x | ((uint64_t)w1.y << 32));
        e1[a][1] = gauss_from_u64((uint64_t)w1.z | ((uint64_t)w1.w << 32));
    }
#pragma unroll 1
    for (uint32_t j = 0; j < c.L; j++) {
        const LimbDev &lb = c.limb[j];
#pragma unroll 1
        for (uint32_t comp = 0; comp < 2; comp++) {
            uint64_t *p = ct + ((tl * 2 + comp) * c.L + j) * c.N + col;
            FEDHE_FOR_ARITH(lb, (enc_outer_inverse_add_limb<M_, A>(lb, p, B, comp == 0, me0, e1)));
        }
    }
}

template <class L, int V, bool TWO_GROUPS, bool NTT_OUT>
static cudaError_t launch_encrypt_fused(const CtxDev &c, const KeysDev &k, const int64_t *m, uint32_t t0,
                                        size_t T, uint64_t seed, uint32_t client, uint64_t *ct,
                                        cudaStream_t s) {
    const size_t smem = ((sizeof(uint64_t) << L::LOGB) + (3u << L::LOGB)) * (TWO_GROUPS ? 2 : 1);
    auto kern = TWO_GROUPS ? encrypt_fused2_kernel<L, V, NTT_OUT> : encrypt_fused_kernel<L, V, NTT_OUT>;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    // one block per SM (the kernel's shared memory allows no more), fewer if there is less work
    int dev = 0, n_sm = 0;
    if ((e = cudaGetDevice(&dev)) || (e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev))) return e;
    const size_t per_sm = (size_t)(227 * 1024) / smem;               // blocks that fit one SM
    size_t grid = (size_t)n_sm * (per_sm ? per_sm : 1);
    if (grid > T * c.L) grid = T * c.L;
    kern<<<(unsigned)grid, (TWO_GROUPS ? 2 : 1) * L::NT / V, smem, s>>>(c, k, m, t0, seed, client, ct, (uint32_t)T);
    return FEDHE_LAUNCHED();
}

// launches the block forward kernel of the long-ring paths
template <bool ACC>
static cudaError_t launch_enc_block_forward(const CtxDev &c, const KeysDev &k, const uint64_t *ubuf, size_t T,
                                            uint64_t *ct, cudaStream_t s) {
    using L = Lay<13, 3>;                                 // long rings are cut into 2^13 blocks
    constexpr int V = 2;
    const size_t smem = sizeof(uint64_t) << L::LOGB;
    auto kern = enc_block_forward_kernel<L, V, ACC>;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    kern<<<(unsigned)((T * c.L) << c.A), L::NT / V, smem, s>>>(c, k, ubuf, ct);
    return FEDHE_LAUNCHED();
}

cudaError_t launch_encrypt(const CtxDev &c, const KeysDev &k, const int64_t *m, uint32_t t0, size_t T,
                           uint64_t seed, uint32_t client, uint64_t *ct, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    if (c.A == 0) {
        if (c.LOGB == 13)
            return launch_encrypt_fused<Lay<13, 3>, 2, false, false>(c, k, m, t0, T, seed, client, ct, s);
        return launch_encrypt_fused<Lay<13, 3>, 2, true, false>(c, k, m, t0, T, seed, client, ct, s);
    }
    cudaError_t e;
    const size_t cols = T * ((size_t)1 << (c.LOGB - 1));      // pairs of columns
    const size_t LN = (size_t)c.L * c.N;
    FEDHE_FOR_A(c, (enc_outer_sample_kernel<A_><<<blocks_for(cols, 256), 256, 0, s>>>(c, t0, seed, client, ct + LN,
                                                                                     2 * LN, cols)));
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_enc_block_forward<false>(c, k, nullptr, T, ct, s))) return e;
    if ((e = launch_ntt_inner(c, false, ct, 2 * T, LN, 0, c.L, s))) return e;
    FEDHE_FOR_A(c, (enc_outer_inverse_add_kernel<A_><<<blocks_for(cols, 256), 256, 0, s>>>(c, m, t0, seed, client, ct,
                                                                                          cols)));
    return FEDHE_LAUNCHED();
}

// Transform-domain wire format: the same ciphertext with every limb polynomial
// stored as its negacyclic transform.  N <= 2^14: the fused kernels with three
// forward transforms per limb.  Longer rings: the error terms go into the
// ciphertext slots and are transformed there; u is transformed in the work
// buffer `ubuf` ([T][L][N]) and its key products are added on the way out.
cudaError_t launch_encrypt_ntt(const CtxDev &c, const KeysDev &k, const int64_t *m, uint32_t t0, size_t T,
                               uint64_t seed, uint32_t client, uint64_t *ubuf, uint64_t *ct, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    if (c.A == 0) {
        if (c.LOGB == 13)
            return launch_encrypt_fused<Lay<13, 3>, 2, false, true>(c, k, m, t0, T, seed, client, ct, s);
        return launch_encrypt_fused<Lay<13, 3>, 2, true, true>(c, k, m, t0, T, seed, client, ct, s);
    }
    cudaError_t e;
    const size_t LN = (size_t)c.L * c.N;
    const size_t pairs = T * (size_t)(c.N >> 1);
    enc_fill_errors_kernel<<<blocks_for(pairs, 256), 256, 0, s>>>(c, m, t0, seed, client, ct, pairs);
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_ntt(c, true, ct, 2 * T, LN, 0, c.L, s))) return e;
    const size_t cols = T * ((size_t)1 << (c.LOGB - 1));
    FEDHE_FOR_A(c, (enc_outer_sample_kernel<A_><<<blocks_for(cols, 256), 256, 0, s>>>(c, t0, seed, client, ubuf, LN,
                                                                                     cols)));
    if ((e = FEDHE_LAUNCHED())) return e;
    return launch_enc_block_forward<true>(c, k, ubuf, T, ct, s);
}

// ===========================================================================
// server: weighted ciphertext sum over all clients fused with the rescale
// ===========================================================================

// One thread per pair of neighbouring coefficients of one (ciphertext,
// component).  The last limb is accumulated first: its centred value is the
// rounding term of every other limb.  The pass is bound by HBM reads
// (32 L C bytes per parameter), so the client pointers and weights are
// staged in shared memory once per block and the loads of four clients are
// issued before their multiply-adds to keep enough bytes in flight.
__device__ __forceinline__ void weighted_sum_pair(const uint64_t *const *sp, const tw_t *sw, int C, uint32_t L,
                                                  uint32_t j, size_t off, uint64_t q, uint64_t &ax,
                                                  uint64_t &ay) {
    const uint64_t q2 = 2 * q;
    ax = 0;
    ay = 0;
    int cl = 0;
    for (; cl + 4 <= C; cl += 4) {
        ulonglong2 v[4];
#pragma unroll
        for (int u = 0; u < 4; u++) v[u] = __ldg(reinterpret_cast<const ulonglong2 *>(sp[cl + u] + off));
#pragma unroll
        for (int u = 0; u < 4; u++) {
            const tw_t w = sw[(cl + u) * L + j];
            ax = csub(ax + shoup_lazy(v[u].x, w.w, w.wp, q), q2);
            ay = csub(ay + shoup_lazy(v[u].y, w.w, w.wp, q), q2);
        }
    }
    for (; cl < C; cl++) {
        const ulonglong2 v = __ldg(reinterpret_cast<const ulonglong2 *>(sp[cl] + off));
        const tw_t w = sw[cl * L + j];
        ax = csub(ax + shoup_lazy(v.x, w.w, w.wp, q), q2);
        ay = csub(ay + shoup_lazy(v.y, w.w, w.wp, q), q2);
    }
    ax = csub(ax, q);
    ay = csub(ay, q);
}

__global__ void __launch_bounds__(256)
aggregate_rescale_kernel(const __grid_constant__ CtxDev c, const uint64_t *const *ptrs, const tw_t *wtab,
                         int C, uint64_t *out, size_t total) {
    extern __shared__ __align__(16) unsigned char agg_sm[];
    const uint32_t L = c.L;
    tw_t *sw = reinterpret_cast<tw_t *>(agg_sm);                                    // [C][L]
    const uint64_t **sp = reinterpret_cast<const uint64_t **>(sw + (size_t)C * L);  // [C]
    for (int e = threadIdx.x; e < C * (int)L; e += blockDim.x) sw[e] = wtab[e];
    for (int e = threadIdx.x; e < C; e += blockDim.x) sp[e] = ptrs[e];
    __syncthreads();
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t pairs = c.N >> 1;
    const uint32_t i = (uint32_t)(g % pairs) * 2;
    const size_t tc = g / pairs;                 // t * 2 + component
    const uint64_t ql = c.limb[L - 1].q;
    uint64_t rx, ry;
    weighted_sum_pair(sp, sw, C, L, L - 1, (tc * L + (L - 1)) * c.N + i, ql, rx, ry);
    const bool negx = rx > ql / 2, negy = ry > ql / 2;
    const uint64_t mx = negx ? ql - rx : rx, my = negy ? ql - ry : ry;   // |centred remainder|
    for (uint32_t j = 0; j + 1 < L; j++) {
        const LimbDev &lb = c.limb[j];
        const uint64_t q = lb.q;
        uint64_t ax, ay;
        weighted_sum_pair(sp, sw, C, L, j, (tc * L + j) * c.N + i, q, ax, ay);
        const uint64_t sx = barrett64(mx, q, lb.mu), sy = barrett64(my, q, lb.mu);
        // acc - r: subtracting a negative remainder adds its magnitude
        const uint64_t dx = negx ? addmod(ax, sx, q) : submod(ax, sx, q);
        const uint64_t dy = negy ? addmod(ay, sy, q) : submod(ay, sy, q);
        ulonglong2 o;
        o.x = shoup(dx, lb.qlinv.w, lb.qlinv.wp, q);
        o.y = shoup(dy, lb.qlinv.w, lb.qlinv.wp, q);
        *reinterpret_cast<ulonglong2 *>(out + (tc * (L - 1) + j) * c.N + i) = o;
    }
}

cudaError_t launch_aggregate(const CtxDev &c, const uint64_t *const *ptrs, const tw_t *wtab, int C,
                             size_t T, uint64_t *out, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    const size_t total = T * 2 * (c.N >> 1);
    const size_t smem = (size_t)C * c.L * sizeof(tw_t) + (size_t)C * sizeof(void *);
    cudaError_t e;
    if (smem > 48 * 1024 &&
        (e = cudaFuncSetAttribute(aggregate_rescale_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)))
        return e;
    aggregate_rescale_kernel<<<blocks_for(total, 256), 256, smem, s>>>(c, ptrs, wtab, C, out, total);
    return FEDHE_LAUNCHED();
}

// ---------------------------------------------------------------------------
// The same on transform-domain ciphertexts.  The weighted sum is pointwise in
// either domain; the rounding term of the rescale is not: the last limb is
// brought back to coefficients, centred, and its residues are transformed
// for every other limb (2L limb transforms per ciphertext index that the
// coefficient format does not need).
// ---------------------------------------------------------------------------

// acc_j = sum_i W_i ct_i for all limbs: limbs below the last go to `out`
// ([T][2][L-1][N]), the last limb to `last` ([T][2][N])
__global__ void __launch_bounds__(256)
aggregate_sum_kernel(const __grid_constant__ CtxDev c, const uint64_t *const *ptrs, const tw_t *wtab, int C,
                     uint64_t *out, uint64_t *last, size_t total) {
    extern __shared__ __align__(16) unsigned char agg_sm[];
    const uint32_t L = c.L;
    tw_t *sw = reinterpret_cast<tw_t *>(agg_sm);
    const uint64_t **sp = reinterpret_cast<const uint64_t **>(sw + (size_t)C * L);
    for (int e = threadIdx.x; e < C * (int)L; e += blockDim.x) sw[e] = wtab[e];
    for (int e = threadIdx.x; e < C; e += blockDim.x) sp[e] = ptrs[e];
    __syncthreads();
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t pairs = c.N >> 1;
    const uint32_t i = (uint32_t)(g % pairs) * 2;
    const size_t tc = g / pairs;
    for (uint32_t j = 0; j < L; j++) {
        u64x2 o;
        weighted_sum_pair(sp, sw, C, L, j, (tc * L + j) * c.N + i, c.limb[j].q, o.x, o.y);
        uint64_t *dst = j + 1 < L ? out + (tc * (L - 1) + j) * c.N + i : last + tc * c.N + i;
        *reinterpret_cast<u64x2 *>(dst) = o;
    }
}

// residues modulo every remaining prime of the centred last-limb coefficients
__global__ void __launch_bounds__(256)
aggregate_spread_kernel(const __grid_constant__ CtxDev c, const uint64_t *last, uint64_t *rem, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t i = (uint32_t)(g % c.N);
    const size_t tc = g / c.N;
    const uint32_t L = c.L;
    const uint64_t ql = c.limb[L - 1].q, r = last[g];
    const bool neg = r > ql / 2;
    const uint64_t mag = neg ? ql - r : r;
    for (uint32_t j = 0; j + 1 < L; j++) {
        const LimbDev &lb = c.limb[j];
        const uint64_t v = barrett64(mag, lb.q, lb.mu);
        rem[(tc * (L - 1) + j) * c.N + i] = (neg && v) ? lb.q - v : v;
    }
}

// out_j = (acc_j - rem_j) / q_{L-1}
__global__ void __launch_bounds__(256)
aggregate_finish_kernel(const __grid_constant__ CtxDev c, const uint64_t *rem, uint64_t *out, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t j = (uint32_t)((g / c.N) % (c.L - 1));
    const LimbDev &lb = c.limb[j];
    out[g] = shoup(submod(out[g], rem[g], lb.q), lb.qlinv.w, lb.qlinv.wp, lb.q);
}

// scratch: [T][2][N] + [T][2][L-1][N] words
cudaError_t launch_aggregate_ntt(const CtxDev &c, const uint64_t *const *ptrs, const tw_t *wtab, int C,
                                 size_t T, uint64_t *scratch, uint64_t *out, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    uint64_t *last = scratch, *rem = scratch + 2 * T * c.N;
    const size_t smem = (size_t)C * c.L * sizeof(tw_t) + (size_t)C * sizeof(void *);
    cudaError_t e;
    if (smem > 48 * 1024 &&
        (e = cudaFuncSetAttribute(aggregate_sum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)))
        return e;
    const size_t pairs = T * 2 * (c.N >> 1);
    aggregate_sum_kernel<<<blocks_for(pairs, 256), 256, smem, s>>>(c, ptrs, wtab, C, out, last, pairs);
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_ntt(c, false, last, 2 * T, c.N, c.L - 1, 1, s))) return e;
    if (c.L > 1) {
        const size_t n_last = 2 * T * c.N, n_out = n_last * (c.L - 1);
        aggregate_spread_kernel<<<blocks_for(n_last, 256), 256, 0, s>>>(c, last, rem, n_last);
        if ((e = FEDHE_LAUNCHED())) return e;
        if ((e = launch_ntt(c, true, rem, 2 * T, (size_t)(c.L - 1) * c.N, 0, c.L - 1, s))) return e;
        aggregate_finish_kernel<<<blocks_for(n_out, 256), 256, 0, s>>>(c, rem, out, n_out);
        if ((e = FEDHE_LAUNCHED())) return e;
    }
    return cudaSuccess;
}

// plaintext remainder: out = sum_i alpha_i * (double) rest_i, client order,
// separate multiply and add
__global__ void __launch_bounds__(256)
plain_aggregate_kernel(const float *const *ptrs, const double *alpha, int C, size_t len, double *out) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= len) return;
    double a = 0.0;
    for (int cl = 0; cl < C; cl++) a = __dadd_rn(a, __dmul_rn(alpha[cl], (double)__ldg(ptrs[cl] + g)));
    out[g] = a;
}

cudaError_t launch_plain_aggregate(const float *const *ptrs, const double *alpha, int C, size_t len,
                                   double *out, cudaStream_t s) {
    if (len == 0) return cudaSuccess;
    plain_aggregate_kernel<<<blocks_for(len, 256), 256, 0, s>>>(ptrs, alpha, C, len, out);
    return FEDHE_LAUNCHED();
}

// ===========================================================================
// decryption: d = c0 + c1 s on limb 0, centred
// ===========================================================================

__global__ void __launch_bounds__(256)
dec_gather_kernel(const __grid_constant__ CtxDev c, const uint64_t *ct, uint32_t level, uint64_t *scratch,
                  size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t i = (uint32_t)(g % c.N);
    const size_t t = g / c.N;
    scratch[g] = ct[((t * 2 + 1) * level + 0) * c.N + i];
}

__global__ void __launch_bounds__(256)
dec_pointwise_kernel(const __grid_constant__ CtxDev c, const KeysDev k, uint64_t *scratch, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t i = (uint32_t)(g % c.N);
    const tw_t s = load_tw(k.s_hat + i);
    scratch[g] = shoup_lazy(scratch[g], s.w, s.wp, c.limb[0].q);
}

// transform-domain ciphertext: scratch = c0^ + c1^ s^ on limb 0
__global__ void __launch_bounds__(256)
dec_pointwise_ntt_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const uint64_t *ct, uint32_t level,
                         uint64_t *scratch, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t i = (uint32_t)(g % c.N);
    const size_t t = g / c.N;
    const uint64_t q = c.limb[0].q;
    const tw_t s = load_tw(k.s_hat + i);
    const uint64_t p = shoup(ct[((t * 2 + 1) * level + 0) * c.N + i], s.w, s.wp, q);
    scratch[g] = addmod(p, ct[((t * 2 + 0) * level + 0) * c.N + i], q);
}

// centred d = scratch (+ c0 when the ciphertext is in the coefficient domain: ct != null)
__global__ void __launch_bounds__(256)
dec_finish_kernel(const __grid_constant__ CtxDev c, const uint64_t *ct, uint32_t level, uint64_t *scratch,
                  size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t i = (uint32_t)(g % c.N);
    const size_t t = g / c.N;
    const uint64_t q = c.limb[0].q;
    const uint64_t r = ct ? addmod(scratch[g], ct[((t * 2 + 0) * level + 0) * c.N + i], q) : scratch[g];
    const int64_t d = r > q / 2 ? -(int64_t)(q - r) : (int64_t)r;
    reinterpret_cast<int64_t *>(scratch)[g] = d;
}

cudaError_t launch_decrypt(const CtxDev &c, const KeysDev &k, const uint64_t *ct, uint32_t level,
                           size_t T, uint64_t *scratch, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    cudaError_t e;
    const size_t total = T * c.N;
    dec_gather_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, ct, level, scratch, total);
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_ntt(c, true, scratch, T, c.N, 0, 1, s))) return e;
    dec_pointwise_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, k, scratch, total);
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_ntt(c, false, scratch, T, c.N, 0, 1, s))) return e;
    dec_finish_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, ct, level, scratch, total);
    return FEDHE_LAUNCHED();
}

cudaError_t launch_decrypt_ntt(const CtxDev &c, const KeysDev &k, const uint64_t *ct, uint32_t level,
                               size_t T, uint64_t *scratch, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    cudaError_t e;
    const size_t total = T * c.N;
    dec_pointwise_ntt_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, k, ct, level, scratch, total);
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_ntt(c, false, scratch, T, c.N, 0, 1, s))) return e;
    dec_finish_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, nullptr, level, scratch, total);
    return FEDHE_LAUNCHED();
}

// Fused path for N <= 2^14: one thread block per ciphertext transforms c1
// (limb 0), multiplies by the secret key, transforms back, adds c0, centres,
// and runs the slot transform on the result without leaving the SM; only the
// two limb-0 polynomials are read and the n decoded values written.
// L: layout of the length-N integer transform (played by L::NT / V threads),
// LF: layout of the length-n complex transform with LF::NT == L::NT / V.
// NTT_IN: the ciphertext is in the transform domain, so the forward transform
// falls away and c0^ + c1^ s^ feeds the inverse transform directly.
template <class L, int V, class LF, bool NTT_IN>
__global__ void __launch_bounds__(L::NT / V, (L::NT / V) <= 512 ? 2 : 1)
decrypt_fused_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const uint64_t *ct, uint32_t level,
                     double *z) {
    static_assert(LF::NT == L::NT / V && LF::LOGB + 1 == L::LOGB, "thread counts and sizes must match");
    extern __shared__ __align__(16) uint64_t sm[];
    constexpr uint32_t B = 1u << L::LOGB, n = B >> 1;
    const uint32_t tid = threadIdx.x;
    const size_t t = blockIdx.x;
    const LimbDev &lb = c.limb[0];
    const uint64_t q = lb.q, q2 = 2 * q;
    const uint64_t *c0 = ct + ((t * 2 + 0) * level) * B, *c1 = ct + ((t * 2 + 1) * level) * B;
    if constexpr (!NTT_IN) {
        const NttArgs fa = LimbOf<ModInt>::args(lb, true, 0, 0);   // limb 0 carries the message
        smem_ntt_forward<L, V>(
            sm, tid, fa, [&](uint32_t i) { return c1[i]; },
            [&](uint32_t p, uint64_t a, uint64_t b) {
                const tw_t s0 = load_tw(k.s_hat + p), s1 = load_tw(k.s_hat + p + 1);
                sm[swz(p)] = shoup_lazy(a, s0.w, s0.wp, q);
                sm[swz(p + 1)] = shoup_lazy(b, s1.w, s1.wp, q);
            });
    }
    int64_t *d = reinterpret_cast<int64_t *>(sm);
    {
        const NttArgs ia = LimbOf<ModInt>::args(lb, false, 0, 0);
        smem_ntt_inverse<L, V, true>(
            sm, tid, ia, lb.ninv, lb.wn,
            [&](uint32_t p) {
                if constexpr (NTT_IN) {
                    const u64x2 a = *reinterpret_cast<const u64x2 *>(c0 + p), b = *reinterpret_cast<const u64x2 *>(c1 + p);
                    const tw_t s0 = load_tw(k.s_hat + p), s1 = load_tw(k.s_hat + p + 1);
                    return u64x2{csub(a.x + shoup_lazy(b.x, s0.w, s0.wp, q), q2),
                                 csub(a.y + shoup_lazy(b.y, s1.w, s1.wp, q), q2)};
                } else {
                    return u64x2{sm[swz(p)], sm[swz(p + 1)]};
                }
            },
            [&](uint32_t i, uint64_t v) {
                const uint64_t r = NTT_IN ? csub(v, q) : addmod(csub(v, q), c0[i], q);
                d[swz(i)] = r > q / 2 ? -(int64_t)(q - r) : (int64_t)r;
            });
    }
    __syncthreads();
    // slot transform: bit-reversed load of (d_k + i d_{k+n}) / Delta from shared memory
    const double inv_delta = __longlong_as_double((long long)(1023 - c.log2_delta) << 52);
    cpx x[LF::E];
#pragma unroll
    for (int r = 0; r < LF::E; r++) {
        const uint32_t kk = bitrev(LF::template idx<LF::NPH - 1>(tid, r), LF::LOGB);
        x[r] = cpx{(double)d[swz(kk)] * inv_delta, (double)d[swz(kk + n)] * inv_delta};
    }
    __syncthreads();                      // all inputs are in registers: the buffer becomes the exchange buffer
    block_dit<LF>(x, reinterpret_cast<cpx *>(sm), tid, c.ftw);
#pragma unroll
    for (int r = 0; r < LF::E; r++) z[t * n + LF::template idx<0>(tid, r)] = x[r].re;
}

template <class L, int V, class LF, bool NTT_IN>
static cudaError_t launch_decrypt_fused_t(const CtxDev &c, const KeysDev &k, const uint64_t *ct, uint32_t level,
                                          size_t T, double *z, cudaStream_t s) {
    const size_t smem = sizeof(uint64_t) << L::LOGB;
    auto kern = decrypt_fused_kernel<L, V, LF, NTT_IN>;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    kern<<<(unsigned)T, L::NT / V, smem, s>>>(c, k, ct, level, z);
    return FEDHE_LAUNCHED();
}

cudaError_t launch_decrypt_fused(const CtxDev &c, const KeysDev &k, const uint64_t *ct, uint32_t level,
                                 size_t T, bool ntt_in, double *z, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    if (c.logN == 13) {
        if (ntt_in) return launch_decrypt_fused_t<Lay<13, 3>, 2, Lay<12, 3>, true>(c, k, ct, level, T, z, s);
        return launch_decrypt_fused_t<Lay<13, 3>, 2, Lay<12, 3>, false>(c, k, ct, level, T, z, s);
    }
    if (ntt_in) return launch_decrypt_fused_t<Lay<14, 3>, 2, Lay<13, 3>, true>(c, k, ct, level, T, z, s);
    return launch_decrypt_fused_t<Lay<14, 3>, 2, Lay<13, 3>, false>(c, k, ct, level, T, z, s);
}

// ===========================================================================
// two-party threshold decryption: dealer split of the secret, partial
// decryption with smudging noise, merge
// ===========================================================================

// tmp[0] = uniform share, tmp[1] = s - share, as residues [L][N]
__global__ void __launch_bounds__(256)
threshold_split_kernel(const __grid_constant__ CtxDev c, const int8_t *s8, uint64_t seed, uint64_t *tmp) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= c.N) return;
    const int sv = s8[i];
    const size_t LN = (size_t)c.L * c.N;
    for (uint32_t j = 0; j < c.L; j++) {
        const uint64_t q = c.limb[j].q;
        u32x4 wa = stream_block(seed, i, 0, 0, TAG_SHARE | (j << 8));
        const uint64_t lo = (uint64_t)wa.x | ((uint64_t)wa.y << 32), hi = (uint64_t)wa.z | ((uint64_t)wa.w << 32);
        const uint64_t a = mod_u128(hi, lo, q);
        tmp[(size_t)j * c.N + i] = a;
        tmp[LN + (size_t)j * c.N + i] = submod(small_residue(sv, q), a, q);
    }
}

__global__ void __launch_bounds__(256)
share_tables_kernel(const __grid_constant__ CtxDev c, const uint64_t *share_hat, tw_t *s_hat) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= (size_t)c.L * c.N) return;
    const uint64_t v = share_hat[g];
    s_hat[g] = tw_t{v, shoup_companion(v, c.limb[g / c.N].q)};
}

// part += E (mod q_0), E uniform in [-2^bits, 2^bits): one thread per pair of coefficients
__global__ void __launch_bounds__(256)
partial_finish_kernel(const __grid_constant__ CtxDev c, uint32_t party, uint64_t seed, uint32_t bits,
                      uint64_t *part, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t pairs = c.N >> 1;
    const uint32_t b = (uint32_t)(g % pairs);
    const size_t t = g / pairs;
    const uint64_t q = c.limb[0].q, mu = c.limb[0].mu;
    u32x4 w = stream_block(seed, b, (uint32_t)t, party, TAG_SMUDGE);
    const uint64_t r0 = (uint64_t)w.x | ((uint64_t)w.y << 32), r1 = (uint64_t)w.z | ((uint64_t)w.w << 32);
    const int64_t e0 = (int64_t)(r0 >> (63 - bits)) - ((int64_t)1 << bits);
    const int64_t e1 = (int64_t)(r1 >> (63 - bits)) - ((int64_t)1 << bits);
    u64x2 *p = reinterpret_cast<u64x2 *>(part + t * c.N + 2 * (size_t)b);
    u64x2 v = *p;
    v.x = addmod(csub(v.x, q), signed_residue(e0, q, mu), q);
    v.y = addmod(csub(v.y, q), signed_residue(e1, q, mu), q);
    *p = v;
}

__global__ void __launch_bounds__(256)
threshold_combine_kernel(const __grid_constant__ CtxDev c, const uint64_t *ct, uint32_t level,
                         const PartPtrs parts, int nparts, int64_t *d, size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t i = (uint32_t)(g % c.N);
    const size_t t = g / c.N;
    const uint64_t q = c.limb[0].q;
    uint64_t r = ct[((t * 2 + 0) * level + 0) * c.N + i];
    for (int p = 0; p < nparts; p++) r = addmod(r, parts.p[p][g], q);
    d[g] = r > q / 2 ? -(int64_t)(q - r) : (int64_t)r;
}

cudaError_t launch_threshold_split(const CtxDev &c, const int8_t *s8, uint64_t seed, uint64_t *tmp,
                                   cudaStream_t s) {
    threshold_split_kernel<<<blocks_for(c.N, 256), 256, 0, s>>>(c, s8, seed, tmp);
    return FEDHE_LAUNCHED();
}

cudaError_t launch_share_tables(const CtxDev &c, const uint64_t *share_hat, tw_t *s_hat, cudaStream_t s) {
    share_tables_kernel<<<blocks_for((size_t)c.L * c.N, 256), 256, 0, s>>>(c, share_hat, s_hat);
    return FEDHE_LAUNCHED();
}

cudaError_t launch_partial_decrypt(const CtxDev &c, const KeysDev &share, uint32_t party, const uint64_t *ct,
                                   uint32_t level, size_t T, uint64_t seed, uint32_t bits, uint64_t *part,
                                   cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    cudaError_t e;
    const size_t total = T * c.N;
    dec_gather_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, ct, level, part, total);
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_ntt(c, true, part, T, c.N, 0, 1, s))) return e;
    dec_pointwise_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, share, part, total);
    if ((e = FEDHE_LAUNCHED())) return e;
    if ((e = launch_ntt(c, false, part, T, c.N, 0, 1, s))) return e;
    const size_t pairs = T * (c.N >> 1);
    partial_finish_kernel<<<blocks_for(pairs, 256), 256, 0, s>>>(c, party, seed, bits, part, pairs);
    return FEDHE_LAUNCHED();
}

cudaError_t launch_threshold_combine(const CtxDev &c, const uint64_t *ct, uint32_t level, const PartPtrs &parts,
                                     int nparts, size_t T, int64_t *d, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    const size_t total = T * c.N;
    threshold_combine_kernel<<<blocks_for(total, 256), 256, 0, s>>>(c, ct, level, parts, nparts, d, total);
    return FEDHE_LAUNCHED();
}

// ===========================================================================
// selective-encryption mask
// ===========================================================================

// ordering key of a sensitivity score: its bit pattern when it is a
// non-negative number, 0 for negatives, -0 and NaN
__device__ __forceinline__ uint32_t score_key(float s) {
    const uint32_t b = __float_as_uint(s);
    return ((b & 0x80000000u) || b > 0x7f800000u) ? 0u : b;
}

// histogram of the next `digit_bits` key bits among the keys whose leading
// `prefix_bits` bits equal `prefix`
__global__ void __launch_bounds__(512)
key_histogram_kernel(const float *score, size_t P, uint32_t prefix, int prefix_bits, int digit_bits,
                     uint32_t *hist) {
    extern __shared__ uint32_t sh[];
    const uint32_t bins = 1u << digit_bits;
    for (uint32_t b = threadIdx.x; b < bins; b += blockDim.x) sh[b] = 0;
    __syncthreads();
    const int shift = 32 - prefix_bits - digit_bits;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < P; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t key = score_key(__ldg(score + i));
        if (prefix_bits == 0 || (key >> (32 - prefix_bits)) == prefix)
            atomicAdd(&sh[(key >> shift) & (bins - 1u)], 1u);
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b < bins; b += blockDim.x)
        if (sh[b]) atomicAdd(&hist[b], sh[b]);
}

cudaError_t launch_key_histogram(const float *score, size_t P, uint32_t prefix, int prefix_bits,
                                 int digit_bits, uint32_t *hist, cudaStream_t s) {
    unsigned grid = blocks_for(P, 512);
    if (grid > 148 * 8) grid = 148 * 8;
    if (grid == 0) grid = 1;
    key_histogram_kernel<<<grid, 512, sizeof(uint32_t) << digit_bits, s>>>(score, P, prefix, prefix_bits,
                                                                          digit_bits, hist);
    return FEDHE_LAUNCHED();
}

// number of keys equal to tau in every block of MASK_BLOCK parameters
__global__ void __launch_bounds__(MASK_BLOCK)
mask_count_eq_kernel(const float *score, size_t P, uint32_t tau, uint32_t *blk_eq) {
    const size_t i = (size_t)blockIdx.x * MASK_BLOCK + threadIdx.x;
    const bool eq = i < P && score_key(__ldg(score + i)) == tau;
    const int n = __syncthreads_count(eq);
    if (threadIdx.x == 0) blk_eq[blockIdx.x] = (uint32_t)n;
}

cudaError_t launch_mask_count_eq(const float *score, size_t P, uint32_t tau, uint32_t *blk_eq,
                                 cudaStream_t s) {
    mask_count_eq_kernel<<<blocks_for(P, MASK_BLOCK), MASK_BLOCK, 0, s>>>(score, P, tau, blk_eq);
    return FEDHE_LAUNCHED();
}

// exclusive prefix sum inside a block of 1024 threads; returns the block total
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t *warp_sums, uint32_t &total) {
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= (uint32_t)d) inc += o;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = warp_sums[lane], winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, winc, d);
            if (lane >= (uint32_t)d) winc += o;
        }
        warp_sums[lane] = winc - w;          // exclusive warp offsets
        if (lane == 31) warp_sums[32] = winc;
    }
    __syncthreads();
    const uint32_t res = warp_sums[warp] + inc - v;
    total = warp_sums[32];
    __syncthreads();
    return res;
}

// single-block exclusive scan of an array (block totals: at most a few
// hundred thousand entries)
__global__ void __launch_bounds__(1024) scan_kernel(uint32_t *a, size_t count, uint32_t *total_out) {
    __shared__ uint32_t warp_sums[33];
    uint32_t carry = 0;
    for (size_t base = 0; base < count; base += 1024) {
        const size_t i = base + threadIdx.x;
        const uint32_t v = i < count ? a[i] : 0u;
        uint32_t tot;
        const uint32_t ex = block_exclusive_scan(v, warp_sums, tot);
        if (i < count) a[i] = carry + ex;
        carry += tot;
    }
    if (threadIdx.x == 0) *total_out = carry;
}

cudaError_t launch_scan(uint32_t *a, size_t count, uint32_t *total, cudaStream_t s) {
    scan_kernel<<<1, 1024, 0, s>>>(a, count, total);
    return FEDHE_LAUNCHED();
}

// membership bits: key > tau, or key == tau and fewer than `need` equal keys
// at lower indices, or inside a forced index range
__global__ void __launch_bounds__(MASK_BLOCK)
mask_select_kernel(const float *score, size_t P, uint32_t tau, uint32_t need, const uint64_t *ranges,
                   uint32_t nranges, const uint32_t *blk_eq_prefix, uint32_t *bits, uint32_t *blk_sel) {
    __shared__ uint32_t warp_sums[33];
    const size_t i = (size_t)blockIdx.x * MASK_BLOCK + threadIdx.x;
    const uint32_t key = i < P ? score_key(__ldg(score + i)) : 0u;
    const bool eq = i < P && key == tau;
    uint32_t tot;
    const uint32_t eq_before = blk_eq_prefix[blockIdx.x] + block_exclusive_scan(eq ? 1u : 0u, warp_sums, tot);
    bool sel = i < P && (key > tau || (eq && eq_before < need));
    if (i < P && !sel) {
        for (uint32_t r = 0; r < nranges; r++)
            if (i >= ranges[2 * r] && i < ranges[2 * r + 1]) sel = true;
    }
    const uint32_t word = __ballot_sync(0xffffffffu, sel);
    if ((threadIdx.x & 31) == 0 && i < P) bits[i >> 5] = word;
    const int n = __syncthreads_count(sel);
    if (threadIdx.x == 0) blk_sel[blockIdx.x] = (uint32_t)n;
}

cudaError_t launch_mask_select(const float *score, size_t P, uint32_t tau, uint32_t need,
                               const uint64_t *ranges, uint32_t nranges, const uint32_t *blk_eq_prefix,
                               uint32_t *bits, uint32_t *blk_sel, cudaStream_t s) {
    mask_select_kernel<<<blocks_for(P, MASK_BLOCK), MASK_BLOCK, 0, s>>>(score, P, tau, need, ranges, nranges,
                                                                        blk_eq_prefix, bits, blk_sel);
    return FEDHE_LAUNCHED();
}

// per-word prefix counts and the ascending index list
__global__ void __launch_bounds__(MASK_BLOCK)
mask_write_kernel(size_t P, const uint32_t *bits, const uint32_t *blk_sel_prefix, uint32_t *wpre,
                  uint32_t *idx) {
    __shared__ uint32_t warp_sums[33];
    const size_t i = (size_t)blockIdx.x * MASK_BLOCK + threadIdx.x;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t word = i < P ? bits[i >> 5] : 0u;      // same for the whole warp
    const bool sel = i < P && ((word >> lane) & 1u);
    uint32_t tot;
    const uint32_t before = blk_sel_prefix[blockIdx.x] + block_exclusive_scan(sel ? 1u : 0u, warp_sums, tot);
    if (lane == 0 && i < P) wpre[i >> 5] = before;
    if (sel) idx[before] = (uint32_t)i;
}

cudaError_t launch_mask_write(size_t P, const uint32_t *bits, const uint32_t *blk_sel_prefix,
                              uint32_t *wpre, uint32_t *idx, cudaStream_t s) {
    mask_write_kernel<<<blocks_for(P, MASK_BLOCK), MASK_BLOCK, 0, s>>>(P, bits, blk_sel_prefix, wpre, idx);
    return FEDHE_LAUNCHED();
}

// ===========================================================================
// packing and merging
// ===========================================================================

// one pass over the update: masked parameters go to their slot, the others to
// the compacted remainder; the tail of the last ciphertext is zeroed
__global__ void __launch_bounds__(256)
pack_kernel(const uint32_t *bits, const uint32_t *wpre, const float *x, size_t P, size_t k, size_t padded,
            float *sel, float *rest) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < P) {
        const float v = __ldg(x + i);
        if (bits == nullptr) {
            sel[i] = v;
        } else {
            const uint32_t w = bits[i >> 5], lane = (uint32_t)(i & 31);
            const size_t before = (size_t)wpre[i >> 5] + __popc(w & ((1u << lane) - 1u));
            if ((w >> lane) & 1u) sel[before] = v;
            else rest[i - before] = v;
        }
    }
    if (i < padded - k) sel[k + i] = 0.0f;
}

cudaError_t launch_pack(const he_mask *mask, const float *x, size_t P, size_t k, size_t padded,
                        float *sel, float *rest, cudaStream_t s) {
    size_t threads = P > padded - k ? P : padded - k;
    if (threads == 0) return cudaSuccess;
    pack_kernel<<<blocks_for(threads, 256), 256, 0, s>>>(mask ? mask->bits : nullptr, mask ? mask->wpre : nullptr,
                                                          x, P, k, padded, sel, rest);
    return FEDHE_LAUNCHED();
}

__global__ void __launch_bounds__(256)
unpack_kernel(const uint32_t *bits, const uint32_t *wpre, const double *z, const double *rest_avg, size_t P,
              double *w_glob) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= P) return;
    if (bits == nullptr) {
        w_glob[i] = z[i];
        return;
    }
    const uint32_t w = bits[i >> 5], lane = (uint32_t)(i & 31);
    const size_t before = (size_t)wpre[i >> 5] + __popc(w & ((1u << lane) - 1u));
    w_glob[i] = ((w >> lane) & 1u) ? z[before] : rest_avg[i - before];
}

cudaError_t launch_unpack(const he_mask *mask, const double *z, const double *rest_avg, size_t P,
                          double *w_glob, cudaStream_t s) {
    if (P == 0) return cudaSuccess;
    unpack_kernel<<<blocks_for(P, 256), 256, 0, s>>>(mask ? mask->bits : nullptr, mask ? mask->wpre : nullptr, z,
                                                     rest_avg, P, w_glob);
    return FEDHE_LAUNCHED();
}

}  // namespace fedhe
