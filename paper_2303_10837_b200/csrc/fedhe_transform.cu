// CUDA kernels (sm_100a) of the FedML-HE secure-aggregation hot path, part 1:
// the batched negacyclic transforms and key generation.  Nothing in the
// library is a dense floating-point contraction, so no tensor-core path
// exists: the transforms are bound by the issue rate of integer multiplies
// (limbs with large primes) and double-precision operations (limbs with
// primes below 2^46), the pointwise passes by HBM bandwidth.
#include "fedhe_kernels.cuh"

namespace fedhe {

std::atomic<uint64_t> g_launches{0};
uint64_t launch_count() { return g_launches.load(); }

// ===========================================================================
// batched negacyclic NTT
// ===========================================================================
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
    extern __shared__ __align__(128) uint64_t sm[];
    uint32_t b = blockIdx.x;
    const uint32_t blk = b & ((1u << c.A) - 1u);
    b >>= c.A;
    const uint32_t limb = b % nlimbs;
    const size_t poly = b / nlimbs;
    const LimbDev &lb = c.limb[limb0 + limb];
    uint64_t *p = data + poly * poly_stride + (size_t)limb * c.N + ((size_t)blk << L::LOGB);
    FEDHE_FOR_ARITH(lb, (ntt_block<M_, L, V, FWD, SCALED>(c, lb, sm, p, blk)));
}

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
cudaError_t launch_ntt_inner(const CtxDev &c, bool forward, uint64_t *data, size_t npoly, size_t poly_stride,
                             uint32_t limb0, uint32_t nlimbs, cudaStream_t s) {
    if (c.LOGB == 13) return launch_ntt_blocks<WLay<13>, 2>(c, forward, data, npoly, poly_stride, limb0, nlimbs, s);
    return launch_ntt_blocks<WLay<14>, 2>(c, forward, data, npoly, poly_stride, limb0, nlimbs, s);
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

}  // namespace fedhe
