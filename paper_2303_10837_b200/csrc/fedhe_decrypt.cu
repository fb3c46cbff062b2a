// Decryption kernels, single-key and two-party threshold (part 5 of the kernels).
#include "fedhe_kernels.cuh"
#include "fedhe_slots.cuh"

namespace fedhe {

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
    extern __shared__ __align__(128) uint64_t sm[];
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
            [&](uint32_t p, uint64_t a, uint64_t b, uint64_t *wa, uint64_t *wb) {
                const tw_t s0 = load_tw(k.s_hat + p), s1 = load_tw(k.s_hat + p + 1);
                *wa = shoup_lazy(a, s0.w, s0.wp, q);         // words wswz(p), wswz(p + 1)
                *wb = shoup_lazy(b, s1.w, s1.wp, q);
            });
    }
    int64_t *d = reinterpret_cast<int64_t *>(sm);
    {
        const NttArgs ia = LimbOf<ModInt>::args(lb, false, 0, 0);
        smem_ntt_inverse<L, V, true>(
            sm, tid, ia, lb.ninv, lb.wn,
            [&](uint32_t p, const uint64_t *wa, const uint64_t *wb) {
                if constexpr (NTT_IN) {
                    const u64x2 a = *reinterpret_cast<const u64x2 *>(c0 + p), b = *reinterpret_cast<const u64x2 *>(c1 + p);
                    const tw_t s0 = load_tw(k.s_hat + p), s1 = load_tw(k.s_hat + p + 1);
                    return u64x2{csub(a.x + shoup_lazy(b.x, s0.w, s0.wp, q), q2),
                                 csub(a.y + shoup_lazy(b.y, s1.w, s1.wp, q), q2)};
                } else {
                    return u64x2{*wa, *wb};
                }
            },
            [&](uint32_t i, uint64_t v, uint64_t *wv) {
                const uint64_t r = NTT_IN ? csub(v, q) : addmod(csub(v, q), c0[i], q);
                *reinterpret_cast<int64_t *>(wv) = r > q / 2 ? -(int64_t)(q - r) : (int64_t)r;     // d[wswz(i)]
            });
    }
    __syncthreads();
    // slot transform: bit-reversed load of (d_k + i d_{k+n}) / Delta from shared memory
    const double inv_delta = __longlong_as_double((long long)(1023 - c.log2_delta) << 52);
    cpx x[LF::E];
#pragma unroll
    for (int r = 0; r < LF::E; r++) {
        const uint32_t kk = bitrev(LF::template idx<LF::NPH - 1>(tid, r), LF::LOGB);
        x[r] = cpx{(double)d[wswz(kk)] * inv_delta, (double)d[wswz(kk + n)] * inv_delta};
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
        if (ntt_in) return launch_decrypt_fused_t<WLay<13>, 2, Lay<12, 3>, true>(c, k, ct, level, T, z, s);
        return launch_decrypt_fused_t<WLay<13>, 2, Lay<12, 3>, false>(c, k, ct, level, T, z, s);
    }
    if (ntt_in) return launch_decrypt_fused_t<WLay<14>, 2, Lay<13, 3>, true>(c, k, ct, level, T, z, s);
    return launch_decrypt_fused_t<WLay<14>, 2, Lay<13, 3>, false>(c, k, ct, level, T, z, s);
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

}  // namespace fedhe
