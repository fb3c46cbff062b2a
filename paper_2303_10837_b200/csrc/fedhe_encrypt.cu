// Encryption kernels (part 3 of the kernels).
#include <cooperative_groups.h>

#include "fedhe_kernels.cuh"
#include "fedhe_slots.cuh"

namespace fedhe {

// ===========================================================================
// encryption:  c0 = pk0 u + e0 + m,  c1 = pk1 u + e1   (mod every q_j)
// ===========================================================================

// Index swizzle of the one-byte sample arrays in shared memory (banks of four
// bytes, i.e. index bits 2..6): the first phase of a transform reads them with
// lanes that differ in index bits 0, 1, 7, 8 and 9, the epilogues with
// consecutive lanes; folding bits 7..9 into bits 2..4 keeps both patterns free
// of bank conflicts, leaves aligned groups of four intact, and does not involve
// the first phase's register bits (10 and up), so a thread computes it once.
__device__ __forceinline__ uint32_t bswz(uint32_t i) { return i ^ (((i >> 7) & 7u) << 2); }

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
                    if (h == 0) return ar.small(su[bswz(i)]);
                    if (h == 2) return ar.small(se[bswz(i)]);
                    return ar.from_residue(signed_residue(__ldcg(mt + i) + (int64_t)se[bswz(i)], q, lb.mu));
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
        static_assert(L::reg_bit(0, 0) >= 10, "the sample swizzle stays clear of the first phase's register bits");
        smem_ntt_forward<L, V>(
            sm, tid, fa, [&](uint32_t base, uint32_t reg) { return ar.small((su + bswz(base))[reg]); },
            [&](uint32_t p, val a, val b, uint64_t *wa, uint64_t *wb) {
                const auto a0 = M::load_key(p1 + p), a1 = M::load_key(p1 + p + 1);
                u64x2 v;
                v.x = M::bits(ar.mul_key(a, a0));
                v.y = M::bits(ar.mul_key(b, a1));
                *reinterpret_cast<u64x2 *>(c1 + p) = v;
                const auto b0 = M::load_key(p0 + p), b1 = M::load_key(p0 + p + 1);
                *wa = M::bits(ar.mul_key(a, b0));            // words wswz(p), wswz(p + 1)
                *wb = M::bits(ar.mul_key(b, b1));
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
            [&](uint32_t p, const uint64_t *wa, const uint64_t *wb) {
                if (h == 0) return pair_of<val>{M::from_bits(*wa), M::from_bits(*wb)};
                const u64x2 t = *reinterpret_cast<const u64x2 *>(cc + p);
                return pair_of<val>{M::from_bits(t.x), M::from_bits(t.y)};
            },
            [&](uint32_t i, val v) {
                // e1 is a small value; e0 + m needs a full reduction
                const uint64_t add = h == 0 ? signed_residue(__ldcg(mt + i) + (int64_t)se[bswz(i)], q, lb.mu)
                                            : small_residue(se[bswz(i)], q);
                cc[i] = ar.canon_add(v, add);
            });
        __syncthreads();   // phase-0 readers are done before the next transform writes
    }
}

// Fused path for N <= 2^14 (one block holds a whole limb): a thread block
// draws u, e0, e1 of a ciphertext once into shared memory and encodes the
// ciphertext's slots (the slot transform runs in the limb buffer; the rounded
// message goes to a scratch of N words that belongs to this block alone and is
// read back once per limb, so it lives in L2), then for every limb of it
// transforms u, multiplies by both halves of the public key, transforms back
// and adds the error and message terms.  HBM sees the slots once and the
// ciphertext once; the second product waits, in transform order, in the c1
// slot it will finally occupy.  A block whose range of units begins in the
// middle of a ciphertext encodes that ciphertext again for itself (no block
// waits for another).
template <class L, int V, bool NTT_OUT>
__global__ void __launch_bounds__(L::NT / V, (L::NT / V) <= 512 ? 2 : 1)
encrypt_fused_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const float *sel, int64_t *mscr,
                     uint32_t t0, uint64_t seed, uint32_t client, uint64_t *ct, uint32_t T) {
    using LF = Lay<L::LOGB - 1, 3>;                  // the slot transform of the same ring
    static_assert(LF::NT == L::NT / V, "the encoder is played by the same threads");
    extern __shared__ __align__(128) uint64_t sm[];
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
    int64_t *mblk = mscr + (size_t)blockIdx.x * B;   // this block's encoded message (stays in L2)
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
                *reinterpret_cast<char4 *>(su + bswz(4 * b)) = v;
            }
            for (uint32_t b = tid; b < B / 2; b += RT) {
                u32x4 w0 = stream_block(seed, b, t, client, TAG_ENC_E0);
                u32x4 w1 = stream_block(seed, b, t, client, TAG_ENC_E1);
                char2 a = make_char2((signed char)gauss_from_u64(gt, (uint64_t)w0.x | ((uint64_t)w0.y << 32)),
                                     (signed char)gauss_from_u64(gt, (uint64_t)w0.z | ((uint64_t)w0.w << 32)));
                char2 e = make_char2((signed char)gauss_from_u64(gt, (uint64_t)w1.x | ((uint64_t)w1.y << 32)),
                                     (signed char)gauss_from_u64(gt, (uint64_t)w1.z | ((uint64_t)w1.w << 32)));
                *reinterpret_cast<char2 *>(se0 + bswz(2 * b)) = a;
                *reinterpret_cast<char2 *>(se1 + bswz(2 * b)) = e;
            }
            // the ciphertext's message: slot transform, scaling and rounding in the limb buffer
            if (encode_in_block<LF>(c, sel + (size_t)tl * (B / 2), sm, mblk)) atomicOr(c.status, 1);
        }
        const LimbDev &lb = c.limb[j];
        uint64_t *cbase = ct + (((size_t)tl * 2 + 0) * c.L + j) * B;
        FEDHE_FOR_ARITH_SEL(lb, (encrypt_unit<M_, L, V, NTT_OUT>(lb, k.pk0_hat + (size_t)j * B, k.pk1_hat + (size_t)j * B, sm, su,
                                                    se0, mblk, cbase, cstride)));
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
        // sample of element i = base | reg: the swizzle of the sample arrays only involves index
        // bits below the first phase's register bits, so it is taken of base once
        auto src2 = [&](uint32_t base, uint32_t reg) {
            // u is ternary: the twiddle product is 0, w or -w
            const int8_t *sb = su + bswz(base);
            const int b = sb[reg + H];
            if constexpr (std::is_same<M, ModF64>::value) {
                return f64_fma(grp == 0 ? (double)b : (double)-b, w0, (double)sb[reg]);
            } else {
                const uint64_t u = small_residue(sb[reg], q);
                const uint64_t v = b == 0 ? 0 : (b > 0 ? w0.w : q - w0.w);
                return grp == 0 ? u + v : u - v + ar.q2;
            }
        };
        auto src = [&](uint32_t i) { return src2(i, 0u); };
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
                    if (h == 2) return ar.small(se[bswz(i)]);
                    return ar.from_residue(signed_residue(__ldcg(mt + i) + (int64_t)se[bswz(i)], q, lb.mu));
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
        auto dst = [&](uint32_t p, val a, val b, uint64_t *wa, uint64_t *wb) {
            const auto a0 = M::load_key(p1 + p), a1 = M::load_key(p1 + p + 1);
            u64x2 v;
            v.x = M::bits(ar.mul_key(a, a0));
            v.y = M::bits(ar.mul_key(b, a1));
            *reinterpret_cast<u64x2 *>(c1 + p) = v;      // parked until the second pass
            const auto b0 = M::load_key(p0 + p), b1 = M::load_key(p0 + p + 1);
            *wa = M::bits(ar.mul_key(a, b0));            // words wswz(p), wswz(p + 1) of this group's half
            *wb = M::bits(ar.mul_key(b, b1));
        };
        static_assert(L::reg_bit(0, 0) >= 10, "the sample swizzle stays clear of the first phase's register bits");
        smem_ntt_forward<L, V>(smg, gt, fa, src2, dst, gsync);
    }
#pragma unroll 1
    for (int h = 0; h < 2; h++) {
        uint64_t *cc = cbase + h * cstride;
        const int8_t *se = se0 + h * B;
        const auto ia = LimbOf<M>::args(lb, false, 1, grp);
        const M &ar = ia.m;
        const auto ninv = LimbOf<M>::ninv(lb), wn = LimbOf<M>::wn(lb);
        auto isrc = [&](uint32_t p, const uint64_t *wa, const uint64_t *wb) {
            if (h == 0) return pair_of<val>{M::from_bits(*wa), M::from_bits(*wb)};
            const u64x2 t = *reinterpret_cast<const u64x2 *>(cc + grp * H + p);
            return pair_of<val>{M::from_bits(t.x), M::from_bits(t.y)};
        };
        auto idst = [&](uint32_t, val v, uint64_t *wv) { *wv = M::bits(v); };
        smem_ntt_inverse<L, V, false>(smg, gt, ia, ninv, wn, isrc, idst, gsync);
        __syncthreads();
        // last stage across the halves with 1/N folded in, then the error / message terms; the
        // message words of four rounds are requested before the first of them is used
        constexpr uint32_t ROUNDS = H / RT, AHEAD = ROUNDS < 4 ? ROUNDS : 4;
        // element tid + r RT = tid ^ r RT sits at word wswz(tid) ^ wswz(r RT): a constant XOR into
        // the low nibble and a constant offset above it
        const uint32_t w_tid = word_address(sm, wswz(tid));
        auto word_of_round = [&](uint32_t r) {
            const uint32_t c = wswz(r * RT);
            const uint32_t a = (w_tid ^ ((c & 15u) << 3)) + ((c & ~15u) << 3);
            return reinterpret_cast<const uint64_t *>(__cvta_shared_to_generic((size_t)a));
        };
        // (the byte swizzle involves index bits 7..9 only: of tid, not of the round)
        static_assert(RT % 1024 == 0, "a round advances the index above the swizzled bits");
        const int8_t *se_tid = se + bswz(tid);
        const int64_t *mt_tid = mt + tid;
        uint64_t *cc_tid = cc + tid;
#pragma unroll
        for (uint32_t k0 = 0; k0 < ROUNDS; k0 += AHEAD) {
            int64_t m_lo[AHEAD], m_hi[AHEAD];
            if (h == 0) {
#pragma unroll
                for (uint32_t k = 0; k < AHEAD; k++) {
                    m_lo[k] = __ldcg(mt_tid + (k0 + k) * RT);
                    m_hi[k] = __ldcg(mt_tid + (k0 + k) * RT + H);
                }
            }
#pragma unroll
            for (uint32_t k = 0; k < AHEAD; k++) {
                const uint32_t er = (k0 + k) * RT;             // element tid + er
                const uint64_t *wl = word_of_round(k0 + k);
                val lo = M::from_bits(wl[0]), hi = M::from_bits(wl[H]);
                ar.inv_scaled(lo, hi, ninv, wn);
                uint64_t add_lo, add_hi;
                if (h == 0) {
                    add_lo = signed_residue(m_lo[k] + (int64_t)se_tid[er], q, lb.mu);
                    add_hi = signed_residue(m_hi[k] + (int64_t)se_tid[er + H], q, lb.mu);
                } else {
                    add_lo = small_residue(se_tid[er], q);
                    add_hi = small_residue(se_tid[er + H], q);
                }
                cc_tid[er] = ar.canon_add(lo, add_lo);
                cc_tid[er + H] = ar.canon_add(hi, add_hi);
            }
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
encrypt_fused2_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const float *sel, int64_t *mscr,
                      uint32_t t0, uint64_t seed, uint32_t client, uint64_t *ct, uint32_t T) {
    using LF = Lay<L::LOGB, 3>;                      // the slot transform of the ring (n = half a limb)
    static_assert(LF::NT == 2 * L::NT / V, "the encoder is played by the whole block");
    extern __shared__ __align__(128) uint64_t sm[];
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
    int64_t *mblk = mscr + (size_t)blockIdx.x * B;   // this block's encoded message (stays in L2)
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
                *reinterpret_cast<char4 *>(su + bswz(4 * b)) = v;
            }
            for (uint32_t b = tid; b < B / 2; b += RT) {
                u32x4 w0 = stream_block(seed, b, t, client, TAG_ENC_E0);
                u32x4 w1 = stream_block(seed, b, t, client, TAG_ENC_E1);
                char2 a = make_char2((signed char)gauss_from_u64(gt_tab, (uint64_t)w0.x | ((uint64_t)w0.y << 32)),
                                     (signed char)gauss_from_u64(gt_tab, (uint64_t)w0.z | ((uint64_t)w0.w << 32)));
                char2 e = make_char2((signed char)gauss_from_u64(gt_tab, (uint64_t)w1.x | ((uint64_t)w1.y << 32)),
                                     (signed char)gauss_from_u64(gt_tab, (uint64_t)w1.z | ((uint64_t)w1.w << 32)));
                *reinterpret_cast<char2 *>(se0 + bswz(2 * b)) = a;
                *reinterpret_cast<char2 *>(se1 + bswz(2 * b)) = e;
            }
            // the ciphertext's message: slot transform, scaling and rounding in the limb buffer
            if (encode_in_block<LF>(c, sel + (size_t)tl * H, sm, mblk)) atomicOr(c.status, 1);
        }
        const LimbDev &lb = c.limb[j];
        uint64_t *cbase = ct + (((size_t)tl * 2 + 0) * c.L + j) * B;
        FEDHE_FOR_ARITH_SEL(lb, (encrypt_unit2<M_, L, V, NTT_OUT>(lb, k.pk0_hat + (size_t)j * B, k.pk1_hat + (size_t)j * B, sm, su,
                                                     se0, mblk, cbase, cstride)));
    }
}

// ===========================================================================
// Long rings on thread-block clusters: a limb of 256 KB (N = 2^15) does not fit
// one SM's shared memory, but it fits the shared memories of a cluster of
// CS = 2 thread blocks.  (The code is written for CS = 2^CL; with CS = 4, for
// N = 2^16, the device holds only 33 clusters at once, 132 of its 148 SMs, and
// the kernel measured 25 % slower than the multi-pass path, which N = 2^16
// therefore keeps.)  The limb is cut into ROWS = 2 CS
// pieces of HB = 2^13 residues; block `rank` of the cluster holds pieces
// 2 rank and 2 rank + 1, and each of its two groups of 512 threads transforms
// one piece as a sub-block of the long transform on its own schedule (named
// barriers), as in the two-group kernel above.  The log2 ROWS outer stages,
// which pair elements of different pieces, are done where all pieces are at
// hand:
//   forward, on the way in: the input u is ternary, so an output of the outer
//     stages is a signed sum of ROWS constants (one row of the outer butterfly
//     network applied to unit vectors, computed once per unit), picked by the
//     samples -- no multiplication;
//   inverse, after the sub-transforms: block `rank` takes the columns
//     [rank HB / CS, (rank + 1) HB / CS) of the ROWS x HB view, reads the
//     elements of a column from the shared memories of all blocks of the
//     cluster (distributed shared memory, plain loads), runs the outer stages
//     with 1/N folded in, adds the error and message terms and writes the
//     ciphertext.
// HBM sees the encoded message and the ciphertext once (the second key
// product waits in its final slot), instead of the six passes over the
// ciphertext of the multi-kernel path below.  The cluster's blocks meet at a
// cluster barrier before and after every read of each other's shared memory;
// all of them run the same units, so every block reaches every barrier.
// ===========================================================================

namespace cg = cooperative_groups;

template <class M, int CL>
__device__ __forceinline__ void encrypt_unit_cluster(const LimbDev &lb, const tw_t *pk0, const tw_t *pk1, uint64_t *sm,
                                                     uint64_t *consts, const int8_t *su, const int8_t *se,
                                                     const int64_t *mt, uint64_t *cbase, size_t cstride,
                                                     uint32_t rank, cg::cluster_group &cluster) {
    using L = WLay<13>;
    constexpr int V = 2;
    using val = typename M::val;
    constexpr uint32_t HB = 1u << 13, CS = 1u << CL, ROWS = 2 * CS, AO = CL + 1, COLS = HB / CS;
    constexpr uint32_t GT = L::NT / V, RT = 2 * GT;            // threads per group, per block
    const uint32_t tid = threadIdx.x, grp = tid / GT, gt = tid % GT;
    const uint32_t row = 2 * rank + grp;                       // the piece this group transforms
    uint64_t *smg = sm + grp * HB;
    const GroupSync gsync = {1 + grp, GT};
    const uint64_t q = lb.q;
    // row `row` of the outer forward stages applied to the unit vectors
    if (gt < ROWS) {
        const auto fo = LimbOf<M>::args(lb, true, 0, 0);
        val x[ROWS], y[ROWS];
#pragma unroll
        for (uint32_t a = 0; a < ROWS; a++) {
            x[a] = fo.m.small(a == gt ? 1 : 0);
            y[a] = fo.m.small(0);
        }
        outer_forward<AO>(x, y, fo);
        val r = x[0];
#pragma unroll
        for (uint32_t a = 1; a < ROWS; a++)
            if (a == row) r = x[a];
        consts[grp * ROWS + gt] = M::bits(fo.m.from_residue(fo.m.canon_wide(r)));       // in [0, q)
    }
    gsync();
    {
        const tw_t *p0 = pk0 + row * HB, *p1 = pk1 + row * HB;
        uint64_t *c1 = cbase + cstride + row * HB;
        const auto fa = LimbOf<M>::args(lb, true, AO, row);
        const M &ar = fa.m;
        val cst[ROWS];
#pragma unroll
        for (uint32_t k = 0; k < ROWS; k++) cst[k] = M::from_bits(consts[grp * ROWS + k]);
        smem_ntt_forward<L, V>(
            smg, gt, fa,
            // element base | reg of the piece: the sample swizzle (index bits 7..9) is taken of base once
            [&](uint32_t base, uint32_t reg) {
                const int8_t *sb = su + bswz(base) + reg;
                if constexpr (std::is_same<M, ModF64>::value) {
                    double acc = 0.0;                                // |acc| < ROWS q
#pragma unroll
                    for (uint32_t k = 0; k < ROWS; k++) acc = f64_fma((double)sb[k * HB], cst[k], acc);
                    return ROWS > 4 ? ar.settle(acc) : acc;
                } else {
                    uint64_t acc = 0;                                // below ROWS q
#pragma unroll
                    for (uint32_t k = 0; k < ROWS; k++) {
                        const int b = sb[k * HB];
                        acc += b == 0 ? 0 : (b > 0 ? cst[k] : q - cst[k]);
                    }
                    return ROWS > 4 ? csub_as<true>(acc, 2 * ar.q2) : acc;      // below 4q
                }
            },
            [&](uint32_t p, val a, val b, uint64_t *wa, uint64_t *wb) {
                const auto a0 = M::load_key(p1 + p), a1 = M::load_key(p1 + p + 1);
                u64x2 v;
                v.x = M::bits(ar.mul_key(a, a0));
                v.y = M::bits(ar.mul_key(b, a1));
                *reinterpret_cast<u64x2 *>(c1 + p) = v;      // parked until the second pass
                const auto b0 = M::load_key(p0 + p), b1 = M::load_key(p0 + p + 1);
                *wa = M::bits(ar.mul_key(a, b0));            // words wswz(p), wswz(p + 1) of this group's piece
                *wb = M::bits(ar.mul_key(b, b1));
            },
            gsync);
    }
    const uint64_t *piece[CS];                                   // the same buffer in every block of the cluster
#pragma unroll
    for (uint32_t a = 0; a < CS; a++) piece[a] = cluster.map_shared_rank(sm, a);
#pragma unroll 1
    for (int h = 0; h < 2; h++) {
        uint64_t *cc = cbase + h * cstride;
        const int8_t *seh = se + h * 2 * HB;
        const auto ia = LimbOf<M>::args(lb, false, AO, row);
        const auto ninv = LimbOf<M>::ninv(lb), wn = LimbOf<M>::wn(lb);
        smem_ntt_inverse<L, V, false>(
            smg, gt, ia, ninv, wn,
            [&](uint32_t p, const uint64_t *wa, const uint64_t *wb) {
                if (h == 0) return pair_of<val>{M::from_bits(*wa), M::from_bits(*wb)};
                const u64x2 t = *reinterpret_cast<const u64x2 *>(cc + row * HB + p);
                return pair_of<val>{M::from_bits(t.x), M::from_bits(t.y)};
            },
            [&](uint32_t, val v, uint64_t *wv) { *wv = M::bits(v); }, gsync);
        cluster.sync();                                          // every piece is transformed and visible
        const auto to = LimbOf<M>::args(lb, false, 0, 0);
#pragma unroll 1
        for (uint32_t c2 = tid; c2 < COLS / 2; c2 += RT) {
            const uint32_t lc = 2 * c2, i = rank * COLS + lc;    // two neighbouring columns
            val x[ROWS], y[ROWS];
#pragma unroll
            for (uint32_t a = 0; a < ROWS; a++) {
                const uint64_t *src = piece[a >> 1] + (a & 1u) * HB;
                x[a] = M::from_bits(src[wswz(i)]);
                y[a] = M::from_bits(src[wswz(i + 1)]);
            }
            outer_inverse<AO>(x, y, to, ninv, wn);
#pragma unroll
            for (uint32_t a = 0; a < ROWS; a++) {
                const int ex = seh[a * COLS + lc], ey = seh[a * COLS + lc + 1];
                uint64_t ax, ay;
                if (h == 0) {
                    const longlong2 mm = __ldcg(reinterpret_cast<const longlong2 *>(mt + a * HB + i));
                    ax = signed_residue(mm.x + (int64_t)ex, q, lb.mu);
                    ay = signed_residue(mm.y + (int64_t)ey, q, lb.mu);
                } else {
                    ax = small_residue(ex, q);
                    ay = small_residue(ey, q);
                }
                // streaming store: the finished ciphertext should not push the waiting products out of L2
                __stcs(reinterpret_cast<ulonglong2 *>(cc + a * HB + i),
                       make_ulonglong2(to.m.canon_add(x[a], ax), to.m.canon_add(y[a], ay)));
            }
        }
        cluster.sync();                                          // nobody still reads this block's pieces
    }
}

template <int CL>
__global__ void __launch_bounds__(1024, 1)
encrypt_cluster_kernel(const __grid_constant__ CtxDev c, const KeysDev k, const float *sel, int64_t *mscr,
                       uint32_t t0, uint64_t seed, uint32_t client, uint64_t *ct, uint32_t T) {
    using LF = Lay<14 - CL, 3>;                                  // this block's share of the slot transform
    static_assert(CL == 1, "the encoder is split over a cluster of two blocks");
    extern __shared__ __align__(128) uint64_t sm[];
    constexpr uint32_t HB = 1u << 13, CS = 1u << CL, ROWS = 2 * CS, N = ROWS * HB, COLS = HB / CS, RT = 1024;
    int8_t *su = reinterpret_cast<int8_t *>(sm + 2 * HB);        // u, all N coefficients
    int8_t *se = su + N;                                         // e0 then e1: this block's columns of every row
    const uint32_t tid = threadIdx.x;
    __shared__ GaussTables gt;
    __shared__ uint64_t consts[2 * 8];
    gauss_tables_init(gt, tid);
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = cluster.block_rank();
    const uint32_t cid = blockIdx.x / CS, nclusters = gridDim.x / CS;

    // (ciphertext, limb) units in ciphertext-major order, dealt evenly to the clusters
    const uint64_t units = (uint64_t)T * c.L;
    const uint32_t u_begin = (uint32_t)(units * cid / nclusters);
    const uint32_t u_end = (uint32_t)(units * (cid + 1) / nclusters);
    const size_t cstride = (size_t)c.L * N;
    int64_t *mcl = mscr + (size_t)cid * N;                        // this cluster's encoded message (stays in L2)
    uint32_t sampled = 0xffffffffu;
    for (uint32_t unit = u_begin; unit < u_end; unit++) {
        const uint32_t tl = unit / c.L, j = unit % c.L;
        if (tl != sampled) {
            sampled = tl;
            const uint32_t t = t0 + tl;
            __syncthreads();
            for (uint32_t b = tid; b < N / 4; b += RT) {
                u32x4 w = stream_block(seed, b, t, client, TAG_ENC_U);
                char4 v = make_char4((signed char)ternary_from_word(w.x), (signed char)ternary_from_word(w.y),
                                     (signed char)ternary_from_word(w.z), (signed char)ternary_from_word(w.w));
                *reinterpret_cast<char4 *>(su + bswz(4 * b)) = v;
            }
            // the error terms of the coefficients this block finishes: columns [rank COLS, (rank + 1) COLS) of every row
            for (uint32_t pp = tid; pp < HB; pp += RT) {
                const uint32_t a = pp / (COLS / 2), lc = 2 * (pp % (COLS / 2));
                const uint32_t coef = a * HB + rank * COLS + lc;         // even: one Philox block per pair
                u32x4 w0 = stream_block(seed, coef >> 1, t, client, TAG_ENC_E0);
                u32x4 w1 = stream_block(seed, coef >> 1, t, client, TAG_ENC_E1);
                char2 e0 = make_char2((signed char)gauss_from_u64(gt, (uint64_t)w0.x | ((uint64_t)w0.y << 32)),
                                      (signed char)gauss_from_u64(gt, (uint64_t)w0.z | ((uint64_t)w0.w << 32)));
                char2 e1 = make_char2((signed char)gauss_from_u64(gt, (uint64_t)w1.x | ((uint64_t)w1.y << 32)),
                                      (signed char)gauss_from_u64(gt, (uint64_t)w1.z | ((uint64_t)w1.w << 32)));
                *reinterpret_cast<char2 *>(se + a * COLS + lc) = e0;
                *reinterpret_cast<char2 *>(se + 2 * HB + a * COLS + lc) = e1;
            }
            // The ciphertext's message.  The slot transform of n = N/2 values is split over the
            // two blocks: the first stage pairs slot i with slot i + n/2, and each block computes
            // its own half of that stage straight from the slots (real inputs, no exchange), then
            // runs the remaining stages on its half in the limb buffer.  Block `rank` produces the
            // coefficients of parity `rank`; both write to the cluster's scratch.
            {
                constexpr uint32_t half = N / 4;                 // n / 2
                const float *slots = sel + (size_t)tl * (N / 2);
                const double2 *ftw = c.ftw;
                const bool bad = encode_block_in_place<LF>(
                    c,
                    [&](uint32_t i) {
                        const cpx U = cpx{(double)__ldg(slots + i), 0.0}, V = cpx{(double)__ldg(slots + i + half), 0.0};
                        if (rank == 0) return cadd_rn(U, V);
                        cpx w = load_ftw(ftw, half + i);
                        w.im = -w.im;
                        return cmul_rn(csub_rn(U, V), w);
                    },
                    sm, mcl, 1, rank);
                if (bad) atomicOr(c.status, 1);
            }
            cluster.sync();                                      // both halves of the message are written
        }
        const LimbDev &lb = c.limb[j];
        uint64_t *cbase = ct + (((size_t)tl * 2 + 0) * c.L + j) * N;
        FEDHE_FOR_ARITH_SEL(lb, (encrypt_unit_cluster<M_, CL>(lb, k.pk0_hat + (size_t)j * N, k.pk1_hat + (size_t)j * N, sm,
                                                             consts, su, se, mcl, cbase, cstride, rank, cluster)));
    }
}

// Launches the cluster kernel with as many clusters as the device holds at
// once (74 pairs or 37 quadruples on 148 SMs); *launched is false, and nothing
// was launched, when the device cannot hold such a cluster.
template <int CL>
static cudaError_t launch_encrypt_cluster(const CtxDev &c, const KeysDev &k, const float *sel, int64_t *mscr,
                                          size_t max_clusters, uint32_t t0, size_t T, uint64_t seed, uint32_t client,
                                          uint64_t *ct, cudaStream_t s, bool *launched) {
    constexpr unsigned CS = 1u << CL;
    const size_t smem = ((size_t)8 << 14) + (size_t)c.N + ((size_t)2 << 14);
    auto kern = encrypt_cluster_kernel<CL>;
    *launched = false;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = CS;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS, 1, 1);
    cfg.blockDim = dim3(1024, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg) != cudaSuccess || clusters < 1) {
        cudaGetLastError();                                      // reported by the caller
        return cudaSuccess;
    }
    const size_t units = T * c.L;
    if ((size_t)clusters > units) clusters = (int)units;
    if ((size_t)clusters > max_clusters) clusters = (int)max_clusters;     // the message scratch has room for so many
    cfg.gridDim = dim3((unsigned)clusters * CS, 1, 1);
    const uint32_t T32 = (uint32_t)T;
    if ((e = cudaLaunchKernelEx(&cfg, kern, c, k, sel, mscr, t0, seed, client, ct, T32))) return e;
    *launched = true;
    return FEDHE_LAUNCHED();
}

// Long rings without clusters (N = 2^16 in the coefficient format, both long rings in
// the transform-domain format): kernels over the 2^A x 2^13 view of a limb.

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

// one thread per pair of neighbouring columns of one ciphertext, all limbs: draws u and runs the outer forward stages;
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
    extern __shared__ __align__(128) uint64_t sm[];
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
    __shared__ GaussTables gt;
    gauss_tables_init(gt, threadIdx.x);
    __syncthreads();
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t pairs = c.N >> 1;
    const uint32_t b = (uint32_t)(g % pairs), i = 2 * b;   // one Philox block per pair
    const size_t tl = g / pairs;
    const uint32_t t = t0 + (uint32_t)tl;
    const u32x4 w0 = stream_block(seed, b, t, client, TAG_ENC_E0);
    const u32x4 w1 = stream_block(seed, b, t, client, TAG_ENC_E1);
    const longlong2 mm = *reinterpret_cast<const longlong2 *>(m + tl * c.N + i);
    const int64_t ax = mm.x + gauss_from_u64(gt, (uint64_t)w0.x | ((uint64_t)w0.y << 32));
    const int64_t ay = mm.y + gauss_from_u64(gt, (uint64_t)w0.z | ((uint64_t)w0.w << 32));
    const int ex = gauss_from_u64(gt, (uint64_t)w1.x | ((uint64_t)w1.y << 32));
    const int ey = gauss_from_u64(gt, (uint64_t)w1.z | ((uint64_t)w1.w << 32));
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
__device__ __forceinline__ void enc_outer_inverse_add_limb(const LimbDev &lb, uint64_t *p, uint32_t B,
                                                           const int64_t (&add)[1u << A][2]) {
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
        o.x = t.m.canon_add(x[a], signed_residue(add[a][0], q, lb.mu));
        o.y = t.m.canon_add(y[a], signed_residue(add[a][1], q, lb.mu));
        *reinterpret_cast<u64x2 *>(p + (size_t)a * B) = o;
    }
}

// (4) one thread per pair of neighbouring columns of one ciphertext: for each
// component draws its error terms once (e0 + m, then e1), then finishes every limb
template <uint32_t A>
__global__ void __launch_bounds__(256, A == 3 ? 2 : 4)
enc_outer_inverse_add_kernel(const __grid_constant__ CtxDev c, const int64_t *m, uint32_t t0, uint64_t seed,
                             uint32_t client, uint64_t *ct, size_t total) {
    __shared__ GaussTables gt;
    gauss_tables_init(gt, threadIdx.x);
    __syncthreads();
    size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t B = 1u << c.LOGB, half = B >> 1;
    constexpr uint32_t rows = 1u << A;
    const uint32_t col = (uint32_t)(g % half) * 2;
    const size_t tl = g / half;
    const uint32_t t = t0 + (uint32_t)tl;
#pragma unroll 1
    for (uint32_t comp = 0; comp < 2; comp++) {
        int64_t add[rows][2];                          // e0 + m, or e1
#pragma unroll
        for (uint32_t a = 0; a < rows; a++) {
            const uint32_t i = a * B + col;           // one Philox block per pair of coefficients
            const u32x4 w = stream_block(seed, i >> 1, t, client, comp == 0 ? TAG_ENC_E0 : TAG_ENC_E1);
            add[a][0] = gauss_from_u64(gt, (uint64_t)w.x | ((uint64_t)w.y << 32));
            add[a][1] = gauss_from_u64(gt, (uint64_t)w.z | ((uint64_t)w.w << 32));
            if (comp == 0) {
                const longlong2 mm = *reinterpret_cast<const longlong2 *>(m + tl * c.N + i);
                add[a][0] += mm.x;
                add[a][1] += mm.y;
            }
        }
#pragma unroll 1
        for (uint32_t j = 0; j < c.L; j++) {
            const LimbDev &lb = c.limb[j];
            uint64_t *p = ct + ((tl * 2 + comp) * c.L + j) * c.N + col;
            FEDHE_FOR_ARITH(lb, (enc_outer_inverse_add_limb<M_, A>(lb, p, B, add)));
        }
    }
}

// shared memory of a block of the fused kernels: the limb and three one-byte sample arrays
static size_t fused_smem(const CtxDev &c) { return ((size_t)c.N << 3) + 3 * (size_t)c.N; }

// The fused kernels run one block per SM for N = 2^14 and two for N = 2^13 (what
// their shared memory allows); every block owns N words of message scratch.
size_t encrypt_fused_blocks(const CtxDev &c, int n_sm) {
    const size_t per_sm = (size_t)(227 * 1024) / fused_smem(c);
    return (size_t)n_sm * (per_sm ? per_sm : 1);
}

template <class L, int V, bool TWO_GROUPS, bool NTT_OUT>
static cudaError_t launch_encrypt_fused(const CtxDev &c, const KeysDev &k, const float *sel, int64_t *mscr,
                                        int n_sm, uint32_t t0, size_t T, uint64_t seed, uint32_t client,
                                        uint64_t *ct, cudaStream_t s) {
    const size_t smem = fused_smem(c);
    auto kern = TWO_GROUPS ? encrypt_fused2_kernel<L, V, NTT_OUT> : encrypt_fused_kernel<L, V, NTT_OUT>;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    size_t grid = encrypt_fused_blocks(c, n_sm);                     // fewer if there is less work
    if (grid > T * c.L) grid = T * c.L;
    kern<<<(unsigned)grid, (TWO_GROUPS ? 2 : 1) * L::NT / V, smem, s>>>(c, k, sel, mscr, t0, seed, client, ct,
                                                                        (uint32_t)T);
    return FEDHE_LAUNCHED();
}

// launches the block forward kernel of the long-ring paths
template <bool ACC>
static cudaError_t launch_enc_block_forward(const CtxDev &c, const KeysDev &k, const uint64_t *ubuf, size_t T,
                                            uint64_t *ct, cudaStream_t s) {
    using L = WLay<13>;                                 // long rings are cut into 2^13 blocks
    constexpr int V = 2;
    const size_t smem = sizeof(uint64_t) << L::LOGB;
    auto kern = enc_block_forward_kernel<L, V, ACC>;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return e;
    kern<<<(unsigned)((T * c.L) << c.A), L::NT / V, smem, s>>>(c, k, ubuf, ct);
    return FEDHE_LAUNCHED();
}

size_t encrypt_work_bytes(const CtxDev &c, int n_sm, size_t T, bool ntt_out) {
    if (c.A == 0) return encrypt_fused_blocks(c, n_sm) * c.N * sizeof(int64_t);
    if (c.logN == 15 && !ntt_out) return (size_t)(n_sm / 2) * c.N * sizeof(int64_t);      // N words per cluster of two blocks
    // long rings: the encoded messages and the encoder's complex buffer; the
    // transform-domain format transforms u in a buffer of its own
    return (2 * T * c.N + (ntt_out ? T * (size_t)c.L * c.N : 0)) * sizeof(uint64_t);
}

cudaError_t launch_encrypt(const CtxDev &c, const KeysDev &k, const float *sel, void *work, int n_sm,
                           uint32_t t0, size_t T, uint64_t seed, uint32_t client, uint64_t *ct,
                           cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    int64_t *m = static_cast<int64_t *>(work);
    if (c.A == 0) {
        if (c.LOGB == 13)
            return launch_encrypt_fused<WLay<13>, 2, false, false>(c, k, sel, m, n_sm, t0, T, seed, client, ct, s);
        return launch_encrypt_fused<WLay<13>, 2, true, false>(c, k, sel, m, n_sm, t0, T, seed, client, ct, s);
    }
    cudaError_t e;
    if (c.logN == 15) {
        // N = 2^15: clusters of two thread blocks, 74 of them on 148 SMs, encoder inside
        bool launched = false;
        if ((e = launch_encrypt_cluster<1>(c, k, sel, m, (size_t)(n_sm / 2), t0, T, seed, client, ct, s, &launched)))
            return e;
        return launched ? cudaSuccess : cudaErrorLaunchOutOfResources;     // a device that cannot hold such a cluster
    }
    if ((e = launch_encode(c, sel, T, reinterpret_cast<double2 *>(m + T * c.N), m, s))) return e;
    // N = 2^16 would need clusters of four blocks, of which the device holds only 33 at once
    // (132 of its 148 SMs; measured 25 % slower than the passes below): the ciphertext buffer
    // itself is the work space, and every pass over it does as much as it can.
    // (1) draw u and run the outer forward stages into the c1 slots; (2) block transforms of the
    // c1 slots whose last phase writes both products u^ pk0^ -> c0 and u^ pk1^ -> c1; (3) inverse
    // block transforms of all slots; (4) outer inverse stages fused with the error and message terms.
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
cudaError_t launch_encrypt_ntt(const CtxDev &c, const KeysDev &k, const float *sel, void *work, int n_sm,
                               uint32_t t0, size_t T, uint64_t seed, uint32_t client, uint64_t *ct,
                               cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    int64_t *m = static_cast<int64_t *>(work);
    if (c.A == 0) {
        if (c.LOGB == 13)
            return launch_encrypt_fused<WLay<13>, 2, false, true>(c, k, sel, m, n_sm, t0, T, seed, client, ct, s);
        return launch_encrypt_fused<WLay<13>, 2, true, true>(c, k, sel, m, n_sm, t0, T, seed, client, ct, s);
    }
    cudaError_t e;
    uint64_t *ubuf = reinterpret_cast<uint64_t *>(m + 2 * T * c.N);
    if ((e = launch_encode(c, sel, T, reinterpret_cast<double2 *>(m + T * c.N), m, s))) return e;
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

}  // namespace fedhe
