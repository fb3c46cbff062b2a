// Device code of the CKKS slot transform: complex arithmetic with one rounding
// per operation, the register-tiled butterfly network and its shared-memory
// exchange.  Used by the encode / decode kernels and by the fused decrypt.
#pragma once

#include "fedhe_kernels.cuh"

namespace fedhe {

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

// The encoder of one block of 2^LF::LOGB slots inside a thread block of LF::NT
// threads: the network, the scaling by Delta/n, the rounding and the
// bit-reversal.  `in(i)` gives the complex value at position i of the block as
// it enters the block's stages (the slot itself when the block is the whole
// vector, the output of the earlier stages otherwise); `sm` is a buffer of
// 2^LF::LOGB cpx values, used first for the exchanges between phases and then
// to put the rounded integers in order; coefficient kk of the block (kk its
// bit-reversed position) goes to m_out[(kk << A) | rb] and its imaginary
// partner to m_out[((kk << A) | rb) + n], where the whole vector has
// n = 2^(LF::LOGB + A) slots and rb is the bit-reversed block number.  Ends with
// a block barrier after which `sm` is free and m_out may be read by the block.
// Returns whether a coefficient left the range (the caller raises the status word).
template <class LF, class In>
__device__ __forceinline__ bool encode_block_in_place(const CtxDev &c, const In &in, uint64_t *sm, int64_t *m_out,
                                                      uint32_t A, uint32_t rb) {
    constexpr uint32_t NB = 1u << LF::LOGB;
    const uint32_t tid = threadIdx.x, n = NB << A;
    cpx x[LF::E];
#pragma unroll
    for (int r = 0; r < LF::E; r++) x[r] = in(LF::template idx<0>(tid, r));
    block_dif<LF>(x, reinterpret_cast<cpx *>(sm), tid, c.ftw);
    // Delta / n is a power of two: one exact multiplication
    const double scale = __longlong_as_double((long long)(1023 + c.log2_delta - (int)(LF::LOGB + A)) << 52);
    const double lim = 4611686018427387904.0;   // 2^62
    bool bad = false;
    int64_t *stage = reinterpret_cast<int64_t *>(sm);
    __syncthreads();                             // the exchange buffer is free again
#pragma unroll
    for (int r = 0; r < LF::E; r++) {
        const uint32_t kk = bitrev(LF::template idx<LF::NPH - 1>(tid, r), LF::LOGB);
        double re = __dmul_rn(x[r].re, scale), im = __dmul_rn(x[r].im, scale);
        if (!(fabs(re) < lim) || !(fabs(im) < lim)) { bad = true; re = 0.0; im = 0.0; }
        stage[stage_swz(kk)] = __double2ll_rn(re);
        stage[NB + stage_swz(kk)] = __double2ll_rn(im);
    }
    __syncthreads();
    for (uint32_t kk = tid; kk < NB; kk += LF::NT) {
        const uint32_t k = (kk << A) | rb;
        m_out[k] = stage[stage_swz(kk)];
        m_out[k + n] = stage[NB + stage_swz(kk)];
    }
    __syncthreads();
    return bad;
}

// the whole encoder of one slot vector of 2^LF::LOGB slots
template <class LF>
__device__ __forceinline__ bool encode_in_block(const CtxDev &c, const float *slots, uint64_t *sm, int64_t *m_out) {
    return encode_block_in_place<LF>(c, [&](uint32_t i) { return cpx{(double)__ldg(slots + i), 0.0}; }, sm, m_out, 0, 0);
}

}  // namespace fedhe
