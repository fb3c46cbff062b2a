// Encode and decode kernels: the CKKS slot transform in fp64 (part 2 of the kernels).
#include "fedhe_kernels.cuh"
#include "fedhe_slots.cuh"

namespace fedhe {

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

}  // namespace fedhe
