// Mask selection, packing and merging kernels (part 6 of the kernels).
#include "fedhe_kernels.cuh"

namespace fedhe {

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
// the compacted remainder; the tail of the last ciphertext is zeroed.  A
// thread takes four neighbouring parameters (one 16-byte load when the
// pointers allow it; they always share one word of the bit mask).
__global__ void __launch_bounds__(256)
pack_kernel(const uint32_t *bits, const uint32_t *wpre, const float *x, size_t P, size_t k, size_t padded,
            float *sel, float *rest, bool vec) {
    const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t i0 = t * 4;
    if (i0 < P) {
        float v[4];
        const uint32_t cnt = P - i0 < 4 ? (uint32_t)(P - i0) : 4u;
        if (vec && cnt == 4) {
            const float4 q = __ldg(reinterpret_cast<const float4 *>(x + i0));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
#pragma unroll
            for (uint32_t j = 0; j < 4; j++) v[j] = j < cnt ? __ldg(x + i0 + j) : 0.0f;
        }
        if (bits == nullptr) {
            if (vec && cnt == 4) {
                *reinterpret_cast<float4 *>(sel + i0) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (uint32_t j = 0; j < 4; j++)
                    if (j < cnt) sel[i0 + j] = v[j];
            }
        } else {
            const uint32_t w = bits[i0 >> 5], lane = (uint32_t)(i0 & 31);
            size_t before = (size_t)wpre[i0 >> 5] + __popc(w & ((1u << lane) - 1u));
#pragma unroll
            for (uint32_t j = 0; j < 4; j++) {
                if (j < cnt) {
                    if ((w >> (lane + j)) & 1u) sel[before++] = v[j];
                    else rest[i0 + j - before] = v[j];
                }
            }
        }
    }
    if (t < padded - k) sel[k + t] = 0.0f;
}

cudaError_t launch_pack(const he_mask *mask, const float *x, size_t P, size_t k, size_t padded,
                        float *sel, float *rest, cudaStream_t s) {
    const size_t quads = (P + 3) / 4;
    size_t threads = quads > padded - k ? quads : padded - k;
    if (threads == 0) return cudaSuccess;
    const bool vec = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(sel)) & 15u) == 0;
    pack_kernel<<<blocks_for(threads, 256), 256, 0, s>>>(mask ? mask->bits : nullptr, mask ? mask->wpre : nullptr,
                                                          x, P, k, padded, sel, rest, vec);
    return FEDHE_LAUNCHED();
}

// the reverse: two neighbouring parameters per thread (one 16-byte store)
__global__ void __launch_bounds__(256)
unpack_kernel(const uint32_t *bits, const uint32_t *wpre, const double *z, const double *rest_avg, size_t P,
              double *w_glob, bool vec) {
    const size_t i0 = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 2;
    if (i0 >= P) return;
    const bool two = i0 + 1 < P;
    double a, b = 0.0;
    if (bits == nullptr) {
        if (vec && two) {
            *reinterpret_cast<double2 *>(w_glob + i0) = *reinterpret_cast<const double2 *>(z + i0);
            return;
        }
        a = z[i0];
        if (two) b = z[i0 + 1];
    } else {
        const uint32_t w = bits[i0 >> 5], lane = (uint32_t)(i0 & 31);
        size_t before = (size_t)wpre[i0 >> 5] + __popc(w & ((1u << lane) - 1u));
        const bool s0 = (w >> lane) & 1u;
        a = s0 ? z[before] : rest_avg[i0 - before];
        before += s0 ? 1 : 0;
        if (two) b = ((w >> (lane + 1)) & 1u) ? z[before] : rest_avg[i0 + 1 - before];
    }
    if (vec && two) {
        *reinterpret_cast<double2 *>(w_glob + i0) = make_double2(a, b);
    } else {
        w_glob[i0] = a;
        if (two) w_glob[i0 + 1] = b;
    }
}

cudaError_t launch_unpack(const he_mask *mask, const double *z, const double *rest_avg, size_t P,
                          double *w_glob, cudaStream_t s) {
    if (P == 0) return cudaSuccess;
    const bool vec = ((reinterpret_cast<uintptr_t>(z) | reinterpret_cast<uintptr_t>(w_glob)) & 15u) == 0;
    unpack_kernel<<<blocks_for((P + 1) / 2, 256), 256, 0, s>>>(mask ? mask->bits : nullptr,
                                                               mask ? mask->wpre : nullptr, z, rest_avg, P, w_glob, vec);
    return FEDHE_LAUNCHED();
}

}  // namespace fedhe
