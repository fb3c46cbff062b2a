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

// exclusive prefix sum over the threads of a block (any whole number of warps up to 32); the block total goes to `total`
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
        uint32_t w = lane < ((blockDim.x + 31u) >> 5) ? warp_sums[lane] : 0u, winc = w;
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

// histogram of the next `digit_bits` key bits among the keys whose leading
// `prefix_bits` bits equal the prefix found so far (state->prefix)
__global__ void __launch_bounds__(512)
key_histogram_kernel(const float *score, size_t P, const SelectState *state, int prefix_bits, int digit_bits,
                     uint32_t *hist) {
    extern __shared__ uint32_t sh[];
    const uint32_t bins = 1u << digit_bits;
    const uint32_t prefix = prefix_bits ? state->prefix : 0u;
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

cudaError_t launch_key_histogram(const float *score, size_t P, const SelectState *state, int prefix_bits,
                                 int digit_bits, int n_sm, uint32_t *hist, cudaStream_t s) {
    unsigned grid = blocks_for(P, 512);
    const unsigned resident = (unsigned)n_sm * 4u;       // four blocks of 512 threads fit one SM
    if (grid > resident) grid = resident;
    if (grid == 0) grid = 1;
    key_histogram_kernel<<<grid, 512, sizeof(uint32_t) << digit_bits, s>>>(score, P, state, prefix_bits,
                                                                          digit_bits, hist);
    return FEDHE_LAUNCHED();
}

// One step of the radix selection on the device: walks the digits of a
// histogram from the largest down until `need` keys are covered, appends the
// digit found to the prefix and takes the keys above it off `need`.  One block;
// after the last step prefix is the threshold key tau and need the number of
// keys equal to tau that belong to the mask.
__global__ void __launch_bounds__(1024)
radix_pick_kernel(const uint32_t *hist, int digit_bits, SelectState *state) {
    __shared__ uint32_t warp_sums[33];
    const uint32_t bins = 1u << digit_bits;
    const uint32_t need = state->need;
    // thread t looks at digits b = bins - 1 - (2 t), bins - 2 - (2 t): descending order
    const uint32_t per = bins / 1024u ? bins / 1024u : 1u;       // 2 for 11 bits, 1 for 10 bits
    uint32_t h[2] = {0u, 0u}, mine = 0u;
    for (uint32_t j = 0; j < per; j++) {
        const uint32_t pos = threadIdx.x * per + j;              // position in descending order
        h[j] = pos < bins ? hist[bins - 1u - pos] : 0u;
        mine += h[j];
    }
    uint32_t tot;
    uint32_t above = block_exclusive_scan(mine, warp_sums, tot);   // keys in digits above this thread's
    __syncthreads();
    for (uint32_t j = 0; j < per; j++) {
        const uint32_t pos = threadIdx.x * per + j;
        // the digit where the running count first reaches `need` (digit 0 if it never does)
        if (pos < bins && above < need && (above + h[j] >= need || pos == bins - 1u)) {
            state->prefix = (state->prefix << digit_bits) | (bins - 1u - pos);
            state->need = need - above;
        }
        above += h[j];
    }
}

cudaError_t launch_radix_pick(const uint32_t *hist, int digit_bits, SelectState *state, cudaStream_t s) {
    radix_pick_kernel<<<1, 1024, 0, s>>>(hist, digit_bits, state);
    return FEDHE_LAUNCHED();
}

// Keys of the four neighbouring parameters a thread takes (one 16-byte load
// where the pointer allows and all four exist; key 0 beyond the end).
__device__ __forceinline__ void load_keys4(const float *score, size_t P, size_t i0, bool vec, uint32_t (&key)[4]) {
    if (vec && i0 + 4 <= P) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(score + i0));
        key[0] = score_key(v.x); key[1] = score_key(v.y); key[2] = score_key(v.z); key[3] = score_key(v.w);
    } else {
#pragma unroll
        for (int j = 0; j < 4; j++) key[j] = i0 + j < P ? score_key(__ldg(score + i0 + j)) : 0u;
    }
}

// number of keys equal to tau in every block of MASK_BLOCK parameters (four per thread)
__global__ void __launch_bounds__(MASK_BLOCK / 4)
mask_count_eq_kernel(const float *score, size_t P, const SelectState *state, uint32_t *blk_eq, bool vec) {
    __shared__ uint32_t warp_sums[33];
    const uint32_t tau = state->prefix;
    const size_t i0 = (size_t)blockIdx.x * MASK_BLOCK + 4 * threadIdx.x;
    uint32_t key[4];
    load_keys4(score, P, i0, vec, key);
    uint32_t cnt = 0;
#pragma unroll
    for (int j = 0; j < 4; j++) cnt += (i0 + j < P && key[j] == tau) ? 1u : 0u;
    uint32_t tot;
    block_exclusive_scan(cnt, warp_sums, tot);
    if (threadIdx.x == 0) blk_eq[blockIdx.x] = tot;
}

cudaError_t launch_mask_count_eq(const float *score, size_t P, const SelectState *state, uint32_t *blk_eq,
                                 cudaStream_t s) {
    const bool vec = (reinterpret_cast<uintptr_t>(score) & 15u) == 0;
    mask_count_eq_kernel<<<blocks_for(P, MASK_BLOCK), MASK_BLOCK / 4, 0, s>>>(score, P, state, blk_eq, vec);
    return FEDHE_LAUNCHED();
}

// single-block exclusive scan of an array (block totals: about a hundred
// thousand entries for the largest model): every thread sums a contiguous
// chunk, the chunk sums are scanned across the block, and the thread writes
// the running prefix back over its chunk
__global__ void __launch_bounds__(1024) scan_kernel(uint32_t *a, size_t count, uint32_t *total_out) {
    __shared__ uint32_t warp_sums[33];
    const size_t per = (count + 1023) / 1024;
    const size_t b = threadIdx.x * per, e = b + per < count ? b + per : count;
    uint32_t sum = 0;
    for (size_t i = b; i < e; i++) sum += a[i];
    uint32_t tot;
    uint32_t run = block_exclusive_scan(sum, warp_sums, tot);
    for (size_t i = b; i < e; i++) {
        const uint32_t v = a[i];
        a[i] = run;
        run += v;
    }
    if (threadIdx.x == 0) *total_out = tot;
}

cudaError_t launch_scan(uint32_t *a, size_t count, uint32_t *total, cudaStream_t s) {
    scan_kernel<<<1, 1024, 0, s>>>(a, count, total);
    return FEDHE_LAUNCHED();
}

// membership bits: key > tau, or key == tau and fewer than `need` equal keys
// at lower indices, or inside a forced index range.  A thread takes four
// neighbouring parameters; eight neighbouring lanes put their four bits
// together into one word of the bit mask.
__global__ void __launch_bounds__(MASK_BLOCK / 4)
mask_select_kernel(const float *score, size_t P, const SelectState *state, const uint64_t *ranges,
                   uint32_t nranges, const uint32_t *blk_eq_prefix, uint32_t *bits, uint32_t *blk_sel, bool vec) {
    __shared__ uint32_t warp_sums[33];
    const uint32_t tau = state->prefix, need = state->need;
    const size_t i0 = (size_t)blockIdx.x * MASK_BLOCK + 4 * threadIdx.x;
    uint32_t key[4];
    load_keys4(score, P, i0, vec, key);
    uint32_t eqs = 0;
#pragma unroll
    for (int j = 0; j < 4; j++) eqs += (i0 + j < P && key[j] == tau) ? 1u : 0u;
    uint32_t tot;
    uint32_t eq_before = blk_eq_prefix[blockIdx.x] + block_exclusive_scan(eqs, warp_sums, tot);
    uint32_t nibble = 0, cnt = 0;
#pragma unroll
    for (int j = 0; j < 4; j++) {
        const size_t i = i0 + j;
        if (i >= P) continue;
        const bool eq = key[j] == tau;
        bool sel = key[j] > tau || (eq && eq_before < need);
        eq_before += eq ? 1u : 0u;
        if (!sel)
            for (uint32_t r = 0; r < nranges; r++)
                if (i >= ranges[2 * r] && i < ranges[2 * r + 1]) sel = true;
        nibble |= sel ? (1u << j) : 0u;
        cnt += sel ? 1u : 0u;
    }
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t word = nibble << (4u * (lane & 7u));
    word |= __shfl_xor_sync(0xffffffffu, word, 1);
    word |= __shfl_xor_sync(0xffffffffu, word, 2);
    word |= __shfl_xor_sync(0xffffffffu, word, 4);
    if ((lane & 7u) == 0 && i0 < P) bits[i0 >> 5] = word;
    block_exclusive_scan(cnt, warp_sums, tot);
    if (threadIdx.x == 0) blk_sel[blockIdx.x] = tot;
}

cudaError_t launch_mask_select(const float *score, size_t P, const SelectState *state,
                               const uint64_t *ranges, uint32_t nranges, const uint32_t *blk_eq_prefix,
                               uint32_t *bits, uint32_t *blk_sel, cudaStream_t s) {
    const bool vec = (reinterpret_cast<uintptr_t>(score) & 15u) == 0;
    mask_select_kernel<<<blocks_for(P, MASK_BLOCK), MASK_BLOCK / 4, 0, s>>>(score, P, state, ranges, nranges,
                                                                            blk_eq_prefix, bits, blk_sel, vec);
    return FEDHE_LAUNCHED();
}

// per-word prefix counts and the ascending index list: a thread takes one word
// of the bit mask (32 parameters), a block the MASK_BLOCK / 32 words of one
// counted block
__global__ void __launch_bounds__(MASK_BLOCK / 32)
mask_write_kernel(size_t P, const uint32_t *bits, const uint32_t *blk_sel_prefix, uint32_t *wpre,
                  uint32_t *idx) {
    __shared__ uint32_t warp_sums[33];
    const size_t word = (size_t)blockIdx.x * (MASK_BLOCK / 32) + threadIdx.x, nwords = (P + 31) >> 5;
    uint32_t w = word < nwords ? bits[word] : 0u;
    uint32_t tot;
    uint32_t before = blk_sel_prefix[blockIdx.x] + block_exclusive_scan((uint32_t)__popc(w), warp_sums, tot);
    if (word < nwords) wpre[word] = before;
    const uint32_t base = (uint32_t)(word << 5);
    while (w) {
        idx[before++] = base + (uint32_t)(__ffs((int)w) - 1);
        w &= w - 1u;
    }
}

cudaError_t launch_mask_write(size_t P, const uint32_t *bits, const uint32_t *blk_sel_prefix,
                              uint32_t *wpre, uint32_t *idx, cudaStream_t s) {
    mask_write_kernel<<<blocks_for(P, MASK_BLOCK), MASK_BLOCK / 32, 0, s>>>(P, bits, blk_sel_prefix, wpre, idx);
    return FEDHE_LAUNCHED();
}

// ===========================================================================
// packing and merging
// ===========================================================================
//
// These are single passes over the update, bound by HBM.  With a mask, a warp
// takes PACK_WORDS consecutive words of the bit mask at a time and lane l the
// parameter of bit l of each: loads and stores of a warp instruction are then
// consecutive addresses (the compacted outputs as well, because the lanes'
// positions are consecutive among the selected / unselected bits of the word),
// and all of a thread's loads are issued before the first store.  Without a
// mask the steps are copies with 16-byte accesses where the pointers allow.

constexpr int PACK_WORDS = 8;       // mask words (256 parameters) per warp
constexpr int COPY_VECS = 4;        // 16-byte vectors per thread of the copies

// masked parameters go to their slot, the others to the compacted remainder
__global__ void __launch_bounds__(256)
pack_masked_kernel(const uint32_t *bits, const uint32_t *wpre, const float *x, size_t P, float *sel, float *rest) {
    const uint32_t lane = threadIdx.x & 31u;
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const size_t word0 = warp * PACK_WORDS, nwords = (P + 31) >> 5;
    if (word0 >= nwords) return;
    float v[PACK_WORDS];
    uint32_t w[PACK_WORDS], pre[PACK_WORDS];
#pragma unroll
    for (int j = 0; j < PACK_WORDS; j++) {
        const size_t word = word0 + j, i = (word << 5) + lane;
        v[j] = i < P ? __ldg(x + i) : 0.0f;
        w[j] = word < nwords ? __ldg(bits + word) : 0u;
        pre[j] = word < nwords ? __ldg(wpre + word) : 0u;
    }
#pragma unroll
    for (int j = 0; j < PACK_WORDS; j++) {
        const size_t i = ((word0 + j) << 5) + lane;
        if (i >= P) continue;
        const size_t before = (size_t)pre[j] + __popc(w[j] & ((1u << lane) - 1u));
        if ((w[j] >> lane) & 1u) sel[before] = v[j];
        else rest[i - before] = v[j];
    }
}

// dst[i] = src[i] for i < count, dst[i] = 0 for count <= i < padded (T may be float or double)
template <class T, class V>
__global__ void __launch_bounds__(256)
copy_pad_kernel(const T *src, size_t count, size_t padded, T *dst, bool vec) {
    constexpr size_t per = sizeof(V) / sizeof(T);
    const size_t base = (size_t)blockIdx.x * blockDim.x * COPY_VECS * per;
    if (vec && base + (size_t)blockDim.x * COPY_VECS * per <= count) {
        V t[COPY_VECS];
#pragma unroll
        for (int j = 0; j < COPY_VECS; j++)
            t[j] = __ldg(reinterpret_cast<const V *>(src + base) + j * blockDim.x + threadIdx.x);
#pragma unroll
        for (int j = 0; j < COPY_VECS; j++)
            reinterpret_cast<V *>(dst + base)[j * blockDim.x + threadIdx.x] = t[j];
        return;
    }
    // ragged end of the input, unaligned pointers, and the zero padding
    for (size_t i = base + threadIdx.x; i < base + (size_t)blockDim.x * COPY_VECS * per && i < padded; i += blockDim.x)
        dst[i] = i < count ? src[i] : (T)0;
}

template <class T, class V>
static cudaError_t launch_copy_pad(const T *src, size_t count, size_t padded, T *dst, cudaStream_t s) {
    if (padded == 0) return cudaSuccess;
    const bool vec = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & (sizeof(V) - 1)) == 0;
    const size_t per_block = 256 * COPY_VECS * (sizeof(V) / sizeof(T));
    copy_pad_kernel<T, V><<<blocks_for(padded, (unsigned)per_block), 256, 0, s>>>(src, count, padded, dst, vec);
    return FEDHE_LAUNCHED();
}

__global__ void __launch_bounds__(256) zero_tail_kernel(float *dst, size_t count) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) dst[i] = 0.0f;
}

cudaError_t launch_pack(const he_mask *mask, const float *x, size_t P, size_t k, size_t padded,
                        float *sel, float *rest, cudaStream_t s) {
    if (!mask) return launch_copy_pad<float, float4>(x, P, padded, sel, s);     // k = P: a copy and the zero tail
    if (P) {
        const size_t warps = (((P + 31) >> 5) + PACK_WORDS - 1) / PACK_WORDS;
        pack_masked_kernel<<<blocks_for(warps * 32, 256), 256, 0, s>>>(mask->bits, mask->wpre, x, P, sel, rest);
        const cudaError_t e = FEDHE_LAUNCHED();
        if (e) return e;
    }
    if (padded > k) {                                                            // tail of the last ciphertext
        zero_tail_kernel<<<blocks_for(padded - k, 256), 256, 0, s>>>(sel + k, padded - k);
        return FEDHE_LAUNCHED();
    }
    return cudaSuccess;
}

// the reverse with a mask: w_glob[i] = z[r] for the r-th masked parameter, the remainder's
// average in order elsewhere
__global__ void __launch_bounds__(256)
unpack_masked_kernel(const uint32_t *bits, const uint32_t *wpre, const double *z, const double *rest_avg, size_t P,
                     double *w_glob) {
    const uint32_t lane = threadIdx.x & 31u;
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const size_t word0 = warp * PACK_WORDS, nwords = (P + 31) >> 5;
    if (word0 >= nwords) return;
    double v[PACK_WORDS];
#pragma unroll
    for (int j = 0; j < PACK_WORDS; j++) {
        const size_t word = word0 + j, i = (word << 5) + lane;
        v[j] = 0.0;
        if (i < P) {
            const uint32_t w = __ldg(bits + word);
            const size_t before = (size_t)__ldg(wpre + word) + __popc(w & ((1u << lane) - 1u));
            v[j] = ((w >> lane) & 1u) ? __ldg(z + before) : __ldg(rest_avg + (i - before));
        }
    }
#pragma unroll
    for (int j = 0; j < PACK_WORDS; j++) {
        const size_t i = ((word0 + j) << 5) + lane;
        if (i < P) w_glob[i] = v[j];
    }
}

cudaError_t launch_unpack(const he_mask *mask, const double *z, const double *rest_avg, size_t P,
                          double *w_glob, cudaStream_t s) {
    if (P == 0) return cudaSuccess;
    if (!mask) return launch_copy_pad<double, double2>(z, P, P, w_glob, s);
    const size_t warps = (((P + 31) >> 5) + PACK_WORDS - 1) / PACK_WORDS;
    unpack_masked_kernel<<<blocks_for(warps * 32, 256), 256, 0, s>>>(mask->bits, mask->wpre, z, rest_avg, P, w_glob);
    return FEDHE_LAUNCHED();
}

}  // namespace fedhe
