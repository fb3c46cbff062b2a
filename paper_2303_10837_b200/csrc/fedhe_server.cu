// Server-side kernels: weighted ciphertext sum with rescale, plaintext remainder (part 4 of the kernels).
#include "fedhe_kernels.cuh"

namespace fedhe {

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

// The same sum for a limb whose prime is below 2^46, in the exact double-precision arithmetic of
// the transforms: a product costs the shared multiply / double-precision pipe 6 slots instead of
// about 19, which matters because this pass keeps that pipe two thirds busy beside HBM.  Every
// product has magnitude at most 3q/4 and the running sum is brought back below q after every 32
// clients, so it stays below 25 q < 2^51 and every addition is exact.
__device__ __forceinline__ void weighted_sum_pair_f64(const uint64_t *const *sp, const tw_t *sw, int C, uint32_t L,
                                                      uint32_t j, size_t off, double q, double qi, uint64_t &ax,
                                                      uint64_t &ay) {
    double sx = 0.0, sy = 0.0;
    int cl = 0;
    for (; cl + 4 <= C; cl += 4) {
        ulonglong2 v[4];
#pragma unroll
        for (int u = 0; u < 4; u++) v[u] = __ldg(reinterpret_cast<const ulonglong2 *>(sp[cl + u] + off));
#pragma unroll
        for (int u = 0; u < 4; u++) {
            const double w = f64_from_u64(sw[(cl + u) * L + j].w);
            sx = f64_add(sx, f64_mulmod(f64_from_u64(v[u].x), w, q, qi));
            sy = f64_add(sy, f64_mulmod(f64_from_u64(v[u].y), w, q, qi));
        }
        if ((cl & 31) == 28) {
            sx = f64_reduce(sx, q, qi);
            sy = f64_reduce(sy, q, qi);
        }
    }
    for (; cl < C; cl++) {
        const ulonglong2 v = __ldg(reinterpret_cast<const ulonglong2 *>(sp[cl] + off));
        const double w = f64_from_u64(sw[cl * L + j].w);
        sx = f64_add(sx, f64_mulmod(f64_from_u64(v.x), w, q, qi));
        sy = f64_add(sy, f64_mulmod(f64_from_u64(v.y), w, q, qi));
    }
    ax = f64_canonical(f64_reduce(sx, q, qi), q);
    ay = f64_canonical(f64_reduce(sy, q, qi), q);
}

// a limb's sum in whichever arithmetic its prime allows
__device__ __forceinline__ void weighted_sum_limb(const LimbDev &lb, const uint64_t *const *sp, const tw_t *sw, int C,
                                                  uint32_t L, uint32_t j, size_t off, uint64_t &ax, uint64_t &ay) {
    if (lb.fwd_d) weighted_sum_pair_f64(sp, sw, C, L, j, off, lb.qd, lb.qi, ax, ay);
    else weighted_sum_pair(sp, sw, C, L, j, off, lb.q, ax, ay);
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
    weighted_sum_limb(c.limb[L - 1], sp, sw, C, L, L - 1, (tc * L + (L - 1)) * c.N + i, rx, ry);
    const bool negx = rx > ql / 2, negy = ry > ql / 2;
    const uint64_t mx = negx ? ql - rx : rx, my = negy ? ql - ry : ry;   // |centred remainder|
    for (uint32_t j = 0; j + 1 < L; j++) {
        const LimbDev &lb = c.limb[j];
        const uint64_t q = lb.q;
        uint64_t ax, ay;
        weighted_sum_limb(lb, sp, sw, C, L, j, (tc * L + j) * c.N + i, ax, ay);
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
// ([T][2][L-1][N]), the last limb to `last` ([T][2][N]); with `last` null all L
// limbs go to `out` ([T][2][L][N]): the partial sum of a subset of the clients
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
        weighted_sum_limb(c.limb[j], sp, sw, C, L, j, (tc * L + j) * c.N + i, o.x, o.y);
        uint64_t *dst = !last ? out + (tc * L + j) * c.N + i
                              : (j + 1 < L ? out + (tc * (L - 1) + j) * c.N + i : last + tc * c.N + i);
        *reinterpret_cast<u64x2 *>(dst) = o;
    }
}

// Rescale of a sum of partial sums.  `parts` names P buffers uint64 [T][2][L][N]
// whose words are added here (P = 1: the caller has added them already); every
// word is a sum of canonical residues that does not overflow 64 bits.  Reduce,
// then as in the fused kernel.  The buffers are read with plain loads, so they
// may be peer memory that other GPUs' he_weighted_partial calls wrote into.
__global__ void __launch_bounds__(256)
rescale_partial_sum_kernel(const __grid_constant__ CtxDev c, const uint64_t *const *parts, int P, uint64_t *out,
                           size_t total) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const uint32_t L = c.L, pairs = c.N >> 1;
    const uint32_t i = (uint32_t)(g % pairs) * 2;
    const size_t tc = g / pairs;
    auto summed = [&](uint32_t j) {
        const size_t off = (tc * L + j) * c.N + i;
        ulonglong2 a = *reinterpret_cast<const ulonglong2 *>(parts[0] + off);
        for (int p = 1; p < P; p++) {
            const ulonglong2 b = *reinterpret_cast<const ulonglong2 *>(parts[p] + off);
            a.x += b.x;
            a.y += b.y;
        }
        return a;
    };
    const LimbDev &ll = c.limb[L - 1];
    const uint64_t ql = ll.q;
    const ulonglong2 rl = summed(L - 1);
    const uint64_t rx = barrett64(rl.x, ql, ll.mu), ry = barrett64(rl.y, ql, ll.mu);
    const bool negx = rx > ql / 2, negy = ry > ql / 2;
    const uint64_t mx = negx ? ql - rx : rx, my = negy ? ql - ry : ry;
    for (uint32_t j = 0; j + 1 < L; j++) {
        const LimbDev &lb = c.limb[j];
        const uint64_t q = lb.q;
        const ulonglong2 a = summed(j);
        const uint64_t ax = barrett64(a.x, q, lb.mu), ay = barrett64(a.y, q, lb.mu);
        const uint64_t sx = barrett64(mx, q, lb.mu), sy = barrett64(my, q, lb.mu);
        const uint64_t dx = negx ? addmod(ax, sx, q) : submod(ax, sx, q);
        const uint64_t dy = negy ? addmod(ay, sy, q) : submod(ay, sy, q);
        ulonglong2 o;
        o.x = shoup(dx, lb.qlinv.w, lb.qlinv.wp, q);
        o.y = shoup(dy, lb.qlinv.w, lb.qlinv.wp, q);
        *reinterpret_cast<ulonglong2 *>(out + (tc * (L - 1) + j) * c.N + i) = o;
    }
}

cudaError_t launch_aggregate_partial(const CtxDev &c, const uint64_t *const *ptrs, const tw_t *wtab, int C,
                                     size_t T, uint64_t *out, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    const size_t smem = (size_t)C * c.L * sizeof(tw_t) + (size_t)C * sizeof(void *);
    cudaError_t e;
    if (smem > 48 * 1024 &&
        (e = cudaFuncSetAttribute(aggregate_sum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)))
        return e;
    const size_t pairs = T * 2 * (c.N >> 1);
    aggregate_sum_kernel<<<blocks_for(pairs, 256), 256, smem, s>>>(c, ptrs, wtab, C, out, nullptr, pairs);
    return FEDHE_LAUNCHED();
}

cudaError_t launch_rescale_partial_sum(const CtxDev &c, const uint64_t *const *parts, int P, size_t T,
                                       uint64_t *out, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    const size_t pairs = T * 2 * (c.N >> 1);
    rescale_partial_sum_kernel<<<blocks_for(pairs, 256), 256, 0, s>>>(c, parts, P, out, pairs);
    return FEDHE_LAUNCHED();
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

// out[k] = sum_i alpha_i * rest_i[k] in fp64, clients in order, separate
// multiply and add.  A thread takes four neighbouring entries (one 16-byte
// load per client, two 16-byte stores) when every pointer allows it, and the
// loads of several clients are in flight at once.
__global__ void __launch_bounds__(256)
plain_aggregate_kernel(const float *const *ptrs, const double *alpha, int C, size_t len, double *out, bool vec) {
    const size_t g = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (g >= len) return;
    double a[4] = {0.0, 0.0, 0.0, 0.0};
    if (vec && g + 4 <= len) {
#pragma unroll 5
        for (int cl = 0; cl < C; cl++) {
            const float4 v = __ldg(reinterpret_cast<const float4 *>(ptrs[cl] + g));
            const double al = alpha[cl];
            a[0] = __dadd_rn(a[0], __dmul_rn(al, (double)v.x));
            a[1] = __dadd_rn(a[1], __dmul_rn(al, (double)v.y));
            a[2] = __dadd_rn(a[2], __dmul_rn(al, (double)v.z));
            a[3] = __dadd_rn(a[3], __dmul_rn(al, (double)v.w));
        }
        *reinterpret_cast<double2 *>(out + g) = make_double2(a[0], a[1]);
        *reinterpret_cast<double2 *>(out + g + 2) = make_double2(a[2], a[3]);
        return;
    }
    const uint32_t cnt = len - g < 4 ? (uint32_t)(len - g) : 4u;
    for (int cl = 0; cl < C; cl++) {
        const double al = alpha[cl];
        for (uint32_t j = 0; j < cnt; j++) a[j] = __dadd_rn(a[j], __dmul_rn(al, (double)__ldg(ptrs[cl] + g + j)));
    }
    for (uint32_t j = 0; j < cnt; j++) out[g + j] = a[j];
}

// aligned16: every client's pointer is 16-byte aligned
cudaError_t launch_plain_aggregate(const float *const *ptrs, const double *alpha, int C, size_t len,
                                   double *out, bool aligned16, cudaStream_t s) {
    if (len == 0) return cudaSuccess;
    const bool vec = aligned16 && (reinterpret_cast<uintptr_t>(out) & 15u) == 0;
    plain_aggregate_kernel<<<blocks_for((len + 3) / 4, 256), 256, 0, s>>>(ptrs, alpha, C, len, out, vec);
    return FEDHE_LAUNCHED();
}

}  // namespace fedhe
