// Microbenchmark of the transform core alone: every SM loads one block of
// residues into shared memory, runs forward + inverse transforms on it in a
// loop without touching global memory, and stores it back (the round trip must
// reproduce the input).  Reports the time of one transform on one SM for both
// limb arithmetics and both block sizes: what a kernel built on the core can
// reach at best once its global traffic is hidden.
//
//   ./transform_loop_bench        (built by build.py next to the library)
#include <cstdio>
#include <vector>
#include <cuda_runtime.h>
#include "fedhe_ntt.cuh"
#include "fedhe_host.h"
using namespace fedhe;

template <class M, class L, int V>
__global__ void __launch_bounds__(L::NT / V, 1) loop_kernel(NttArgsT<M> fa, NttArgsT<M> ia, typename M::tab ninv, typename M::tab wn, uint64_t *data, int iters) {
    extern __shared__ __align__(16) uint64_t sm[];
    const uint32_t tid = threadIdx.x;
    uint64_t *p = data + ((size_t)blockIdx.x << L::LOGB);
    for (uint32_t i = tid; i < (1u << L::LOGB); i += blockDim.x) sm[wswz(i)] = M::bits(fa.m.from_residue(p[i]));
    __syncthreads();
    for (int it = 0; it < iters; it++) {
        smem_ntt_forward<L, V>(sm, tid, fa, [&](uint32_t i) { return M::from_bits(sm[wswz(i)]); },
            [&](uint32_t i, typename M::val a, typename M::val b) { sm[wswz(i)] = M::bits(fa.m.from_residue(fa.m.canon_wide(a))); sm[wswz(i + 1)] = M::bits(fa.m.from_residue(fa.m.canon_wide(b))); });
        __syncthreads();
        smem_ntt_inverse<L, V, true>(sm, tid, ia, ninv, wn,
            [&](uint32_t i) { return pair_of<typename M::val>{M::from_bits(sm[wswz(i)]), M::from_bits(sm[wswz(i + 1)])}; },
            [&](uint32_t i, typename M::val v) { sm[wswz(i)] = M::bits(ia.m.from_residue(ia.m.canon(v))); });
        __syncthreads();
    }
    for (uint32_t i = tid; i < (1u << L::LOGB); i += blockDim.x) p[i] = fa.m.to_residue(M::from_bits(sm[wswz(i)]));
}

template <class M> struct Tab;
template <> struct Tab<ModInt> { static tw_t cv(HostTw t) { return tw_t{t.w, t.wp}; } static ModInt m(uint64_t q) { return ModInt{q, 2 * q}; } };
template <> struct Tab<ModF64> { static double cv(HostTw t) { return (double)t.w; } static ModF64 m(uint64_t q) { return ModF64{(double)q, 1.0 / (double)q}; } };

template <class M, class L, int V>
void run(const char *name, uint64_t q, int iters) {
    const uint32_t N = 1u << L::LOGB;
    HostLimb hl; host_build_limb(N, q, hl);
    std::vector<typename M::tab> f(N), iv(N);
    for (uint32_t i = 0; i < N; i++) { f[i] = Tab<M>::cv(hl.fwd[i]); iv[i] = Tab<M>::cv(hl.inv[i]); }
    typename M::tab *df, *di; cudaMalloc(&df, N * sizeof(f[0])); cudaMalloc(&di, N * sizeof(f[0]));
    cudaMemcpy(df, f.data(), N * sizeof(f[0]), cudaMemcpyHostToDevice); cudaMemcpy(di, iv.data(), N * sizeof(f[0]), cudaMemcpyHostToDevice);
    int nsm; cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, 0);
    std::vector<uint64_t> h((size_t)nsm * N); for (size_t i = 0; i < h.size(); i++) h[i] = (i * 0x9E3779B97F4A7C15ull >> 8) % q;
    uint64_t *d; cudaMalloc(&d, h.size() * 8); cudaMemcpy(d, h.data(), h.size() * 8, cudaMemcpyHostToDevice);
    NttArgsT<M> fa{df, Tab<M>::m(q), 0, 0}, ia{di, Tab<M>::m(q), 0, 0};
    auto k = loop_kernel<M, L, V>;
    const size_t smem = sizeof(uint64_t) << L::LOGB;
    cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    k<<<nsm, L::NT / V, smem>>>(fa, ia, Tab<M>::cv(hl.ninv), Tab<M>::cv(hl.wn), d, 2);
    cudaDeviceSynchronize();
    cudaEventRecord(e0);
    k<<<nsm, L::NT / V, smem>>>(fa, ia, Tab<M>::cv(hl.ninv), Tab<M>::cv(hl.wn), d, iters);
    cudaEventRecord(e1); cudaDeviceSynchronize();
    float ms; cudaEventElapsedTime(&ms, e0, e1);
    std::vector<uint64_t> back(h.size()); cudaMemcpy(back.data(), d, h.size() * 8, cudaMemcpyDeviceToHost);
    size_t bad = 0; for (size_t i = 0; i < h.size(); i++) bad += back[i] != h[i];
    const double us = ms * 1e3 / (2.0 * iters);
    const double bf = (double)(N / 2) * L::LOGB;
    printf("%-28s %8.2f us per transform per SM  (%.2f butterflies per SM and clock at 1.965 GHz)  round-trip mismatches %zu  err %s\n",
           name, us, bf / (us * 1965.0), bad, cudaGetErrorString(cudaGetLastError()));
    cudaFree(d); cudaFree(df); cudaFree(di);
}

int main() {
    const uint64_t q60 = 0xffffffffffc0001ull, q45 = 0x1fffffc20001ull;
    run<ModInt, WLay<14>, 2>("int  2^14 1024 thr", q60, 50);
    run<ModF64, WLay<14>, 2>("f64  2^14 1024 thr", q45, 50);
    run<ModInt, WLay<14>, 4>("int  2^14  512 thr", q60, 50);
    run<ModF64, WLay<14>, 4>("f64  2^14  512 thr", q45, 50);
    run<ModInt, WLay<13>, 2>("int  2^13  512 thr", q60, 50);
    run<ModF64, WLay<13>, 2>("f64  2^13  512 thr", q45, 50);
    return 0;
}
