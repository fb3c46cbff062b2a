// Internal types shared by the kernels and the C ABI of the CUDA library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/fedhe.h"
#include "fedhe_ntt.cuh"

namespace fedhe {

// Per-prime constants and table pointers, passed to kernels by value.
struct LimbDev {
    uint64_t q;          // the prime
    uint64_t mu;         // floor(2^64 / q), Barrett
    tw_t ninv;           // 1/N
    tw_t wn;             // (inverse twiddle of stage 0) / N
    tw_t qlinv;          // 1 / q_{L-1} mod q (unused for the last prime)
    const tw_t *fwd;     // psi^brev(i)
    const tw_t *inv;     // psi^-brev(i)
    // primes below F64_PRIME_LIMIT also carry what the double-precision
    // transforms need (fwd_d is null for the others)
    const double *fwd_d; // the same twiddles as doubles
    const double *inv_d;
    double qd, qi;       // q and 1/q rounded
    double ninv_d, wn_d; // 1/N and (inverse twiddle of stage 0)/N
};

// the pieces of a limb that a transform in arithmetic M needs
template <class M>
struct LimbOf;
template <bool SEL>
struct LimbOf<ModIntT<SEL>> {
    static HD NttArgsT<ModIntT<SEL>> args(const LimbDev &lb, bool fwd, uint32_t A, uint32_t blk) {
        return NttArgsT<ModIntT<SEL>>{fwd ? lb.fwd : lb.inv, ModIntT<SEL>{lb.q, 2 * lb.q}, A, blk};
    }
    static HD tw_t ninv(const LimbDev &lb) { return lb.ninv; }
    static HD tw_t wn(const LimbDev &lb) { return lb.wn; }
};
template <>
struct LimbOf<ModF64> {
    static HD NttArgsF args(const LimbDev &lb, bool fwd, uint32_t A, uint32_t blk) {
        return NttArgsF{fwd ? lb.fwd_d : lb.inv_d, ModF64{lb.qd, lb.qi}, A, blk};
    }
    static HD double ninv(const LimbDev &lb) { return lb.ninv_d; }
    static HD double wn(const LimbDev &lb) { return lb.wn_d; }
};

struct CtxDev {
    uint32_t N, logN, L;
    uint32_t LOGB, A;    // a length-N transform = 2^A blocks of 2^LOGB
    int32_t log2_delta;
    LimbDev limb[HE_MAX_LIMBS];
    const LimbDev *limb_dev;   // the same table in device memory, for kernels that loop over limbs
    const double2 *ftw;  // slot-transform twiddles, entry [len/2 + j]
    int *status;         // sticky anomaly word
};

struct KeysDev {
    const tw_t *pk0_hat; // [L][N] transform-domain public key with Shoup companions
    const tw_t *pk1_hat;
    const tw_t *s_hat;   // [L][N] transform-domain secret key
    const int8_t *s;     // [N]
};

}  // namespace fedhe

struct he_ctx {
    uint32_t magic;
    int device;
    fedhe::CtxDev dev;
    he_params params;
    std::vector<void *> owned;     // device allocations freed with the context
    // growable work buffers (device)
    void *ws = nullptr;            // encode output / decrypt scratch
    size_t ws_bytes = 0;
    void *tab = nullptr;           // per-call pointer and weight tables
    size_t tab_bytes = 0;
    void *round_buf = nullptr;     // buffers of he_round_host
    size_t round_bytes = 0;
    int sm_count = 0;
    cudaStream_t copy_stream = nullptr;   // uploads of he_round_host, overlapped with compute
    cudaStream_t down_stream = nullptr;   // downloads of he_round_host (PCIe carries both directions at once)
    cudaEvent_t ev_ready[2] = {nullptr, nullptr}, ev_free[2] = {nullptr, nullptr};
    cudaEvent_t ev_chunk = nullptr;       // a chunk's result is ready for download
};

struct he_keys {
    uint32_t magic;
    he_ctx *ctx;
    fedhe::KeysDev dev;
    void *storage;
    bool is_share = false;   // a party's share of the secret (no public key, no small secret)
};

struct he_mask {
    uint32_t magic;
    size_t P, k;
    uint32_t *idx;       // [k] ascending
    uint32_t *bits;      // [ceil(P/32)] bit i of word i/32 set if parameter i is encrypted
    uint32_t *wpre;      // [ceil(P/32)] number of encrypted parameters before the word
};

namespace fedhe {
constexpr uint32_t CTX_MAGIC = 0x48454358u, KEYS_MAGIC = 0x48454b59u, MASK_MAGIC = 0x48454d4bu;
}
