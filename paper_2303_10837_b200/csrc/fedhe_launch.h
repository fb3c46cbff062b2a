// Launch wrappers of the CUDA kernels (implemented in fedhe_transform.cu, fedhe_slots.cu, fedhe_encrypt.cu, fedhe_server.cu, fedhe_decrypt.cu and fedhe_mask.cu),
// called by the C ABI in fedhe_api.cu.  All of them enqueue work on `s` and
// return the launch status; none synchronises.
#pragma once

#include "fedhe_internal.cuh"

namespace fedhe {

uint64_t launch_count();

// In-place negacyclic transforms of `npoly` polynomials.  Polynomial p, limb
// l (0 <= l < nlimbs, using prime limb0 + l) starts at data + p*poly_stride
// + l*N.  Forward input may lie in [0, 4q), inverse input in [0, 2q);
// outputs are canonical.
cudaError_t launch_ntt(const CtxDev &c, bool forward, uint64_t *data, size_t npoly, size_t poly_stride,
                       uint32_t limb0, uint32_t nlimbs, cudaStream_t s);

// keygen pieces: tmp is uint64 [3][L][N]
cudaError_t launch_keygen_sample(const CtxDev &c, uint64_t seed, int8_t *s8, uint64_t *tmp, cudaStream_t s);
cudaError_t launch_keygen_combine(const CtxDev &c, const uint64_t *tmp, tw_t *pk0_hat, tw_t *pk1_hat,
                                  tw_t *s_hat, cudaStream_t s);
cudaError_t launch_extract_values(const tw_t *src, uint64_t *dst, size_t count, cudaStream_t s);

// slot transform.  cplx: scratch of T*n double2, used only when n > 8192
cudaError_t launch_encode(const CtxDev &c, const float *sel, size_t T, double2 *cplx, int64_t *m,
                          cudaStream_t s);
cudaError_t launch_decode(const CtxDev &c, const int64_t *d, size_t T, double2 *cplx, double *z,
                          cudaStream_t s);

// Encode + encrypt ciphertexts t0 .. t0+T-1 (sel and ct point at the first of
// them).  `work` is scratch of encrypt_work_bytes() bytes: for N <= 2^14 N words
// per thread block of the fused kernel (the block's encoded message), for
// longer rings the encoded messages of all T ciphertexts and the encoder's
// complex buffer.  n_sm: the device's SM count.
size_t encrypt_work_bytes(const CtxDev &c, int n_sm, size_t T, bool ntt_out);
cudaError_t launch_encrypt(const CtxDev &c, const KeysDev &k, const float *sel, void *work, int n_sm,
                           uint32_t t0, size_t T, uint64_t seed, uint32_t client, uint64_t *ct,
                           cudaStream_t s);

// the same with every limb polynomial of the result in the transform domain
cudaError_t launch_encrypt_ntt(const CtxDev &c, const KeysDev &k, const float *sel, void *work, int n_sm,
                               uint32_t t0, size_t T, uint64_t seed, uint32_t client, uint64_t *ct,
                               cudaStream_t s);

// ptrs: device array of C ciphertext pointers; wtab: device [C][L] weights
cudaError_t launch_aggregate(const CtxDev &c, const uint64_t *const *ptrs, const tw_t *wtab, int C,
                             size_t T, uint64_t *out, cudaStream_t s);
// transform-domain ciphertexts in and out; scratch: uint64 [T][2][L][N]
cudaError_t launch_aggregate_ntt(const CtxDev &c, const uint64_t *const *ptrs, const tw_t *wtab, int C,
                                 size_t T, uint64_t *scratch, uint64_t *out, cudaStream_t s);
// aligned16: every client's pointer is 16-byte aligned (the caller knows the host copies)
// the clients' weighted sum on all L limbs without the rescale, and the rescale of a sum of such sums
cudaError_t launch_aggregate_partial(const CtxDev &c, const uint64_t *const *ptrs, const tw_t *wtab, int C,
                                     size_t T, uint64_t *out, cudaStream_t s);
cudaError_t launch_rescale_partial_sum(const CtxDev &c, const uint64_t *const *parts, int P, size_t T,
                                       uint64_t *out, cudaStream_t s);
cudaError_t launch_plain_aggregate(const float *const *ptrs, const double *alpha, int C, size_t len,
                                   double *out, bool aligned16, cudaStream_t s);

// scratch: uint64 [T][N]; on return it holds the centred integers as int64
cudaError_t launch_decrypt(const CtxDev &c, const KeysDev &k, const uint64_t *ct, uint32_t level,
                           size_t T, uint64_t *scratch, cudaStream_t s);

// the same for a transform-domain ciphertext
cudaError_t launch_decrypt_ntt(const CtxDev &c, const KeysDev &k, const uint64_t *ct, uint32_t level,
                               size_t T, uint64_t *scratch, cudaStream_t s);

// fused decrypt + decode for N <= 2^14 (no scratch): z double [T][n];
// ntt_in: the ciphertext is in the transform domain
cudaError_t launch_decrypt_fused(const CtxDev &c, const KeysDev &k, const uint64_t *ct, uint32_t level,
                                 size_t T, bool ntt_in, double *z, cudaStream_t s);

// two-party threshold decryption.  tmp: uint64 [2][L][N] (shares as residues)
cudaError_t launch_threshold_split(const CtxDev &c, const int8_t *s8, uint64_t seed, uint64_t *tmp,
                                   cudaStream_t s);
cudaError_t launch_share_tables(const CtxDev &c, const uint64_t *share_hat, tw_t *s_hat, cudaStream_t s);
// part: uint64 [T][N], work space and result (canonical residues mod q_0)
cudaError_t launch_partial_decrypt(const CtxDev &c, const KeysDev &share, uint32_t party, const uint64_t *ct,
                                   uint32_t level, size_t T, uint64_t seed, uint32_t bits, uint64_t *part,
                                   cudaStream_t s);
struct PartPtrs { const uint64_t *p[8]; };
cudaError_t launch_threshold_combine(const CtxDev &c, const uint64_t *ct, uint32_t level, const PartPtrs &parts,
                                     int nparts, size_t T, int64_t *d, cudaStream_t s);

// context-owned work space for T ciphertexts (2 * T * N words); implemented in fedhe_api.cu
int ctx_workspace(he_ctx *ctx, size_t T, void **out);

// mask construction (blocks of MASK_BLOCK consecutive parameters)
constexpr uint32_t MASK_BLOCK = 4096;
// progress of the radix selection, in device memory: the key prefix found so far (tau after
// the last step) and how many keys are still to be covered (after the last step: how many keys
// equal to tau belong to the mask)
struct SelectState { uint32_t prefix, need; };
cudaError_t launch_key_histogram(const float *score, size_t P, const SelectState *state, int prefix_bits,
                                 int digit_bits, int n_sm, uint32_t *hist, cudaStream_t s);
cudaError_t launch_radix_pick(const uint32_t *hist, int digit_bits, SelectState *state, cudaStream_t s);
cudaError_t launch_mask_count_eq(const float *score, size_t P, const SelectState *state, uint32_t *blk_eq,
                                 cudaStream_t s);
// in-place exclusive scan of a[0..count); the grand total goes to *total
cudaError_t launch_scan(uint32_t *a, size_t count, uint32_t *total, cudaStream_t s);
cudaError_t launch_mask_select(const float *score, size_t P, const SelectState *state,
                               const uint64_t *ranges, uint32_t nranges, const uint32_t *blk_eq_prefix,
                               uint32_t *bits, uint32_t *blk_sel, cudaStream_t s);
cudaError_t launch_mask_write(size_t P, const uint32_t *bits, const uint32_t *blk_sel_prefix,
                              uint32_t *wpre, uint32_t *idx, cudaStream_t s);

cudaError_t launch_pack(const he_mask *mask, const float *x, size_t P, size_t k, size_t padded,
                        float *sel, float *rest, cudaStream_t s);
cudaError_t launch_unpack(const he_mask *mask, const double *z, const double *rest_avg, size_t P,
                          double *w_glob, cudaStream_t s);

}  // namespace fedhe
