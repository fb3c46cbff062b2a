/*
 * fedhe_oracle.h -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * Plain, slow, single-purpose CPU restatement of the FedML-HE secure
 * aggregation round (paper Algorithm 1 and the aggregation equation of the
 * section "Algorithm for HE-Based Federated Aggregation"), with CKKS (the
 * scheme the paper's preliminaries name) written out in RNS form.  It exists
 * so that the CUDA library can be checked coefficient by coefficient.  It
 * shares no code, table generator or header with the CUDA path.  Only tests,
 * the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Every function follows the algorithm step by step: no blocking, fusion or
 * reordering.  Integer arithmetic is exact (unsigned __int128 products and
 * the % operator); floating point is IEEE binary64 with no contraction
 * (compile with -ffp-contract=off).
 *
 * Pins (tests marked "not gpu"): every function below is pinned by a test
 * against something other than itself (brute-force definitions in Python
 * big integers, the published Philox known-answer vectors, a 60-digit
 * recomputation of the Gaussian table, closed forms of the canonical
 * embedding, big-integer CRT, full sorts).  No function is "parity unpinned".
 */
#ifndef FEDHE_ORACLE_H
#define FEDHE_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_MAX_L 16

typedef struct orc_ctx orc_ctx;

/* ---- modular arithmetic and parameter checks ---------------------------- */
uint64_t orc_mulmod(uint64_t a, uint64_t b, uint64_t q);
uint64_t orc_powmod(uint64_t a, uint64_t e, uint64_t q);
uint64_t orc_invmod(uint64_t a, uint64_t q);              /* q prime */
int orc_is_prime(uint64_t q);                              /* deterministic Miller-Rabin */
/* smallest psi in [1,q) with psi^N = -1 (mod q); 0 if q != 1 mod 2N */
uint64_t orc_min_root_2n(uint64_t q, uint32_t N);

/* ---- context: ring degree N, L primes, scale 2^log2_delta ---------------- */
/* returns NULL if N is not a power of two in [4, 65536], L out of range, a
 * modulus is not prime, not 1 mod 2N, repeated, or >= 2^62. */
orc_ctx *orc_ctx_create(uint32_t N, uint32_t L, const uint64_t *q, int log2_delta);
void orc_ctx_destroy(orc_ctx *c);
uint64_t orc_ctx_psi(const orc_ctx *c, uint32_t limb);
/* copies the 2N (cos, sin) pairs of exp(2 pi i t / 2N), t < 2N */
void orc_twiddle_table(const orc_ctx *c, double *out);

/* ---- negacyclic transforms ---------------------------------------------- */
/* forward: A[k] = sum_j a_j psi^{(2 brev(k)+1) j} mod q, in place */
void orc_ntt_forward(const orc_ctx *c, uint32_t limb, uint64_t *a);
void orc_ntt_inverse(const orc_ctx *c, uint32_t limb, uint64_t *a);
void orc_negacyclic_mul_ntt(const orc_ctx *c, uint32_t limb, const uint64_t *a,
                            const uint64_t *b, uint64_t *out);
/* O(N^2) definition of the product in Z_q[X]/(X^N+1) */
void orc_negacyclic_mul_schoolbook(uint32_t N, uint64_t q, const uint64_t *a,
                                   const uint64_t *b, uint64_t *out);

/* ---- randomness: Philox4x32-10 (Salmon et al., SC'11) -------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
void orc_gauss_table(uint64_t out[38]);  /* thresholds T[x], x = -19..18, sigma 3.2 */
/* tags: 1 secret s, 2 public a, 3 key error, 4 enc u, 5 enc e0, 6 enc e1 */
void orc_sample_ternary(uint64_t seed, uint32_t t, uint32_t client, uint32_t tag,
                        uint32_t N, int8_t *out);
void orc_sample_gauss(uint64_t seed, uint32_t t, uint32_t client, uint32_t tag,
                      uint32_t N, int8_t *out);
void orc_sample_uniform(uint64_t seed, uint32_t t, uint32_t client, uint32_t tag,
                        uint32_t limb, uint64_t q, uint32_t N, uint64_t *out);

/* ---- scheme ---------------------------------------------------------------- */
/* s[N] in {-1,0,1}; pk[2][L][N] coefficient domain, canonical residues */
void orc_keygen(const orc_ctx *c, uint64_t seed, int8_t *s, uint64_t *pk);
/* slots[n] (n = N/2) -> m[N]; returns 1 if some |m_k| >= 2^62, else 0 */
int orc_encode(const orc_ctx *c, const float *slots, int64_t *m);
void orc_encrypt_one(const orc_ctx *c, const uint64_t *pk, const int64_t *m,
                     uint64_t seed, uint32_t client, uint32_t t, uint64_t *ct);
/* sel[T*n] -> ct[T][2][L][N]; returns number of ciphertexts that overflowed */
int orc_encrypt(const orc_ctx *c, const uint64_t *pk, const float *sel, size_t T,
                uint64_t seed, uint32_t client, uint64_t *ct);
void orc_weights(const orc_ctx *c, const double *alpha, uint32_t C, uint64_t *W);
/* acc[T][2][L][N] = sum_i (W_i mod q_j) ct_i mod q_j */
void orc_weighted_sum(const orc_ctx *c, const uint64_t *const *cts, const uint64_t *W,
                      uint32_t C, size_t T, uint64_t *acc);
/* drop the last prime with rounding: out[T][2][L-1][N] */
void orc_rescale(const orc_ctx *c, const uint64_t *acc, size_t T, uint64_t *out);
void orc_plain_aggregate(const float *const *rests, const double *alpha, uint32_t C,
                         size_t len, double *out);
/* residues of c0 + c1 s on one limb of a ciphertext with `level` limbs */
void orc_decrypt_limb(const orc_ctx *c, const int8_t *s, const uint64_t *ct,
                      uint32_t level, uint32_t limb, uint64_t *out);
/* limb-0 decryption, centred: d[T][N] */
void orc_decrypt(const orc_ctx *c, const int8_t *s, const uint64_t *ct, uint32_t level,
                 size_t T, int64_t *d);
void orc_decode(const orc_ctx *c, const int64_t *d, double *z);

/* ---- two-party threshold decryption (appendix "Key Management And Threshold HE") ---- */
/* dealer split of the secret: share0[L][N] uniform mod q_j (stream tag 7),
 * share1 = s - share0 (mod q_j) */
void orc_threshold_split(const orc_ctx *c, const int8_t *s, uint64_t seed, uint64_t *share0,
                         uint64_t *share1);
/* smudging noise of `party` for ciphertext index t: uniform integers in
 * [-2^bits, 2^bits) from stream tag 8 */
void orc_sample_smudge(uint64_t seed, uint32_t t, uint32_t party, uint32_t bits, uint32_t N, int64_t *out);
/* partial decryption of one ciphertext on limb 0: c1 share + E (mod q_0);
 * share points at the party's [L][N] residues */
void orc_partial_decrypt(const orc_ctx *c, const uint64_t *share, uint32_t party, const uint64_t *ct,
                         uint32_t level, uint64_t seed, uint32_t t, uint32_t bits, uint64_t *out);
/* d = c0 + sum of the parts (mod q_0), centred */
void orc_threshold_combine(const orc_ctx *c, const uint64_t *ct, uint32_t level,
                           const uint64_t *const *parts, uint32_t nparts, int64_t *d);

/* ---- selective-encryption mask, packing ---------------------------------- */
/* indices of the k largest keys (ties: lower index first), ascending */
void orc_select_mask(const float *score, size_t P, size_t k, uint32_t *idx);
/* idx == NULL means full encryption (k = P). sel has T*n entries, rest P-k */
void orc_pack(const orc_ctx *c, const uint32_t *idx, size_t k, const float *x, size_t P,
              float *sel, float *rest);
void orc_unpack(const uint32_t *idx, size_t k, const double *z, const double *rest_avg,
                size_t P, double *w_glob);

/* ---- one whole round, for the timed CPU baseline ------------------------- */
/* xs[C][P] client updates; idx/k the mask (NULL = full); w_glob[P] out.
 * t_begin..t_end restricts the ciphertext indices processed (a bounded
 * sample); the plaintext remainder is aggregated only if do_rest != 0.
 * returns 0, or -1 on allocation failure. */
int orc_round(const orc_ctx *c, const float *const *xs, const double *alpha, uint32_t C,
              size_t P, const uint32_t *idx, size_t k, uint64_t key_seed, uint64_t enc_seed,
              size_t t_begin, size_t t_end, int do_rest, double *w_glob);
int orc_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
