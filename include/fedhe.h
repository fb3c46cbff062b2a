/*
 * fedhe.h -- C ABI of the B200 (sm_100a) library for the hot path of FedML-HE
 * secure aggregation: selective-encryption mask, CKKS packing/encoding,
 * public-key encryption, server-side weighted ciphertext sum with rescale,
 * decryption/decoding and merge with the plaintext-averaged remainder.
 *
 * The entry points follow the paper's statement of the problem:
 *   Algorithm 1 ("HE-Based Federated Aggregation"), the aggregation equation
 *   [W_glob] = sum_i a_i [[M (.) W_i]] + sum_i a_i ((1-M) (.) W_i), "Step 2"
 *   of Selective Parameter Encryption (mask = ratio p of the most sensitive
 *   parameters), and the framework API table (key_gen, enc, he_aggregate,
 *   dec; flatten/reshape stay with the caller).
 *
 * Conventions
 *   - Every call returns an int: HE_OK (0) or a negative HE_ERR_* code; no
 *     exception crosses this boundary.  he_strerror() names a code.
 *   - "dev" pointers are device pointers on the context's GPU, owned by the
 *     caller, never freed by the library; "host" pointers are ordinary host
 *     memory.  Handles (he_ctx, he_keys, he_mask) are owned by the library
 *     and released by the matching *_destroy.
 *   - Alignment: every dev pointer to uint64 words (ciphertexts, aggregates,
 *     partial decryptions, exported keys, the polynomials of he_ntt_*) must be
 *     16-byte aligned, because the kernels move two words per access; a
 *     pointer that is not is refused with HE_ERR_INVALID_ARG before anything is
 *     launched.  float, double, int64 and index buffers need only their
 *     natural alignment (the kernels fall back to narrower accesses).
 *   - The library cannot see how large a caller's buffer is: every size below
 *     is a requirement on the caller (the Python binding checks them).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls are asynchronous on it unless stated otherwise.  A context keeps
 *     library-owned work buffers; calls that share a context must be issued
 *     on one stream at a time.  A call that needs more work space than the
 *     context holds (he_encode, he_encrypt*, he_decrypt* on rings above
 *     N = 16384, he_threshold_combine, he_weighted_aggregate_ntt,
 *     he_select_mask*, he_round_host with a larger problem than before) frees
 *     and reallocates it, which synchronises the whole device once;
 *     he_ctx_reserve does that ahead of time.
 *   - Kernels never trap or assert.  A numeric anomaly (an encoded
 *     coefficient of magnitude >= 2^62, or a non-finite input) sets a sticky
 *     status word read by he_ctx_status().
 *   - Ring R = Z[X]/(X^N+1), N a power of two, RNS primes q_0..q_{L-1} (all
 *     of them ciphertext limbs; the rescale drops q_{L-1}); n = N/2 real
 *     slots per ciphertext; scale Delta = 2^log2_delta.
 *   - Ciphertext layout: uint64 [T][2][level][N], coefficient domain, natural
 *     coefficient order, canonical residues in [0, q_j); level = L for fresh
 *     ciphertexts and L-1 after he_weighted_aggregate.
 */
#ifndef FEDHE_H
#define FEDHE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HE_MAX_LIMBS 16
#define HE_MAX_CLIENTS 256

enum {
    HE_OK = 0,
    HE_ERR_INVALID_ARG = -1, /* null pointer, zero size, k > P, bad handle */
    HE_ERR_PARAMS = -2,      /* N, L, primes or scale not usable */
    HE_ERR_ALLOC = -3,       /* device or host allocation failed */
    HE_ERR_CUDA = -4,        /* a CUDA runtime call failed */
    HE_ERR_OVERFLOW = -5,    /* status: an encoded coefficient left the range */
    HE_ERR_LEVEL = -6,       /* operation needs a level the context lacks */
    HE_ERR_SIZE = -7         /* size beyond what the call supports */
};

typedef struct he_ctx he_ctx;
typedef struct he_keys he_keys;
typedef struct he_mask he_mask;

/* Crypto context = the public configuration every party holds (Algorithm 1,
 * key generation; the server receives only this). */
typedef struct he_params {
    uint32_t N;                  /* ring degree: power of two, 8192..65536 */
    uint32_t L;                  /* number of RNS primes, 2..HE_MAX_LIMBS */
    uint64_t q[HE_MAX_LIMBS];    /* distinct primes < 2^61 with q = 1 mod 2N */
    int32_t log2_delta;          /* scale bits, 1 <= log2_delta, 2^log2_delta < q_0 / 4 */
} he_params;

const char *he_strerror(int code);

/* Creates a context on the current CUDA device: validates the parameters
 * (HE_ERR_PARAMS), builds the root/twiddle tables on the host and uploads
 * them.  Synchronous. */
int he_ctx_create(const he_params *params, he_ctx **out);
int he_ctx_destroy(he_ctx *ctx);
/* Synchronises the device, returns the sticky status (HE_OK or
 * HE_ERR_OVERFLOW) in *status and clears it. */
int he_ctx_status(he_ctx *ctx, int *status);
/* Pre-sizes the library-owned work buffers for encryptions/decryptions of up
 * to max_k encrypted parameters so that later calls allocate nothing.
 * Synchronous. */
int he_ctx_reserve(he_ctx *ctx, size_t max_k);

size_t he_slots(const he_ctx *ctx);                       /* n = N/2 */
size_t he_num_ct(const he_ctx *ctx, size_t k);            /* T = ceil(k / n): a short vector still costs a ciphertext */
size_t he_ct_words(const he_ctx *ctx, uint32_t level);    /* 2 * level * N uint64 words per ciphertext */

/* HE.KeyGen (Algorithm 1, first step; API table "key_gen").  s uniform
 * ternary, a_j uniform mod q_j, e discrete Gaussian (sigma 3.2), all from
 * Philox4x32-10 streams of `seed`;  pk = (-a s + e, a).  Both keys stay on
 * the device inside the handle. */
int he_keygen(he_ctx *ctx, uint64_t seed, he_keys **out, void *stream);
int he_keys_destroy(he_keys *keys);
/* Writes the public key (dev uint64 [2][L][N], coefficient domain, canonical)
 * and/or the secret key (dev int8 [N], values -1,0,1); either may be NULL. */
int he_keys_export(he_ctx *ctx, const he_keys *keys, uint64_t *pk_dev, int8_t *s_dev, void *stream);

/* Select(., p) of Algorithm 1 / "Step 2": the k parameters with the highest
 * sensitivity score.  key(score) = its fp32 bit pattern if the sign bit is
 * clear and it is not NaN, else 0; order by key descending, index ascending;
 * the first k form the mask.  score: dev float[P], P < 2^32, 0 <= k <= P.
 * Synchronous (the result sizes are needed on the host).  The mask's device
 * buffers come from a per-device memory pool that the library creates on
 * first use and keeps until the process ends; he_mask_destroy returns them
 * to the pool, which holds at most 256 MiB of unused memory. */
int he_select_mask(he_ctx *ctx, const float *score_dev, size_t P, size_t k, he_mask **out, void *stream);
/* Variant for the paper's empirical selection recipe (the top-p most
 * sensitive parameters as well as whole layers, e.g. the first and last):
 * the mask is the union of the top-k set above and of the half-open index
 * ranges [ranges[2i], ranges[2i+1]) (host array, at most 64 ranges, each
 * within [0, P]); its final size is reported by he_mask_indices. */
int he_select_mask_ranges(he_ctx *ctx, const float *score_dev, size_t P, size_t k,
                          const uint64_t *ranges_host, size_t num_ranges, he_mask **out, void *stream);
/* Selected indices, ascending: dev uint32 [k]; pointer owned by the mask. */
int he_mask_indices(const he_mask *mask, const uint32_t **idx_dev, size_t *k);
/* Copies the k selected indices into a caller-owned buffer: dev uint32 [k]. */
int he_mask_copy_indices(const he_mask *mask, uint32_t *out_dev, void *stream);
int he_mask_destroy(he_mask *mask);

/* Client side of  [W_i] = Enc(pk, M (.) W_i) + (1-M) (.) W_i : gathers the
 * masked parameters into slot order and compacts the complement.
 *   x: dev float[P];  sel: dev float[T*n], entries k..T*n-1 are zeroed;
 *   rest: dev float[P-k] (ascending index order), may be NULL when mask is
 *   NULL.  mask == NULL means full encryption (k = P). */
int he_pack(he_ctx *ctx, const he_mask *mask, const float *x_dev, size_t P, float *sel_dev,
            float *rest_dev, void *stream);

/* CKKS encoding alone (parity hook): m = round(Delta * sigma^{-1}(z)) for the
 * T = ceil(k/n) slot vectors of sel (dev float[T*n]); m: dev int64 [T][N]. */
int he_encode(he_ctx *ctx, const float *sel_dev, size_t k, int64_t *m_dev, void *stream);

/* HE.Enc(pk, .) of Algorithm 1 (API table "enc"): encodes and encrypts the T
 * slot vectors of sel.  Ciphertext t of client `client_id` draws u (ternary),
 * e0, e1 (Gaussian) from Philox streams of (seed, t, client_id):
 *   c0 = pk0 u + e0 + m,  c1 = pk1 u + e1  (mod q_j).
 * ct: dev uint64 [T][2][L][N].  A (seed, client_id, t) triple must not be
 * reused across rounds. */
int he_encrypt(he_ctx *ctx, const he_keys *keys, const float *sel_dev, size_t k, uint64_t seed,
               uint32_t client_id, uint64_t *ct_dev, void *stream);

/* Same for the ciphertext indices t_begin .. t_begin+t_count-1 only (a caller
 * that streams a large model in chunks): sel points at the slots of
 * ciphertext t_begin, ct at uint64 [t_count][2][L][N]; the Philox streams are
 * those of the absolute index, so chunked and whole encryption agree. */
int he_encrypt_range(he_ctx *ctx, const he_keys *keys, const float *sel_dev, size_t t_begin, size_t t_count,
                     uint64_t seed, uint32_t client_id, uint64_t *ct_dev, void *stream);

/* Server step  sum_i a_i [[M (.) W_i]]  with plaintext weights and one
 * multiplicative level (API table "he_aggregate"): W_i = rint(a_i q_{L-1}) as
 * a constant polynomial, acc = sum_i W_i ct_i mod q_j, then the rescale by
 * q_{L-1} with rounding, which returns exactly to scale Delta.
 *   cts: host array of C dev pointers, each uint64 [T][2][L][N];
 *   alpha: host double[C] (caller normalises: sum = 1), 1 <= C <= HE_MAX_CLIENTS;
 *   agg: dev uint64 [T][2][L-1][N]. */
int he_weighted_aggregate(he_ctx *ctx, const uint64_t *const *cts_host, const double *alpha_host,
                          int C, size_t T, uint64_t *agg_dev, void *stream);

/* The same server step in two halves, for a server whose clients' ciphertexts
 * sit on several GPUs (Algorithm 1's aggregation is a sum over clients, so it
 * splits over any partition of them).  he_weighted_partial gives
 *   partial = sum over the C given clients of W_i ct_i mod q_j
 * on all L limbs, canonical residues, dev uint64 [T][2][L][N], no rescale;
 * alpha are the clients' weights of the WHOLE round (normalised over all
 * clients, not over this subset).  The caller adds the partial sums of all
 * subsets word by word as plain 64-bit integers (e.g. a reduce-scatter with a
 * sum over uint64/int64) -- at most floor(2^64 / max_j q_j) of them, 16 for
 * 60-bit primes -- and he_rescale_partial_sum reduces that sum modulo every
 * q_j and applies the rescale:  agg, dev uint64 [T][2][L-1][N], is then word
 * for word what he_weighted_aggregate gives on all clients at once.
 * `parts` is the number of partial sums that were added (HE_ERR_SIZE if that
 * many could overflow 64 bits). */
int he_weighted_partial(he_ctx *ctx, const uint64_t *const *cts_host, const double *alpha_host, int C, size_t T,
                        uint64_t *partial_dev, void *stream);
int he_rescale_partial_sum(he_ctx *ctx, const uint64_t *sum_dev, uint32_t parts, size_t T, uint64_t *agg_dev,
                           void *stream);
/* The same without a separate addition: parts is a host array of P dev
 * pointers, each a result of he_weighted_partial for the same T ciphertext
 * indices (uint64 [T][2][L][N]); the kernel adds them while it reads.  The
 * buffers are read with plain loads only, so they may be peer-mapped memory
 * that he_weighted_partial calls on other GPUs wrote into (each GPU calls
 * he_weighted_partial once per owner, on that owner's range of ciphertext
 * indices, with partial_dev inside the owner's buffer); the caller orders
 * those writes before this call.  1 <= P <= min(HE_MAX_CLIENTS,
 * floor(2^64 / max_j q_j)). */
int he_rescale_partial_parts(he_ctx *ctx, const uint64_t *const *parts_host, int P, size_t T, uint64_t *agg_dev,
                             void *stream);

/* Plaintext part  sum_i a_i ((1-M) (.) W_i): out[k] = sum_i alpha_i * rest_i[k]
 * in fp64, client order, separate multiply and add.
 *   rests: host array of C dev pointers float[len]; out: dev double[len]. */
int he_plain_aggregate(he_ctx *ctx, const float *const *rests_host, const double *alpha_host, int C,
                       size_t len, double *out_dev, void *stream);

/* HE.Dec(sk, .) of Algorithm 1 (API table "dec") on ciphertexts of level L-1:
 * d = c0 + c1 s mod q_0 centred, decoded to the n slots.
 *   agg: dev uint64 [T][2][L-1][N];  z: dev double[T*n]. */
int he_decrypt(he_ctx *ctx, const he_keys *keys, const uint64_t *agg_dev, size_t T, double *z_dev,
               void *stream);
/* Same with an explicit level (1..L) so that fresh ciphertexts can be opened. */
int he_decrypt_level(he_ctx *ctx, const he_keys *keys, const uint64_t *ct_dev, uint32_t level, size_t T,
                     double *z_dev, void *stream);

/* Transform-domain wire format (an alternative to the coefficient-domain
 * ciphertexts above; the paper leaves the ciphertext representation to its HE
 * library, Section 3.2 / API table).  Same layout and sizes, but every limb
 * polynomial is stored as its negacyclic transform
 *   A^[k] = sum_j a_j psi^((2 brev(k) + 1) j) mod q,
 * psi the smallest primitive 2N-th root of unity, brev over log2 N bits, i.e.
 * exactly he_ntt_forward of the coefficient-domain ciphertext.  The three
 * calls mirror he_encrypt, he_weighted_aggregate and he_decrypt_level:
 * encryption costs the same 3L limb transforms (all forward), the server's
 * weighted sum stays pointwise but its rescale needs 2L limb transforms per
 * ciphertext index (last limb back, rounding term forward for every other
 * limb), decryption saves one transform.  Arguments, ownership and errors as
 * for the coefficient-domain calls; mixing the two formats in one call is not
 * detected (the bytes are valid residues either way). */
int he_encrypt_ntt(he_ctx *ctx, const he_keys *keys, const float *sel_dev, size_t k, uint64_t seed,
                   uint32_t client_id, uint64_t *ct_dev, void *stream);
int he_weighted_aggregate_ntt(he_ctx *ctx, const uint64_t *const *cts_host, const double *alpha_host,
                              int C, size_t T, uint64_t *agg_dev, void *stream);
int he_decrypt_level_ntt(he_ctx *ctx, const he_keys *keys, const uint64_t *ct_dev, uint32_t level, size_t T,
                         double *z_dev, void *stream);

/* (No counterpart in the paper.)  Decryption for callers that must not
 * allocate: a process that has given all free device memory to its own pool,
 * or a latency-critical loop that cannot take the device-wide synchronisation
 * of cudaMalloc/cudaFree.  Same arguments and result as he_decrypt.  It runs
 * the multi-kernel decryption path (the one he_decrypt takes on rings above
 * N = 16384, where it may grow the context's work buffer), with the work
 * buffer a fixed 16 MiB array inside the library image (present on every GPU
 * that loads the library until the process exits), so the call issues no
 * cudaMalloc, cudaFree or allocating library routine whatever kernels the
 * library picks.  On the rings it accepts, he_decrypt itself is one fused
 * kernel without a work buffer, allocates nothing either and is faster; this
 * call costs about three more passes over T * N words.
 *   A cudaDeviceReset by the caller invalidates the cached address of the
 *   array together with every handle of the library.
 *   Limits: N <= 16384 and T * N <= HE_NOALLOC_MAX_WORDS (T <= 128 at
 *   N = 16384, T <= 256 at N = 8192); anything larger returns HE_ERR_SIZE.
 *   The context's GPU must be the current device (HE_ERR_INVALID_ARG).
 *   The first call on a device looks up the array's device address
 *   (cudaGetSymbolAddress), which is also the latest moment at which the CUDA
 *   runtime loads the library's device image, array included, on that GPU;
 *   make that first call before any stream capture.
 *   Every call on a device shares the one array, which keeps the previous
 *   call's contents (none of it needs to start at zero); calls that overlap
 *   on the GPU, e.g. on two streams, race on it. */
#define HE_NOALLOC_MAX_WORDS (1u << 21)
int he_decrypt_noalloc(he_ctx *ctx, const he_keys *keys, const uint64_t *agg_dev, size_t T, double *z_dev,
                       void *stream);

/* Client merge  Dec(sk, M (.) [W_glob]) + (1-M) (.) [W_glob]:
 * w_glob[idx[r]] = z[r], complement positions take rest_avg in order.
 *   z: dev double[>= k]; rest_avg: dev double[P-k] (NULL if mask NULL);
 *   w_glob: dev double[P]. */
int he_unpack(he_ctx *ctx, const he_mask *mask, const double *z_dev, const double *rest_avg_dev,
              size_t P, double *w_glob_dev, void *stream);

/* Two-party threshold decryption (paper appendix "Key Management And
 * Threshold HE": every party holds a share of the secret key, decrypts the
 * final ciphertext partially, and the partial results are merged).  The
 * interactive key agreement is out of scope: a dealer splits an existing
 * secret additively, share0 uniform mod q_j (Philox stream of `seed`),
 * share1 = s - share0.  The share handles are released with he_keys_destroy
 * and are accepted only by he_partial_decrypt.  Synchronous. */
int he_threshold_split(he_ctx *ctx, const he_keys *keys, uint64_t seed, he_keys **share0, he_keys **share1,
                       void *stream);
/* Party `party`'s partial decryption of T ciphertexts of `level` limbs:
 * part = c1 * share + E (mod q_0), E uniform in [-2^smudge_bits, 2^smudge_bits)
 * per coefficient from the Philox stream of (seed, t, party); smudge_bits <= 40.
 *   ct: dev uint64 [T][2][level][N]; part: dev uint64 [T][N], canonical residues. */
int he_partial_decrypt(he_ctx *ctx, const he_keys *share, uint32_t party, const uint64_t *ct_dev, uint32_t level,
                       size_t T, uint64_t seed, uint32_t smudge_bits, uint64_t *part_dev, void *stream);
/* Merge: d = c0 + sum of the parts (mod q_0), centred and decoded like
 * he_decrypt.  parts: host array of nparts (<= 8) dev pointers uint64 [T][N];
 * z: dev double[T*n]. */
int he_threshold_combine(he_ctx *ctx, const uint64_t *ct_dev, uint32_t level, const uint64_t *const *parts_host,
                         int nparts, size_t T, double *z_dev, void *stream);

/* Batched negacyclic transforms on raw residues (kernel sweep; no paper
 * counterpart): polys dev uint64 [B][L][N] in place, canonical residues in,
 * canonical residues out.  Forward: A[k] = sum_j a_j psi^((2 brev(k)+1) j)
 * mod q (bit-reversed output order), psi the smallest primitive 2N-th root
 * of unity mod q; inverse undoes it. */
int he_ntt_forward(he_ctx *ctx, uint64_t *polys_dev, size_t B, void *stream);
int he_ntt_inverse(he_ctx *ctx, uint64_t *polys_dev, size_t B, void *stream);

/* One whole round from host memory, the call an application makes when its
 * updates live on the host: copies every client's update to the device,
 * runs pack -> encrypt (all clients) -> weighted aggregate + plaintext
 * remainder -> decrypt -> unpack in chunks of ciphertext indices, and copies
 * the merged global model back.
 *   xs: host array of C host pointers float[P]; alpha: host double[C];
 *   mask: NULL = full encryption; w_glob: host double[P].
 * Synchronous; allocates its device buffers through the context.  Uploads and
 * downloads run on two streams of their own beside the arithmetic: with full
 * encryption the slots of the next chunk of ciphertext indices (a contiguous
 * piece of every update) go up while the current chunk is computed, and the
 * decoded slots of a finished chunk go home while the next is computed; with
 * a mask the whole update of the next client goes up while the current one is
 * packed and encrypted.  They overlap the arithmetic only when xs and w_glob
 * are page-locked (pinned) host memory; pageable memory is correct but
 * serialises.  With full encryption parts of w_glob are written
 * before the call returns; after an error return its contents are unspecified.
 * Bad arguments (a NULL xs[i], a weight outside [0, 1]) are refused before
 * anything is queued.  On every return, error or not, all streams have been
 * waited for: no copy is still reading xs or writing w_glob. */
int he_round_host(he_ctx *ctx, const he_keys *keys, const he_mask *mask, const float *const *xs_host,
                  const double *alpha_host, int C, size_t P, uint64_t enc_seed, double *w_glob_host,
                  void *stream);

/* Number of kernel launches issued by this library since it was loaded. */
uint64_t he_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FEDHE_H */
