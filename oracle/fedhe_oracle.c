/*
 * fedhe_oracle.c -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * Plain CPU restatement of the FedML-HE secure-aggregation round; see
 * fedhe_oracle.h for scope, rules and pins.  Passages followed:
 *   - Algorithm 1 (key generation, client encryption of M (.) W_i, server
 *     aggregation, client decryption and merge);
 *   - the aggregation equation  [W_glob] = sum_i a_i [[M (.) W_i]]
 *     + sum_i a_i ((1-M) (.) W_i)  with plaintext weights a_i and exactly one
 *     multiplicative level;
 *   - "Step 2" of Selective Parameter Encryption (mask = the ratio p of the
 *     most sensitive parameters);
 *   - the HE interface of the appendix figure (KeyGen, Enc, Eval, Dec), with
 *     CKKS as the scheme (appendix, "Homomorphic Encryption");
 *   - the packing behaviour (a short vector still costs a full ciphertext).
 * The paper does not spell out CKKS itself.  The readings taken here:
 * RNS over L word-sized primes q_0..q_{L-1} (all of them ciphertext limbs),
 * real values in n = N/2 slots ordered by the powers of 5, uniform ternary
 * secret and ephemeral keys, discrete Gaussian errors with sigma 3.2 on
 * [-19, 19] sampled from a 64-bit cumulative table, Philox4x32-10 streams
 * indexed by (seed; coefficient block, ciphertext, client, tag|limb<<8),
 * weights encoded as the constant polynomial rint(a_i q_{L-1}) so that the
 * rescale by q_{L-1} returns exactly to scale Delta, decryption from limb 0.
 */
#include "fedhe_oracle.h"

#include <math.h>
#include <quadmath.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef unsigned __int128 u128;

struct orc_ctx {
    uint32_t N, L, logN;
    int log2_delta;
    uint64_t q[ORC_MAX_L];
    uint64_t psi[ORC_MAX_L];
    uint64_t inv_n[ORC_MAX_L];
    uint64_t *psi_br[ORC_MAX_L];      /* psi^{brev(i)} , i < N */
    uint64_t *ipsi_br[ORC_MAX_L];     /* their inverses */
    double *tw;                        /* [2N][2] : cos, sin of 2 pi t / 2N */
};

/* ------------------------------------------------------------------------- */
/* modular arithmetic                                                         */
/* ------------------------------------------------------------------------- */

uint64_t orc_mulmod(uint64_t a, uint64_t b, uint64_t q) {
    return (uint64_t)(((u128)a * (u128)b) % (u128)q);
}

uint64_t orc_powmod(uint64_t a, uint64_t e, uint64_t q) {
    uint64_t r = 1 % q;
    a %= q;
    while (e) {
        if (e & 1) r = orc_mulmod(r, a, q);
        a = orc_mulmod(a, a, q);
        e >>= 1;
    }
    return r;
}

uint64_t orc_invmod(uint64_t a, uint64_t q) { return orc_powmod(a, q - 2, q); }

static uint64_t addmod(uint64_t a, uint64_t b, uint64_t q) {
    uint64_t s = a + b; /* a, b < q < 2^63: no wrap */
    return s >= q ? s - q : s;
}

static uint64_t submod(uint64_t a, uint64_t b, uint64_t q) { return a >= b ? a - b : a + q - b; }

/* residue in [0,q) of a signed integer */
static uint64_t from_signed(int64_t v, uint64_t q) {
    if (v >= 0) return (uint64_t)v % q;
    uint64_t a = (uint64_t)(-(v + 1)) + 1u; /* |v| without overflow at INT64_MIN */
    uint64_t r = a % q;
    return r ? q - r : 0;
}

int orc_is_prime(uint64_t n) {
    static const uint64_t bases[12] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    if (n < 2) return 0;
    for (int i = 0; i < 12; i++) {
        if (n == bases[i]) return 1;
        if (n % bases[i] == 0) return 0;
    }
    uint64_t d = n - 1;
    int r = 0;
    while ((d & 1) == 0) { d >>= 1; r++; }
    for (int i = 0; i < 12; i++) {
        uint64_t x = orc_powmod(bases[i], d, n);
        if (x == 1 || x == n - 1) continue;
        int comp = 1;
        for (int k = 1; k < r; k++) {
            x = orc_mulmod(x, x, n);
            if (x == n - 1) { comp = 0; break; }
        }
        if (comp) return 0;
    }
    return 1;
}

uint64_t orc_min_root_2n(uint64_t q, uint32_t N) {
    uint64_t two_n = 2ull * N;
    if ((q - 1) % two_n != 0) return 0;
    /* any element of order exactly 2N: x^((q-1)/2N) whose N-th power is -1 */
    uint64_t g = 0;
    for (uint64_t x = 2; x < q; x++) {
        uint64_t c = orc_powmod(x, (q - 1) / two_n, q);
        if (orc_powmod(c, N, q) == q - 1) { g = c; break; }
    }
    /* the primitive 2N-th roots are the odd powers of g: take the least */
    uint64_t g2 = orc_mulmod(g, g, q), cur = g, best = g;
    for (uint32_t k = 1; k < N; k++) {
        cur = orc_mulmod(cur, g2, q);
        if (cur < best) best = cur;
    }
    return best;
}

static uint32_t brev(uint32_t x, uint32_t bits) {
    uint32_t r = 0;
    for (uint32_t i = 0; i < bits; i++) r |= ((x >> i) & 1u) << (bits - 1 - i);
    return r;
}

/* ------------------------------------------------------------------------- */
/* context                                                                    */
/* ------------------------------------------------------------------------- */

/* cos and sin of 2 pi t / M rounded to binary64, using the eight-fold
 * symmetry so that exact values (0, 1) and mirror pairs come out exact */
static void unit_root(uint32_t t, uint32_t M, double *co, double *si) {
    uint32_t e = M / 8;         /* M >= 8 always here */
    uint32_t oct = t / e, r = t % e;
    /* angle within the octant, measured from the nearer axis */
    uint32_t a = (oct & 1) ? e - r : r;
    __float128 ang = (2.0Q * M_PIq * (__float128)a) / (__float128)M;
    double c = (double)cosq(ang), s = (double)sinq(ang);
    if (a == 0) { c = 1.0; s = 0.0; }
    double x, y;
    switch (oct) {
    case 0: x = c;  y = s;  break;
    case 1: x = s;  y = c;  break;
    case 2: x = -s; y = c;  break;
    case 3: x = -c; y = s;  break;
    case 4: x = -c; y = -s; break;
    case 5: x = -s; y = -c; break;
    case 6: x = s;  y = -c; break;
    default: x = c; y = -s; break;
    }
    *co = x + 0.0; /* turn -0.0 into +0.0 */
    *si = y + 0.0;
}

orc_ctx *orc_ctx_create(uint32_t N, uint32_t L, const uint64_t *q, int log2_delta) {
    if (N < 4 || N > 65536 || (N & (N - 1))) return NULL;
    if (L < 1 || L > ORC_MAX_L) return NULL;
    if (log2_delta < 1 || log2_delta > 60) return NULL;
    for (uint32_t j = 0; j < L; j++) {
        if (q[j] >= (1ull << 62) || !orc_is_prime(q[j]) || (q[j] - 1) % (2ull * N)) return NULL;
        for (uint32_t i = 0; i < j; i++)
            if (q[i] == q[j]) return NULL;
    }
    orc_ctx *c = (orc_ctx *)calloc(1, sizeof(orc_ctx));
    if (!c) return NULL;
    c->N = N; c->L = L; c->log2_delta = log2_delta;
    while ((1u << c->logN) < N) c->logN++;
    for (uint32_t j = 0; j < L; j++) {
        c->q[j] = q[j];
        c->psi[j] = orc_min_root_2n(q[j], N);
        c->inv_n[j] = orc_invmod(N, q[j]);
        c->psi_br[j] = (uint64_t *)malloc(sizeof(uint64_t) * N);
        c->ipsi_br[j] = (uint64_t *)malloc(sizeof(uint64_t) * N);
        uint64_t p = 1;
        for (uint32_t i = 0; i < N; i++) {          /* p = psi^i */
            uint32_t r = brev(i, c->logN);
            c->psi_br[j][r] = p;
            c->ipsi_br[j][r] = orc_invmod(p, q[j]);
            p = orc_mulmod(p, c->psi[j], q[j]);
        }
    }
    uint32_t M = 2 * N;
    c->tw = (double *)malloc(sizeof(double) * 2 * M);
    for (uint32_t t = 0; t < M; t++) unit_root(t, M, &c->tw[2 * t], &c->tw[2 * t + 1]);
    return c;
}

void orc_ctx_destroy(orc_ctx *c) {
    if (!c) return;
    for (uint32_t j = 0; j < c->L; j++) { free(c->psi_br[j]); free(c->ipsi_br[j]); }
    free(c->tw);
    free(c);
}

uint64_t orc_ctx_psi(const orc_ctx *c, uint32_t limb) { return c->psi[limb]; }

void orc_twiddle_table(const orc_ctx *c, double *out) {
    memcpy(out, c->tw, sizeof(double) * 4 * c->N);
}

/* ------------------------------------------------------------------------- */
/* negacyclic number-theoretic transform                                      */
/* ------------------------------------------------------------------------- */

/* Decimation in time with the powers of psi merged into the butterflies;
 * natural-order input, bit-reversed output. */
void orc_ntt_forward(const orc_ctx *c, uint32_t limb, uint64_t *a) {
    const uint64_t q = c->q[limb];
    const uint64_t *w = c->psi_br[limb];
    uint32_t t = c->N;
    for (uint32_t m = 1; m < c->N; m <<= 1) {
        t >>= 1;
        for (uint32_t i = 0; i < m; i++) {
            uint32_t j1 = 2 * i * t;
            uint64_t W = w[m + i];
            for (uint32_t j = j1; j < j1 + t; j++) {
                uint64_t U = a[j];
                uint64_t V = orc_mulmod(a[j + t], W, q);
                a[j] = addmod(U, V, q);
                a[j + t] = submod(U, V, q);
            }
        }
    }
}

/* exact inverse of the above: bit-reversed input, natural-order output */
void orc_ntt_inverse(const orc_ctx *c, uint32_t limb, uint64_t *a) {
    const uint64_t q = c->q[limb];
    const uint64_t *w = c->ipsi_br[limb];
    uint32_t t = 1;
    for (uint32_t m = c->N; m > 1; m >>= 1) {
        uint32_t h = m >> 1, j1 = 0;
        for (uint32_t i = 0; i < h; i++) {
            uint64_t W = w[h + i];
            for (uint32_t j = j1; j < j1 + t; j++) {
                uint64_t U = a[j], V = a[j + t];
                a[j] = addmod(U, V, q);
                a[j + t] = orc_mulmod(submod(U, V, q), W, q);
            }
            j1 += 2 * t;
        }
        t <<= 1;
    }
    for (uint32_t j = 0; j < c->N; j++) a[j] = orc_mulmod(a[j], c->inv_n[limb], q);
}

void orc_negacyclic_mul_ntt(const orc_ctx *c, uint32_t limb, const uint64_t *a,
                            const uint64_t *b, uint64_t *out) {
    uint32_t N = c->N;
    uint64_t *ta = (uint64_t *)malloc(sizeof(uint64_t) * N);
    uint64_t *tb = (uint64_t *)malloc(sizeof(uint64_t) * N);
    memcpy(ta, a, sizeof(uint64_t) * N);
    memcpy(tb, b, sizeof(uint64_t) * N);
    orc_ntt_forward(c, limb, ta);
    orc_ntt_forward(c, limb, tb);
    for (uint32_t j = 0; j < N; j++) ta[j] = orc_mulmod(ta[j], tb[j], c->q[limb]);
    orc_ntt_inverse(c, limb, ta);
    memcpy(out, ta, sizeof(uint64_t) * N);
    free(ta); free(tb);
}

void orc_negacyclic_mul_schoolbook(uint32_t N, uint64_t q, const uint64_t *a,
                                   const uint64_t *b, uint64_t *out) {
    for (uint32_t k = 0; k < N; k++) out[k] = 0;
    for (uint32_t i = 0; i < N; i++)
        for (uint32_t j = 0; j < N; j++) {
            uint64_t p = orc_mulmod(a[i] % q, b[j] % q, q);
            uint32_t k = i + j;
            if (k < N) out[k] = addmod(out[k], p, q);
            else out[k - N] = submod(out[k - N], p, q);   /* X^N = -1 */
        }
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 and the three samplers                                       */
/* ------------------------------------------------------------------------- */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;   /* round multipliers */
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;   /* key increments (Weyl) */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; r++) {
        uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* T[x] = floor(2^64 Pr[X <= x]), x = -19..18, for Pr[x] ~ exp(-x^2 / (2 3.2^2))
 * on the integers of [-19, 19] */
static const uint64_t GAUSS_T[38] = {
    0x0000000bd798c7acull, 0x00000053f5e234f7ull, 0x000001e24b89625aull, 0x000009adbc7900e1ull,
    0x00002d17ca1e3a82ull, 0x0000bf05ff772ee2ull, 0x0002e06843bbf95dull, 0x000a19062dceb033ull,
    0x00204c0ded173b17ull, 0x005e3163ffc656a8ull, 0x00fab6a7e614dfaeull, 0x0261b16e99bc14f8ull,
    0x054c69348bbc9867ull, 0x0acd276539458231ull, 0x143796b3c337f00bull, 0x22d43df09de40e7aull,
    0x37651d96aa4fb429ull, 0x51a5da2b40f1bff1ull, 0x700ad4bf5a6e80e2ull, 0x8ff52b40a5917f1dull,
    0xae5a25d4bf0e400eull, 0xc89ae26955b04bd6ull, 0xdd2bc20f621bf185ull, 0xebc8694c3cc80ff4ull,
    0xf532d89ac6ba7dceull, 0xfab396cb74436798ull, 0xfd9e4e916643eb07ull, 0xff05495819eb2051ull,
    0xffa1ce9c0039a957ull, 0xffdfb3f212e8c4e8ull, 0xfff5e6f9d2314fccull, 0xfffd1f97bc4406a2ull,
    0xffff40fa0088d11dull, 0xffffd2e835e1c57dull, 0xfffff6524386ff1eull, 0xfffffe1db4769da5ull,
    0xffffffac0a1dcb08ull, 0xfffffff428673853ull};

void orc_gauss_table(uint64_t out[38]) { memcpy(out, GAUSS_T, sizeof(GAUSS_T)); }

static void stream_block(uint64_t seed, uint32_t block, uint32_t t, uint32_t client,
                         uint32_t tag, uint32_t limb, uint32_t w[4]) {
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t ctr[4] = {block, t, client, tag | (limb << 8)};
    orc_philox4x32_10(ctr, key, w);
}

/* coefficient j: word j&3 of block j>>2, mapped to {-1,0,1} by floor(3 w / 2^32) - 1 */
void orc_sample_ternary(uint64_t seed, uint32_t t, uint32_t client, uint32_t tag,
                        uint32_t N, int8_t *out) {
    for (uint32_t j = 0; j < N; j++) {
        uint32_t w[4];
        stream_block(seed, j >> 2, t, client, tag, 0, w);
        out[j] = (int8_t)((int)(((uint64_t)w[j & 3] * 3u) >> 32) - 1);
    }
}

/* coefficient j: the 64-bit r made of words 2(j&1), 2(j&1)+1 of block j>>1;
 * value = -19 + #{x : r >= T[x]} */
void orc_sample_gauss(uint64_t seed, uint32_t t, uint32_t client, uint32_t tag,
                      uint32_t N, int8_t *out) {
    for (uint32_t j = 0; j < N; j++) {
        uint32_t w[4];
        stream_block(seed, j >> 1, t, client, tag, 0, w);
        uint64_t r = (uint64_t)w[2 * (j & 1)] | ((uint64_t)w[2 * (j & 1) + 1] << 32);
        int v = -19;
        for (int x = 0; x < 38; x++) v += (r >= GAUSS_T[x]);
        out[j] = (int8_t)v;
    }
}

/* coefficient j: the 128-bit value of block j, reduced mod q */
void orc_sample_uniform(uint64_t seed, uint32_t t, uint32_t client, uint32_t tag,
                        uint32_t limb, uint64_t q, uint32_t N, uint64_t *out) {
    for (uint32_t j = 0; j < N; j++) {
        uint32_t w[4];
        stream_block(seed, j, t, client, tag, limb, w);
        u128 v = (u128)w[0] | ((u128)w[1] << 32) | ((u128)w[2] << 64) | ((u128)w[3] << 96);
        out[j] = (uint64_t)(v % (u128)q);
    }
}

/* ------------------------------------------------------------------------- */
/* key generation (Algorithm 1, "Key Authority Generate Key")                 */
/* ------------------------------------------------------------------------- */

void orc_keygen(const orc_ctx *c, uint64_t seed, int8_t *s, uint64_t *pk) {
    uint32_t N = c->N, L = c->L;
    int8_t *e = (int8_t *)malloc(N);
    uint64_t *sq = (uint64_t *)malloc(sizeof(uint64_t) * N);
    uint64_t *as = (uint64_t *)malloc(sizeof(uint64_t) * N);
    orc_sample_ternary(seed, 0, 0, 1, N, s);
    orc_sample_gauss(seed, 0, 0, 3, N, e);
    for (uint32_t j = 0; j < L; j++) {
        uint64_t q = c->q[j];
        uint64_t *pk0 = pk + (size_t)(0 * L + j) * N, *pk1 = pk + (size_t)(1 * L + j) * N;
        orc_sample_uniform(seed, 0, 0, 2, j, q, N, pk1);          /* a_j */
        for (uint32_t i = 0; i < N; i++) sq[i] = from_signed(s[i], q);
        orc_negacyclic_mul_ntt(c, j, pk1, sq, as);                /* a_j s */
        for (uint32_t i = 0; i < N; i++)                           /* -a s + e */
            pk0[i] = addmod(submod(0, as[i], q), from_signed(e[i], q), q);
    }
    free(e); free(sq); free(as);
}

/* ------------------------------------------------------------------------- */
/* CKKS encode / decode: the canonical embedding on the orbit of 5            */
/* ------------------------------------------------------------------------- */

typedef struct { double re, im; } cplx;

/* (a+bi)(c+di) with four multiplications and two additions, data first */
static cplx cmul(cplx x, cplx w) {
    cplx r;
    r.re = x.re * w.re - x.im * w.im;
    r.im = x.re * w.im + x.im * w.re;
    return r;
}

static cplx cadd(cplx a, cplx b) { cplx r = {a.re + b.re, a.im + b.im}; return r; }
static cplx csub(cplx a, cplx b) { cplx r = {a.re - b.re, a.im - b.im}; return r; }

static void bitrev_permute(cplx *x, uint32_t n) {
    uint32_t bits = 0;
    while ((1u << bits) < n) bits++;
    for (uint32_t i = 0; i < n; i++) {
        uint32_t r = brev(i, bits);
        if (r > i) { cplx tmp = x[i]; x[i] = x[r]; x[r] = tmp; }
    }
}

/* zeta_{4 len}^{5^j mod 4 len} taken from the table of 2N-th roots */
static cplx rot_root(const orc_ctx *c, uint32_t len, uint32_t pow5) {
    uint32_t M = 2 * c->N;
    uint32_t idx = pow5 * (M / (4 * len));
    cplx w = {c->tw[2 * idx], c->tw[2 * idx + 1]};
    return w;
}

int orc_encode(const orc_ctx *c, const float *slots, int64_t *m) {
    uint32_t N = c->N, n = N / 2;
    cplx *x = (cplx *)malloc(sizeof(cplx) * n);
    for (uint32_t i = 0; i < n; i++) { x[i].re = (double)slots[i]; x[i].im = 0.0; }
    /* inverse of the slot map: stages len = n, n/2, ..., 2 */
    for (uint32_t len = n; len >= 2; len >>= 1) {
        uint32_t h = len / 2, mod = 4 * len;
        for (uint32_t b = 0; b < n; b += len) {
            uint32_t p5 = 1;                                   /* 5^j mod 4 len */
            for (uint32_t j = 0; j < h; j++) {
                cplx w = rot_root(c, len, p5);
                w.im = -w.im;                                  /* conjugate */
                cplx U = x[b + j], V = x[b + j + h];
                x[b + j] = cadd(U, V);
                x[b + j + h] = cmul(csub(U, V), w);
                p5 = (uint32_t)(((uint64_t)p5 * 5u) % mod);
            }
        }
    }
    bitrev_permute(x, n);
    /* Delta / n is a power of two: one exact multiplication */
    double scale = ldexp(1.0, c->log2_delta) / (double)n;
    int overflow = 0;
    const double lim = 4611686018427387904.0; /* 2^62 */
    for (uint32_t k = 0; k < n; k++) {
        double re = rint(x[k].re * scale), im = rint(x[k].im * scale);
        if (!(fabs(re) < lim) || !(fabs(im) < lim)) { overflow = 1; re = 0.0; im = 0.0; }
        m[k] = (int64_t)re;
        m[k + n] = (int64_t)im;
    }
    free(x);
    return overflow;
}

void orc_decode(const orc_ctx *c, const int64_t *d, double *z) {
    uint32_t N = c->N, n = N / 2;
    cplx *x = (cplx *)malloc(sizeof(cplx) * n);
    double inv_delta = ldexp(1.0, -c->log2_delta);
    for (uint32_t k = 0; k < n; k++) {
        x[k].re = (double)d[k] * inv_delta;
        x[k].im = (double)d[k + n] * inv_delta;
    }
    bitrev_permute(x, n);
    for (uint32_t len = 2; len <= n; len <<= 1) {
        uint32_t h = len / 2, mod = 4 * len;
        for (uint32_t b = 0; b < n; b += len) {
            uint32_t p5 = 1;
            for (uint32_t j = 0; j < h; j++) {
                cplx w = rot_root(c, len, p5);
                cplx U = x[b + j], V = cmul(x[b + j + h], w);
                x[b + j] = cadd(U, V);
                x[b + j + h] = csub(U, V);
                p5 = (uint32_t)(((uint64_t)p5 * 5u) % mod);
            }
        }
    }
    for (uint32_t j = 0; j < n; j++) z[j] = x[j].re;
    free(x);
}

/* ------------------------------------------------------------------------- */
/* encryption (Algorithm 1: HE.Enc(pk, M (.) W_i))                            */
/* ------------------------------------------------------------------------- */

void orc_encrypt_one(const orc_ctx *c, const uint64_t *pk, const int64_t *m,
                     uint64_t seed, uint32_t client, uint32_t t, uint64_t *ct) {
    uint32_t N = c->N, L = c->L;
    int8_t *u = (int8_t *)malloc(N), *e0 = (int8_t *)malloc(N), *e1 = (int8_t *)malloc(N);
    uint64_t *uq = (uint64_t *)malloc(sizeof(uint64_t) * N);
    uint64_t *pr = (uint64_t *)malloc(sizeof(uint64_t) * N);
    orc_sample_ternary(seed, t, client, 4, N, u);
    orc_sample_gauss(seed, t, client, 5, N, e0);
    orc_sample_gauss(seed, t, client, 6, N, e1);
    for (uint32_t j = 0; j < L; j++) {
        uint64_t q = c->q[j];
        const uint64_t *pk0 = pk + (size_t)(0 * L + j) * N, *pk1 = pk + (size_t)(1 * L + j) * N;
        uint64_t *c0 = ct + (size_t)(0 * L + j) * N, *c1 = ct + (size_t)(1 * L + j) * N;
        for (uint32_t i = 0; i < N; i++) uq[i] = from_signed(u[i], q);
        orc_negacyclic_mul_ntt(c, j, pk0, uq, pr);                 /* pk0 u */
        for (uint32_t i = 0; i < N; i++)
            c0[i] = addmod(addmod(pr[i], from_signed(e0[i], q), q), from_signed(m[i], q), q);
        orc_negacyclic_mul_ntt(c, j, pk1, uq, pr);                 /* pk1 u */
        for (uint32_t i = 0; i < N; i++) c1[i] = addmod(pr[i], from_signed(e1[i], q), q);
    }
    free(u); free(e0); free(e1); free(uq); free(pr);
}

int orc_encrypt(const orc_ctx *c, const uint64_t *pk, const float *sel, size_t T,
                uint64_t seed, uint32_t client, uint64_t *ct) {
    uint32_t N = c->N, n = N / 2, L = c->L;
    int bad = 0;
#pragma omp parallel for schedule(dynamic) reduction(+ : bad)
    for (size_t t = 0; t < T; t++) {
        int64_t *m = (int64_t *)malloc(sizeof(int64_t) * N);
        bad += orc_encode(c, sel + t * n, m);
        orc_encrypt_one(c, pk, m, seed, client, (uint32_t)t, ct + t * 2 * (size_t)L * N);
        free(m);
    }
    return bad;
}

/* ------------------------------------------------------------------------- */
/* server: weighted sum with plaintext weights, then rescale                  */
/* ------------------------------------------------------------------------- */

/* weight a_i as the constant polynomial rint(a_i q_{L-1}): a constant slot
 * vector encodes to a constant, and scale q_{L-1} makes the rescale exact */
void orc_weights(const orc_ctx *c, const double *alpha, uint32_t C, uint64_t *W) {
    double ql = (double)c->q[c->L - 1];
    for (uint32_t i = 0; i < C; i++) {
        double p = alpha[i] * ql;
        W[i] = (uint64_t)rint(p);
    }
}

void orc_weighted_sum(const orc_ctx *c, const uint64_t *const *cts, const uint64_t *W,
                      uint32_t C, size_t T, uint64_t *acc) {
    uint32_t N = c->N, L = c->L;
#pragma omp parallel for schedule(static)
    for (size_t t = 0; t < T; t++)
        for (uint32_t comp = 0; comp < 2; comp++)
            for (uint32_t j = 0; j < L; j++) {
                uint64_t q = c->q[j];
                size_t off = ((t * 2 + comp) * L + j) * (size_t)N;
                for (uint32_t k = 0; k < N; k++) {
                    uint64_t a = 0;
                    for (uint32_t i = 0; i < C; i++)
                        a = addmod(a, orc_mulmod(W[i] % q, cts[i][off + k], q), q);
                    acc[off + k] = a;
                }
            }
}

/* out_j = (acc_j - r) / q_{L-1} mod q_j, r = acc_{L-1} centred in (-q/2, q/2] */
void orc_rescale(const orc_ctx *c, const uint64_t *acc, size_t T, uint64_t *out) {
    uint32_t N = c->N, L = c->L;
    uint64_t ql = c->q[L - 1];
#pragma omp parallel for schedule(static)
    for (size_t t = 0; t < T; t++)
        for (uint32_t comp = 0; comp < 2; comp++) {
            const uint64_t *last = acc + ((t * 2 + comp) * L + (L - 1)) * (size_t)N;
            for (uint32_t j = 0; j + 1 < L; j++) {
                uint64_t q = c->q[j];
                uint64_t qlinv = orc_invmod(ql % q, q);
                const uint64_t *src = acc + ((t * 2 + comp) * L + j) * (size_t)N;
                uint64_t *dst = out + ((t * 2 + comp) * (L - 1) + j) * (size_t)N;
                for (uint32_t k = 0; k < N; k++) {
                    uint64_t r = last[k];
                    uint64_t rj;                         /* centred r, mod q_j */
                    if (r > ql / 2) rj = submod(0, (ql - r) % q, q);   /* r - ql < 0 */
                    else rj = r % q;
                    dst[k] = orc_mulmod(submod(src[k], rj, q), qlinv, q);
                }
            }
        }
}

void orc_plain_aggregate(const float *const *rests, const double *alpha, uint32_t C,
                         size_t len, double *out) {
#pragma omp parallel for schedule(static)
    for (size_t k = 0; k < len; k++) {
        double a = 0.0;
        for (uint32_t i = 0; i < C; i++) {
            double p = alpha[i] * (double)rests[i][k];
            a = a + p;
        }
        out[k] = a;
    }
}

/* ------------------------------------------------------------------------- */
/* decryption (Algorithm 1: HE.Dec(sk, M (.) [W_glob]))                       */
/* ------------------------------------------------------------------------- */

void orc_decrypt_limb(const orc_ctx *c, const int8_t *s, const uint64_t *ct,
                      uint32_t level, uint32_t limb, uint64_t *out) {
    uint32_t N = c->N;
    uint64_t q = c->q[limb];
    const uint64_t *c0 = ct + (size_t)(0 * level + limb) * N;
    const uint64_t *c1 = ct + (size_t)(1 * level + limb) * N;
    uint64_t *sq = (uint64_t *)malloc(sizeof(uint64_t) * N);
    for (uint32_t i = 0; i < N; i++) sq[i] = from_signed(s[i], q);
    orc_negacyclic_mul_ntt(c, limb, c1, sq, out);
    for (uint32_t i = 0; i < N; i++) out[i] = addmod(out[i], c0[i], q);
    free(sq);
}

void orc_decrypt(const orc_ctx *c, const int8_t *s, const uint64_t *ct, uint32_t level,
                 size_t T, int64_t *d) {
    uint32_t N = c->N;
    uint64_t q = c->q[0];
#pragma omp parallel for schedule(dynamic)
    for (size_t t = 0; t < T; t++) {
        uint64_t *r = (uint64_t *)malloc(sizeof(uint64_t) * N);
        orc_decrypt_limb(c, s, ct + t * 2 * (size_t)level * N, level, 0, r);
        for (uint32_t i = 0; i < N; i++)         /* centre into (-q/2, q/2] */
            d[t * N + i] = r[i] > q / 2 ? -(int64_t)(q - r[i]) : (int64_t)r[i];
        free(r);
    }
}

/* ------------------------------------------------------------------------- */
/* two-party threshold decryption: each party decrypts partially with its    */
/* share of the key and the partial results are merged (paper, appendix      */
/* "Key Management And Threshold HE").  The interactive key agreement is     */
/* replaced by a dealer that splits an existing secret additively.           */
/* ------------------------------------------------------------------------- */

void orc_threshold_split(const orc_ctx *c, const int8_t *s, uint64_t seed, uint64_t *share0,
                         uint64_t *share1) {
    uint32_t N = c->N;
    for (uint32_t j = 0; j < c->L; j++) {
        uint64_t q = c->q[j];
        uint64_t *a = share0 + (size_t)j * N, *b = share1 + (size_t)j * N;
        orc_sample_uniform(seed, 0, 0, 7, j, q, N, a);
        for (uint32_t i = 0; i < N; i++) b[i] = submod(from_signed(s[i], q), a[i], q);
    }
}

/* coefficient j: the 64-bit r of words 2(j&1), 2(j&1)+1 of block j>>1;
 * value = (r >> (63 - bits)) - 2^bits */
void orc_sample_smudge(uint64_t seed, uint32_t t, uint32_t party, uint32_t bits, uint32_t N, int64_t *out) {
    for (uint32_t j = 0; j < N; j++) {
        uint32_t w[4];
        stream_block(seed, j >> 1, t, party, 8, 0, w);
        uint64_t r = (uint64_t)w[2 * (j & 1)] | ((uint64_t)w[2 * (j & 1) + 1] << 32);
        out[j] = (int64_t)(r >> (63 - bits)) - ((int64_t)1 << bits);
    }
}

void orc_partial_decrypt(const orc_ctx *c, const uint64_t *share, uint32_t party, const uint64_t *ct,
                         uint32_t level, uint64_t seed, uint32_t t, uint32_t bits, uint64_t *out) {
    uint32_t N = c->N;
    uint64_t q = c->q[0];
    const uint64_t *c1 = ct + (size_t)(1 * level + 0) * N;
    int64_t *e = (int64_t *)malloc(sizeof(int64_t) * N);
    orc_sample_smudge(seed, t, party, bits, N, e);
    orc_negacyclic_mul_ntt(c, 0, c1, share, out);             /* limb 0 of the share */
    for (uint32_t i = 0; i < N; i++) out[i] = addmod(out[i], from_signed(e[i], q), q);
    free(e);
}

void orc_threshold_combine(const orc_ctx *c, const uint64_t *ct, uint32_t level,
                           const uint64_t *const *parts, uint32_t nparts, int64_t *d) {
    uint32_t N = c->N;
    uint64_t q = c->q[0];
    const uint64_t *c0 = ct + (size_t)(0 * level + 0) * N;
    for (uint32_t i = 0; i < N; i++) {
        uint64_t r = c0[i];
        for (uint32_t p = 0; p < nparts; p++) r = addmod(r, parts[p][i], q);
        d[i] = r > q / 2 ? -(int64_t)(q - r) : (int64_t)r;
    }
}

/* ------------------------------------------------------------------------- */
/* selective-encryption mask ("Step 2"), packing, merge                       */
/* ------------------------------------------------------------------------- */

static uint32_t score_key(float s) {
    uint32_t b;
    memcpy(&b, &s, 4);
    if (b & 0x80000000u) return 0;      /* negative (and -0): lowest */
    if (b > 0x7f800000u) return 0;      /* NaN: lowest */
    return b;
}

typedef struct { uint32_t key, idx; } kv;

static int kv_cmp(const void *a, const void *b) {
    const kv *x = (const kv *)a, *y = (const kv *)b;
    if (x->key != y->key) return x->key > y->key ? -1 : 1;   /* key descending */
    if (x->idx != y->idx) return x->idx < y->idx ? -1 : 1;   /* index ascending */
    return 0;
}

static int u32_cmp(const void *a, const void *b) {
    uint32_t x = *(const uint32_t *)a, y = *(const uint32_t *)b;
    return x < y ? -1 : (x > y);
}

void orc_select_mask(const float *score, size_t P, size_t k, uint32_t *idx) {
    kv *v = (kv *)malloc(sizeof(kv) * (P ? P : 1));
    for (size_t i = 0; i < P; i++) { v[i].key = score_key(score[i]); v[i].idx = (uint32_t)i; }
    qsort(v, P, sizeof(kv), kv_cmp);
    for (size_t r = 0; r < k; r++) idx[r] = v[r].idx;
    qsort(idx, k, sizeof(uint32_t), u32_cmp);
    free(v);
}

void orc_pack(const orc_ctx *c, const uint32_t *idx, size_t k, const float *x, size_t P,
              float *sel, float *rest) {
    size_t n = c->N / 2, T = (k + n - 1) / n;
    for (size_t r = 0; r < T * n; r++) sel[r] = 0.0f;
    if (!idx) {
        for (size_t r = 0; r < k; r++) sel[r] = x[r];
        return;
    }
    for (size_t r = 0; r < k; r++) sel[r] = x[idx[r]];
    size_t next = 0, o = 0;
    for (size_t i = 0; i < P; i++) {
        if (next < k && idx[next] == i) next++;
        else rest[o++] = x[i];
    }
}

void orc_unpack(const uint32_t *idx, size_t k, const double *z, const double *rest_avg,
                size_t P, double *w_glob) {
    if (!idx) {
        for (size_t r = 0; r < k; r++) w_glob[r] = z[r];
        return;
    }
    size_t next = 0, o = 0;
    for (size_t i = 0; i < P; i++) {
        if (next < k && idx[next] == i) { w_glob[i] = z[next]; next++; }
        else w_glob[i] = rest_avg[o++];
    }
}

/* ------------------------------------------------------------------------- */
/* one whole round                                                            */
/* ------------------------------------------------------------------------- */

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int orc_round(const orc_ctx *c, const float *const *xs, const double *alpha, uint32_t C,
              size_t P, const uint32_t *idx, size_t k, uint64_t key_seed, uint64_t enc_seed,
              size_t t_begin, size_t t_end, int do_rest, double *w_glob) {
    uint32_t N = c->N, L = c->L;
    size_t n = N / 2, ctw = 2 * (size_t)L * N;
    int8_t *s = (int8_t *)malloc(N);
    uint64_t *pk = (uint64_t *)malloc(sizeof(uint64_t) * ctw);
    uint64_t *W = (uint64_t *)malloc(sizeof(uint64_t) * C);
    if (!s || !pk || !W) return -1;
    orc_keygen(c, key_seed, s, pk);
    orc_weights(c, alpha, C, W);
    int fail = 0;
    /* ciphertext indices are independent units of work */
#pragma omp parallel for schedule(dynamic)
    for (size_t t = t_begin; t < t_end; t++) {
        float *slots = (float *)malloc(sizeof(float) * n);
        int64_t *m = (int64_t *)malloc(sizeof(int64_t) * N);
        uint64_t *cts = (uint64_t *)malloc(sizeof(uint64_t) * ctw * C);
        uint64_t *acc = (uint64_t *)malloc(sizeof(uint64_t) * ctw);
        uint64_t *agg = (uint64_t *)malloc(sizeof(uint64_t) * ctw);
        double *z = (double *)malloc(sizeof(double) * n);
        const uint64_t **ptr = (const uint64_t **)malloc(sizeof(uint64_t *) * C);
        if (!slots || !m || !cts || !acc || !agg || !z || !ptr) {
            fail = 1;
        } else {
            for (uint32_t i = 0; i < C; i++) {                 /* clients: pack, encode, encrypt */
                for (size_t r = 0; r < n; r++) {
                    size_t g = t * n + r;
                    slots[r] = g < k ? xs[i][idx ? idx[g] : g] : 0.0f;
                }
                orc_encode(c, slots, m);
                orc_encrypt_one(c, pk, m, enc_seed, i, (uint32_t)t, cts + ctw * i);
                ptr[i] = cts + ctw * i;
            }
            orc_weighted_sum(c, ptr, W, C, 1, acc);            /* server */
            orc_rescale(c, acc, 1, agg);
            orc_decrypt(c, s, agg, L - 1, 1, m);               /* client */
            orc_decode(c, m, z);
            for (size_t r = 0; r < n; r++) {                   /* scatter back */
                size_t g = t * n + r;
                if (g < k) w_glob[idx ? idx[g] : g] = z[r];
            }
        }
        free(slots); free(m); free(cts); free(acc); free(agg); free(z); free(ptr);
    }
    if (do_rest && idx && !fail) {                             /* plaintext remainder */
        size_t next = 0;
        for (size_t i = 0; i < P; i++) {
            if (next < k && idx[next] == i) { next++; continue; }
            double a = 0.0;
            for (uint32_t cidx = 0; cidx < C; cidx++) {
                double p = alpha[cidx] * (double)xs[cidx][i];
                a = a + p;
            }
            w_glob[i] = a;
        }
    }
    free(s); free(pk); free(W);
    return fail ? -1 : 0;
}
