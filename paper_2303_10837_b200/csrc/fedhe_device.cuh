// Device-side primitives: 64-bit modular arithmetic (Shoup / Barrett, lazy
// Harvey ranges), Philox4x32-10 and the samplers built on it.
//
// Functions marked HD also compile for the host so that the thread-level
// index arithmetic of the transforms can be exercised without a GPU.
#pragma once

#include <stdint.h>
#include <string.h>

#if !defined(__CUDA_ARCH__)
#include <cmath>
#endif

#if defined(__CUDACC__)
#define HD __host__ __device__ __forceinline__
#else
#define HD inline
#endif

namespace fedhe {

// ---------------------------------------------------------------------------
// 64-bit modular arithmetic
// ---------------------------------------------------------------------------

HD uint64_t mulhi64(uint64_t a, uint64_t b) {
#if defined(__CUDA_ARCH__)
    return __umul64hi(a, b);
#else
    return (uint64_t)(((unsigned __int128)a * b) >> 64);
#endif
}

// 64-bit add / subtract / conditional subtract.  On the device they are
// written as 32-bit carry chains: left to itself the compiler puts the high
// halves of 64-bit additions on the integer multiply-add pipe, which is the
// pipe the transforms saturate; carry chains stay on the plain ALU pipe
// (measured: +9 % butterflies per clock).
HD uint64_t add64(uint64_t a, uint64_t b) {
#if defined(__CUDA_ARCH__)
    uint32_t rl, rh;
    asm("add.cc.u32 %0, %2, %4; addc.u32 %1, %3, %5;"
        : "=r"(rl), "=r"(rh)
        : "r"((uint32_t)a), "r"((uint32_t)(a >> 32)), "r"((uint32_t)b), "r"((uint32_t)(b >> 32)));
    return ((uint64_t)rh << 32) | rl;
#else
    return a + b;
#endif
}

HD uint64_t sub64(uint64_t a, uint64_t b) {
#if defined(__CUDA_ARCH__)
    uint32_t rl, rh;
    asm("sub.cc.u32 %0, %2, %4; subc.u32 %1, %3, %5;"
        : "=r"(rl), "=r"(rh)
        : "r"((uint32_t)a), "r"((uint32_t)(a >> 32)), "r"((uint32_t)b), "r"((uint32_t)(b >> 32)));
    return ((uint64_t)rh << 32) | rl;
#else
    return a - b;
#endif
}

// x - m if x >= m (the borrow of x - m decides)
HD uint64_t csub(uint64_t x, uint64_t m) {
#if defined(__CUDA_ARCH__)
    uint32_t rl, rh, borrow;
    asm("sub.cc.u32 %0, %3, %5; subc.cc.u32 %1, %4, %6; subc.u32 %2, 0, 0;"
        : "=r"(rl), "=r"(rh), "=r"(borrow)
        : "r"((uint32_t)x), "r"((uint32_t)(x >> 32)), "r"((uint32_t)m), "r"((uint32_t)(m >> 32)));
    return borrow ? x : (((uint64_t)rh << 32) | rl);
#else
    return x >= m ? x - m : x;
#endif
}

// The same for x, m < 2^63 (every modulus is below 2^61 and every lazy value
// below 4q) without predicated moves: the sign of the 64-bit difference,
// spread to a mask, picks x or the difference with two bitwise selects.  The
// compiler issues the two predicated moves of the version above to the
// multiply pipe; where that pipe is the bound (the fused encrypt) the selects
// win (-3.6 % with 60-bit primes), where memory is (the server's weighted sum,
// the standalone transform) the extra logic operations lose 2-3 %.
HD uint64_t csub_sel(uint64_t x, uint64_t m) {
#if defined(__CUDA_ARCH__)
    uint32_t rl, rh;
    asm("{\n\t"
        ".reg .u32 dl, dh, k;\n\t"
        "sub.cc.u32 dl, %2, %4;\n\t"
        "subc.u32 dh, %3, %5;\n\t"
        "shr.s32 k, dh, 31;\n\t"                  // all ones if x < m
        "lop3.b32 %0, %2, dl, k, 0xE4;\n\t"      // k ? x : difference
        "lop3.b32 %1, %3, dh, k, 0xE4;\n\t"
        "}"
        : "=r"(rl), "=r"(rh)
        : "r"((uint32_t)x), "r"((uint32_t)(x >> 32)), "r"((uint32_t)m), "r"((uint32_t)(m >> 32)));
    return ((uint64_t)rh << 32) | rl;
#else
    return x >= m ? x - m : x;
#endif
}
template <bool SEL>
HD uint64_t csub_as(uint64_t x, uint64_t m) { return SEL ? csub_sel(x, m) : csub(x, m); }

// Shoup product with a fixed operand w < q and wp = floor(w 2^64 / q):
// returns x w mod q up to one extra q, i.e. a value in [0, 2q), for any x.
//
// On the device the product is written out in 32-bit pieces.  The quotient
// hi = floor(x wp / 2^64) comes from the three upper partial products chained
// through the carry flag (of x0 wp0 only the high word matters); the result is
// x w + hi (2^64 - q) mod 2^64, accumulated by two wide multiply-adds into one
// 64-bit register pair plus four narrow ones into its high word, so that no
// separate subtraction and no carry additions remain.  Measured on whole
// transforms in shared memory against `x * w - __umul64hi(x, wp) * q`: 6 %
// faster, 30.5 instead of 34.5 instructions per butterfly.
HD uint64_t shoup_lazy(uint64_t x, uint64_t w, uint64_t wp, uint64_t q) {
#if defined(__CUDA_ARCH__)
    const uint64_t nq = 0 - q;
    uint64_t r;
    asm("{\n\t"
        ".reg .u32 x0, x1, p0, p1, w0, w1, n0, n1, t1, t2, t3, r0, r1;\n\t"
        ".reg .u64 acc;\n\t"
        "mov.b64 {x0, x1}, %1;\n\t"
        "mov.b64 {w0, w1}, %2;\n\t"
        "mov.b64 {p0, p1}, %3;\n\t"
        "mov.b64 {n0, n1}, %4;\n\t"
        "mul.hi.u32 t1, x0, p0;\n\t"
        "mad.lo.cc.u32 t1, x0, p1, t1;\n\t"
        "madc.hi.u32 t2, x0, p1, 0;\n\t"
        "mad.lo.cc.u32 t1, x1, p0, t1;\n\t"
        "madc.hi.cc.u32 t2, x1, p0, t2;\n\t"
        "addc.u32 t3, 0, 0;\n\t"
        "mad.lo.cc.u32 t2, x1, p1, t2;\n\t"
        "madc.hi.u32 t3, x1, p1, t3;\n\t"            // hi = t3 : t2
        "mul.wide.u32 acc, x0, w0;\n\t"
        "mad.wide.u32 acc, t2, n0, acc;\n\t"
        "mov.b64 {r0, r1}, acc;\n\t"
        "mad.lo.u32 r1, x0, w1, r1;\n\t"
        "mad.lo.u32 r1, x1, w0, r1;\n\t"
        "mad.lo.u32 r1, t2, n1, r1;\n\t"
        "mad.lo.u32 r1, t3, n0, r1;\n\t"
        "mov.b64 %0, {r0, r1};\n\t"
        "}"
        : "=l"(r)
        : "l"(x), "l"(w), "l"(wp), "l"(nq));
    return r;
#else
    uint64_t hi = mulhi64(x, wp);
    return sub64(x * w, hi * q);
#endif
}

HD uint64_t shoup(uint64_t x, uint64_t w, uint64_t wp, uint64_t q) {
    return csub(shoup_lazy(x, w, wp, q), q);
}

// Barrett reduction of any 64-bit x with mu = floor(2^64 / q): result in [0, q)
HD uint64_t barrett64(uint64_t x, uint64_t q, uint64_t mu) {
    uint64_t t = mulhi64(x, mu);
    uint64_t r = x - t * q;           // in [0, 3q)
    r = csub(r, 2 * q);
    return csub(r, q);
}

// residue in [0, q) of a signed 64-bit integer
HD uint64_t signed_residue(int64_t v, uint64_t q, uint64_t mu) {
    uint64_t a = v < 0 ? (uint64_t)0 - (uint64_t)v : (uint64_t)v;
    // encoded updates are far below the primes, so a warp rarely needs the reduction
    uint64_t r = a;
    if (a >= q) r = barrett64(a, q, mu);
    return (v < 0 && r != 0) ? q - r : r;
}

// residue of a small signed value |v| < q
HD uint64_t small_residue(int v, uint64_t q) { return v < 0 ? q - (uint64_t)(-v) : (uint64_t)v; }

// Harvey butterflies.  Forward (Cooley-Tukey): inputs and outputs in [0, 4q).
template <bool SEL = false>
HD void ct_butterfly(uint64_t &x, uint64_t &y, uint64_t w, uint64_t wp, uint64_t q, uint64_t q2) {
    uint64_t u = csub_as<SEL>(x, q2);
    uint64_t v = shoup_lazy(y, w, wp, q);
    x = add64(u, v);
    y = add64(sub64(u, v), q2);
}

// Inverse (Gentleman-Sande): inputs and outputs in [0, 2q).
template <bool SEL = false>
HD void gs_butterfly(uint64_t &x, uint64_t &y, uint64_t w, uint64_t wp, uint64_t q, uint64_t q2) {
    uint64_t u = x, v = y;
    x = csub_as<SEL>(add64(u, v), q2);
    y = shoup_lazy(add64(sub64(u, v), q2), w, wp, q);
}

// ---------------------------------------------------------------------------
// Residues of a prime below 2^46 as integers held in doubles
//
// The double-precision pipe of the SM is separate from the integer multiply
// pipe that the 64-bit Shoup products saturate, and a modular product costs it
// six operations against about nineteen 32-bit multiply slots, so limbs whose
// prime is small enough run their transforms in this arithmetic.  Values are
// signed integers of magnitude at most 2^50 (exact in a double); every
// operation below is a single correctly rounded instruction, written with the
// rounding intrinsics so that nothing is contracted or reordered.
// ---------------------------------------------------------------------------

constexpr uint64_t F64_PRIME_LIMIT = 1ull << 46;
constexpr double F64_TWO52 = 4503599627370496.0;

HD double f64_fma(double a, double b, double c) {
#if defined(__CUDA_ARCH__)
    return __fma_rn(a, b, c);
#else
    return std::fma(a, b, c);
#endif
}
HD double f64_mul(double a, double b) {
#if defined(__CUDA_ARCH__)
    return __dmul_rn(a, b);
#else
    return a * b;
#endif
}
HD double f64_add(double a, double b) {
#if defined(__CUDA_ARCH__)
    return __dadd_rn(a, b);
#else
    return a + b;
#endif
}
HD double f64_sub(double a, double b) { return f64_add(a, -b); }

HD double f64_from_bits(uint64_t b) {
#if defined(__CUDA_ARCH__)
    return __longlong_as_double((long long)b);
#else
    double d;
    memcpy(&d, &b, 8);
    return d;
#endif
}
HD uint64_t f64_bits(double d) {
#if defined(__CUDA_ARCH__)
    return (uint64_t)__double_as_longlong(d);
#else
    uint64_t b;
    memcpy(&b, &d, 8);
    return b;
#endif
}

// exact conversions of integers 0 <= x < 2^52 through the exponent of 2^52
HD double f64_from_u64(uint64_t x) { return f64_sub(f64_from_bits(x | 0x4330000000000000ull), F64_TWO52); }
HD uint64_t f64_to_u64(double r) { return f64_bits(f64_add(r, F64_TWO52)) & 0x000fffffffffffffull; }

// x - q rint(x / q) for |x| < 2^51 with qi = 1/q rounded: exact, magnitude at most q/2 + 1
// round to the nearest integer: the conversion instruction, which leaves the double-precision
// arithmetic pipe free (adding and subtracting 1.5 * 2^52 costs that pipe two operations:
// 1.6 % slower on a limb set in doubles)
HD double f64_rint(double x) {
#if defined(__CUDA_ARCH__)
    double r;
    asm("cvt.rni.f64.f64 %0, %1;" : "=d"(r) : "d"(x));
    return r;
#else
    return std::nearbyint(x);
#endif
}
HD double f64_reduce(double x, double q, double qi) {
    const double k = f64_rint(f64_mul(x, qi));
    return f64_fma(-k, q, x);
}

// y w mod q for integers |y| <= 2^50 and 0 <= w < q < 2^46.  The product is
// taken exactly as h + l; k = rint(fl(h qi)) differs from y w / q by at most
// 1/2 (the rounding to an integer) + 2 * 2^50 2^-53 (the rounded reciprocal and
// the rounded product, each 2^-53 of a quotient below 2^50) = 3/4, so the
// result, which both fused operations deliver exactly (h - k q is an integer
// below 2^53), has magnitude at most 3q/4.
HD double f64_mulmod(double y, double w, double q, double qi) {
    const double h = f64_mul(y, w);
    const double l = f64_fma(y, w, -h);
    const double k = f64_rint(f64_mul(h, qi));
    return f64_add(f64_fma(-k, q, h), l);
}

// the residue in [0, q) of an integer |r| < q
HD uint64_t f64_canonical(double r, double q) { return f64_to_u64(r < 0.0 ? f64_add(r, q) : r); }

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11)
// ---------------------------------------------------------------------------

struct u32x4 { uint32_t x, y, z, w; };

HD void mulhilo32(uint32_t a, uint32_t b, uint32_t &hi, uint32_t &lo) {
#if defined(__CUDA_ARCH__)
    lo = a * b;
    hi = __umulhi(a, b);
#else
    uint64_t p = (uint64_t)a * b;
    lo = (uint32_t)p;
    hi = (uint32_t)(p >> 32);
#endif
}

HD u32x4 philox4x32_10(u32x4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; r++) {
        uint32_t h0, l0, h1, l1;
        mulhilo32(0xD2511F53u, c.x, h0, l0);
        mulhilo32(0xCD9E8D57u, c.z, h1, l1);
        u32x4 n;
        n.x = h1 ^ c.y ^ k0;
        n.y = l1;
        n.z = h0 ^ c.w ^ k1;
        n.w = l0;
        c = n;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c;
}

// Stream coordinates: counter = (block, ciphertext index, client, tag | limb << 8),
// key = the two halves of the seed.
enum : uint32_t {
    TAG_SK = 1, TAG_PK_A = 2, TAG_PK_E = 3, TAG_ENC_U = 4, TAG_ENC_E0 = 5, TAG_ENC_E1 = 6,
    TAG_SHARE = 7, TAG_SMUDGE = 8
};

HD u32x4 stream_block(uint64_t seed, uint32_t block, uint32_t t, uint32_t client, uint32_t tag_limb) {
    u32x4 c = {block, t, client, tag_limb};
    return philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
}

// uniform ternary value from one 32-bit word: floor(3 w / 2^32) - 1
HD int ternary_from_word(uint32_t w) {
#if defined(__CUDA_ARCH__)
    return (int)__umulhi(w, 3u) - 1;
#else
    return (int)(((uint64_t)w * 3u) >> 32) - 1;
#endif
}

}  // namespace fedhe
