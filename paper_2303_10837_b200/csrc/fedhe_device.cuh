// Device-side primitives: 64-bit modular arithmetic (Shoup / Barrett, lazy
// Harvey ranges), Philox4x32-10 and the samplers built on it.
//
// Functions marked HD also compile for the host so that the thread-level
// index arithmetic of the transforms can be exercised without a GPU.
#pragma once

#include <stdint.h>

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

// Shoup product with a fixed operand w < q and wp = floor(w 2^64 / q):
// returns x w mod q up to one extra q, i.e. a value in [0, 2q), for any x.
HD uint64_t shoup_lazy(uint64_t x, uint64_t w, uint64_t wp, uint64_t q) {
    uint64_t hi = mulhi64(x, wp);
    return sub64(x * w, hi * q);
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
    uint64_t r = barrett64(a, q, mu);
    return (v < 0 && r != 0) ? q - r : r;
}

// residue of a small signed value |v| < q
HD uint64_t small_residue(int v, uint64_t q) { return v < 0 ? q - (uint64_t)(-v) : (uint64_t)v; }

// Harvey butterflies.  Forward (Cooley-Tukey): inputs and outputs in [0, 4q).
HD void ct_butterfly(uint64_t &x, uint64_t &y, uint64_t w, uint64_t wp, uint64_t q, uint64_t q2) {
    uint64_t u = csub(x, q2);
    uint64_t v = shoup_lazy(y, w, wp, q);
    x = add64(u, v);
    y = add64(sub64(u, v), q2);
}

// The same butterflies without any conditional subtraction, for primes small
// enough that the values may simply grow: forward, every stage adds at most
// 2q to the bound; inverse, the sum doubles it, and the difference is kept
// non-negative by adding `bound`, a multiple of q not below the inputs.
HD void ct_butterfly_grow(uint64_t &x, uint64_t &y, uint64_t w, uint64_t wp, uint64_t q, uint64_t q2) {
    const uint64_t u = x, v = shoup_lazy(y, w, wp, q);
    x = add64(u, v);
    y = add64(sub64(u, v), q2);
}
HD void gs_butterfly_grow(uint64_t &x, uint64_t &y, uint64_t w, uint64_t wp, uint64_t q, uint64_t bound) {
    const uint64_t u = x, v = y;
    x = add64(u, v);
    y = shoup_lazy(add64(sub64(u, v), bound), w, wp, q);
}

// Inverse (Gentleman-Sande): inputs and outputs in [0, 2q).
HD void gs_butterfly(uint64_t &x, uint64_t &y, uint64_t w, uint64_t wp, uint64_t q, uint64_t q2) {
    uint64_t u = x, v = y;
    x = csub(add64(u, v), q2);
    y = shoup_lazy(add64(sub64(u, v), q2), w, wp, q);
}

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
