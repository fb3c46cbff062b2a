// Host-side table construction for the CUDA library (see fedhe_host.h).
#include "fedhe_host.h"

#include <quadmath.h>

namespace fedhe {

typedef unsigned __int128 u128;

uint64_t host_mulmod(uint64_t a, uint64_t b, uint64_t q) { return (uint64_t)((u128)a * b % q); }

uint64_t host_powmod(uint64_t a, uint64_t e, uint64_t q) {
    uint64_t r = 1 % q;
    a %= q;
    for (; e; e >>= 1) {
        if (e & 1) r = host_mulmod(r, a, q);
        a = host_mulmod(a, a, q);
    }
    return r;
}

uint64_t host_invmod(uint64_t a, uint64_t q) { return host_powmod(a, q - 2, q); }

HostTw host_shoup(uint64_t w, uint64_t q) {
    HostTw t;
    t.w = w;
    t.wp = (uint64_t)(((u128)w << 64) / q);
    return t;
}

// Miller-Rabin with the first twelve primes as witnesses: exact below 3.3e24
bool host_is_prime(uint64_t n) {
    const uint64_t wit[12] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    if (n < 2) return false;
    for (uint64_t p : wit) {
        if (n == p) return true;
        if (n % p == 0) return false;
    }
    uint64_t d = n - 1;
    int r = 0;
    while (!(d & 1)) { d >>= 1; r++; }
    for (uint64_t a : wit) {
        uint64_t x = host_powmod(a, d, n);
        if (x == 1 || x == n - 1) continue;
        bool witness = true;
        for (int i = 1; i < r && witness; i++) {
            x = host_mulmod(x, x, n);
            if (x == n - 1) witness = false;
        }
        if (witness) return false;
    }
    return true;
}

const char *host_check_params(uint32_t N, uint32_t L, const uint64_t *q, int log2_delta) {
    if (N < 8192 || N > 65536 || (N & (N - 1))) return "N must be a power of two in [8192, 65536]";
    if (L < 2 || L > 16) return "L must be in [2, 16]";
    if (log2_delta < 1 || log2_delta > 58) return "log2_delta out of range";
    for (uint32_t j = 0; j < L; j++) {
        if (q[j] >= (1ull << 61) || q[j] < (1ull << 20)) return "prime out of range";
        if ((q[j] - 1) % (2ull * N)) return "prime is not 1 mod 2N";
        if (!host_is_prime(q[j])) return "modulus is not prime";
        for (uint32_t i = 0; i < j; i++)
            if (q[i] == q[j]) return "repeated prime";
    }
    if ((1ull << log2_delta) >= q[0] / 4) return "scale too large for q_0";
    return nullptr;
}

static uint32_t bit_reverse(uint32_t x, int bits) {
    uint32_t r = 0;
    for (int i = 0; i < bits; i++) r |= ((x >> i) & 1u) << (bits - 1 - i);
    return r;
}

static uint64_t smallest_root_2n(uint64_t q, uint32_t N) {
    // an element of order exactly 2N, then the least of its odd powers
    uint64_t g = 0, cof = (q - 1) / (2ull * N);
    for (uint64_t x = 2;; x++) {
        uint64_t c = host_powmod(x, cof, q);
        if (host_powmod(c, N, q) == q - 1) { g = c; break; }
    }
    uint64_t sq = host_mulmod(g, g, q), cur = g, best = g;
    for (uint32_t k = 1; k < N; k++) {
        cur = host_mulmod(cur, sq, q);
        if (cur < best) best = cur;
    }
    return best;
}

void host_build_limb(uint32_t N, uint64_t q, HostLimb &out) {
    int logN = 0;
    while ((1u << logN) < N) logN++;
    out.q = q;
    out.psi = smallest_root_2n(q, N);
    out.mu = (uint64_t)((((u128)1) << 64) / q);
    out.fwd.resize(N);
    out.inv.resize(N);
    uint64_t ipsi = host_invmod(out.psi, q);
    uint64_t p = 1, ip = 1;
    for (uint32_t i = 0; i < N; i++) {
        uint32_t r = bit_reverse(i, logN);
        out.fwd[r] = host_shoup(p, q);
        out.inv[r] = host_shoup(ip, q);
        p = host_mulmod(p, out.psi, q);
        ip = host_mulmod(ip, ipsi, q);
    }
    uint64_t ninv = host_invmod(N, q);
    out.ninv = host_shoup(ninv, q);
    out.wn = host_shoup(host_mulmod(out.inv[1].w, ninv, q), q);
}

// cos/sin of 2 pi a / M for 0 <= a <= M/8 in quad precision, rounded once
static void first_octant(uint32_t a, uint32_t M, double &c, double &s) {
    if (a == 0) { c = 1.0; s = 0.0; return; }
    const __float128 pi = 4 * atanq((__float128)1);
    __float128 ang = (2 * pi * (__float128)a) / (__float128)M;
    c = (double)cosq(ang);
    s = (double)sinq(ang);
}

void host_unit_roots(uint32_t N, std::vector<double> &roots) {
    const uint32_t M = 2 * N, e = M / 8;
    roots.assign(2 * (size_t)M, 0.0);
    for (uint32_t t = 0; t < M; t++) {
        uint32_t oct = t / e, r = t % e;
        uint32_t a = (oct & 1) ? e - r : r;      // distance to the nearer axis
        double c, s, x, y;
        first_octant(a, M, c, s);
        switch (oct) {
        case 0: x = c; y = s; break;
        case 1: x = s; y = c; break;
        case 2: x = -s; y = c; break;
        case 3: x = -c; y = s; break;
        case 4: x = -c; y = -s; break;
        case 5: x = -s; y = -c; break;
        case 6: x = s; y = -c; break;
        default: x = c; y = -s; break;
        }
        roots[2 * t] = x + 0.0;
        roots[2 * t + 1] = y + 0.0;
    }
}

void host_slot_twiddles(uint32_t N, const std::vector<double> &roots, std::vector<double> &out) {
    const uint32_t n = N / 2, M = 2 * N;
    out.assign(2 * (size_t)n, 0.0);
    for (uint32_t len = 2; len <= n; len <<= 1) {
        uint32_t h = len / 2, mod = 4 * len, step = M / mod;
        uint32_t p5 = 1;
        for (uint32_t j = 0; j < h; j++) {
            uint32_t t = p5 * step;
            out[2 * (size_t)(h + j)] = roots[2 * (size_t)t];
            out[2 * (size_t)(h + j) + 1] = roots[2 * (size_t)t + 1];
            p5 = (uint32_t)(((uint64_t)p5 * 5u) % mod);
        }
    }
}

}  // namespace fedhe
