// Host-side check of the CUDA library's transform core (no GPU): the header
// that the kernels are built from is compiled for the CPU, every lane of every
// virtual warp of a block is played in turn with a plain array as shared memory,
// and the result is compared with the transform's definition
//   A^[k] = sum_j a_j psi^((2 brev(k) + 1) j) mod q
// evaluated directly.  Covers both limb arithmetics (64-bit integers, and
// signed integers in doubles for primes below 2^46), whole blocks and the
// pieces of a longer transform, the scaled inverse, the bounds that the
// double-precision arithmetic relies on, the shared-memory swizzle, and that a
// virtual warp keeps to its own words between the phases that only a
// warp-level barrier separates.
//
// Built and run by tests/test_host_transform.py:  prints "ok" and exits 0.
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <algorithm>
#include <vector>

#include "../paper_2303_10837_b200/csrc/fedhe_host.h"
#include "../paper_2303_10837_b200/csrc/fedhe_ntt.cuh"

using namespace fedhe;
typedef unsigned __int128 u128;

static uint64_t rng_state = 0x243F6A8885A308D3ull;
static uint64_t rnd() {   // splitmix64
    uint64_t z = (rng_state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

#define CHECK(cond, ...)                                  \
    do {                                                  \
        if (!(cond)) {                                    \
            printf("FAILED %s:%d: ", __FILE__, __LINE__); \
            printf(__VA_ARGS__);                          \
            printf("\n");                                 \
            exit(1);                                      \
        }                                                 \
    } while (0)

static uint32_t brev(uint32_t x, int bits) {
    uint32_t r = 0;
    for (int i = 0; i < bits; i++) r |= ((x >> i) & 1u) << (bits - 1 - i);
    return r;
}

// ---- the arithmetic in doubles against exact integers ------------------------
static void check_f64_primitives(uint64_t q) {
    const double qd = (double)q, qi = 1.0 / qd;
    const double bound = std::ldexp(1.0, 50);
    for (int it = 0; it < 400000; it++) {
        // |y| up to 2^50 (the documented limit), w anywhere in [0, q), with edge values mixed in
        int64_t y = (int64_t)(rnd() >> 13) - ((int64_t)1 << 50);
        uint64_t w = rnd() % q;
        switch (it & 15) {
        case 0: y = ((int64_t)1 << 50); break;
        case 1: y = -((int64_t)1 << 50); break;
        case 2: w = q - 1; break;
        case 3: w = 0; break;
        case 4: y = 0; break;
        case 5: y = (int64_t)q; break;
        case 6: y = ((int64_t)1 << 50); w = q - 1; break;
        default: break;
        }
        const double r = f64_mulmod((double)y, (double)w, qd, qi);
        CHECK(r == std::floor(r) && std::fabs(r) <= 0.75 * qd + 1, "mulmod range y=%lld w=%llu r=%.1f",
              (long long)y, (unsigned long long)w, r);
        // congruence: (y w - r) mod q == 0 in exact arithmetic
        const __int128 exact = (__int128)y * (__int128)w - (__int128)(int64_t)r;
        CHECK(exact % (__int128)q == 0, "mulmod congruence y=%lld w=%llu", (long long)y, (unsigned long long)w);
        CHECK(std::fabs((double)y) <= bound, "test input out of range");
        // reduction
        const int64_t x = (int64_t)(rnd() >> 13) - ((int64_t)1 << 50);
        const double s = f64_reduce((double)x, qd, qi);
        CHECK(std::fabs(s) <= 0.5 * qd + 1 && ((__int128)x - (__int128)(int64_t)s) % (__int128)q == 0,
              "reduce x=%lld", (long long)x);
        // conversions and canonical form
        const uint64_t u = rnd() >> 12;
        CHECK(f64_to_u64(f64_from_u64(u)) == u, "u64 <-> double %llu", (unsigned long long)u);
        const int64_t v = (int64_t)(rnd() % (2 * q - 1)) - (int64_t)(q - 1);   // |v| < q
        const uint64_t c = f64_canonical((double)v, qd);
        CHECK(c < q && c == (uint64_t)((v % (int64_t)q + (int64_t)q) % (int64_t)q), "canonical %lld", (long long)v);
    }
}

// ---- definition of the transform --------------------------------------------
static uint64_t eval_definition(const std::vector<uint64_t> &a, uint64_t psi, uint64_t q, uint32_t k, int logN) {
    const uint64_t root = host_powmod(psi, 2 * (uint64_t)brev(k, logN) + 1, q);
    uint64_t acc = 0, p = 1;
    for (size_t j = 0; j < a.size(); j++) {
        acc = (uint64_t)(((u128)a[j] * p + acc) % q);
        p = host_mulmod(p, root, q);
    }
    return acc;
}

template <class M>
struct Tables;
template <>
struct Tables<ModInt> {
    std::vector<tw_t> fwd, inv;
    tw_t ninv, wn;
    ModInt m;
    explicit Tables(const HostLimb &hl) : m{hl.q, 2 * hl.q} {
        for (auto &t : hl.fwd) fwd.push_back(tw_t{t.w, t.wp});
        for (auto &t : hl.inv) inv.push_back(tw_t{t.w, t.wp});
        ninv = tw_t{hl.ninv.w, hl.ninv.wp};
        wn = tw_t{hl.wn.w, hl.wn.wp};
    }
};
template <>
struct Tables<ModF64> {
    std::vector<double> fwd, inv;
    double ninv, wn;
    ModF64 m;
    explicit Tables(const HostLimb &hl) : m{(double)hl.q, 1.0 / (double)hl.q} {
        for (auto &t : hl.fwd) fwd.push_back((double)t.w);
        for (auto &t : hl.inv) inv.push_back((double)t.w);
        ninv = (double)hl.ninv.w;
        wn = (double)hl.wn.w;
    }
};

// the shared-memory words one virtual warp touches in phase P (sorted)
template <class L, int P>
static std::vector<uint32_t> warp_words(uint32_t vw) {
    std::vector<uint32_t> w;
    for (uint32_t lane = 0; lane < 32; lane++)
        for (int r = 0; r < L::E; r++) w.push_back(wswz(L::template base<P>(vw, lane) | L::template reg<P>(r)));
    std::sort(w.begin(), w.end());
    return w;
}

// Inside a super-phase only a warp-level barrier separates the phases, so a
// virtual warp must work on the same words in all of them.
template <class L, int P = 0>
static void check_closure() {
    if constexpr (P + 1 < L::NPH && P + 1 != L::SPLIT) {
        for (uint32_t vw = 0; vw < (uint32_t)L::NW; vw++)
        {
            const std::vector<uint32_t> here = warp_words<L, P>(vw), next = warp_words<L, P + 1>(vw);
            CHECK(here == next, "warp %u leaves its words between phases %d and %d", vw, P, P + 1);
        }
    }
    if constexpr (P + 1 < L::NPH) check_closure<L, P + 1>();
}

// one block of 2^LOGB values, piece `blk` of a transform cut into 2^A blocks, all phases
template <class L, class M, int P = 0>
static void forward_block(std::vector<uint64_t> &sm, const NttArgsT<M> &a, double *max_abs) {
    std::vector<uint64_t> out(sm.size());
    std::vector<int> writers(sm.size(), 0);
    for (uint32_t vw = 0; vw < (uint32_t)L::NW; vw++)
        for (uint32_t lane = 0; lane < 32; lane++) {
            const uint32_t base = L::template base<P>(vw, lane);
            typename M::val x[L::E];
            for (int r = 0; r < L::E; r++) {
                CHECK((base & L::template reg<P>(r)) == 0, "register bits overlap the thread's bits");
                x[r] = M::from_bits(sm[wswz(base | L::template reg<P>(r))]);
            }
            fwd_phase<L, P>(x, base, a);
            for (int r = 0; r < L::E; r++) {
                const uint32_t i = wswz(base | L::template reg<P>(r));
                CHECK(i < sm.size(), "index out of the block");
                writers[i]++;
                out[i] = M::bits(x[r]);
                if (max_abs) *max_abs = std::fmax(*max_abs, std::fabs((double)x[r]));
            }
            if (P == L::NPH - 1)
                for (int r = 0; r < L::E; r += 2)
                    CHECK((L::template reg<P>(r) & 1u) == 0 && L::template reg<P>(r + 1) == (L::template reg<P>(r) | 1u),
                          "the last phase hands out pairs of neighbours");
        }
    for (int wcount : writers) CHECK(wcount == 1, "every word has exactly one owner per phase");
    sm = out;
    if constexpr (P + 1 < L::NPH) forward_block<L, M, P + 1>(sm, a, max_abs);
}

template <class L, class M, class T, bool SCALED, int P = L::NPH - 1>
static void inverse_block(std::vector<uint64_t> &sm, const NttArgsT<M> &a, const T &ninv, const T &wn,
                          double *max_abs) {
    std::vector<uint64_t> out(sm.size());
    for (uint32_t vw = 0; vw < (uint32_t)L::NW; vw++)
        for (uint32_t lane = 0; lane < 32; lane++) {
            const uint32_t base = L::template base<P>(vw, lane);
            typename M::val x[L::E];
            for (int r = 0; r < L::E; r++) x[r] = M::from_bits(sm[wswz(base | L::template reg<P>(r))]);
            if constexpr (P == 0 && SCALED) {
                inv_phase<L, 0, 1>(x, base, a);
                inv_stage0_scaled<L>(x, a.m, ninv, wn);
            } else {
                inv_phase<L, P, 0>(x, base, a);
            }
            for (int r = 0; r < L::E; r++) {
                out[wswz(base | L::template reg<P>(r))] = M::bits(x[r]);
                if (max_abs) *max_abs = std::fmax(*max_abs, std::fabs((double)x[r]));
            }
        }
    sm = out;
    if constexpr (P > 0) inverse_block<L, M, T, SCALED, P - 1>(sm, a, ninv, wn, max_abs);
}

// whole transform of length N = 2^A * 2^LOGB: outer stages done plainly here
// (pairs at distance N/2, N/4, ...), block stages by the code under test
template <class L, class M>
static void check_transform(uint32_t A, uint64_t q, int samples) {
    const int logN = L::LOGB + (int)A;
    const uint32_t N = 1u << logN, B = 1u << L::LOGB;
    HostLimb hl;
    host_build_limb(N, q, hl);
    Tables<M> tab(hl);
    std::vector<uint64_t> a(N);
    for (auto &v : a) v = rnd() % q;
    a[0] = q - 1;
    a[N - 1] = q - 1;

    // forward
    std::vector<typename M::val> x(N);
    for (uint32_t i = 0; i < N; i++) x[i] = tab.m.from_residue(a[i]);
    for (uint32_t s = 0; s < A; s++) {
        const uint32_t half = N >> (s + 1);
        for (uint32_t i = 0; i < N; i++) {
            if (i & half) continue;
            tab.m.fwd(x[i], x[i | half], tab.fwd[(1u << s) + (i >> (logN - s))]);
        }
    }
    std::vector<uint64_t> hat(N);
    double max_fwd = 0;
    for (uint32_t blk = 0; blk < (1u << A); blk++) {
        std::vector<uint64_t> sm(B);
        for (uint32_t i = 0; i < B; i++) sm[wswz(i)] = M::bits(x[blk * B + i]);
        const NttArgsT<M> args{tab.fwd.data(), tab.m, A, blk};
        forward_block<L, M>(sm, args, &max_fwd);
        for (uint32_t i = 0; i < B; i++) hat[blk * B + i] = tab.m.canon_wide(M::from_bits(sm[wswz(i)]));
    }
    if (std::is_same<M, ModF64>::value)
        CHECK(max_fwd <= 13.0 * (double)q, "forward values stay below 13 q (%.2f q)", max_fwd / (double)q);
    for (int t = 0; t < samples; t++) {
        const uint32_t k = t == 0 ? 0 : (t == 1 ? N - 1 : (uint32_t)(rnd() % N));
        CHECK(hat[k] == eval_definition(a, hl.psi, q, k, logN), "forward output %u (N=%u, A=%u)", k, N, A);
    }

    // inverse: block stages, then the outer stages with 1/N folded into stage 0
    std::vector<typename M::val> y(N);
    double max_inv = 0;
    for (uint32_t blk = 0; blk < (1u << A); blk++) {
        std::vector<uint64_t> sm(B);
        for (uint32_t i = 0; i < B; i++) sm[wswz(i)] = M::bits(tab.m.from_residue(hat[blk * B + i]));
        const NttArgsT<M> args{tab.inv.data(), tab.m, A, blk};
        if (A == 0) inverse_block<L, M, decltype(tab.ninv), true>(sm, args, tab.ninv, tab.wn, &max_inv);
        else inverse_block<L, M, decltype(tab.ninv), false>(sm, args, tab.ninv, tab.wn, &max_inv);
        for (uint32_t i = 0; i < B; i++) y[blk * B + i] = M::from_bits(sm[wswz(i)]);
    }
    if (std::is_same<M, ModF64>::value)
        CHECK(max_inv <= (double)q, "inverse values are back below q after every phase (%.2f q)", max_inv / (double)q);
    for (int s = (int)A - 1; s >= 0; s--) {
        const uint32_t half = N >> (s + 1);
        for (uint32_t i = 0; i < N; i++) {
            if (i & half) continue;
            if (s == 0) tab.m.inv_scaled(y[i], y[i | half], tab.ninv, tab.wn);
            else tab.m.inv(y[i], y[i | half], tab.inv[(1u << s) + (i >> (logN - s))]);
        }
    }
    for (uint32_t i = 0; i < N; i++) CHECK(tab.m.canon(y[i]) == a[i], "round trip at %u (N=%u, A=%u)", i, N, A);
}

// the swizzle keeps the 16 lanes of every half-warp on 16 different banks of
// 8 bytes in every phase layout, and permutes every aligned group of 16 words
template <class L, int P = 0>
static void check_banks() {
    for (uint32_t vw = 0; vw < (uint32_t)L::NW; vw++)
        for (int r = 0; r < L::E; r++)
            for (int halfwarp = 0; halfwarp < 2; halfwarp++) {
                uint32_t seen = 0;
                for (uint32_t l = 0; l < 16; l++) {
                    const uint32_t i = L::template base<P>(vw, halfwarp * 16 + l) | L::template reg<P>(r);
                    const uint32_t bank = wswz(i) & 15u;   // 16 banks of 8 bytes
                    CHECK(!(seen & (1u << bank)), "bank conflict in phase %d", P);
                    seen |= 1u << bank;
                }
            }
    if constexpr (P + 1 < L::NPH) check_banks<L, P + 1>();
}

int main() {
    for (uint32_t g = 0; g < (1u << 14); g += 16) {
        uint32_t seen = 0;
        for (uint32_t i = 0; i < 16; i++) {
            CHECK((wswz(g + i) & ~15u) == g, "swizzle leaves its group");
            seen |= 1u << (wswz(g + i) & 15u);
        }
        CHECK(seen == 0xffffu, "swizzle is not a permutation");
    }
    const uint64_t q60 = 0xffffffffffc0001ull, q45 = 0x1fffffc20001ull, q40 = 0xffffe80001ull;
    check_f64_primitives(q45);
    check_f64_primitives(q40);
    check_f64_primitives((1ull << 46) - 2 * 65536 * 3 + 1);   // any odd modulus below 2^46 serves the arithmetic
    check_banks<WLay<13>>();
    check_banks<WLay<14>>();
    check_closure<WLay<13>>();
    check_closure<WLay<14>>();
    // whole blocks
    check_transform<WLay<13>, ModInt>(0, q60, 24);
    check_transform<WLay<13>, ModF64>(0, q45, 24);
    check_transform<WLay<14>, ModInt>(0, q60, 12);
    check_transform<WLay<14>, ModF64>(0, q40, 12);
    check_transform<WLay<13>, ModInt>(0, q40, 12);          // a small prime in integer arithmetic
    // pieces of longer transforms (the two-group encrypt and the long rings)
    check_transform<WLay<13>, ModInt>(1, q60, 8);
    check_transform<WLay<13>, ModF64>(1, q40, 8);
    check_transform<WLay<13>, ModF64>(2, q45, 6);
    check_transform<WLay<13>, ModInt>(3, q60, 4);
    check_transform<WLay<13>, ModF64>(3, q45, 4);
    printf("ok\n");
    return 0;
}
