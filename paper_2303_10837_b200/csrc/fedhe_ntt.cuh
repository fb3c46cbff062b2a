// Register-tiled negacyclic NTT of one block of B = 2^LOGB residues held by
// one thread block in shared memory: a thread takes E = 8 residues into
// registers, does up to three butterfly stages on them and puts them back;
// between such phases the elements change hands, inside a warp where the
// layout allows it and across the block once per transform.
//
// Index conventions (forward transform, natural order in, bit-reversed out):
// stage s (0-based) of a length-N transform pairs the elements whose indices
// differ in bit logN-1-s and uses the twiddle  tw[2^s + (index >> (logN - s))],
// tw[i] = psi^brev(i).  The inverse transform runs the stages backwards with
// the inverse table.  A block may be one of 2^A consecutive pieces of a
// longer transform (N = 2^A B) whose first A stages were done elsewhere; then
// the local stage s' is the global stage A + s' and the block index enters
// the twiddle index.
#pragma once

#include <type_traits>

#include "fedhe_device.cuh"

namespace fedhe {

struct tw_t { uint64_t w, wp; };   // twiddle and its Shoup companion floor(w 2^64 / q)

#if defined(__CUDACC__)
// 16-byte read-only load of a table entry
__device__ __forceinline__ tw_t load_tw(const tw_t *p) {
    ulonglong2 v = __ldg(reinterpret_cast<const ulonglong2 *>(p));
    tw_t t = {v.x, v.y};
    return t;
}
#endif
#if defined(__CUDA_ARCH__)
#define FEDHE_LD_TW(p) load_tw(p)
#else
#define FEDHE_LD_TW(p) (*(p))
#endif

struct alignas(16) u64x2 { uint64_t x, y; };   // two neighbouring residues
template <class V>
struct pair_of { V x, y; };                      // two neighbouring values of an arithmetic

// Index swizzle and thread layout of the complex slot transform (its kernels
// keep their values in registers across phases and exchange them through
// shared memory between phases).  XOR-ing t ^ (t << 1), t = index bits 4..6,
// into the low nibble spreads the accesses of every phase layout over the
// banks; the map permutes every aligned group of 16 words.
HD uint32_t swz(uint32_t i) {
    const uint32_t t = (i >> 4) & 7u;
    return i ^ t ^ ((t << 1) & 15u);
}

// Phase p < NPH-1 keeps in registers the elements that differ in index bits
// [lo, lo+LE), lo = LOGB - (p+1) LE; the last phase holds the remaining R low
// bits plus the LE-R top bits.
template <int LOGB_, int LE_>
struct Lay {
    static constexpr int LOGB = LOGB_, LE = LE_;
    static constexpr int E = 1 << LE;
    static constexpr int NT = 1 << (LOGB - LE);
    static constexpr int NPH = (LOGB + LE - 1) / LE;
    static constexpr int R = LOGB - (NPH - 1) * LE;   // stages of the last phase, 1..LE
    static constexpr int HB = LE - R;                 // top bits held in the last phase

    // element index held in register r of thread tid during phase P
    template <int P>
    static HD uint32_t idx(uint32_t tid, int r) {
        if constexpr (P < NPH - 1) {
            constexpr int lo = LOGB - (P + 1) * LE;
            return ((tid >> lo) << (lo + LE)) | ((uint32_t)r << lo) | (tid & ((1u << lo) - 1u));
        } else {
            uint32_t rl = (uint32_t)r & ((1u << R) - 1u), rh = (uint32_t)r >> R;
            return (rh << (LOGB - HB)) | (tid << R) | rl;
        }
    }

    // index >> (LOGB - s) for the butterflies of local stage s = P LE + i whose
    // lower register has the given group number g (the register bits above the
    // pair bit)
    template <int P, int I>
    static HD uint32_t top(uint32_t tid, int r) {
        constexpr int s = P * LE + I;
        return idx<P>(tid, r) >> (LOGB - s);
    }
};

// ---- runs of consecutive table entries ---------------------------------------
//
// Inside a phase the twiddles of stage I of one thread are 2^I consecutive
// table entries starting at a multiple of 2^I, so they come in with 16- and
// 32-byte loads (one address computation each) instead of one load per entry.
template <int K>
HD void load_run(const double *p, double (&w)[K]) {
#if defined(__CUDA_ARCH__)
    if constexpr (K == 1) {
        w[0] = __ldg(p);
    } else if constexpr (K == 2) {
        const double2 v = __ldg(reinterpret_cast<const double2 *>(p));
        w[0] = v.x;
        w[1] = v.y;
    } else {
#pragma unroll
        for (int i = 0; i < K; i += 4)
            asm("ld.global.nc.v4.f64 {%0,%1,%2,%3}, [%4];"
                : "=d"(w[i]), "=d"(w[i + 1]), "=d"(w[i + 2]), "=d"(w[i + 3])
                : "l"(p + i));
    }
#else
    for (int i = 0; i < K; i++) w[i] = p[i];
#endif
}
template <int K>
HD void load_run(const tw_t *p, tw_t (&w)[K]) {
#if defined(__CUDA_ARCH__)
    if constexpr (K == 1) {
        w[0] = load_tw(p);
    } else {
#pragma unroll
        for (int i = 0; i < K; i += 2)
            asm("ld.global.nc.v4.u64 {%0,%1,%2,%3}, [%4];"
                : "=l"(w[i].w), "=l"(w[i].wp), "=l"(w[i + 1].w), "=l"(w[i + 1].wp)
                : "l"(p + i));
    }
#else
    for (int i = 0; i < K; i++) w[i] = p[i];
#endif
}

// ---- arithmetic of one limb ---------------------------------------------------
//
// ModInt: any prime below 2^61; 64-bit integers in the lazy Harvey ranges
// (forward [0, 4q), inverse [0, 2q)), table entries {w, floor(w 2^64 / q)}.
// ModF64: primes below 2^46; signed integers in doubles, table entries the
// twiddles as doubles.  Forward, every stage adds at most 3q/4 to the bound
// (q at the input, at most 13q after 16 stages); inverse, sums double and
// differences go through the product, so after the at most three stages of a
// phase the sums are brought back below q (settle) before they are stored.

// SEL: conditional subtractions by bitwise selects (csub_sel) instead of predicated moves
template <bool SEL>
struct ModIntT {
    static constexpr int UNROLL_V = 1;   // virtual threads of a phase one after the other
    using val = uint64_t;
    using tab = tw_t;
    uint64_t q, q2;
    static HD val from_bits(uint64_t b) { return b; }
    static HD uint64_t bits(val v) { return v; }
    static HD tw_t load(const tw_t *p) { return FEDHE_LD_TW(p); }
    HD void fwd(val &x, val &y, const tw_t &w) const { ct_butterfly<SEL>(x, y, w.w, w.wp, q, q2); }
    HD void inv(val &x, val &y, const tw_t &w) const { gs_butterfly<SEL>(x, y, w.w, w.wp, q, q2); }
    // x <- (x + y) a, y <- (x - y) b for inputs below 2q; outputs below 2q
    HD void inv_scaled(val &x, val &y, const tw_t &a, const tw_t &b) const {
        const uint64_t u = x, v = y;
        x = shoup_lazy(u + v, a.w, a.wp, q);
        y = shoup_lazy(u - v + q2, b.w, b.wp, q);
    }
    HD val settle(val v) const { return v; }
    // conversions: a residue below 2q <-> the value; a small signed integer -> the value
    HD val from_residue(uint64_t r) const { return r; }
    HD uint64_t to_residue(val v) const { return v; }
    HD val small(int v) const { return small_residue(v, q); }
    // canonical residue of a forward output (below 4q) / of an inverse output (below 2q),
    // and of an inverse output plus a residue in [0, q)
    HD uint64_t canon_wide(val v) const { return csub_as<SEL>(csub_as<SEL>(v, q2), q); }
    HD uint64_t canon(val v) const { return csub_as<SEL>(v, q); }
    HD uint64_t canon_add(val v, uint64_t add) const { return csub_as<SEL>(csub_as<SEL>(v, q) + add, q); }
    // canonical residue of a forward output plus a key product
    HD uint64_t canon_sum(val a, val b) const { return csub_as<SEL>(canon_wide(a) + csub_as<SEL>(b, q), q); }
    // product with an entry of a key table, below 2q for any v
    using key = tw_t;
    static HD key load_key(const tw_t *p) { return FEDHE_LD_TW(p); }
    HD val mul_key(val v, const key &k) const { return shoup_lazy(v, k.w, k.wp, q); }
};

using ModInt = ModIntT<false>;
using ModIntSel = ModIntT<true>;

struct ModF64 {
    static constexpr int UNROLL_V = 2;
    using val = double;
    using tab = double;
    double q, qi;        // the prime and its rounded reciprocal
    static HD val from_bits(uint64_t b) { return f64_from_bits(b); }
    static HD uint64_t bits(val v) { return f64_bits(v); }
    static HD double load(const double *p) {
#if defined(__CUDA_ARCH__)
        return __ldg(p);
#else
        return *p;
#endif
    }
    HD double mul(double y, double w) const { return f64_mulmod(y, w, q, qi); }
    HD void fwd(val &x, val &y, double w) const {
        const double u = x, t = mul(y, w);
        x = f64_add(u, t);
        y = f64_sub(u, t);
    }
    HD void inv(val &x, val &y, double w) const {
        const double u = x, v = y;
        x = f64_add(u, v);
        y = mul(f64_sub(u, v), w);
    }
    HD void inv_scaled(val &x, val &y, double a, double b) const {
        const double u = x, v = y;
        x = mul(f64_add(u, v), a);
        y = mul(f64_sub(u, v), b);
    }
    HD val settle(val v) const { return f64_reduce(v, q, qi); }
    HD val from_residue(uint64_t r) const { return f64_from_u64(r); }
    HD uint64_t to_residue(val v) const { return f64_canonical(v, q); }          // |v| < q
    HD val small(int v) const { return (double)v; }
    HD uint64_t canon_wide(val v) const { return f64_canonical(f64_reduce(v, q, qi), q); }
    HD uint64_t canon(val v) const { return f64_canonical(v, q); }               // |v| < q
    HD uint64_t canon_add(val v, uint64_t add) const {                           // |v| < q
        const double r = f64_add(v, f64_from_u64(add));
        return f64_canonical(r >= q ? f64_sub(r, q) : r, q);
    }
    HD uint64_t canon_sum(val a, val b) const { return canon_wide(f64_add(a, b)); }
    // only the value of a key-table entry is read; |result| <= 3q/4
    using key = double;
    static HD key load_key(const tw_t *p) {
#if defined(__CUDA_ARCH__)
        return f64_from_u64(__ldg(&p->w));
#else
        return f64_from_u64(p->w);
#endif
    }
    HD val mul_key(val v, key k) const { return mul(v, k); }
};

// ---- warp-local layout --------------------------------------------------------
//
// The 3 * 4 + R stages of a block run in five phases of (3, 3, 3, 3, R) stages,
// R = LOGB - 12.  In every phase a virtual thread holds E = 8 elements that
// differ in three index bits (the register bits: the bits the phase's
// butterflies pair, plus 3 - R idle bits in the last phase), the 32 lanes of
// its virtual warp differ in five more (the lane bits), and the remaining
// LOGB - 8 bits number the virtual warp.  Register and lane bits are chosen so
// that a virtual warp works on one and the same set of 256 elements
// throughout phases 0-1 and on another throughout phases 2-4: inside such a
// super-phase the elements change hands between the lanes of one warp only, a
// warp-level barrier orders the exchange, and the warps of a block drift apart
// (one warp's shared-memory traffic overlaps another's arithmetic).  Only the
// step from phase 1 to phase 2 needs a barrier over the whole block.
//
// Register bits:  phase P < 4: LOGB - 3 (P + 1) + {0, 1, 2};
//                 phase 4: {0 .. R-1} (paired) and the top 3 - R bits below bit 8.
// Lane bits (lane bit 0 first) and virtual-warp bits:
//   LOGB 14: {0,1,8,9,10} {0,1,11,12,13} | {0,1,2,3,4} {0,1,5,6,7} {2,3,4,5,6};  warp: 2..7 | 8..13
//   LOGB 13: {0,1,8,9,7}  {0,1,11,12,10} | {0,1,2,3,7} {0,4,5,6,7} {1,2,3,4,5};  warp: 2..6 | 8..12
// In the last phase a thread owns runs of 2^R neighbouring elements and the
// lanes of a warp follow one another, so that a warp reads and writes whole
// lines of global memory.

// Shared-memory index swizzle for 8-byte words.  A 64-bit access of a warp is
// served half-warp by half-warp from 16 banks of 8 bytes (the low four index
// bits); the 16 lanes of a half-warp differ in the index bits named first in
// the lists above.  The map XORs into the low nibble, as linear maps over
// GF(2), the columns 0011, 0110, 1100 for index bits 4, 5, 6 and 0100, 1000
// for bits 8, 9 and again for bits 11, 12, which makes the bank a bijection of
// each of those sets of four bits; it permutes every aligned group of 16 words.
HD uint32_t wswz(uint32_t i) {
    const uint32_t t = (i >> 4) & 7u;
    return i ^ t ^ ((t << 1) & 15u) ^ ((((i >> 8) ^ (i >> 11)) & 3u) << 2);
}

template <int LOGB_>
struct WLay {
    static_assert(LOGB_ == 13 || LOGB_ == 14, "blocks of 2^13 or 2^14 elements");
    static constexpr int LOGB = LOGB_, LE = 3, E = 8, NPH = 5;
    static constexpr int SPLIT = 2;                       // phases [0, SPLIT) and [SPLIT, NPH) are the super-phases
    static constexpr int NT = 1 << (LOGB - LE);           // virtual threads
    static constexpr int NW = NT / 32;                    // virtual warps
    static constexpr int WB = LOGB - 8;                   // index bits that number the virtual warp
    static constexpr int R = LOGB - 12;                   // stages of the last phase

    static HD constexpr int nst(int P) { return P < NPH - 1 ? LE : R; }
    static HD constexpr int reg_bit(int P, int k) {
        if (P < NPH - 1) return LOGB - LE * (P + 1) + k;
        return k < R ? k : 8 - (LE - R) + (k - R);
    }
    static HD constexpr int lane_bit(int P, int k) {
        constexpr int t14[5][5] = {{0, 1, 8, 9, 10}, {0, 1, 11, 12, 13}, {0, 1, 2, 3, 4}, {0, 1, 5, 6, 7}, {2, 3, 4, 5, 6}};
        constexpr int t13[5][5] = {{0, 1, 8, 9, 7}, {0, 1, 11, 12, 10}, {0, 1, 2, 3, 7}, {0, 4, 5, 6, 7}, {1, 2, 3, 4, 5}};
        return LOGB == 14 ? t14[P][k] : t13[P][k];
    }
    static HD constexpr int warp_bit(int P, int k) { return (P < SPLIT ? 2 : 8) + k; }

    // bits [K, K + len) of x go to consecutive index bits: one shift and mask per run
    template <int P, bool LANE, int K>
    static HD constexpr int run() {
        constexpr int NB = LANE ? 5 : WB;
        int len = 1;
        while (K + len < NB &&
               (LANE ? lane_bit(P, K + len) : warp_bit(P, K + len)) == (LANE ? lane_bit(P, K) : warp_bit(P, K)) + len)
            len++;
        return len;
    }
    template <int P, bool LANE, int K = 0>
    static HD uint32_t deposit(uint32_t x) {
        constexpr int NB = LANE ? 5 : WB;
        if constexpr (K >= NB) {
            return 0u;
        } else {
            constexpr int len = run<P, LANE, K>();
            constexpr int pos = LANE ? lane_bit(P, K) : warp_bit(P, K);
            return (((x >> K) & ((1u << len) - 1u)) << pos) | deposit<P, LANE, K + len>(x);
        }
    }
    // index of the element in register 0 of a lane of a virtual warp in phase P
    template <int P>
    static HD uint32_t base(uint32_t vwarp, uint32_t lane) {
        return deposit<P, true>(lane) | deposit<P, false>(vwarp);
    }
    // what register r adds to that index
    template <int P>
    static HD constexpr uint32_t reg(int r) {
        uint32_t i = 0;
        for (int k = 0; k < LE; k++) i |= (uint32_t)((r >> k) & 1) << reg_bit(P, k);
        return i;
    }
};

// ---- phases ----------------------------------------------------------------

template <class M>
struct NttArgsT {
    const typename M::tab *tw;   // table of this limb and direction, indexed by the global twiddle index
    M m;                         // the limb's arithmetic
    uint32_t A;                  // log2 of the number of blocks the whole transform is cut into
    uint32_t blk;                // which block this is
};
using NttArgs = NttArgsT<ModInt>;
using NttArgsF = NttArgsT<ModF64>;

// Local stage s = 3 P + I pairs the elements that differ in index bit
// LOGB - 1 - s and uses the twiddle with index 2^(A+s) + (blk << s) +
// (index >> (LOGB - s)).  In the phases before the last, the indices of a
// thread's registers agree above the register bits, so the 2^I twiddles of
// stage I are consecutive table entries: w[g] serves the butterflies whose
// lower register has r >> (3 - I) == g.
template <class L, int P, int I, class M>
HD void stage_twiddles(typename M::tab (&w)[1 << I], uint32_t base, const NttArgsT<M> &a) {
    static_assert(P < L::NPH - 1, "in the last phase the registers of a group are far apart in the index");
    constexpr int s = P * L::LE + I;
    constexpr int above = L::reg_bit(P, 0) + L::LE;        // index bits above the register bits
    load_run<1 << I>(a.tw + (1u << (a.A + s)) + (a.blk << s) + ((base >> above) << I), w);
}

// twiddle of a butterfly of the last phase whose lower element has index i
template <class L, int I, class M>
HD auto last_twiddle(uint32_t i, const NttArgsT<M> &a) {
    constexpr int s = (L::NPH - 1) * L::LE + I;
    return M::load(a.tw + (1u << (a.A + s)) + (a.blk << s) + (i >> (L::LOGB - s)));
}

template <class L, int P, int I, class M>
HD void fwd_stage(typename M::val (&x)[L::E], uint32_t base, const NttArgsT<M> &a) {
    constexpr int nst = L::nst(P);
    constexpr int bit = nst - 1 - I;              // register bit of the pair
    if constexpr (P < L::NPH - 1) {
        typename M::tab w[1 << I];
        stage_twiddles<L, P, I>(w, base, a);
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            a.m.fwd(x[r], x[r | (1 << bit)], w[r >> (nst - I)]);
        }
    } else {
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            // registers that agree above the pair bit share one twiddle; the
            // compiler merges the equal loads of an unrolled group
            a.m.fwd(x[r], x[r | (1 << bit)], last_twiddle<L, I>(base + L::template reg<P>(r), a));
        }
    }
}

template <class L, int P, int I, class M>
HD void inv_stage(typename M::val (&x)[L::E], uint32_t base, const NttArgsT<M> &a) {
    constexpr int nst = L::nst(P);
    constexpr int bit = nst - 1 - I;
    if constexpr (P < L::NPH - 1) {
        typename M::tab w[1 << I];
        stage_twiddles<L, P, I>(w, base, a);
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            a.m.inv(x[r], x[r | (1 << bit)], w[r >> (nst - I)]);
        }
    } else {
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            a.m.inv(x[r], x[r | (1 << bit)], last_twiddle<L, I>(base + L::template reg<P>(r), a));
        }
    }
}

// last inverse stage of a whole transform (global stage 0) with the factor
// 1/N folded in: x <- (x + y)/N, y <- (x - y) w /N.  ninv = 1/N, wn = w/N.
template <class L, class M, class T>
HD void inv_stage0_scaled(typename M::val (&x)[L::E], const M &m, const T &ninv, const T &wn) {
    constexpr int bit = L::LE - 1;
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        if (r & (1 << bit)) continue;
        m.inv_scaled(x[r], x[r | (1 << bit)], ninv, wn);
    }
}

template <class L, int P, int I = 0, class M>
HD void fwd_phase(typename M::val (&x)[L::E], uint32_t base, const NttArgsT<M> &a) {
    if constexpr (I < L::nst(P)) {
        fwd_stage<L, P, I>(x, base, a);
        fwd_phase<L, P, I + 1>(x, base, a);
    }
}

// inverse phase: stages nst-1 down to STOP (STOP = 1 leaves stage 0 of the
// phase to the caller); a phase that ends with an ordinary stage settles the
// sums of that stage (the registers whose pair bit is clear)
template <class L, int P, int STOP, int I, class M>
HD void inv_phase_from(typename M::val (&x)[L::E], uint32_t base, const NttArgsT<M> &a) {
    if constexpr (I >= STOP) {
        inv_stage<L, P, I>(x, base, a);
        inv_phase_from<L, P, STOP, I - 1>(x, base, a);
    } else if constexpr (STOP == 0) {
#pragma unroll
        for (int r = 0; r < L::E; r++)
            if (!(r & (1 << (L::nst(P) - 1)))) x[r] = a.m.settle(x[r]);
    }
}

template <class L, int P, int STOP = 0, class M>
HD void inv_phase(typename M::val (&x)[L::E], uint32_t base, const NttArgsT<M> &a) {
    inv_phase_from<L, P, STOP, L::nst(P) - 1>(x, base, a);
}

#if defined(__CUDACC__)
// ---------------------------------------------------------------------------
// Whole-block transforms.  The block's residues stay in shared memory
// (swizzled) and every warp plays V virtual warps per phase; a virtual thread
// loads its E residues, does the phase's butterflies in registers and stores
// them back to the same places, so that only E residues are live per thread
// at a time (E = 8 keeps a 1024-thread block within 64 registers with no
// spills) and no separate exchange buffer is needed.  The first phase takes
// its input from `src`, the last hands its output to `dst`:
//   forward:  src(i) -> residue i;            dst(i, a, b): residues i, i+1
//   inverse:  src(i) -> residues i, i+1 (members x, y);   dst(i, a): residue i
// all in the value type of the limb's arithmetic (pairs always start at an
// even index and are neighbours in memory).  The thread that hands element i
// to `dst` is the one that read it from `src` or from shared memory word
// wswz(i) in the same phase, so `dst` may overwrite that word.
// ---------------------------------------------------------------------------

// Barrier over the whole thread block, or over one of its halves / quarters
// when several groups of threads transform separate sub-blocks on their own
// schedules (named barrier 1 + group; every thread of the group must call it).
struct BlockSync {
    __device__ __forceinline__ void operator()() const { __syncthreads(); }
};
struct GroupSync {
    uint32_t id, nthreads;
    __device__ __forceinline__ void operator()() const {
        asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
    }
};

// Word of register r of a thread, given the 32-bit shared-memory address `a0`
// of its register-0 word (sm + wswz(base)).  The swizzle is linear over GF(2)
// and `base` is zero at the register bits, so the word index is
// wswz(base) ^ wswz(reg(r)); of that constant the part above the low nibble
// only sets bits that are clear in wswz(base), i.e. it adds and folds into the
// instruction's offset, while the nibble is XOR-ed into the address itself
// (which needs `sm` on a 128-byte boundary): one logic operation per distinct
// nibble instead of an XOR and a scaled add per access.
template <class L, int P>
__device__ __forceinline__ uint64_t *reg_word(uint32_t a0, int r) {
    const uint32_t k = wswz(L::template reg<P>(r));
    const uint32_t a = (a0 ^ ((k & 15u) << 3)) + ((k & ~15u) << 3);
    return reinterpret_cast<uint64_t *>(__cvta_shared_to_generic((size_t)a));
}
__device__ __forceinline__ uint32_t word_address(const uint64_t *sm, uint32_t word) {
    return (uint32_t)__cvta_generic_to_shared(sm) + (word << 3);
}

// phases [P, PEND) of a forward transform, a warp-level barrier between them
template <class L, int V, int P, int PEND, class M, class Src, class Dst>
__device__ __forceinline__ void forward_phases(uint64_t *sm, uint32_t warp, uint32_t lane, const NttArgsT<M> &a,
                                               const Src &src, const Dst &dst) {
    constexpr int LAST = L::NPH - 1;
#pragma unroll M::UNROLL_V
    for (int v = 0; v < V; v++) {
        const uint32_t base = L::template base<P>(warp + v * (L::NW / V), lane);
        const uint32_t a0 = word_address(sm, wswz(base));
        typename M::val x[L::E];
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if constexpr (P == 0) {
                // a source may take the index in two parts, base (zero at the register bits, the
                // same for all E calls) and the register's constant, to hoist what depends on base
                if constexpr (std::is_invocable<Src, uint32_t, uint32_t>::value) x[r] = src(base, L::template reg<P>(r));
                else x[r] = src(base + L::template reg<P>(r));
            } else {
                x[r] = M::from_bits(*reg_word<L, P>(a0, r));
            }
        }
        fwd_phase<L, P>(x, base, a);
        if constexpr (P == LAST) {
#pragma unroll
            for (int r = 0; r < L::E; r += 2) {
                // a sink that keeps the pair in this buffer may take the two words' addresses
                // (one logic operation each) instead of swizzling the index itself
                if constexpr (std::is_invocable<Dst, uint32_t, typename M::val, typename M::val, uint64_t *, uint64_t *>::value)
                    dst(base + L::template reg<P>(r), x[r], x[r + 1], reg_word<L, P>(a0, r), reg_word<L, P>(a0, r + 1));
                else
                    dst(base + L::template reg<P>(r), x[r], x[r + 1]);
            }
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) *reg_word<L, P>(a0, r) = M::bits(x[r]);
        }
    }
    if constexpr (P + 1 < PEND) {
        __syncwarp();
        forward_phases<L, V, P + 1, PEND>(sm, warp, lane, a, src, dst);
    }
}

template <class L, int V, class M, class Src, class Dst, class Sync = BlockSync>
__device__ __forceinline__ void smem_ntt_forward(uint64_t *sm, uint32_t tid, const NttArgsT<M> &a, const Src &src,
                                                 const Dst &dst, const Sync &sync = Sync()) {
    const uint32_t warp = tid >> 5, lane = tid & 31u;
    forward_phases<L, V, 0, L::SPLIT>(sm, warp, lane, a, src, dst);
    sync();
    forward_phases<L, V, L::SPLIT, L::NPH>(sm, warp, lane, a, src, dst);
}

// phases P down to PEND of an inverse transform
template <class L, int V, bool SCALED, int P, int PEND, class M, class T, class Src, class Dst>
__device__ __forceinline__ void inverse_phases(uint64_t *sm, uint32_t warp, uint32_t lane, const NttArgsT<M> &a,
                                               const T &ninv, const T &wn, const Src &src, const Dst &dst) {
    constexpr int LAST = L::NPH - 1;
#pragma unroll M::UNROLL_V
    for (int v = 0; v < V; v++) {
        const uint32_t base = L::template base<P>(warp + v * (L::NW / V), lane);
        const uint32_t a0 = word_address(sm, wswz(base));
        typename M::val x[L::E];
        if constexpr (P == LAST) {
#pragma unroll
            for (int r = 0; r < L::E; r += 2) {
                if constexpr (std::is_invocable<Src, uint32_t, const uint64_t *, const uint64_t *>::value) {
                    const auto t = src(base + L::template reg<P>(r), reg_word<L, P>(a0, r), reg_word<L, P>(a0, r + 1));
                    x[r] = t.x;
                    x[r + 1] = t.y;
                } else {
                    const auto t = src(base + L::template reg<P>(r));
                    x[r] = t.x;
                    x[r + 1] = t.y;
                }
            }
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) x[r] = M::from_bits(*reg_word<L, P>(a0, r));
        }
        if constexpr (P == 0 && SCALED) {
            inv_phase<L, 0, 1>(x, base, a);
            inv_stage0_scaled<L>(x, a.m, ninv, wn);
        } else {
            inv_phase<L, P, 0>(x, base, a);
        }
        if constexpr (P == 0) {
#pragma unroll
            for (int r = 0; r < L::E; r++) {
                if constexpr (std::is_invocable<Dst, uint32_t, typename M::val, uint64_t *>::value)
                    dst(base + L::template reg<P>(r), x[r], reg_word<L, P>(a0, r));
                else
                    dst(base + L::template reg<P>(r), x[r]);
            }
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) *reg_word<L, P>(a0, r) = M::bits(x[r]);
        }
    }
    if constexpr (P > PEND) {
        __syncwarp();
        inverse_phases<L, V, SCALED, P - 1, PEND>(sm, warp, lane, a, ninv, wn, src, dst);
    }
}

template <class L, int V, bool SCALED, class M, class T, class Src, class Dst, class Sync = BlockSync>
__device__ __forceinline__ void smem_ntt_inverse(uint64_t *sm, uint32_t tid, const NttArgsT<M> &a, const T &ninv,
                                                 const T &wn, const Src &src, const Dst &dst,
                                                 const Sync &sync = Sync()) {
    const uint32_t warp = tid >> 5, lane = tid & 31u;
    inverse_phases<L, V, SCALED, L::NPH - 1, L::SPLIT>(sm, warp, lane, a, ninv, wn, src, dst);
    sync();
    inverse_phases<L, V, SCALED, L::SPLIT - 1, 0>(sm, warp, lane, a, ninv, wn, src, dst);
}
#endif

}  // namespace fedhe
