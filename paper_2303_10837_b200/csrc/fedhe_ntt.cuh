// Register-tiled negacyclic NTT of one block of B = 2^LOGB residues held by
// one thread block in shared memory: a thread takes E = 2^LE residues into
// registers, does LE butterfly stages on them and puts them back; between
// such phases the index bits are re-dealt among the threads.
//
// Index conventions (forward transform, natural order in, bit-reversed out):
// stage s (0-based) of a length-N transform pairs the elements whose indices
// differ in bit logN-1-s and uses the twiddle  tw[2^s + (index >> (logN - s))],
// tw[i] = psi^brev(i).  The inverse transform runs the stages backwards with
// the inverse table.  A block may be one of 2^A consecutive pieces of a
// longer transform (N = 2^A B) whose first A stages were done elsewhere; then
// the local stage s' is the global stage A + s' and the block index enters
// the twiddle index.
//
// Phase p < NPH-1 keeps in registers the elements that differ in index bits
// [lo, lo+LE), lo = LOGB - (p+1) LE; the last phase holds the remaining R low
// bits plus the LE-R top bits (so that a thread owns runs of 2^R consecutive
// elements and a warp covers whole 128-byte lines).
#pragma once

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

// Shared-memory index swizzle.  A 64-bit access of a warp is served half-warp
// by half-warp from 16 banks of 8 bytes (the low four index bits), and the 16
// lanes of a half-warp differ in four index bits that depend on the phase:
// bits {0,1,2,3}, {0,4,5,6}, {1,2,3,4}, {0,1,5,6} or {2,3,4,5} for the layouts
// in use.  XOR-ing t ^ (t << 1), t = index bits 4..6, into the low nibble makes
// the bank a bijection of each of these sets (as linear maps over GF(2): the
// columns 0011, 0110, 1100 for bits 4, 5, 6 next to the identity), so no
// phase has bank conflicts; the map permutes every aligned group of 16 words.
HD uint32_t swz(uint32_t i) {
    const uint32_t t = (i >> 4) & 7u;
    return i ^ t ^ ((t << 1) & 15u);
}

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
// ModInt: any prime below 2^62; 64-bit integers in the lazy Harvey ranges
// (forward [0, 4q), inverse [0, 2q)), table entries {w, floor(w 2^64 / q)}.
// ModF64: primes below 2^46; signed integers in doubles, table entries the
// twiddles as doubles.  Forward, every stage adds at most 3q/4 to the bound
// (q at the input, at most 13q after 16 stages); inverse, sums double and
// differences go through the product, so after the at most three stages of a
// phase the sums are brought back below q (settle) before they are stored.

struct ModInt {
    static constexpr int UNROLL_V = 1;   // virtual threads of a phase one after the other
    using val = uint64_t;
    using tab = tw_t;
    uint64_t q, q2;
    static HD val from_bits(uint64_t b) { return b; }
    static HD uint64_t bits(val v) { return v; }
    static HD tw_t load(const tw_t *p) { return FEDHE_LD_TW(p); }
    HD void fwd(val &x, val &y, const tw_t &w) const { ct_butterfly(x, y, w.w, w.wp, q, q2); }
    HD void inv(val &x, val &y, const tw_t &w) const { gs_butterfly(x, y, w.w, w.wp, q, q2); }
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
    HD uint64_t canon_wide(val v) const { return csub(csub(v, q2), q); }
    HD uint64_t canon(val v) const { return csub(v, q); }
    HD uint64_t canon_add(val v, uint64_t add) const { return csub(csub(v, q) + add, q); }
    // canonical residue of a forward output plus a key product
    HD uint64_t canon_sum(val a, val b) const { return csub(canon_wide(a) + csub(b, q), q); }
    // product with an entry of a key table, below 2q for any v
    using key = tw_t;
    static HD key load_key(const tw_t *p) { return FEDHE_LD_TW(p); }
    HD val mul_key(val v, const key &k) const { return shoup_lazy(v, k.w, k.wp, q); }
};

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

// twiddles of local stage s = P LE + I for the registers of one thread:
// w[g] serves the butterflies whose lower register has r >> (nst - I) == g
template <class L, int P, int I, class M>
HD void stage_twiddles(typename M::tab (&w)[1 << I], uint32_t tid, const NttArgsT<M> &a) {
    constexpr int s = P * L::LE + I;
    const uint32_t base = (1u << (a.A + s)) + (a.blk << s);
    static_assert(P < L::NPH - 1, "in the last phase the registers of a group are far apart in the index");
    constexpr int lo = L::LOGB - (P + 1) * L::LE;
    load_run<1 << I>(a.tw + base + ((tid >> lo) << I), w);
}

template <class L, int P, int I, class M>
HD void fwd_stage(typename M::val (&x)[L::E], uint32_t tid, const NttArgsT<M> &a) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    constexpr int bit = nst - 1 - I;              // register bit of the pair
    if constexpr (P < L::NPH - 1) {
        typename M::tab w[1 << I];
        stage_twiddles<L, P, I>(w, tid, a);
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            a.m.fwd(x[r], x[r | (1 << bit)], w[r >> (nst - I)]);
        }
    } else {
        constexpr int s = P * L::LE + I;
        const uint32_t base = (1u << (a.A + s)) + (a.blk << s);
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            // registers that agree above the pair bit share one twiddle; the
            // compiler merges the equal loads of an unrolled group
            const auto w = M::load(a.tw + base + L::template top<P, I>(tid, r));
            a.m.fwd(x[r], x[r | (1 << bit)], w);
        }
    }
}

template <class L, int P, int I, class M>
HD void inv_stage(typename M::val (&x)[L::E], uint32_t tid, const NttArgsT<M> &a) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    constexpr int bit = nst - 1 - I;
    if constexpr (P < L::NPH - 1) {
        typename M::tab w[1 << I];
        stage_twiddles<L, P, I>(w, tid, a);
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            a.m.inv(x[r], x[r | (1 << bit)], w[r >> (nst - I)]);
        }
    } else {
        constexpr int s = P * L::LE + I;
        const uint32_t base = (1u << (a.A + s)) + (a.blk << s);
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            if (r & (1 << bit)) continue;
            const auto w = M::load(a.tw + base + L::template top<P, I>(tid, r));
            a.m.inv(x[r], x[r | (1 << bit)], w);
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
HD void fwd_phase(typename M::val (&x)[L::E], uint32_t tid, const NttArgsT<M> &a) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    if constexpr (I < nst) {
        fwd_stage<L, P, I>(x, tid, a);
        fwd_phase<L, P, I + 1>(x, tid, a);
    }
}

// inverse phase: stages nst-1 down to STOP (STOP = 1 leaves stage 0 of the
// phase to the caller); a phase that ends with an ordinary stage settles the
// sums of that stage (the registers whose pair bit is clear)
template <class L, int P, int STOP, int I, class M>
HD void inv_phase_from(typename M::val (&x)[L::E], uint32_t tid, const NttArgsT<M> &a) {
    if constexpr (I >= STOP) {
        inv_stage<L, P, I>(x, tid, a);
        inv_phase_from<L, P, STOP, I - 1>(x, tid, a);
    } else if constexpr (STOP == 0) {
        constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
#pragma unroll
        for (int r = 0; r < L::E; r++)
            if (!(r & (1 << (nst - 1)))) x[r] = a.m.settle(x[r]);
    }
}

template <class L, int P, int STOP = 0, class M>
HD void inv_phase(typename M::val (&x)[L::E], uint32_t tid, const NttArgsT<M> &a) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    inv_phase_from<L, P, STOP, nst - 1>(x, tid, a);
}

#if defined(__CUDACC__)
// ---------------------------------------------------------------------------
// Whole-block transforms.  The block's residues stay in shared memory
// (swizzled) and every thread plays V "virtual threads" per phase, each of
// which loads its E residues, does the phase's butterflies in registers and
// stores them back to the same places, so that only E residues are live per
// thread at a time (E = 8 keeps a 1024-thread block within 64 registers with
// no spills) and no separate exchange buffer is needed.  The first phase takes its input
// from `src`, the last hands its output to `dst`:
//   forward:  src(i) -> residue i;            dst(i, a, b): residues i, i+1
//   inverse:  src(i) -> residues i, i+1 (members x, y);   dst(i, a): residue i
// all in the value type of the limb's arithmetic
// (pairs always start at an even index and are neighbours in memory).
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

template <class L, int V, class M, class Src, class Dst, class Sync = BlockSync, int P = 0>
__device__ __forceinline__ void smem_ntt_forward(uint64_t *sm, uint32_t tid, const NttArgsT<M> &a, const Src &src,
                                                 const Dst &dst, const Sync &sync = Sync()) {
    constexpr int RT = L::NT / V, LAST = L::NPH - 1;
#pragma unroll M::UNROLL_V
    for (int v = 0; v < V; v++) {
        const uint32_t vt = tid + v * RT;
        typename M::val x[L::E];
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            const uint32_t i = L::template idx<P>(vt, r);
            if constexpr (P == 0) x[r] = src(i);
            else x[r] = M::from_bits(sm[swz(i)]);
        }
        fwd_phase<L, P>(x, vt, a);
        if constexpr (P == LAST) {
#pragma unroll
            for (int r = 0; r < L::E; r += 2) dst(L::template idx<P>(vt, r), x[r], x[r + 1]);
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) sm[swz(L::template idx<P>(vt, r))] = M::bits(x[r]);
        }
    }
    if constexpr (P < LAST) {
        sync();
        smem_ntt_forward<L, V, M, Src, Dst, Sync, P + 1>(sm, tid, a, src, dst, sync);
    }
}

template <class L, int V, bool SCALED, class M, class T, class Src, class Dst, class Sync = BlockSync,
          int P = L::NPH - 1>
__device__ __forceinline__ void smem_ntt_inverse(uint64_t *sm, uint32_t tid, const NttArgsT<M> &a, const T &ninv,
                                                 const T &wn, const Src &src, const Dst &dst,
                                                 const Sync &sync = Sync()) {
    constexpr int RT = L::NT / V, LAST = L::NPH - 1;
#pragma unroll M::UNROLL_V
    for (int v = 0; v < V; v++) {
        const uint32_t vt = tid + v * RT;
        typename M::val x[L::E];
        if constexpr (P == LAST) {
#pragma unroll
            for (int r = 0; r < L::E; r += 2) {
                const auto t = src(L::template idx<P>(vt, r));
                x[r] = t.x;
                x[r + 1] = t.y;
            }
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) x[r] = M::from_bits(sm[swz(L::template idx<P>(vt, r))]);
        }
        if constexpr (P == 0 && SCALED) {
            inv_phase<L, 0, 1>(x, vt, a);
            inv_stage0_scaled<L>(x, a.m, ninv, wn);
        } else {
            inv_phase<L, P, 0>(x, vt, a);
        }
        if constexpr (P == 0) {
#pragma unroll
            for (int r = 0; r < L::E; r++) dst(L::template idx<0>(vt, r), x[r]);
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) sm[swz(L::template idx<P>(vt, r))] = M::bits(x[r]);
        }
    }
    if constexpr (P > 0) {
        sync();
        smem_ntt_inverse<L, V, SCALED, M, T, Src, Dst, Sync, P - 1>(sm, tid, a, ninv, wn, src, dst, sync);
    }
}
#endif


}  // namespace fedhe
