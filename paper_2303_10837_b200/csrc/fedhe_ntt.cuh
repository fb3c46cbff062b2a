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

// shared-memory index swizzle: makes all phase layouts free of bank conflicts
// for 8-byte accesses (xor the low nibble with the next one)
HD uint32_t swz(uint32_t i) { return i ^ ((i >> 4) & 15u); }

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

// ---- phases ----------------------------------------------------------------

struct NttArgs {
    const tw_t *tw;      // table of this limb and direction, indexed by the global twiddle index
    uint64_t q, q2;      // modulus and twice the modulus
    uint32_t A;          // log2 of the number of blocks the whole transform is cut into
    uint32_t blk;        // which block this is
};

// GROW: no conditional subtractions (small primes only, see the *_grow
// butterflies): a sub-block's inverse input must lie below 2q, and after k
// inverse stages the values lie below 2^(k+1) q.
template <class L, int P, int I, bool GROW = false>
HD void fwd_stage(uint64_t (&x)[L::E], uint32_t tid, const NttArgs &a) {
    constexpr int s = P * L::LE + I;
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    constexpr int bit = nst - 1 - I;              // register bit of the pair
    const uint32_t base = (1u << (a.A + s)) + (a.blk << s);
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        if (r & (1 << bit)) continue;
        // all registers that agree above the pair bit share one twiddle; the
        // compiler merges the equal loads of an unrolled group
        const tw_t *pw = a.tw + base + L::template top<P, I>(tid, r);
        tw_t w = FEDHE_LD_TW(pw);
        if constexpr (GROW) ct_butterfly_grow(x[r], x[r | (1 << bit)], w.w, w.wp, a.q, a.q2);
        else ct_butterfly(x[r], x[r | (1 << bit)], w.w, w.wp, a.q, a.q2);
    }
}

template <class L, int P, int I, bool GROW = false>
HD void inv_stage(uint64_t (&x)[L::E], uint32_t tid, const NttArgs &a) {
    constexpr int s = P * L::LE + I;
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    constexpr int bit = nst - 1 - I;
    const uint32_t base = (1u << (a.A + s)) + (a.blk << s);
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        if (r & (1 << bit)) continue;
        const tw_t *pw = a.tw + base + L::template top<P, I>(tid, r);
        tw_t w = FEDHE_LD_TW(pw);
        // local stage s is the (LOGB - 1 - s)-th to run: inputs lie below 2^(LOGB - s) q
        if constexpr (GROW) gs_butterfly_grow(x[r], x[r | (1 << bit)], w.w, w.wp, a.q, a.q << (L::LOGB - s));
        else gs_butterfly(x[r], x[r | (1 << bit)], w.w, w.wp, a.q, a.q2);
    }
}

// last inverse stage of a whole transform (global stage 0) with the factor
// 1/N folded in: x <- (x + y)/N, y <- (x - y) w /N.  ninv = 1/N, wn = w/N.
template <class L>
HD void inv_stage0_scaled(uint64_t (&x)[L::E], tw_t ninv, tw_t wn, uint64_t q, uint64_t q2) {
    constexpr int bit = L::LE - 1;
#pragma unroll
    for (int r = 0; r < L::E; r++) {
        if (r & (1 << bit)) continue;
        uint64_t u = x[r], v = x[r | (1 << bit)];
        x[r] = shoup_lazy(u + v, ninv.w, ninv.wp, q);
        x[r | (1 << bit)] = shoup_lazy(u - v + q2, wn.w, wn.wp, q);
    }
}

template <class L, int P, int I = 0, bool GROW = false>
HD void fwd_phase(uint64_t (&x)[L::E], uint32_t tid, const NttArgs &a) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    if constexpr (I < nst) {
        fwd_stage<L, P, I, GROW>(x, tid, a);
        fwd_phase<L, P, I + 1, GROW>(x, tid, a);
    }
}

// inverse phase: stages nst-1 down to STOP (STOP = 1 leaves stage 0 of the
// phase to the caller)
template <class L, int P, int STOP, int I, bool GROW = false>
HD void inv_phase_from(uint64_t (&x)[L::E], uint32_t tid, const NttArgs &a) {
    if constexpr (I >= STOP) {
        inv_stage<L, P, I, GROW>(x, tid, a);
        inv_phase_from<L, P, STOP, I - 1, GROW>(x, tid, a);
    }
}

template <class L, int P, int STOP = 0, bool GROW = false>
HD void inv_phase(uint64_t (&x)[L::E], uint32_t tid, const NttArgs &a) {
    constexpr int nst = (P < L::NPH - 1) ? L::LE : L::R;
    inv_phase_from<L, P, STOP, nst - 1, GROW>(x, tid, a);
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
//   inverse:  src(i) -> residues i, i+1;      dst(i, a): residue i
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

template <class L, int V, bool GROW = false, class Src, class Dst, class Sync = BlockSync, int P = 0>
__device__ __forceinline__ void smem_ntt_forward(uint64_t *sm, uint32_t tid, const NttArgs &a, const Src &src,
                                                 const Dst &dst, const Sync &sync = Sync()) {
    constexpr int RT = L::NT / V, LAST = L::NPH - 1;
#pragma unroll 1
    for (int v = 0; v < V; v++) {
        const uint32_t vt = tid + v * RT;
        uint64_t x[L::E];
#pragma unroll
        for (int r = 0; r < L::E; r++) {
            const uint32_t i = L::template idx<P>(vt, r);
            if constexpr (P == 0) x[r] = src(i);
            else x[r] = sm[swz(i)];
        }
        fwd_phase<L, P, 0, GROW>(x, vt, a);
        if constexpr (P == LAST) {
#pragma unroll
            for (int r = 0; r < L::E; r += 2) dst(L::template idx<P>(vt, r), x[r], x[r + 1]);
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) sm[swz(L::template idx<P>(vt, r))] = x[r];
        }
    }
    if constexpr (P < LAST) {
        sync();
        smem_ntt_forward<L, V, GROW, Src, Dst, Sync, P + 1>(sm, tid, a, src, dst, sync);
    }
}

template <class L, int V, bool SCALED, bool GROW = false, class Src, class Dst, class Sync = BlockSync,
          int P = L::NPH - 1>
__device__ __forceinline__ void smem_ntt_inverse(uint64_t *sm, uint32_t tid, const NttArgs &a, tw_t ninv,
                                                 tw_t wn, const Src &src, const Dst &dst,
                                                 const Sync &sync = Sync()) {
    constexpr int RT = L::NT / V, LAST = L::NPH - 1;
#pragma unroll 1
    for (int v = 0; v < V; v++) {
        const uint32_t vt = tid + v * RT;
        uint64_t x[L::E];
        if constexpr (P == LAST) {
#pragma unroll
            for (int r = 0; r < L::E; r += 2) {
                const u64x2 t = src(L::template idx<P>(vt, r));
                x[r] = t.x;
                x[r + 1] = t.y;
            }
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) x[r] = sm[swz(L::template idx<P>(vt, r))];
        }
        static_assert(!(SCALED && GROW), "the scaled last stage expects inputs below 2q");
        if constexpr (P == 0 && SCALED) {
            inv_phase<L, 0, 1>(x, vt, a);
            inv_stage0_scaled<L>(x, ninv, wn, a.q, a.q2);
        } else {
            inv_phase<L, P, 0, GROW>(x, vt, a);
        }
        if constexpr (P == 0) {
#pragma unroll
            for (int r = 0; r < L::E; r++) dst(L::template idx<0>(vt, r), x[r]);
        } else {
#pragma unroll
            for (int r = 0; r < L::E; r++) sm[swz(L::template idx<P>(vt, r))] = x[r];
        }
    }
    if constexpr (P > 0) {
        sync();
        smem_ntt_inverse<L, V, SCALED, GROW, Src, Dst, Sync, P - 1>(sm, tid, a, ninv, wn, src, dst, sync);
    }
}
#endif


}  // namespace fedhe
