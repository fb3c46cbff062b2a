// Host-side table construction for the CUDA library: parameter validation,
// roots of unity, Shoup twiddle tables and the fp64 root table of the slot
// transform.  Plain C++ (compiled by the host compiler, no CUDA).
#pragma once

#include <stdint.h>

#include <vector>

namespace fedhe {

struct HostTw { uint64_t w, wp; };   // value and floor(value * 2^64 / q)

struct HostLimb {
    uint64_t q = 0;
    uint64_t psi = 0;          // smallest primitive 2N-th root of unity mod q
    uint64_t mu = 0;           // floor(2^64 / q)
    HostTw ninv{};             // 1/N
    HostTw wn{};               // (inverse twiddle of stage 0) / N
    std::vector<HostTw> fwd;   // fwd[i] = psi^brev(i), i < N
    std::vector<HostTw> inv;   // inv[i] = psi^-brev(i)
};

uint64_t host_mulmod(uint64_t a, uint64_t b, uint64_t q);
uint64_t host_powmod(uint64_t a, uint64_t e, uint64_t q);
uint64_t host_invmod(uint64_t a, uint64_t q);
HostTw host_shoup(uint64_t w, uint64_t q);
bool host_is_prime(uint64_t n);

// 0 if usable, else a short reason (static string)
const char *host_check_params(uint32_t N, uint32_t L, const uint64_t *q, int log2_delta);
void host_build_limb(uint32_t N, uint64_t q, HostLimb &out);

// roots[2t], roots[2t+1] = cos, sin of 2 pi t / (2N), each the binary64
// nearest to the true value, t < 2N
void host_unit_roots(uint32_t N, std::vector<double> &roots);
// Per-stage twiddles of the slot transform: for len = 2, 4, ..., n (n = N/2)
// and j < len/2, entry [len/2 + j] = exp(2 pi i 5^j / (4 len)) (cos, sin);
// entry [0] is unused.  Size n complex numbers.
void host_slot_twiddles(uint32_t N, const std::vector<double> &roots, std::vector<double> &out);

}  // namespace fedhe
