// he_decrypt_noalloc: the multi-kernel decryption path (gather, transform, key
// product, inverse transform, centring, slot transform), whose intermediate
// polynomials need a work buffer, with that buffer a fixed array inside the
// library image instead of memory obtained from the CUDA allocator.
//
// Who needs it: a caller that has handed all remaining device memory to its
// own pool (a serving process with a pre-partitioned HBM budget, a job under
// a hard memory cap) cannot let a library call cudaMalloc behind its back,
// and a caller inside a latency-critical loop cannot afford the device-wide
// synchronisation that cudaMalloc/cudaFree imply.  For the rings this entry
// point accepts (N <= 16384) he_decrypt itself runs one fused kernel that needs
// no work buffer and allocates nothing either, and is the faster call; the
// multi-kernel path is what he_decrypt uses on the longer rings, where it may
// grow the context's work buffer.  This entry point gives a caller that path
// with a guarantee that does not depend on which kernel the library picks: it
// never allocates, at the price of a size limit and of about three extra
// passes over T * N words.
//
// The array costs HE_NOALLOC_MAX_WORDS * 8 bytes (16 MiB) on every GPU that
// loads the library, until the process exits.  All calls on a device share
// it and it keeps whatever the previous call left there: nothing in it has to
// start at zero (every word that is read was written earlier in the same
// call), but two calls that overlap on the GPU (different streams) race.
// The array's device address is looked up once per device and kept for the
// life of the process; a caller that resets the device (cudaDeviceReset)
// invalidates it together with every context and key handle of the library.
#include <mutex>

#include "fedhe_launch.h"

using namespace fedhe;

namespace {

static __device__ __align__(256) unsigned long long g_noalloc_scratch[HE_NOALLOC_MAX_WORDS];

constexpr int kMaxDevices = 64;
uint64_t *g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// In host code the name of a __device__ array is only a handle; the address a
// kernel can use comes from cudaGetSymbolAddress, once per device, with that
// device current.
int scratch_for_current_device(uint64_t **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return HE_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return HE_ERR_SIZE;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return HE_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<uint64_t *>(p);
    }
    *out = g_scratch_addr[dev];
    return HE_OK;
}

}  // namespace

extern "C" int he_decrypt_noalloc(he_ctx *ctx, const he_keys *keys, const uint64_t *agg_dev, size_t T,
                                  double *z_dev, void *stream) {
    if (!ctx || ctx->magic != CTX_MAGIC || !keys || keys->magic != KEYS_MAGIC || keys->ctx != ctx ||
        keys->is_share)
        return HE_ERR_INVALID_ARG;
    const CtxDev &d = ctx->dev;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return HE_ERR_CUDA;
    if (dev != ctx->device) return HE_ERR_INVALID_ARG;       // the context's GPU must be current
    // sizes beyond the fixed array, and rings whose decoder needs a second buffer
    if (d.N > 16384) return HE_ERR_SIZE;
    if (T > HE_NOALLOC_MAX_WORDS / d.N) return HE_ERR_SIZE;
    if (T == 0) return HE_OK;
    if (!agg_dev || !z_dev || (reinterpret_cast<uintptr_t>(agg_dev) & 15u)) return HE_ERR_INVALID_ARG;
    uint64_t *scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != HE_OK) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (launch_decrypt(d, keys->dev, agg_dev, d.L - 1, T, scratch, st) != cudaSuccess) return HE_ERR_CUDA;
    if (launch_decode(d, reinterpret_cast<const int64_t *>(scratch), T, nullptr, z_dev, st) != cudaSuccess)
        return HE_ERR_CUDA;
    return HE_OK;
}
