// C ABI of the library (see include/fedhe.h): argument validation, handle
// management, host-side table upload and the sequencing of kernel launches.
#include <math.h>
#include <string.h>

#include <mutex>
#include <new>
#include <vector>

#include "fedhe_host.h"
#include "fedhe_launch.h"

using namespace fedhe;

namespace {

inline cudaStream_t as_stream(void *s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool good(const he_ctx *c) { return c && c->magic == CTX_MAGIC; }
inline bool good(const he_keys *k) { return k && k->magic == KEYS_MAGIC; }
inline bool good(const he_mask *m) { return m && m->magic == MASK_MAGIC; }
// ciphertext-like buffers are read and written with 16-byte accesses
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#define CU(expr)                                   \
    do {                                           \
        cudaError_t e__ = (expr);                  \
        if (e__ != cudaSuccess) return e__ == cudaErrorMemoryAllocation ? HE_ERR_ALLOC : HE_ERR_CUDA; \
    } while (0)

// grows a context-owned device buffer; contents are not preserved
int ensure(void **buf, size_t *cap, size_t need) {
    if (need <= *cap) return HE_OK;
    if (*buf) {
        CU(cudaFree(*buf));
        *buf = nullptr;
        *cap = 0;
    }
    CU(cudaMalloc(buf, need));
    *cap = need;
    return HE_OK;
}

template <class T>
int upload(he_ctx *ctx, const T *host, size_t count, const T **dev) {
    void *p = nullptr;
    CU(cudaMalloc(&p, count * sizeof(T)));
    ctx->owned.push_back(p);
    CU(cudaMemcpy(p, host, count * sizeof(T), cudaMemcpyHostToDevice));
    *dev = static_cast<const T *>(p);
    return HE_OK;
}

size_t work_bytes(const he_ctx *ctx, size_t T) { return 2 * T * (size_t)ctx->dev.N * sizeof(uint64_t); }

}  // namespace

namespace fedhe {
int ctx_workspace(he_ctx *ctx, size_t T, void **out) {
    const int rc = ensure(&ctx->ws, &ctx->ws_bytes, work_bytes(ctx, T));
    *out = ctx->ws;
    return rc;
}
}  // namespace fedhe

extern "C" {

const char *he_strerror(int code) {
    switch (code) {
    case HE_OK: return "ok";
    case HE_ERR_INVALID_ARG: return "invalid argument";
    case HE_ERR_PARAMS: return "unusable crypto parameters";
    case HE_ERR_ALLOC: return "allocation failed";
    case HE_ERR_CUDA: return "CUDA runtime error";
    case HE_ERR_OVERFLOW: return "encoded coefficient out of range";
    case HE_ERR_LEVEL: return "ciphertext level mismatch";
    case HE_ERR_SIZE: return "size not supported";
    default: return "unknown error";
    }
}

uint64_t he_launch_count(void) { return launch_count(); }

int he_ctx_create(const he_params *p, he_ctx **out) {
    if (!p || !out) return HE_ERR_INVALID_ARG;
    *out = nullptr;
    if (p->L > HE_MAX_LIMBS) return HE_ERR_PARAMS;
    if (host_check_params(p->N, p->L, p->q, p->log2_delta)) return HE_ERR_PARAMS;
    he_ctx *ctx = new (std::nothrow) he_ctx();
    if (!ctx) return HE_ERR_ALLOC;
    ctx->magic = CTX_MAGIC;
    ctx->params = *p;
    int rc = HE_OK;
    do {
        if (cudaGetDevice(&ctx->device) != cudaSuccess) { rc = HE_ERR_CUDA; break; }
        if (cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess ||
            ctx->sm_count < 1) {
            rc = HE_ERR_CUDA;
            break;
        }
        CtxDev &d = ctx->dev;
        memset(&d, 0, sizeof(d));
        d.N = p->N;
        d.L = p->L;
        d.log2_delta = p->log2_delta;
        while ((1u << d.logN) < d.N) d.logN++;
        d.LOGB = d.logN <= 14 ? d.logN : 13;   // longer transforms: 2^13 blocks, two per SM
        d.A = d.logN - d.LOGB;
        const uint64_t ql = p->q[p->L - 1];
        for (uint32_t j = 0; j < p->L && rc == HE_OK; j++) {
            HostLimb hl;
            host_build_limb(d.N, p->q[j], hl);
            LimbDev &ld = d.limb[j];
            ld.q = hl.q;
            ld.mu = hl.mu;
            ld.ninv = tw_t{hl.ninv.w, hl.ninv.wp};
            ld.wn = tw_t{hl.wn.w, hl.wn.wp};
            if (j + 1 < p->L) {
                HostTw qi = host_shoup(host_invmod(ql % hl.q, hl.q), hl.q);
                ld.qlinv = tw_t{qi.w, qi.wp};
            }
            rc = upload(ctx, reinterpret_cast<const tw_t *>(hl.fwd.data()), hl.fwd.size(), &ld.fwd);
            if (rc == HE_OK) rc = upload(ctx, reinterpret_cast<const tw_t *>(hl.inv.data()), hl.inv.size(), &ld.inv);
            if (rc == HE_OK && hl.q < F64_PRIME_LIMIT) {
                // every value is below 2^46, so the conversions are exact
                std::vector<double> fd(hl.fwd.size()), id(hl.inv.size());
                for (size_t i = 0; i < fd.size(); i++) fd[i] = (double)hl.fwd[i].w;
                for (size_t i = 0; i < id.size(); i++) id[i] = (double)hl.inv[i].w;
                ld.qd = (double)hl.q;
                ld.qi = 1.0 / ld.qd;
                ld.ninv_d = (double)hl.ninv.w;
                ld.wn_d = (double)hl.wn.w;
                rc = upload(ctx, fd.data(), fd.size(), &ld.fwd_d);
                if (rc == HE_OK) rc = upload(ctx, id.data(), id.size(), &ld.inv_d);
            }
        }
        if (rc != HE_OK) break;
        std::vector<double> roots, ftw;
        host_unit_roots(d.N, roots);
        host_slot_twiddles(d.N, roots, ftw);
        rc = upload(ctx, reinterpret_cast<const double2 *>(ftw.data()), ftw.size() / 2, &d.ftw);
        if (rc != HE_OK) break;
        rc = upload(ctx, d.limb, HE_MAX_LIMBS, &d.limb_dev);
        if (rc != HE_OK) break;
        void *st = nullptr;
        if (cudaMalloc(&st, sizeof(int)) != cudaSuccess) { rc = HE_ERR_ALLOC; break; }
        ctx->owned.push_back(st);
        if (cudaMemset(st, 0, sizeof(int)) != cudaSuccess) { rc = HE_ERR_CUDA; break; }
        d.status = static_cast<int *>(st);
        // pointer and weight tables of the aggregation calls
        rc = ensure(&ctx->tab, &ctx->tab_bytes,
                    HE_MAX_CLIENTS * (2 * sizeof(void *) + sizeof(double) + HE_MAX_LIMBS * sizeof(tw_t)));
    } while (0);
    if (rc != HE_OK) {
        he_ctx_destroy(ctx);
        return rc;
    }
    *out = ctx;
    return HE_OK;
}

int he_ctx_destroy(he_ctx *ctx) {
    if (!good(ctx)) return HE_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    for (void *p : ctx->owned) cudaFree(p);
    if (ctx->ws) cudaFree(ctx->ws);
    if (ctx->tab) cudaFree(ctx->tab);
    if (ctx->round_buf) cudaFree(ctx->round_buf);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->down_stream) cudaStreamDestroy(ctx->down_stream);
    for (int i = 0; i < 2; i++) {
        if (ctx->ev_ready[i]) cudaEventDestroy(ctx->ev_ready[i]);
        if (ctx->ev_free[i]) cudaEventDestroy(ctx->ev_free[i]);
    }
    if (ctx->ev_chunk) cudaEventDestroy(ctx->ev_chunk);
    ctx->magic = 0;
    delete ctx;
    return HE_OK;
}

int he_ctx_status(he_ctx *ctx, int *status) {
    if (!good(ctx) || !status) return HE_ERR_INVALID_ARG;
    int word = 0;
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(&word, ctx->dev.status, sizeof(int), cudaMemcpyDeviceToHost));
    if (word) CU(cudaMemset(ctx->dev.status, 0, sizeof(int)));
    *status = word ? HE_ERR_OVERFLOW : HE_OK;
    return HE_OK;
}

int he_ctx_reserve(he_ctx *ctx, size_t max_k) {
    if (!good(ctx)) return HE_ERR_INVALID_ARG;
    const size_t T = he_num_ct(ctx, max_k);
    size_t need = encrypt_work_bytes(ctx->dev, ctx->sm_count, T, true);
    if (ctx->dev.A > 0 && work_bytes(ctx, T) > need) need = work_bytes(ctx, T);     // decryption on the long rings
    return ensure(&ctx->ws, &ctx->ws_bytes, need);
}

size_t he_slots(const he_ctx *ctx) { return good(ctx) ? ctx->dev.N / 2 : 0; }

size_t he_num_ct(const he_ctx *ctx, size_t k) {
    if (!good(ctx)) return 0;
    const size_t n = ctx->dev.N / 2;
    return (k + n - 1) / n;
}

size_t he_ct_words(const he_ctx *ctx, uint32_t level) {
    return good(ctx) ? 2 * (size_t)level * ctx->dev.N : 0;
}

// ---------------------------------------------------------------------------

int he_keygen(he_ctx *ctx, uint64_t seed, he_keys **out, void *stream) {
    if (!good(ctx) || !out) return HE_ERR_INVALID_ARG;
    *out = nullptr;
    const CtxDev &d = ctx->dev;
    const size_t LN = (size_t)d.L * d.N;
    he_keys *k = new (std::nothrow) he_keys();
    if (!k) return HE_ERR_ALLOC;
    k->magic = KEYS_MAGIC;
    k->ctx = ctx;
    k->storage = nullptr;
    const size_t bytes = 3 * LN * sizeof(tw_t) + d.N;
    void *tmp = nullptr;
    int rc = HE_OK;
    do {
        if (cudaMalloc(&k->storage, bytes) != cudaSuccess || cudaMalloc(&tmp, 3 * LN * sizeof(uint64_t)) != cudaSuccess) {
            rc = HE_ERR_ALLOC;
            break;
        }
        tw_t *base = static_cast<tw_t *>(k->storage);
        tw_t *pk0 = base, *pk1 = base + LN, *sh = base + 2 * LN;
        int8_t *s8 = reinterpret_cast<int8_t *>(base + 3 * LN);
        k->dev = KeysDev{pk0, pk1, sh, s8};
        cudaStream_t st = as_stream(stream);
        uint64_t *t64 = static_cast<uint64_t *>(tmp);
        if (launch_keygen_sample(d, seed, s8, t64, st) != cudaSuccess ||
            launch_ntt(d, true, t64, 3, LN, 0, d.L, st) != cudaSuccess ||
            launch_keygen_combine(d, t64, pk0, pk1, sh, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess) {
            rc = HE_ERR_CUDA;
        }
    } while (0);
    if (tmp) cudaFree(tmp);
    if (rc != HE_OK) {
        if (k->storage) cudaFree(k->storage);
        delete k;
        return rc;
    }
    *out = k;
    return HE_OK;
}

int he_keys_destroy(he_keys *keys) {
    if (!good(keys)) return HE_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    cudaFree(keys->storage);
    keys->magic = 0;
    delete keys;
    return HE_OK;
}

int he_keys_export(he_ctx *ctx, const he_keys *keys, uint64_t *pk_dev, int8_t *s_dev, void *stream) {
    if (!good(ctx) || !good(keys) || keys->ctx != ctx || keys->is_share) return HE_ERR_INVALID_ARG;
    const CtxDev &d = ctx->dev;
    const size_t LN = (size_t)d.L * d.N;
    cudaStream_t st = as_stream(stream);
    if (pk_dev) {
        if (!aligned16(pk_dev)) return HE_ERR_INVALID_ARG;
        // pk0^ and pk1^ are adjacent in the key storage
        CU(launch_extract_values(keys->dev.pk0_hat, pk_dev, 2 * LN, st));
        CU(launch_ntt(d, false, pk_dev, 2, LN, 0, d.L, st));
    }
    if (s_dev) CU(cudaMemcpyAsync(s_dev, keys->dev.s, d.N, cudaMemcpyDeviceToDevice, st));
    return HE_OK;
}

// ---------------------------------------------------------------------------
// mask
// ---------------------------------------------------------------------------

// Masks are made and dropped once per round, and a plain device allocation costs more than the
// kernels of the selection.  Their buffers therefore come from one memory pool per device, made
// on first use and kept for the life of the process; the pool hands freed buffers out again and
// gives back to the driver only what it holds beyond MASK_POOL_KEEP bytes.
static constexpr uint64_t MASK_POOL_KEEP = 256ull << 20;
static cudaMemPool_t mask_pool(int device) {
    static std::mutex mu;
    static cudaMemPool_t pools[64] = {};
    if (device < 0 || device >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!pools[device]) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = device;
        cudaMemPool_t pool = nullptr;
        if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        uint64_t keep = MASK_POOL_KEEP;
        cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        pools[device] = pool;
    }
    return pools[device];
}

static int build_mask(he_ctx *ctx, const float *score, size_t P, size_t k, const uint64_t *ranges_host,
                      size_t num_ranges, he_mask **out, void *stream) {
    if (!good(ctx) || !out || (!score && P) || k > P) return HE_ERR_INVALID_ARG;
    *out = nullptr;
    if (P == 0) return HE_ERR_INVALID_ARG;
    if (P >= (1ull << 32)) return HE_ERR_SIZE;
    if (num_ranges > 64 || (num_ranges && !ranges_host)) return HE_ERR_INVALID_ARG;
    size_t forced = 0;                       // upper bound of what the ranges add to the mask
    for (size_t r = 0; r < num_ranges; r++) {
        if (ranges_host[2 * r] > ranges_host[2 * r + 1] || ranges_host[2 * r + 1] > P) return HE_ERR_INVALID_ARG;
        forced += ranges_host[2 * r + 1] - ranges_host[2 * r];
    }
    cudaStream_t st = as_stream(stream);
    const size_t nblocks = (P + MASK_BLOCK - 1) / MASK_BLOCK, nwords = (P + 31) / 32;
    const size_t kmax = k + forced < P ? k + forced : P;

    // Scratch in the context's work space (no allocation, and no free that would wait for the
    // device): selection state (2) | totals (2) | three histograms (2048 each) | blk_a | blk_b | ranges
    const size_t scratch_words = 4 + 3 * 2048 + 2 * nblocks + 4 * 64 + 2;
    {
        const int erc = ensure(&ctx->ws, &ctx->ws_bytes, scratch_words * sizeof(uint32_t));
        if (erc != HE_OK) return erc;
    }
    uint32_t *scratch = static_cast<uint32_t *>(ctx->ws);
    SelectState *state = reinterpret_cast<SelectState *>(scratch);
    uint32_t *totals = scratch + 2, *hist = scratch + 4, *blk_eq = hist + 3 * 2048, *blk_sel = blk_eq + nblocks;
    uint64_t *ranges_dev = reinterpret_cast<uint64_t *>(scratch + ((4 + 3 * 2048 + 2 * nblocks + 1) & ~(size_t)1));
    // The mask owns one allocation: bit mask | per-word prefix counts | index list (its size is
    // known up to the overlap of the forced ranges with the top-k set and with each other).
    uint32_t *bits = nullptr;
    cudaMemPool_t pool = mask_pool(ctx->device);
    if (!pool) return HE_ERR_CUDA;
    if (cudaMallocFromPoolAsync(reinterpret_cast<void **>(&bits), (2 * nwords + (kmax ? kmax : 1)) * sizeof(uint32_t),
                                pool, st) != cudaSuccess) {
        cudaGetLastError();
        return HE_ERR_ALLOC;
    }
    uint32_t *wpre = bits + nwords, *idx = wpre + nwords;
    int rc = HE_OK;
    he_mask *m = nullptr;
    do {
#define MCU(expr) if ((expr) != cudaSuccess) { rc = HE_ERR_CUDA; break; }
        // Radix select of the k-th largest key, 11 + 11 + 10 bits, entirely on the device: the
        // digit walk between two histogram passes is a one-block kernel, so nothing is read
        // back before the end.
        const SelectState init = {k ? 0u : 0xffffffffu, (uint32_t)k};      // k = 0: no key reaches the threshold
        MCU(cudaMemcpyAsync(state, &init, sizeof(init), cudaMemcpyHostToDevice, st));
        if (k) {
            static const int digits[3] = {11, 11, 10};
            MCU(cudaMemsetAsync(hist, 0, 3 * 2048 * sizeof(uint32_t), st));
            int prefix_bits = 0;
            bool fail = false;
            for (int pass = 0; pass < 3 && !fail; pass++) {
                uint32_t *h = hist + pass * 2048;
                fail = launch_key_histogram(score, P, state, prefix_bits, digits[pass], ctx->sm_count, h, st) != cudaSuccess ||
                       launch_radix_pick(h, digits[pass], state, st) != cudaSuccess;
                prefix_bits += digits[pass];
            }
            if (fail) { rc = HE_ERR_CUDA; break; }
        }
        if (num_ranges)
            MCU(cudaMemcpyAsync(ranges_dev, ranges_host, 2 * num_ranges * sizeof(uint64_t), cudaMemcpyHostToDevice, st));
        MCU(launch_mask_count_eq(score, P, state, blk_eq, st));
        MCU(launch_scan(blk_eq, nblocks, totals, st));
        MCU(launch_mask_select(score, P, state, ranges_dev, (uint32_t)num_ranges, blk_eq, bits, blk_sel, st));
        MCU(launch_scan(blk_sel, nblocks, totals + 1, st));
        MCU(launch_mask_write(P, bits, blk_sel, wpre, idx, st));
        uint32_t ksel = 0;
        MCU(cudaMemcpyAsync(&ksel, totals + 1, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
        MCU(cudaStreamSynchronize(st));                                      // the one wait of the call
        if ((num_ranges == 0 && ksel != k) || ksel > kmax) { rc = HE_ERR_CUDA; break; }     // cannot happen
        m = new (std::nothrow) he_mask();
        if (!m) { rc = HE_ERR_ALLOC; break; }
        m->magic = MASK_MAGIC;
        m->P = P;
        m->k = ksel;
        m->idx = idx;
        m->bits = bits;
        m->wpre = wpre;
#undef MCU
    } while (0);
    if (rc != HE_OK) {
        cudaStreamSynchronize(st);           // nothing may still write the allocation
        cudaFreeAsync(bits, st);
        return rc;
    }
    *out = m;
    return HE_OK;
}

int he_select_mask(he_ctx *ctx, const float *score_dev, size_t P, size_t k, he_mask **out, void *stream) {
    return build_mask(ctx, score_dev, P, k, nullptr, 0, out, stream);
}

int he_select_mask_ranges(he_ctx *ctx, const float *score_dev, size_t P, size_t k, const uint64_t *ranges_host,
                          size_t num_ranges, he_mask **out, void *stream) {
    return build_mask(ctx, score_dev, P, k, ranges_host, num_ranges, out, stream);
}

int he_mask_indices(const he_mask *mask, const uint32_t **idx_dev, size_t *k) {
    if (!good(mask)) return HE_ERR_INVALID_ARG;
    if (idx_dev) *idx_dev = mask->idx;
    if (k) *k = mask->k;
    return HE_OK;
}

int he_mask_copy_indices(const he_mask *mask, uint32_t *out_dev, void *stream) {
    if (!good(mask) || (!out_dev && mask->k)) return HE_ERR_INVALID_ARG;
    if (mask->k)
        CU(cudaMemcpyAsync(out_dev, mask->idx, mask->k * sizeof(uint32_t), cudaMemcpyDeviceToDevice, as_stream(stream)));
    return HE_OK;
}

int he_mask_destroy(he_mask *mask) {
    if (!good(mask)) return HE_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    cudaFreeAsync(mask->bits, nullptr);      // back to the pool; prefix counts and index list are parts of this allocation
    mask->magic = 0;
    delete mask;
    return HE_OK;
}

// ---------------------------------------------------------------------------
// client and server steps
// ---------------------------------------------------------------------------

int he_pack(he_ctx *ctx, const he_mask *mask, const float *x_dev, size_t P, float *sel_dev, float *rest_dev,
            void *stream) {
    if (!good(ctx) || !x_dev || P == 0) return HE_ERR_INVALID_ARG;
    size_t k = P;
    if (mask) {
        if (!good(mask) || mask->P != P) return HE_ERR_INVALID_ARG;
        k = mask->k;
        if (k < P && !rest_dev) return HE_ERR_INVALID_ARG;
    }
    const size_t padded = he_num_ct(ctx, k) * he_slots(ctx);
    if (padded && !sel_dev) return HE_ERR_INVALID_ARG;
    CU(launch_pack(mask, x_dev, P, k, padded, sel_dev, rest_dev, as_stream(stream)));
    return HE_OK;
}

int he_encode(he_ctx *ctx, const float *sel_dev, size_t k, int64_t *m_dev, void *stream) {
    if (!good(ctx) || !sel_dev || !m_dev) return HE_ERR_INVALID_ARG;
    const size_t T = he_num_ct(ctx, k);
    if (T == 0) return HE_OK;
    int rc = ensure(&ctx->ws, &ctx->ws_bytes, work_bytes(ctx, T));
    if (rc != HE_OK) return rc;
    CU(launch_encode(ctx->dev, sel_dev, T, static_cast<double2 *>(ctx->ws), m_dev, as_stream(stream)));
    return HE_OK;
}

static int encrypt_range(he_ctx *ctx, const he_keys *keys, const float *sel_dev, size_t t_begin, size_t t_count,
                         uint64_t seed, uint32_t client_id, bool ntt_out, uint64_t *ct_dev, void *stream) {
    if (!good(ctx) || !good(keys) || keys->ctx != ctx || keys->is_share) return HE_ERR_INVALID_ARG;
    if (t_begin + t_count >= (1ull << 32)) return HE_ERR_SIZE;
    if (t_count == 0) return HE_OK;
    if (!sel_dev || !ct_dev || !aligned16(ct_dev)) return HE_ERR_INVALID_ARG;
    const CtxDev &d = ctx->dev;
    int rc = ensure(&ctx->ws, &ctx->ws_bytes, encrypt_work_bytes(d, ctx->sm_count, t_count, ntt_out));
    if (rc != HE_OK) return rc;
    cudaStream_t st = as_stream(stream);
    if (ntt_out)
        CU(launch_encrypt_ntt(d, keys->dev, sel_dev, ctx->ws, ctx->sm_count, (uint32_t)t_begin, t_count, seed,
                              client_id, ct_dev, st));
    else
        CU(launch_encrypt(d, keys->dev, sel_dev, ctx->ws, ctx->sm_count, (uint32_t)t_begin, t_count, seed,
                          client_id, ct_dev, st));
    return HE_OK;
}

int he_encrypt_range(he_ctx *ctx, const he_keys *keys, const float *sel_dev, size_t t_begin, size_t t_count,
                     uint64_t seed, uint32_t client_id, uint64_t *ct_dev, void *stream) {
    return encrypt_range(ctx, keys, sel_dev, t_begin, t_count, seed, client_id, false, ct_dev, stream);
}

int he_encrypt_ntt(he_ctx *ctx, const he_keys *keys, const float *sel_dev, size_t k, uint64_t seed,
                   uint32_t client_id, uint64_t *ct_dev, void *stream) {
    if (!good(ctx)) return HE_ERR_INVALID_ARG;
    return encrypt_range(ctx, keys, sel_dev, 0, he_num_ct(ctx, k), seed, client_id, true, ct_dev, stream);
}

int he_encrypt(he_ctx *ctx, const he_keys *keys, const float *sel_dev, size_t k, uint64_t seed,
               uint32_t client_id, uint64_t *ct_dev, void *stream) {
    if (!good(ctx)) return HE_ERR_INVALID_ARG;
    return he_encrypt_range(ctx, keys, sel_dev, 0, he_num_ct(ctx, k), seed, client_id, ct_dev, stream);
}

enum AggMode { AGG_RESCALE, AGG_NTT, AGG_PARTIAL };

static int weighted_aggregate(he_ctx *ctx, const uint64_t *const *cts_host, const double *alpha_host, int C,
                              size_t T, AggMode mode, uint64_t *agg_dev, void *stream) {
    if (!good(ctx) || !cts_host || !alpha_host || C < 1) return HE_ERR_INVALID_ARG;
    if (C > HE_MAX_CLIENTS) return HE_ERR_SIZE;
    if (T && (!agg_dev || !aligned16(agg_dev))) return HE_ERR_INVALID_ARG;
    const CtxDev &d = ctx->dev;
    const uint32_t L = d.L;
    // weights as constant polynomials at scale q_{L-1}: W_i = rint(alpha_i * q_{L-1})
    const double ql = (double)d.limb[L - 1].q;
    std::vector<unsigned char> host(C * (sizeof(void *) + L * sizeof(tw_t)));
    const uint64_t **ptrs = reinterpret_cast<const uint64_t **>(host.data());
    tw_t *wt = reinterpret_cast<tw_t *>(host.data() + C * sizeof(void *));
    for (int i = 0; i < C; i++) {
        if (T && (!cts_host[i] || !aligned16(cts_host[i]))) return HE_ERR_INVALID_ARG;
        const double a = alpha_host[i];
        if (!(a >= 0.0) || !(a <= 1.0)) return HE_ERR_INVALID_ARG;
        const double prod = a * ql;
        const uint64_t W = (uint64_t)rint(prod);
        ptrs[i] = cts_host[i];
        for (uint32_t j = 0; j < L; j++) {
            const HostTw w = host_shoup(W % d.limb[j].q, d.limb[j].q);
            wt[i * L + j] = tw_t{w.w, w.wp};
        }
    }
    if (T == 0) return HE_OK;
    cudaStream_t st = as_stream(stream);
    CU(cudaMemcpyAsync(ctx->tab, host.data(), host.size(), cudaMemcpyHostToDevice, st));
    const uint64_t *const *dptrs = static_cast<const uint64_t *const *>(ctx->tab);
    const tw_t *dw = reinterpret_cast<const tw_t *>(static_cast<unsigned char *>(ctx->tab) + C * sizeof(void *));
    if (mode == AGG_NTT) {
        int rc = ensure(&ctx->ws, &ctx->ws_bytes, 2 * T * (size_t)L * d.N * sizeof(uint64_t));
        if (rc != HE_OK) return rc;
        CU(launch_aggregate_ntt(d, dptrs, dw, C, T, static_cast<uint64_t *>(ctx->ws), agg_dev, st));
    } else if (mode == AGG_PARTIAL) {
        CU(launch_aggregate_partial(d, dptrs, dw, C, T, agg_dev, st));
    } else {
        CU(launch_aggregate(d, dptrs, dw, C, T, agg_dev, st));
    }
    return HE_OK;
}

int he_weighted_aggregate(he_ctx *ctx, const uint64_t *const *cts_host, const double *alpha_host, int C,
                          size_t T, uint64_t *agg_dev, void *stream) {
    return weighted_aggregate(ctx, cts_host, alpha_host, C, T, AGG_RESCALE, agg_dev, stream);
}

int he_weighted_partial(he_ctx *ctx, const uint64_t *const *cts_host, const double *alpha_host, int C, size_t T,
                        uint64_t *partial_dev, void *stream) {
    return weighted_aggregate(ctx, cts_host, alpha_host, C, T, AGG_PARTIAL, partial_dev, stream);
}

// `added`: how many canonical partial sums every word of the buffers may hold in total
static int rescale_partial(he_ctx *ctx, const uint64_t *const *parts_host, int P, uint64_t added, size_t T,
                           uint64_t *agg_dev, void *stream) {
    if (!good(ctx) || !parts_host || P < 1 || added < 1) return HE_ERR_INVALID_ARG;
    if (P > HE_MAX_CLIENTS) return HE_ERR_SIZE;
    uint64_t qmax = 0;
    for (uint32_t j = 0; j < ctx->dev.L; j++) qmax = ctx->dev.limb[j].q > qmax ? ctx->dev.limb[j].q : qmax;
    if (added > UINT64_MAX / qmax) return HE_ERR_SIZE;         // the 64-bit sums could wrap
    if (T == 0) return HE_OK;
    if (!agg_dev || !aligned16(agg_dev)) return HE_ERR_INVALID_ARG;
    for (int p = 0; p < P; p++)
        if (!parts_host[p] || !aligned16(parts_host[p])) return HE_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    CU(cudaMemcpyAsync(ctx->tab, parts_host, P * sizeof(void *), cudaMemcpyHostToDevice, st));
    CU(launch_rescale_partial_sum(ctx->dev, static_cast<const uint64_t *const *>(ctx->tab), P, T, agg_dev, st));
    return HE_OK;
}

int he_rescale_partial_sum(he_ctx *ctx, const uint64_t *sum_dev, uint32_t parts, size_t T, uint64_t *agg_dev,
                           void *stream) {
    const uint64_t *one[1] = {sum_dev};
    return rescale_partial(ctx, one, 1, parts, T, agg_dev, stream);
}

int he_rescale_partial_parts(he_ctx *ctx, const uint64_t *const *parts_host, int P, size_t T, uint64_t *agg_dev,
                             void *stream) {
    return rescale_partial(ctx, parts_host, P, P < 1 ? 1 : (uint64_t)P, T, agg_dev, stream);
}

int he_weighted_aggregate_ntt(he_ctx *ctx, const uint64_t *const *cts_host, const double *alpha_host, int C,
                              size_t T, uint64_t *agg_dev, void *stream) {
    return weighted_aggregate(ctx, cts_host, alpha_host, C, T, AGG_NTT, agg_dev, stream);
}

int he_plain_aggregate(he_ctx *ctx, const float *const *rests_host, const double *alpha_host, int C,
                       size_t len, double *out_dev, void *stream) {
    if (!good(ctx) || !rests_host || !alpha_host || C < 1) return HE_ERR_INVALID_ARG;
    if (C > HE_MAX_CLIENTS) return HE_ERR_SIZE;
    if (len == 0) return HE_OK;
    if (!out_dev) return HE_ERR_INVALID_ARG;
    std::vector<unsigned char> host(C * (sizeof(void *) + sizeof(double)));
    const float **ptrs = reinterpret_cast<const float **>(host.data());
    double *al = reinterpret_cast<double *>(host.data() + C * sizeof(void *));
    bool aligned = true;
    for (int i = 0; i < C; i++) {
        if (!rests_host[i]) return HE_ERR_INVALID_ARG;
        ptrs[i] = rests_host[i];
        al[i] = alpha_host[i];
        aligned = aligned && aligned16(rests_host[i]);
    }
    cudaStream_t st = as_stream(stream);
    // second half of the table buffer, so that it does not collide with a
    // ciphertext aggregation queued just before
    unsigned char *base = static_cast<unsigned char *>(ctx->tab) + HE_MAX_CLIENTS * (sizeof(void *) + HE_MAX_LIMBS * sizeof(tw_t));
    CU(cudaMemcpyAsync(base, host.data(), host.size(), cudaMemcpyHostToDevice, st));
    CU(launch_plain_aggregate(reinterpret_cast<const float *const *>(base),
                              reinterpret_cast<const double *>(base + C * sizeof(void *)), C, len, out_dev, aligned,
                              st));
    return HE_OK;
}

static int decrypt_level(he_ctx *ctx, const he_keys *keys, const uint64_t *ct_dev, uint32_t level, size_t T,
                         bool ntt_in, double *z_dev, void *stream) {
    if (!good(ctx) || !good(keys) || keys->ctx != ctx || keys->is_share) return HE_ERR_INVALID_ARG;
    if (level < 1 || level > ctx->dev.L) return HE_ERR_LEVEL;
    if (T == 0) return HE_OK;
    if (!ct_dev || !z_dev || !aligned16(ct_dev)) return HE_ERR_INVALID_ARG;
    const CtxDev &d = ctx->dev;
    if (d.logN <= 14) {                 // one fused kernel, no work buffer
        CU(launch_decrypt_fused(d, keys->dev, ct_dev, level, T, ntt_in, z_dev, as_stream(stream)));
        return HE_OK;
    }
    int rc = ensure(&ctx->ws, &ctx->ws_bytes, work_bytes(ctx, T));
    if (rc != HE_OK) return rc;
    uint64_t *scratch = static_cast<uint64_t *>(ctx->ws);
    double2 *cplx = reinterpret_cast<double2 *>(scratch + T * d.N);
    cudaStream_t st = as_stream(stream);
    if (ntt_in) CU(launch_decrypt_ntt(d, keys->dev, ct_dev, level, T, scratch, st));
    else CU(launch_decrypt(d, keys->dev, ct_dev, level, T, scratch, st));
    CU(launch_decode(d, reinterpret_cast<const int64_t *>(scratch), T, cplx, z_dev, st));
    return HE_OK;
}

int he_decrypt_level(he_ctx *ctx, const he_keys *keys, const uint64_t *ct_dev, uint32_t level, size_t T,
                     double *z_dev, void *stream) {
    return decrypt_level(ctx, keys, ct_dev, level, T, false, z_dev, stream);
}

int he_decrypt_level_ntt(he_ctx *ctx, const he_keys *keys, const uint64_t *ct_dev, uint32_t level, size_t T,
                         double *z_dev, void *stream) {
    return decrypt_level(ctx, keys, ct_dev, level, T, true, z_dev, stream);
}

int he_decrypt(he_ctx *ctx, const he_keys *keys, const uint64_t *agg_dev, size_t T, double *z_dev, void *stream) {
    if (!good(ctx)) return HE_ERR_INVALID_ARG;
    return he_decrypt_level(ctx, keys, agg_dev, ctx->dev.L - 1, T, z_dev, stream);
}

int he_unpack(he_ctx *ctx, const he_mask *mask, const double *z_dev, const double *rest_avg_dev, size_t P,
              double *w_glob_dev, void *stream) {
    if (!good(ctx) || !w_glob_dev || P == 0) return HE_ERR_INVALID_ARG;
    if (mask) {
        if (!good(mask) || mask->P != P) return HE_ERR_INVALID_ARG;
        if (mask->k < P && !rest_avg_dev) return HE_ERR_INVALID_ARG;
        if (mask->k && !z_dev) return HE_ERR_INVALID_ARG;
    } else if (!z_dev) {
        return HE_ERR_INVALID_ARG;
    }
    CU(launch_unpack(mask, z_dev, rest_avg_dev, P, w_glob_dev, as_stream(stream)));
    return HE_OK;
}

int he_ntt_forward(he_ctx *ctx, uint64_t *polys_dev, size_t B, void *stream) {
    if (!good(ctx) || !polys_dev || !aligned16(polys_dev)) return HE_ERR_INVALID_ARG;
    const CtxDev &d = ctx->dev;
    if ((B * d.L) >> (31 - d.A)) return HE_ERR_SIZE;
    CU(launch_ntt(d, true, polys_dev, B, (size_t)d.L * d.N, 0, d.L, as_stream(stream)));
    return HE_OK;
}

int he_ntt_inverse(he_ctx *ctx, uint64_t *polys_dev, size_t B, void *stream) {
    if (!good(ctx) || !polys_dev || !aligned16(polys_dev)) return HE_ERR_INVALID_ARG;
    const CtxDev &d = ctx->dev;
    if ((B * d.L) >> (31 - d.A)) return HE_ERR_SIZE;
    CU(launch_ntt(d, false, polys_dev, B, (size_t)d.L * d.N, 0, d.L, as_stream(stream)));
    return HE_OK;
}

// ---------------------------------------------------------------------------
// two-party threshold decryption
// ---------------------------------------------------------------------------

int he_threshold_split(he_ctx *ctx, const he_keys *keys, uint64_t seed, he_keys **share0, he_keys **share1,
                       void *stream) {
    if (!good(ctx) || !good(keys) || keys->ctx != ctx || keys->is_share || !share0 || !share1)
        return HE_ERR_INVALID_ARG;
    *share0 = *share1 = nullptr;
    const CtxDev &d = ctx->dev;
    const size_t LN = (size_t)d.L * d.N;
    cudaStream_t st = as_stream(stream);
    void *tmp = nullptr;
    he_keys *sh[2] = {nullptr, nullptr};
    int rc = HE_OK;
    do {
        if (cudaMalloc(&tmp, 2 * LN * sizeof(uint64_t)) != cudaSuccess) { rc = HE_ERR_ALLOC; break; }
        uint64_t *t64 = static_cast<uint64_t *>(tmp);
        if (launch_threshold_split(d, keys->dev.s, seed, t64, st) != cudaSuccess ||
            launch_ntt(d, true, t64, 2, LN, 0, d.L, st) != cudaSuccess) {
            rc = HE_ERR_CUDA;
            break;
        }
        for (int p = 0; p < 2 && rc == HE_OK; p++) {
            sh[p] = new (std::nothrow) he_keys();
            if (!sh[p]) { rc = HE_ERR_ALLOC; break; }
            sh[p]->magic = KEYS_MAGIC;
            sh[p]->ctx = ctx;
            sh[p]->is_share = true;
            sh[p]->storage = nullptr;
            if (cudaMalloc(&sh[p]->storage, LN * sizeof(tw_t)) != cudaSuccess) { rc = HE_ERR_ALLOC; break; }
            tw_t *tab = static_cast<tw_t *>(sh[p]->storage);
            sh[p]->dev = KeysDev{nullptr, nullptr, tab, nullptr};
            if (launch_share_tables(d, t64 + p * LN, tab, st) != cudaSuccess) rc = HE_ERR_CUDA;
        }
        if (rc == HE_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = HE_ERR_CUDA;
    } while (0);
    if (tmp) cudaFree(tmp);
    if (rc != HE_OK) {
        for (int p = 0; p < 2; p++)
            if (sh[p]) {
                if (sh[p]->storage) cudaFree(sh[p]->storage);
                delete sh[p];
            }
        return rc;
    }
    *share0 = sh[0];
    *share1 = sh[1];
    return HE_OK;
}

int he_partial_decrypt(he_ctx *ctx, const he_keys *share, uint32_t party, const uint64_t *ct_dev, uint32_t level,
                       size_t T, uint64_t seed, uint32_t smudge_bits, uint64_t *part_dev, void *stream) {
    if (!good(ctx) || !good(share) || share->ctx != ctx || !share->is_share) return HE_ERR_INVALID_ARG;
    if (level < 1 || level > ctx->dev.L) return HE_ERR_LEVEL;
    if (smudge_bits > 40 || T >= (1ull << 32)) return HE_ERR_SIZE;
    if (T == 0) return HE_OK;
    if (!ct_dev || !part_dev || !aligned16(ct_dev) || !aligned16(part_dev)) return HE_ERR_INVALID_ARG;
    CU(launch_partial_decrypt(ctx->dev, share->dev, party, ct_dev, level, T, seed, smudge_bits, part_dev,
                              as_stream(stream)));
    return HE_OK;
}

int he_threshold_combine(he_ctx *ctx, const uint64_t *ct_dev, uint32_t level, const uint64_t *const *parts_host,
                         int nparts, size_t T, double *z_dev, void *stream) {
    if (!good(ctx) || !parts_host || nparts < 1) return HE_ERR_INVALID_ARG;
    if (nparts > 8) return HE_ERR_SIZE;
    if (level < 1 || level > ctx->dev.L) return HE_ERR_LEVEL;
    if (T == 0) return HE_OK;
    if (!ct_dev || !z_dev || !aligned16(ct_dev)) return HE_ERR_INVALID_ARG;
    PartPtrs pp = {};
    for (int p = 0; p < nparts; p++) {
        if (!parts_host[p] || !aligned16(parts_host[p])) return HE_ERR_INVALID_ARG;
        pp.p[p] = parts_host[p];
    }
    void *ws = nullptr;
    const int rc = ctx_workspace(ctx, T, &ws);
    if (rc != HE_OK) return rc;
    int64_t *d = static_cast<int64_t *>(ws);
    double2 *cplx = reinterpret_cast<double2 *>(d + T * ctx->dev.N);
    cudaStream_t st = as_stream(stream);
    CU(launch_threshold_combine(ctx->dev, ct_dev, level, pp, nparts, T, d, st));
    CU(launch_decode(ctx->dev, d, T, cplx, z_dev, st));
    return HE_OK;
}

// ---------------------------------------------------------------------------
// whole round from host memory
// ---------------------------------------------------------------------------

static int round_host_streams(he_ctx *ctx) {
    if (ctx->copy_stream) return HE_OK;
    CU(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    CU(cudaStreamCreateWithFlags(&ctx->down_stream, cudaStreamNonBlocking));
    for (int i = 0; i < 2; i++) {
        CU(cudaEventCreateWithFlags(&ctx->ev_ready[i], cudaEventDisableTiming));
        CU(cudaEventCreateWithFlags(&ctx->ev_free[i], cudaEventDisableTiming));
    }
    CU(cudaEventCreateWithFlags(&ctx->ev_chunk, cudaEventDisableTiming));
    return HE_OK;
}

// The queued part of he_round_host with full encryption (no mask): the packed
// slots of a chunk of ciphertext indices are a contiguous piece of every
// client's update, so each chunk's pieces go straight from the host into the
// slot buffers (no staging copy of the whole update, no pack kernel), on the
// upload stream, one chunk ahead of the arithmetic; the decoded slots of a
// chunk go home on the download stream while the next chunk is computed.
// Chunks start at one wave of thread blocks, so that little is uploaded before
// the first kernel can start, and double up to about 8 GiB of ciphertexts.
static int round_host_full(he_ctx *ctx, const he_keys *keys, const float *const *xs_host, const double *alpha_host,
                           int C, size_t P, uint64_t enc_seed, double *w_glob_host, void *stream) {
    const CtxDev &d = ctx->dev;
    const size_t n = d.N / 2, T = he_num_ct(ctx, P);
    const size_t ctw = 2 * (size_t)d.L * d.N, aggw = 2 * (size_t)(d.L - 1) * d.N;
    const size_t sm = (size_t)ctx->sm_count;
    size_t cap = ((size_t)8 << 30) / (C * ctw * sizeof(uint64_t));
    if (cap > sm) cap -= cap % sm;
    if (cap < 1) cap = 1;
    std::vector<size_t> sizes;
    for (size_t done = 0, cur = sm < cap ? sm : cap; done < T;) {
        size_t tc = T - done < cur ? T - done : cur;
        if (T - done - tc < sm / 2) tc = T - done;          // no sliver at the end
        if (tc > cap && cap >= sm) tc = cap;
        sizes.push_back(tc);
        done += tc;
        cur = 2 * cur < cap ? 2 * cur : cap;
    }
    // the download of the last chunk's slots is not hidden behind anything: keep that chunk to one wave
    if (sizes.size() > 1 && sizes.back() >= 2 * sm) {
        sizes.back() -= sm;
        sizes.push_back(sm);
    }
    size_t Tmax = 0;
    for (size_t v : sizes) Tmax = v > Tmax ? v : Tmax;
    auto align = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const size_t b_sel = align(Tmax * n * sizeof(float)), b_cts = align(C * Tmax * ctw * sizeof(uint64_t)),
                 b_agg = align(Tmax * aggw * sizeof(uint64_t)), b_z = align(T * n * sizeof(double));
    int rc = ensure(&ctx->round_buf, &ctx->round_bytes, 2 * C * b_sel + b_cts + b_agg + b_z);
    if (rc != HE_OK) return rc;
    {
        size_t need = encrypt_work_bytes(d, ctx->sm_count, Tmax, false);
        if (d.A > 0 && work_bytes(ctx, Tmax) > need) need = work_bytes(ctx, Tmax);
        rc = ensure(&ctx->ws, &ctx->ws_bytes, need);
    }
    if (rc != HE_OK) return rc;
    if ((rc = round_host_streams(ctx)) != HE_OK) return rc;
    unsigned char *p = static_cast<unsigned char *>(ctx->round_buf);
    unsigned char *selbuf[2];
    selbuf[0] = p; p += C * b_sel;
    selbuf[1] = p; p += C * b_sel;
    uint64_t *cts = reinterpret_cast<uint64_t *>(p); p += b_cts;
    uint64_t *agg = reinterpret_cast<uint64_t *>(p); p += b_agg;
    double *z = reinterpret_cast<double *>(p);
    cudaStream_t st = as_stream(stream);
    CU(cudaEventRecord(ctx->ev_free[0], st));       // earlier work on `st` may still use the buffers
    CU(cudaEventRecord(ctx->ev_free[1], st));

    // one client's slots of the chunk [t0, t0 + tc) into the slot buffers of parity b
    auto upload_client = [&](int b, int i, size_t t0, size_t tc) -> int {
        const size_t first = t0 * n, want = tc * n, have = P - first < want ? P - first : want;
        float *dst = reinterpret_cast<float *>(selbuf[b] + (size_t)i * b_sel);
        CU(cudaMemcpyAsync(dst, xs_host[i] + first, have * sizeof(float), cudaMemcpyHostToDevice, ctx->copy_stream));
        if (have < want)                             // the ragged tail of the last ciphertext
            CU(cudaMemsetAsync(dst + have, 0, (want - have) * sizeof(float), ctx->copy_stream));
        return HE_OK;
    };
    auto upload = [&](size_t c, size_t t0, size_t tc) -> int {
        const int b = (int)(c & 1);
        CU(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_free[b], 0));
        for (int i = 0; i < C; i++) {
            const int urc = upload_client(b, i, t0, tc);
            if (urc != HE_OK) return urc;
        }
        CU(cudaEventRecord(ctx->ev_ready[b], ctx->copy_stream));
        return HE_OK;
    };
    std::vector<const uint64_t *> cptr(C);
    size_t t0 = 0;
    for (size_t c = 0; c < sizes.size(); c++) {
        const size_t tc = sizes[c];
        const int b = (int)(c & 1);
        if (c == 0) CU(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_free[b], 0));
        else CU(cudaStreamWaitEvent(st, ctx->ev_ready[b], 0));
        for (int i = 0; i < C; i++) {
            if (c == 0) {
                // the first chunk client by client: a client's encryption starts as soon as its own
                // slots have arrived (a wait takes the event's latest record at the time of the call)
                if ((rc = upload_client(b, i, t0, tc)) != HE_OK) return rc;
                CU(cudaEventRecord(ctx->ev_ready[b], ctx->copy_stream));
                CU(cudaStreamWaitEvent(st, ctx->ev_ready[b], 0));
            }
            uint64_t *ci = cts + (size_t)i * Tmax * ctw;
            rc = he_encrypt_range(ctx, keys, reinterpret_cast<const float *>(selbuf[b] + (size_t)i * b_sel), t0, tc,
                                  enc_seed, (uint32_t)i, ci, stream);
            if (rc != HE_OK) return rc;
            cptr[i] = ci;
        }
        CU(cudaEventRecord(ctx->ev_free[b], st));   // the slot buffers of this parity may be refilled
        // the next chunk's slots go up while this chunk is computed
        if (c + 1 < sizes.size() && (rc = upload(c + 1, t0 + tc, sizes[c + 1])) != HE_OK) return rc;
        rc = he_weighted_aggregate(ctx, cptr.data(), alpha_host, C, tc, agg, stream);
        if (rc != HE_OK) return rc;
        rc = he_decrypt(ctx, keys, agg, tc, z + t0 * n, stream);
        if (rc != HE_OK) return rc;
        const size_t first = t0 * n, count = P - first < tc * n ? P - first : tc * n;
        CU(cudaEventRecord(ctx->ev_chunk, st));
        CU(cudaStreamWaitEvent(ctx->down_stream, ctx->ev_chunk, 0));
        CU(cudaMemcpyAsync(w_glob_host + first, z + first, count * sizeof(double), cudaMemcpyDeviceToHost,
                           ctx->down_stream));
        t0 += tc;
    }
    return HE_OK;                                    // the caller waits for the streams
}

// The queued part of he_round_host with a mask; every argument has been validated.
static int round_host_queued(he_ctx *ctx, const he_keys *keys, const he_mask *mask, const float *const *xs_host,
                             const double *alpha_host, int C, size_t P, size_t k, uint64_t enc_seed,
                             double *w_glob_host, void *stream) {
    const CtxDev &d = ctx->dev;
    const size_t n = d.N / 2, T = he_num_ct(ctx, k), padded = T * n, restlen = P - k;
    const size_t ctw = 2 * (size_t)d.L * d.N, aggw = 2 * (size_t)(d.L - 1) * d.N;
    // The mask gathers from anywhere in an update, so every client's whole
    // update is uploaded (two staging buffers on the upload stream: the upload of
    // client i+1 overlaps the packing and first encryption of client i).
    // Ciphertext indices are processed in chunks that keep all clients'
    // ciphertexts of a chunk within about 8 GiB; a chunk is a whole number of
    // waves of one thread block per SM.
    const size_t sm = (size_t)ctx->sm_count;
    auto whole_waves = [&](size_t want, size_t cap) {
        size_t v = want < cap ? want : cap;
        if (v > sm) v -= v % sm;
        return v < 1 ? (size_t)1 : v;
    };
    const size_t cap = ((size_t)8 << 30) / (C * ctw * sizeof(uint64_t));
    size_t Tc = (T < 4 * sm && T <= cap) ? T : whole_waves((T + 1) / 2 + sm - 1, cap);   // first chunk, the largest
    if (Tc > T) Tc = T;
    const size_t Tc_rest = T > Tc ? whole_waves((T - Tc + 1) / 2 + sm - 1, Tc) : Tc;
    auto align = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const size_t b_x = align(P * sizeof(float)), b_sel = align(padded * sizeof(float)),
                 b_rest = align(restlen * sizeof(float)), b_cts = align(C * Tc * ctw * sizeof(uint64_t)),
                 b_agg = align(Tc * aggw * sizeof(uint64_t)), b_z = align(padded * sizeof(double)),
                 b_ravg = align(restlen * sizeof(double)), b_out = align(P * sizeof(double));
    const size_t total = 2 * b_x + C * (b_sel + b_rest) + b_cts + b_agg + b_z + b_ravg + b_out;
    int rc = ensure(&ctx->round_buf, &ctx->round_bytes, total);
    if (rc != HE_OK) return rc;
    {
        size_t need = encrypt_work_bytes(d, ctx->sm_count, Tc, false);
        if (d.A > 0 && work_bytes(ctx, Tc) > need) need = work_bytes(ctx, Tc);
        rc = ensure(&ctx->ws, &ctx->ws_bytes, need);
    }
    if (rc != HE_OK) return rc;
    unsigned char *p = static_cast<unsigned char *>(ctx->round_buf);
    float *x[2];
    x[0] = reinterpret_cast<float *>(p); p += b_x;
    x[1] = reinterpret_cast<float *>(p); p += b_x;
    std::vector<float *> sel(C), rest(C);
    for (int i = 0; i < C; i++) { sel[i] = reinterpret_cast<float *>(p); p += b_sel; }
    for (int i = 0; i < C; i++) { rest[i] = reinterpret_cast<float *>(p); p += b_rest; }
    uint64_t *cts = reinterpret_cast<uint64_t *>(p); p += b_cts;
    uint64_t *agg = reinterpret_cast<uint64_t *>(p); p += b_agg;
    double *z = reinterpret_cast<double *>(p); p += b_z;
    double *ravg = reinterpret_cast<double *>(p); p += b_ravg;
    double *out = reinterpret_cast<double *>(p);
    cudaStream_t st = as_stream(stream);

    if ((rc = round_host_streams(ctx)) != HE_OK) return rc;
    CU(cudaEventRecord(ctx->ev_free[0], st));       // earlier work on `st` may still use the buffers
    CU(cudaEventRecord(ctx->ev_free[1], st));
    std::vector<const uint64_t *> cptr(C);
    for (size_t t0 = 0, step = Tc; t0 < T || t0 == 0; t0 += step, step = Tc_rest) {
        const size_t tc = T - t0 < step ? T - t0 : step;
        for (int i = 0; i < C; i++) {
            const int b = i & 1;
            if (t0 == 0) {
                CU(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_free[b], 0));
                CU(cudaMemcpyAsync(x[b], xs_host[i], P * sizeof(float), cudaMemcpyHostToDevice, ctx->copy_stream));
                CU(cudaEventRecord(ctx->ev_ready[b], ctx->copy_stream));
                CU(cudaStreamWaitEvent(st, ctx->ev_ready[b], 0));
                rc = he_pack(ctx, mask, x[b], P, sel[i], restlen ? rest[i] : nullptr, stream);
                if (rc != HE_OK) return rc;
                CU(cudaEventRecord(ctx->ev_free[b], st));
            }
            if (tc == 0) continue;
            uint64_t *ci = cts + (size_t)i * Tc * ctw;
            rc = he_encrypt_range(ctx, keys, sel[i] + t0 * n, t0, tc, enc_seed, (uint32_t)i, ci, stream);
            if (rc != HE_OK) return rc;
            cptr[i] = ci;
        }
        if (tc == 0) break;
        rc = he_weighted_aggregate(ctx, cptr.data(), alpha_host, C, tc, agg, stream);
        if (rc != HE_OK) return rc;
        rc = he_decrypt(ctx, keys, agg, tc, z + t0 * n, stream);
        if (rc != HE_OK) return rc;
    }
    if (restlen) {
        std::vector<const float *> rptr(rest.begin(), rest.end());
        rc = he_plain_aggregate(ctx, rptr.data(), alpha_host, C, restlen, ravg, stream);
        if (rc != HE_OK) return rc;
    }
    rc = he_unpack(ctx, mask, z, restlen ? ravg : nullptr, P, out, stream);
    if (rc != HE_OK) return rc;
    CU(cudaMemcpyAsync(w_glob_host, out, P * sizeof(double), cudaMemcpyDeviceToHost, st));
    return HE_OK;
}

int he_round_host(he_ctx *ctx, const he_keys *keys, const he_mask *mask, const float *const *xs_host,
                  const double *alpha_host, int C, size_t P, uint64_t enc_seed, double *w_glob_host,
                  void *stream) {
    // everything that can be refused is refused here, before anything is queued
    if (!good(ctx) || !good(keys) || keys->ctx != ctx || keys->is_share || !xs_host || !alpha_host || !w_glob_host || C < 1 || P == 0)
        return HE_ERR_INVALID_ARG;
    if (C > HE_MAX_CLIENTS) return HE_ERR_SIZE;
    size_t k = P;
    if (mask) {
        if (!good(mask) || mask->P != P) return HE_ERR_INVALID_ARG;
        k = mask->k;
    }
    for (int i = 0; i < C; i++) {
        if (!xs_host[i]) return HE_ERR_INVALID_ARG;
        if (!(alpha_host[i] >= 0.0) || !(alpha_host[i] <= 1.0)) return HE_ERR_INVALID_ARG;
    }
    const int rc = mask ? round_host_queued(ctx, keys, mask, xs_host, alpha_host, C, P, k, enc_seed, w_glob_host, stream)
                        : round_host_full(ctx, keys, xs_host, alpha_host, C, P, enc_seed, w_glob_host, stream);
    // Success or not, nothing may still be reading xs or writing w_glob when the
    // call returns: wait for both streams (on an error path their status is ignored).
    cudaError_t e0 = ctx->copy_stream ? cudaStreamSynchronize(ctx->copy_stream) : cudaSuccess;
    cudaError_t e1 = cudaStreamSynchronize(as_stream(stream));
    cudaError_t e2 = ctx->down_stream ? cudaStreamSynchronize(ctx->down_stream) : cudaSuccess;
    if (rc != HE_OK) return rc;
    return (e0 == cudaSuccess && e1 == cudaSuccess && e2 == cudaSuccess) ? HE_OK : HE_ERR_CUDA;
}

}  // extern "C"
