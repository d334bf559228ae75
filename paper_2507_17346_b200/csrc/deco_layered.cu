// Per-layer Top-k: the flat vector is cut into layers [offset_l, offset_{l+1}) and every worker
// keeps the k_l = k(delta, d_l) largest entries of each layer.  Layers do not interact anywhere
// in Algorithm 1 (accumulate, select, residual, aggregate and update are all entry-wise or
// per-selection), so the variant is a batch of independent contexts, one per layer, that share
// the policy (delta, tau), the stepsize, the gradient buffer (rows of the full length d, the
// layer's columns starting at its offset) and the parameter vector (the layer's slice).  The
// layers are stepped round-robin on a few internal streams forked from and joined back into
// the caller's stream.
#include "deco_internal.h"

#include <new>
#include <vector>

namespace {
constexpr int LAYER_STREAMS = 4;
}

struct deco_layered {
    uint64_t d = 0;
    uint32_t n = 0;
    int device = 0;
    int grad_dtype = DECO_F32;
    std::vector<deco_ctx *> layers;
    std::vector<uint64_t> offsets;       // n_layers + 1
    float *params = nullptr;
    bool own_params = false;
    cudaStream_t streams[LAYER_STREAMS] = {};
    cudaEvent_t ev_fork = nullptr;
    cudaEvent_t ev_done[LAYER_STREAMS] = {};
    uint64_t t = 0;
};

namespace {

struct Guard {
    int prev = -1;
    bool ok = false;
    explicit Guard(int dev)
    {
        ok = cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess);
    }
    ~Guard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

void release(deco_layered *L)
{
    for (deco_ctx *c : L->layers) deco_destroy(c);
    for (cudaStream_t s : L->streams)
        if (s) cudaStreamDestroy(s);
    for (cudaEvent_t e : L->ev_done)
        if (e) cudaEventDestroy(e);
    if (L->ev_fork) cudaEventDestroy(L->ev_fork);
    if (L->own_params) cudaFree(L->params);
    delete L;
}

}  // namespace

extern "C" deco_status deco_layered_init(deco_layered **out, uint64_t d, uint32_t n,
                                         const uint64_t *layer_offsets, uint32_t n_layers,
                                         double delta, uint32_t tau, float lr,
                                         const deco_options *opt)
{
    if (!out || !layer_offsets || n_layers == 0 || n_layers > (1u << 20)) return DECO_ERR_INVALID_ARG;
    if (layer_offsets[0] != 0 || layer_offsets[n_layers] != d) return DECO_ERR_INVALID_ARG;
    for (uint32_t l = 0; l < n_layers; ++l)
        if (layer_offsets[l + 1] <= layer_offsets[l]) return DECO_ERR_INVALID_ARG;
    deco_options o = {};
    if (opt) o = *opt;
    if (o.params && (reinterpret_cast<uintptr_t>(o.params) & 15u)) return DECO_ERR_INVALID_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || o.device < 0 || o.device >= ndev) {
        cudaGetLastError();
        return DECO_ERR_INVALID_ARG;
    }
    Guard guard(o.device);
    if (!guard.ok) return DECO_ERR_CUDA;
    deco_layered *L = new (std::nothrow) deco_layered();
    if (!L) return DECO_ERR_OOM;
    L->d = d;
    L->n = n;
    L->device = o.device;
    L->grad_dtype = o.grad_dtype;
    try {
        L->offsets.assign(layer_offsets, layer_offsets + n_layers + 1);
        L->layers.reserve(n_layers);
    } catch (...) {
        delete L;
        return DECO_ERR_OOM;
    }
    if (o.params) {
        L->params = o.params;
    } else {
        const cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&L->params), sizeof(float) * d);
        if (err != cudaSuccess || cudaMemset(L->params, 0, sizeof(float) * d) != cudaSuccess) {
            cudaGetLastError();
            release(L);
            return err == cudaErrorMemoryAllocation ? DECO_ERR_OOM : DECO_ERR_CUDA;
        }
        L->own_params = true;
    }
    bool ok = cudaEventCreateWithFlags(&L->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    for (int q = 0; q < LAYER_STREAMS && ok; ++q)
        ok = cudaStreamCreateWithFlags(&L->streams[q], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&L->ev_done[q], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        release(L);
        return DECO_ERR_CUDA;
    }
    for (uint32_t l = 0; l < n_layers; ++l) {
        deco_options ol = o;
        ol.params = L->params + L->offsets[l];
        // Random-k: every layer draws from a priority stream of its own
        const uint64_t seed = ((static_cast<uint64_t>(o.seed_hi) << 32) | o.seed_lo) + l;
        ol.seed_lo = static_cast<uint32_t>(seed);
        ol.seed_hi = static_cast<uint32_t>(seed >> 32);
        deco_ctx *c = nullptr;
        const deco_status st = deco::init_context(&c, L->offsets[l + 1] - L->offsets[l], n, delta, tau,
                                                  lr, &ol, d);
        if (st != DECO_OK) {
            release(L);
            return st;
        }
        L->layers.push_back(c);
    }
    *out = L;
    return DECO_OK;
}

extern "C" void deco_layered_destroy(deco_layered *L)
{
    if (!L) return;
    Guard guard(L->device);
    cudaDeviceSynchronize();
    release(L);
}

extern "C" deco_status deco_layered_step(deco_layered *L, const void *grads, void *stream)
{
    if (!L || !grads) return DECO_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(grads) & 15u) return DECO_ERR_INVALID_ARG;
    Guard guard(L->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaEventRecord(L->ev_fork, s) != cudaSuccess) return DECO_ERR_CUDA;
    for (cudaStream_t q : L->streams)
        if (cudaStreamWaitEvent(q, L->ev_fork, 0) != cudaSuccess) return DECO_ERR_CUDA;
    const size_t esz = L->grad_dtype == DECO_BF16 ? 2 : 4;
    deco_status st = DECO_OK;
    for (size_t l = 0; l < L->layers.size() && st == DECO_OK; ++l)
        st = deco_step(L->layers[l], static_cast<const char *>(grads) + L->offsets[l] * esz,
                       L->streams[l % LAYER_STREAMS]);
    for (int q = 0; q < LAYER_STREAMS; ++q)
        if (cudaEventRecord(L->ev_done[q], L->streams[q]) != cudaSuccess ||
            cudaStreamWaitEvent(s, L->ev_done[q], 0) != cudaSuccess)
            return DECO_ERR_CUDA;
    if (st == DECO_OK) L->t += 1;
    return st;
}

extern "C" deco_status deco_layered_join(deco_layered *L, void *stream)
{
    if (!L) return DECO_ERR_INVALID_ARG;
    deco_status st = DECO_OK;
    for (deco_ctx *c : L->layers)
        if (st == DECO_OK) st = deco_join(c, stream);
    return st;
}

extern "C" deco_status deco_layered_set_policy(deco_layered *L, double delta, uint32_t tau)
{
    if (!L) return DECO_ERR_INVALID_ARG;
    if (!(delta > 0.0) || !(delta <= 1.0)) return DECO_ERR_INVALID_ARG;
    // all or nothing: check every layer's capacity first
    for (deco_ctx *c : L->layers)
        if (tau > c->tau_max || deco_k_from_delta(delta, c->d) > c->k_cap) return DECO_ERR_CAPACITY;
    for (deco_ctx *c : L->layers) {
        const deco_status st = deco_set_policy(c, delta, tau);
        if (st != DECO_OK) return st;
    }
    return DECO_OK;
}

extern "C" deco_status deco_layered_set_lr(deco_layered *L, float lr)
{
    if (!L) return DECO_ERR_INVALID_ARG;
    for (deco_ctx *c : L->layers) {
        const deco_status st = deco_set_lr(c, lr);
        if (st != DECO_OK) return st;
    }
    return DECO_OK;
}

extern "C" deco_status deco_layered_layer(deco_layered *L, uint32_t layer, deco_ctx **ctx,
                                          uint64_t *offset, uint64_t *length)
{
    if (!L || layer >= L->layers.size()) return DECO_ERR_INVALID_ARG;
    if (ctx) *ctx = L->layers[layer];
    if (offset) *offset = L->offsets[layer];
    if (length) *length = L->offsets[layer + 1] - L->offsets[layer];
    return DECO_OK;
}

extern "C" deco_status deco_layered_info(deco_layered *L, uint32_t *n_layers, uint64_t *k_total,
                                         float **params, uint64_t *step)
{
    if (!L) return DECO_ERR_INVALID_ARG;
    if (n_layers) *n_layers = static_cast<uint32_t>(L->layers.size());
    if (k_total) {
        *k_total = 0;
        for (deco_ctx *c : L->layers) *k_total += c->k;
    }
    if (params) *params = L->params;
    if (step) *step = L->t;
    return DECO_OK;
}
