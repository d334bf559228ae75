// Per-layer Top-k: the flat vector is cut into layers [offset_l, offset_{l+1}) and every worker
// keeps the k_l = k(delta, d_l) largest entries of each layer.  Layers do not interact anywhere
// in Algorithm 1 (accumulate, select, residual, aggregate and update are all entry-wise or
// per-selection), so the variant is a batch of independent contexts, one per layer, that share
// the policy (delta, tau), the stepsize, the gradient buffer (rows of the full length d, the
// layer's columns starting at its offset) and the parameter vector (the layer's slice).  The
// layers are stepped round-robin on a few internal streams forked from and joined back into
// the caller's stream.
//
// Layers of at most one tile (Top-k on the streaming route) are not stepped one by one: their
// contexts only hold the buffers, and two launches do the device work of all of them (one CTA
// per layer and worker for the worker side, one CTA per layer for aggregation and update).
#include "deco_internal.h"

#include <algorithm>
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
    // the short layers that are stepped as one batch
    std::vector<uint32_t> small;                 // their layer numbers
    std::vector<uint32_t> big;                   // all other layers
    std::vector<deco::SmallLayer> small_host;    // the table, host copy
    deco::SmallLayer *small_dev = nullptr;
    uint32_t *small_slot_pos = nullptr;          // [small][ring]
    bool small_dirty = true;                     // k changed: upload the table before the next step
    // the other layers' worker side runs in a fixed number of launches when they all use
    // Top-k on the streaming route
    deco::MultiPlan *plan = nullptr;
    std::vector<deco::ServerLayer> server_host;  // one entry per layer of `big`
    deco::ServerLayer *server_dev = nullptr;
    uint32_t *big_tile_layer = nullptr;          // device: layer (position in `big`) of every tile
    uint32_t *big_slot_pos = nullptr;            // device: [big][ring]
    uint32_t big_tiles = 0;
    bool server_dirty = true;
    bool any_dense = false, any_sparse = false;
    uint32_t apply_ctas = 1;
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
    deco::multi_plan_destroy(L->plan);
    cudaFree(L->server_dev);
    cudaFree(L->big_tile_layer);
    cudaFree(L->big_slot_pos);
    cudaFree(L->small_dev);
    cudaFree(L->small_slot_pos);
    if (L->own_params) cudaFree(L->params);
    delete L;
}

// Sort the layers into the batch of short ones and the rest, and build the batch's table.
cudaError_t build_small_batch(deco_layered *L)
{
    for (uint32_t l = 0; l < L->layers.size(); ++l) {
        const deco_ctx *c = L->layers[l];
        const bool is_small = c->d <= static_cast<uint64_t>(deco::TILE) &&
                              c->compressor == DECO_COMPRESSOR_TOPK &&
                              c->select_mode == DECO_SELECT_AUTO && c->n_total == c->n;
        (is_small ? L->small : L->big).push_back(l);
    }
    bool batchable = !L->big.empty();
    std::vector<deco_ctx *> ctxs;
    std::vector<uint64_t> offs;
    for (uint32_t l : L->big) {
        const deco_ctx *c = L->layers[l];
        batchable = batchable && c->compressor == DECO_COMPRESSOR_TOPK &&
                    c->select_mode == DECO_SELECT_AUTO && c->n_total == c->n;
        ctxs.push_back(L->layers[l]);
        offs.push_back(L->offsets[l]);
    }
    if (batchable) {
        L->plan = deco::multi_plan_create(ctxs, offs, L->n, L->grad_dtype);
        if (!L->plan) return cudaErrorMemoryAllocation;
        const uint32_t ring = ctxs[0]->ring;
        std::vector<uint32_t> map;
        L->server_host.resize(ctxs.size());
        for (size_t q = 0; q < ctxs.size(); ++q) {
            L->server_host[q].first_tile = static_cast<uint32_t>(map.size());
            map.insert(map.end(), ctxs[q]->ntiles, static_cast<uint32_t>(q));
        }
        L->big_tiles = static_cast<uint32_t>(map.size());
        cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&L->server_dev),
                                     sizeof(deco::ServerLayer) * ctxs.size());
        if (err == cudaSuccess)
            err = cudaMalloc(reinterpret_cast<void **>(&L->big_tile_layer), sizeof(uint32_t) * map.size());
        if (err == cudaSuccess)
            err = cudaMemcpy(L->big_tile_layer, map.data(), sizeof(uint32_t) * map.size(), cudaMemcpyHostToDevice);
        if (err == cudaSuccess)
            err = cudaMalloc(reinterpret_cast<void **>(&L->big_slot_pos), sizeof(uint32_t) * ctxs.size() * ring);
        if (err == cudaSuccess)
            err = cudaMemset(L->big_slot_pos, 0, sizeof(uint32_t) * ctxs.size() * ring);
        if (err != cudaSuccess) return err;
        for (size_t q = 0; q < ctxs.size(); ++q) {
            const deco_ctx *c = ctxs[q];
            deco::ServerLayer &e = L->server_host[q];
            e.msg = c->msg;
            e.k_cap = c->k_cap;
            e.tile_start = c->tile_start;
            e.slots = c->slots;
            e.params = c->params;
            e.status = c->dev_status;
            e.slot_pos = L->big_slot_pos + q * ring;
            e.d = c->d;
            e.ntiles = c->ntiles;
        }
        L->server_dirty = true;
    }
    if (L->small.empty()) return cudaSuccess;
    const uint32_t ring = L->layers[L->small[0]]->ring;
    cudaError_t err = cudaMalloc(reinterpret_cast<void **>(&L->small_dev),
                                 sizeof(deco::SmallLayer) * L->small.size());
    if (err == cudaSuccess)
        err = cudaMalloc(reinterpret_cast<void **>(&L->small_slot_pos),
                         sizeof(uint32_t) * L->small.size() * ring);
    if (err == cudaSuccess)
        err = cudaMemset(L->small_slot_pos, 0, sizeof(uint32_t) * L->small.size() * ring);
    if (err != cudaSuccess) return err;
    L->small_host.resize(L->small.size());
    for (size_t q = 0; q < L->small.size(); ++q) {
        deco_ctx *c = L->layers[L->small[q]];
        deco::SmallLayer &e = L->small_host[q];
        e.e = c->e;
        e.e_stride = c->e_stride;
        e.g_off = L->offsets[L->small[q]];
        e.msg = c->msg;
        e.k_cap = c->k_cap;
        e.slots = c->slots;
        e.tile_start = c->tile_start;
        e.sel = c->sel;
        e.params = c->params;
        e.status = c->dev_status;
        e.slot_pos = L->small_slot_pos + q * ring;
        e.d = static_cast<uint32_t>(c->d);
        e.k = static_cast<uint32_t>(c->k);
    }
    L->small_dirty = true;
    return cudaSuccess;
}

// One iteration of all short layers on stream s: table upload if k changed, worker side,
// aggregation and update, and the host bookkeeping of every context.
deco_status step_small_batch(deco_layered *L, const void *grads, cudaStream_t s)
{
    if (L->small.empty()) return DECO_OK;
    const uint32_t layers = static_cast<uint32_t>(L->small.size());
    deco_ctx *first = L->layers[L->small[0]];
    for (uint32_t l : L->small)
        if (L->layers[l]->phase != 0) return DECO_ERR_STATE;
    if (L->small_dirty) {
        for (size_t q = 0; q < L->small.size(); ++q)
            L->small_host[q].k = static_cast<uint32_t>(L->layers[L->small[q]]->k);
        // the host table is pageable: the copy has left it when the call returns
        if (cudaMemcpyAsync(L->small_dev, L->small_host.data(), sizeof(deco::SmallLayer) * layers,
                            cudaMemcpyHostToDevice, s) != cudaSuccess)
            return DECO_ERR_CUDA;
        L->small_dirty = false;
    }
    const float alpha = first->lr_at_server ? 1.0f : first->lr;
    const float beta = first->lr_at_server ? first->lr : 1.0f;
    const float neg_scale = -(beta / static_cast<float>(first->n_total));
    if (deco::launch_small_workers(L->small_dev, layers, L->n, grads, L->d, L->grad_dtype, alpha, s) !=
        cudaSuccess)
        return DECO_ERR_CUDA;
    // every layer shares t, tau and the ring size, so the slots due are the same for all
    std::vector<uint32_t> due;
    uint32_t slot_write = 0;
    for (size_t q = 0; q < L->small.size(); ++q)
        slot_write = deco::advance_iteration_external(L->layers[L->small[q]], q == 0 ? &due : nullptr);
    bool aggregate = true;
    size_t at = 0;
    do {
        deco::SmallDue part;
        part.count = 0;
        while (at < due.size() && part.count < deco::SMALL_DUE_MAX) part.slot[part.count++] = due[at++];
        if (deco::launch_small_server(L->small_dev, layers, L->n, aggregate, slot_write, part, neg_scale,
                                      s) != cudaSuccess)
            return DECO_ERR_CUDA;
        aggregate = false;
    } while (at < due.size());
    first->launches += 2;
    return DECO_OK;
}

// Server side of all layers of `big` on stream s (their messages are complete there), and the
// host bookkeeping of every context.
deco_status step_big_server(deco_layered *L, cudaStream_t s)
{
    const uint32_t layers = static_cast<uint32_t>(L->big.size());
    const deco_ctx *first = L->layers[L->big[0]];
    if (L->server_dirty) {
        uint64_t most = 1;
        L->any_dense = L->any_sparse = false;
        for (uint32_t q = 0; q < layers; ++q) {
            const deco_ctx *c = L->layers[L->big[q]];
            L->server_host[q].k = static_cast<uint32_t>(c->k);
            L->server_host[q].dense = deco::aggregate_prefers_dense(c) ? 1u : 0u;
            (L->server_host[q].dense ? L->any_dense : L->any_sparse) = true;
            most = std::max<uint64_t>(most, static_cast<uint64_t>(c->n) * c->k_cap);
        }
        // the host table is pageable: the copy has left it when the call returns
        if (cudaMemcpyAsync(L->server_dev, L->server_host.data(), sizeof(deco::ServerLayer) * layers,
                            cudaMemcpyHostToDevice, s) != cudaSuccess)
            return DECO_ERR_CUDA;
        const uint64_t want = (most + 1023) / 1024, cap = std::max<uint64_t>(1, 148ull * 64 / layers);
        L->apply_ctas = static_cast<uint32_t>(std::min(want, cap));
        L->server_dirty = false;
    }
    const float beta = first->lr_at_server ? first->lr : 1.0f;
    const float neg_scale = -(beta / static_cast<float>(first->n_total));
    // every layer shares t, tau and the ring size, so the slots due are the same for all
    std::vector<uint32_t> due;
    uint32_t slot_write = 0;
    for (uint32_t q = 0; q < layers; ++q)
        slot_write = deco::advance_iteration_external(L->layers[L->big[q]], q == 0 ? &due : nullptr);
    if (deco::launch_multi_aggregate(L->server_dev, L->big_tile_layer, L->big_tiles, L->n, slot_write,
                                     L->any_dense, L->any_sparse, s) != cudaSuccess)
        return DECO_ERR_CUDA;
    for (uint32_t slot_read : due)
        if (deco::launch_multi_apply(L->server_dev, layers, L->n, L->apply_ctas, slot_read, neg_scale, s) !=
            cudaSuccess)
            return DECO_ERR_CUDA;
    L->layers[L->big[0]]->launches += 1 + due.size();
    return DECO_OK;
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
    if (build_small_batch(L) != cudaSuccess) {
        cudaGetLastError();
        release(L);
        return DECO_ERR_OOM;
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
    // the batch of short layers first, then the others
    deco_status st = step_small_batch(L, grads, L->streams[0]);
    if (L->plan && st == DECO_OK) {
        // worker side of all of them in one sequence of launches, then their server side
        for (uint32_t l : L->big)
            if (L->layers[l]->phase != 0) return DECO_ERR_STATE;
        const deco_ctx *first = L->layers[L->big[0]];
        const float alpha = first->lr_at_server ? 1.0f : first->lr;
        cudaStream_t cs = L->streams[1 % LAYER_STREAMS];
        if (deco::multi_compress(L->plan, grads, alpha, cs) != cudaSuccess) return DECO_ERR_CUDA;
        st = step_big_server(L, cs);
    } else {
        for (size_t q = 0; q < L->big.size() && st == DECO_OK; ++q) {
            const uint32_t l = L->big[q];
            st = deco_step(L->layers[l], static_cast<const char *>(grads) + L->offsets[l] * esz,
                           L->streams[(q + 1) % LAYER_STREAMS]);
        }
    }
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
    L->small_dirty = true;
    deco::multi_plan_mark_dirty(L->plan);
    L->server_dirty = true;
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
