// Host side of libdeco: context, memory, iteration state machine, cache (ring) bookkeeping.
#include <cstdio>
#include <cstring>
#include <new>

#include "deco_internal.h"

using namespace deco;

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

template <typename T>
deco_status dev_alloc(deco_ctx *c, T **p, uint64_t count)
{
    const uint64_t bytes = (count ? count : 1) * sizeof(T);
    void *q = nullptr;
    cudaError_t err = cudaMalloc(&q, bytes);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return err == cudaErrorMemoryAllocation ? DECO_ERR_OOM : DECO_ERR_CUDA;
    }
    *p = static_cast<T *>(q);
    c->device_bytes += bytes;
    return DECO_OK;
}

void free_all(deco_ctx *c)
{
    cudaFree(c->e);
    if (c->own_params) cudaFree(c->params);
    cudaFree(c->msg);
    cudaFree(c->xchg);
    cudaFree(c->slots);
    cudaFree(c->stage);
    cudaFree(c->band);
    cudaFree(c->work);
    cudaFree(c->hist);
    cudaFree(c->sel);
    cudaFree(c->tile_gt);
    cudaFree(c->tile_eq);
    cudaFree(c->tile_take);
    cudaFree(c->tile_start);
    cudaFree(c->tile_off);
    cudaFree(c->tile_cnt);
    cudaFree(c->tile_rej);
    cudaFree(c->chunk_cnt);
    cudaFree(c->chunk_rej);
    cudaFree(c->chunk_eq);
    cudaFree(c->chunk_eqb);
    cudaFree(c->chunk_start);
    cudaFree(c->sample_keys);
    cudaFree(c->sample_hist);
    cudaFree(c->sample_win);
    cudaFree(c->done);
    cudaFree(c->dev_status);
    for (int b = 0; b < 2; ++b) {
        cudaFree(c->grads_staging[b]);
        if (c->ev_copied[b]) cudaEventDestroy(c->ev_copied[b]);
        if (c->ev_consumed[b]) cudaEventDestroy(c->ev_consumed[b]);
    }
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    for (cudaEvent_t ev : c->events) cudaEventDestroy(ev);
    c->events.clear();
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->ev_emit) cudaEventDestroy(c->ev_emit);
    if (c->ev_agg) cudaEventDestroy(c->ev_agg);
    if (c->ev_pass) cudaEventDestroy(c->ev_pass);
    if (c->side_stream) cudaStreamDestroy(c->side_stream);
    if (c->agg_stream) cudaStreamDestroy(c->agg_stream);
}

deco_status zero_state(deco_ctx *c, cudaStream_t s)
{
    cudaError_t err = cudaMemsetAsync(c->e, 0, sizeof(float) * c->n * c->e_stride, s);
    if (err == cudaSuccess && c->own_params)
        err = cudaMemsetAsync(c->params, 0, sizeof(float) * c->d, s);
    if (err == cudaSuccess) err = cudaMemsetAsync(c->sel, 0, sizeof(SelectState) * c->n, s);
    if (err == cudaSuccess) err = cudaMemsetAsync(c->dev_status, 0, sizeof(uint32_t) * 4, s);
    if (err == cudaSuccess)
        err = cudaMemsetAsync(c->done, 0, sizeof(uint32_t) * c->n * DONE_SLOTS, s);
    if (err == cudaSuccess)
        err = cudaMemsetAsync(c->sample_hist, 0, sizeof(uint32_t) * c->n * SAMPLE_BINS, s);
    if (err == cudaSuccess)
        err = cudaMemsetAsync(c->sample_win, 0, sizeof(uint32_t) * c->n * WINDOW_WORDS, s);
    if (err == cudaSuccess)
        err = c->packed ? cudaMemsetAsync(c->xchg, 0, sizeof(uint32_t) * c->n_total * c->xrow_cap, s)
                        : cudaMemsetAsync(c->tile_start, 0, sizeof(uint32_t) * c->n * (c->ntiles + 1), s);
    c->launches += 5;
    c->t = 0;
    c->phase = 0;
    for (auto &sl : c->slot_info) sl = Slot();
    return err == cudaSuccess ? DECO_OK : DECO_ERR_CUDA;
}

inline cudaStream_t as_stream(void *s) { return static_cast<cudaStream_t>(s); }

// Host-side wait for whatever deco_step left on the internal stream (for calls that read the
// cache or the device status from the host, or hand out pointers).
inline cudaError_t drain_internal(deco_ctx *c)
{
    if (c->agg_deferred) {
        const cudaError_t err = launch_deferred_aggregate(c);
        if (err != cudaSuccess) return err;
    }
    c->agg_pending = false;
    if (!c->side_stream) return cudaSuccess;
    const cudaError_t err = cudaStreamSynchronize(c->side_stream);
    return err != cudaSuccess ? err : cudaStreamSynchronize(c->agg_stream);
}

constexpr size_t MAX_TIMED_ITERS = 4096;

// Record event `which` (0..7) of the iteration being timed, if timing is on and there is room.
void mark(deco_ctx *c, int which, cudaStream_t s)
{
    if (!c->timing || c->timed_iters >= MAX_TIMED_ITERS) return;
    const size_t need = (c->timed_iters + 1) * 8;
    while (c->events.size() < need) {
        cudaEvent_t ev = nullptr;
        if (cudaEventCreate(&ev) != cudaSuccess) { c->timing = false; return; }
        c->events.push_back(ev);
    }
    cudaEventRecord(c->events[c->timed_iters * 8 + which], s);
}

}  // namespace

cudaError_t deco::launch_deferred_aggregate(deco_ctx *c)
{
    if (!c->agg_deferred) return cudaSuccess;
    c->agg_deferred = false;
    // ev_emit: the messages of that iteration are complete
    cudaError_t err = cudaStreamWaitEvent(c->agg_stream, c->ev_emit, 0);
    if (err != cudaSuccess) return err;
    deco_pair *slot = c->slots + static_cast<uint64_t>(c->agg_slot) * c->slot_pairs;
    mark(c, 3, c->agg_stream);
    err = c->agg_dense ? launch_aggregate_dense(c, reinterpret_cast<float *>(slot), c->agg_stream)
                       : launch_aggregate(c, slot, c->agg_stream);
    if (err != cudaSuccess) return err;
    mark(c, 4, c->agg_stream);
    err = cudaEventRecord(c->ev_agg, c->agg_stream);
    c->agg_pending = true;
    return err;
}

extern "C" const char *deco_status_string(deco_status s)
{
    switch (s) {
    case DECO_OK: return "ok";
    case DECO_ERR_INVALID_ARG: return "invalid argument";
    case DECO_ERR_OOM: return "out of memory";
    case DECO_ERR_CUDA: return "CUDA runtime error";
    case DECO_ERR_STATE: return "call out of order";
    case DECO_ERR_CAPACITY: return "beyond the capacity fixed at deco_init";
    case DECO_ERR_TIMEOUT: return "device-side wait ran out";
    case DECO_ERR_DEVICE_CHECK: return "a kernel self-check failed";
    }
    return "unknown status";
}

extern "C" deco_status deco_init(deco_ctx **out, uint64_t d, uint32_t n, double delta,
                                 uint32_t tau, float lr, const deco_options *opt)
{
    return deco::init_context(out, d, n, delta, tau, lr, opt, 0);
}

deco_status deco::init_context(deco_ctx **out, uint64_t d, uint32_t n, double delta, uint32_t tau,
                               float lr, const deco_options *opt, uint64_t g_stride)
{
    if (!out) return DECO_ERR_INVALID_ARG;
    if (g_stride != 0 && g_stride < d) return DECO_ERR_INVALID_ARG;
    deco_options o;
    std::memset(&o, 0, sizeof o);
    if (opt) o = *opt;
    for (uint32_t r : o.reserved)
        if (r != 0) return DECO_ERR_INVALID_ARG;
    if (d == 0 || d >= 0xFFFFFFFFull - TILE || n == 0 || n > 65535) return DECO_ERR_INVALID_ARG;
    if (o.n_total == 0 && o.worker_base != 0) return DECO_ERR_INVALID_ARG;
    if (o.n_total != 0 && (o.n_total > 65535 || static_cast<uint64_t>(o.worker_base) + n > o.n_total))
        return DECO_ERR_INVALID_ARG;
    if (!(delta > 0.0) || !(delta <= 1.0) || !(lr == lr)) return DECO_ERR_INVALID_ARG;
    if (o.grad_dtype != DECO_F32 && o.grad_dtype != DECO_BF16) return DECO_ERR_INVALID_ARG;
    if (o.select_mode != DECO_SELECT_AUTO && o.select_mode != DECO_SELECT_EXACT_PASSES)
        return DECO_ERR_INVALID_ARG;
    if (o.compressor != DECO_COMPRESSOR_TOPK && o.compressor != DECO_COMPRESSOR_RANDK)
        return DECO_ERR_INVALID_ARG;
    if (o.delta_max != 0.0 && (!(o.delta_max <= 1.0) || o.delta_max < delta))
        return DECO_ERR_INVALID_ARG;
    if (o.tau_max != 0 && o.tau_max < tau) return DECO_ERR_INVALID_ARG;
    if (o.tau_max > (1u << 20) || tau > (1u << 20)) return DECO_ERR_INVALID_ARG;
    if (o.params && (reinterpret_cast<uintptr_t>(o.params) & (g_stride ? 3u : 15u))) return DECO_ERR_INVALID_ARG;

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) {
        cudaGetLastError();
        return DECO_ERR_CUDA;
    }
    if (o.device < 0 || o.device >= ndev) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(o.device);
    if (!guard.ok) return DECO_ERR_CUDA;

    deco_ctx *c = new (std::nothrow) deco_ctx();
    if (!c) return DECO_ERR_OOM;
    c->d = d;
    c->g_stride = g_stride ? g_stride : d;
    c->n = n;
    c->n_total = o.n_total ? o.n_total : n;
    c->worker_base = o.worker_base;
    c->delta = delta;
    c->delta_max = o.delta_max != 0.0 ? o.delta_max : delta;
    c->tau = tau;
    c->tau_max = o.tau_max != 0 ? o.tau_max : tau;
    c->lr = lr;
    c->grad_dtype = o.grad_dtype;
    c->lr_at_server = o.lr_at_server;
    c->select_mode = o.select_mode;
    c->compressor = o.compressor;
    c->seed = (static_cast<uint64_t>(o.seed_hi) << 32) | o.seed_lo;
    c->device = o.device;
    c->k = deco_k_from_delta(delta, d);
    c->k_cap = deco_k_from_delta(c->delta_max, d);
    c->ntiles = static_cast<uint32_t>((d + TILE - 1) / TILE);
    c->e_stride = static_cast<uint64_t>(c->ntiles) * TILE;
    c->nchunks = (c->ntiles + CHUNK_TILES - 1) / CHUNK_TILES;
    c->ring = c->tau_max + 1;
    // staged candidates per worker: six times the message capacity plus slack, at most d
    c->stage_cap = 6 * c->k_cap + 65536;
    if (c->stage_cap > c->e_stride) c->stage_cap = c->e_stride;
    try {
        c->slot_info.resize(c->ring);
    } catch (...) {
        delete c;
        return DECO_ERR_OOM;
    }

    deco_status st = DECO_OK;
    auto need = [&](deco_status s) { if (st == DECO_OK) st = s; };
    need(dev_alloc(c, &c->e, static_cast<uint64_t>(n) * c->e_stride));
    if (o.params) {
        c->params = o.params;
    } else {
        need(dev_alloc(c, &c->params, d));
        c->own_params = (st == DECO_OK);
    }
    c->packed = o.n_total != 0;
    if (c->packed) {
        c->xrow_cap = exchange_row_words(c, c->k_cap);
        need(dev_alloc(c, &c->xchg, static_cast<uint64_t>(c->n_total) * c->xrow_cap));
    } else {
        need(dev_alloc(c, &c->msg, static_cast<uint64_t>(n) * c->k_cap));
    }
    // a cache slot holds the n_total * k_cap pairs of a merged aggregate; where the messages can
    // be dense enough for the plain vector S[e_stride] to be the better layout, it has room for
    // that too (a context that is one layer of a layered one keeps the pair layout only)
    c->slot_pairs = static_cast<uint64_t>(c->n_total) * c->k_cap;
    c->dense_capable = g_stride == 0 && c->slot_pairs * 8 >= d;
    if (c->dense_capable) {
        if (c->slot_pairs < c->e_stride / 2) c->slot_pairs = c->e_stride / 2;
        c->slot_pairs = (c->slot_pairs + 31) & ~31ull;  // vectors start on 256-byte boundaries
    }
    need(dev_alloc(c, &c->slots, static_cast<uint64_t>(c->ring) * c->slot_pairs));
    need(dev_alloc(c, &c->stage, static_cast<uint64_t>(n) * c->stage_cap));
    // slices of 256 staged entries, plus one partial slice for every tile that has any
    c->work_cap = c->stage_cap / 256 + (c->stage_cap / 17 < c->ntiles ? c->stage_cap / 17 : c->ntiles) + 32;
    need(dev_alloc(c, &c->work, static_cast<uint64_t>(n) * c->work_cap));
    need(dev_alloc(c, &c->hist, static_cast<uint64_t>(n) * 2 * RADIX_LEVELS * RADIX_BINS));
    need(dev_alloc(c, &c->done, static_cast<uint64_t>(n) * DONE_SLOTS));
    need(dev_alloc(c, &c->sample_keys, static_cast<uint64_t>(n) * SAMPLE_KEYS));
    need(dev_alloc(c, &c->sample_hist, static_cast<uint64_t>(n) * SAMPLE_BINS));
    need(dev_alloc(c, &c->sample_win, static_cast<uint64_t>(n) * WINDOW_WORDS));
    need(dev_alloc(c, &c->sel, n));
    need(dev_alloc(c, &c->tile_gt, static_cast<uint64_t>(n) * c->ntiles));
    need(dev_alloc(c, &c->tile_eq, static_cast<uint64_t>(n) * c->ntiles));
    need(dev_alloc(c, &c->tile_take, static_cast<uint64_t>(n) * c->ntiles));
    if (!c->packed) need(dev_alloc(c, &c->tile_start, static_cast<uint64_t>(n) * (c->ntiles + 1)));
    set_message_layout(c, c->k);
    need(dev_alloc(c, &c->tile_off, static_cast<uint64_t>(n) * c->ntiles));
    need(dev_alloc(c, &c->tile_cnt, static_cast<uint64_t>(n) * c->ntiles));
    need(dev_alloc(c, &c->tile_rej, static_cast<uint64_t>(n) * c->ntiles));
    need(dev_alloc(c, &c->chunk_cnt, static_cast<uint64_t>(n) * c->nchunks));
    need(dev_alloc(c, &c->chunk_rej, static_cast<uint64_t>(n) * c->nchunks));
    need(dev_alloc(c, &c->chunk_eq, static_cast<uint64_t>(n) * c->nchunks));
    need(dev_alloc(c, &c->chunk_eqb, static_cast<uint64_t>(n) * c->nchunks));
    need(dev_alloc(c, &c->chunk_start, static_cast<uint64_t>(n) * (c->nchunks + 1)));
    need(dev_alloc(c, &c->dev_status, 4));
    // the band list exists only where deco_set_policy can make the messages dense enough for it
    if (c->k_cap * 32 >= d) need(dev_alloc(c, &c->band, static_cast<uint64_t>(n) * c->stage_cap));
    if (st == DECO_OK && query_fallback_grid(c) != cudaSuccess) st = DECO_ERR_CUDA;
    if (st == DECO_OK &&
        (cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
         cudaStreamCreateWithFlags(&c->agg_stream, cudaStreamNonBlocking) != cudaSuccess ||
         cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&c->ev_emit, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&c->ev_agg, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&c->ev_pass, cudaEventDisableTiming) != cudaSuccess))
        st = DECO_ERR_CUDA;
    if (st == DECO_OK) st = zero_state(c, nullptr);
    if (st == DECO_OK && cudaStreamSynchronize(nullptr) != cudaSuccess) st = DECO_ERR_CUDA;
    if (st != DECO_OK) {
        free_all(c);
        delete c;
        cudaGetLastError();
        return st;
    }
    *out = c;
    return DECO_OK;
}

extern "C" void deco_destroy(deco_ctx *c)
{
    if (!c) return;
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    free_all(c);
    delete c;
}

extern "C" deco_status deco_reset(deco_ctx *c, void *stream)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    if (drain_internal(c) != cudaSuccess) return DECO_ERR_CUDA;
    return zero_state(c, as_stream(stream));
}

extern "C" deco_status deco_ef_compress(deco_ctx *c, const void *grads, void *stream)
{
    if (!c || !grads) return DECO_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(grads) & (c->g_stride != c->d ? 1u : 15u)) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    cudaStream_t s = as_stream(stream);
    c->k_of_msg = c->k;
    set_message_layout(c, c->k);
    cudaError_t err = launch_begin_step(c, grads, s);
    mark(c, 0, s);
    if (err == cudaSuccess) err = launch_accumulate(c, grads, s);
    mark(c, 1, s);
    if (err == cudaSuccess) err = launch_selection(c, s);
    mark(c, 2, s);
    if (err != cudaSuccess) return DECO_ERR_CUDA;
    c->phase = 1;
    return DECO_OK;
}

extern "C" deco_status deco_aggregate_stale(deco_ctx *c, void *stream)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    if (c->phase != 1) return DECO_ERR_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    const uint32_t si = static_cast<uint32_t>(c->t % c->ring);
    Slot &sl = c->slot_info[si];
    if (sl.valid) return DECO_ERR_STATE;    // cannot happen while tau <= tau_max
    deco_pair *slot = c->slots + static_cast<uint64_t>(si) * c->slot_pairs;
    const bool dense = aggregate_as_vector(c, c->k_of_msg);
    if (wait_for_aggregate(c, as_stream(stream)) != cudaSuccess) return DECO_ERR_CUDA;
    mark(c, 3, as_stream(stream));
    const cudaError_t err = dense ? launch_aggregate_dense(c, reinterpret_cast<float *>(slot), as_stream(stream))
                                  : launch_aggregate(c, slot, as_stream(stream));
    if (err != cudaSuccess) return DECO_ERR_CUDA;
    mark(c, 4, as_stream(stream));
    sl.step = c->t;
    sl.positions = dense ? c->d : static_cast<uint64_t>(c->n_total) * c->k_of_msg;
    sl.dense = dense;
    sl.valid = true;
    c->phase = 2;
    return DECO_OK;
}

namespace {

// Launch the update for every cached aggregate that is due at iteration t (step <= t - tau),
// oldest first, on stream s.
deco_status apply_due(deco_ctx *c, cudaStream_t s)
{
    const float beta = c->lr_at_server ? c->lr : 1.0f;
    const float neg_scale = -(beta / static_cast<float>(c->n_total));
    if (c->t < c->tau) return DECO_OK;
    const uint64_t due = c->t - c->tau;
    // step ids still cached lie in (t - ring, t]
    const uint64_t lo = c->t + 1 >= c->ring ? c->t + 1 - c->ring : 0;
    for (uint64_t step = lo; step <= due; ++step) {
        Slot &sl = c->slot_info[step % c->ring];
        if (!sl.valid || sl.step != step) continue;
        const deco_pair *slot = c->slots + (step % c->ring) * c->slot_pairs;
        const cudaError_t err = sl.dense ? launch_apply_dense(c, reinterpret_cast<const float *>(slot), neg_scale, s)
                                         : launch_apply(c, slot, sl.positions, neg_scale, s);
        if (err != cudaSuccess) return DECO_ERR_CUDA;
        sl.valid = false;
    }
    return DECO_OK;
}

void finish_iteration(deco_ctx *c)
{
    if (c->timing && c->timed_iters < MAX_TIMED_ITERS) c->timed_iters += 1;
    c->t += 1;
    c->phase = 0;
}

}  // namespace

deco_status deco::mark_compressed_external(deco_ctx *c)
{
    if (c->phase != 0) return DECO_ERR_STATE;
    c->k_of_msg = c->k;
    c->phase = 1;
    return DECO_OK;
}

uint32_t deco::advance_iteration_external(deco_ctx *c, std::vector<uint32_t> *due)
{
    const uint32_t si = static_cast<uint32_t>(c->t % c->ring);
    c->k_of_msg = c->k;
    Slot &now = c->slot_info[si];
    now.step = c->t;
    now.positions = static_cast<uint64_t>(c->n_total) * c->k;
    now.dense = false;
    now.valid = true;
    if (c->t >= c->tau) {
        const uint64_t last = c->t - c->tau;
        const uint64_t lo = c->t + 1 >= c->ring ? c->t + 1 - c->ring : 0;
        for (uint64_t step = lo; step <= last; ++step) {
            Slot &sl = c->slot_info[step % c->ring];
            if (!sl.valid || sl.step != step) continue;
            if (due) due->push_back(static_cast<uint32_t>(step % c->ring));
            sl.valid = false;
        }
    }
    c->t += 1;
    c->phase = 0;
    return si;
}

extern "C" deco_status deco_apply_update(deco_ctx *c, void *stream)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    if (c->phase != 2) return DECO_ERR_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    if (wait_for_aggregate(c, as_stream(stream)) != cudaSuccess) return DECO_ERR_CUDA;
    mark(c, 5, as_stream(stream));
    const deco_status st = apply_due(c, as_stream(stream));
    if (st != DECO_OK) return st;
    mark(c, 6, as_stream(stream));
    finish_iteration(c);
    return DECO_OK;
}

extern "C" deco_status deco_set_kernel_timing(deco_ctx *c, int32_t enabled)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    c->timing = enabled != 0;
    c->timed_iters = 0;
    return DECO_OK;
}

extern "C" deco_status deco_get_kernel_timing(deco_ctx *c, void *stream, double *ms_sum,
                                              uint64_t *iterations)
{
    if (!c || !ms_sum || !iterations) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return DECO_ERR_CUDA;
    if (drain_internal(c) != cudaSuccess) return DECO_ERR_CUDA;
    static const int pairs[4][2] = {{0, 1}, {1, 2}, {3, 4}, {5, 6}};
    for (int p = 0; p < 4; ++p) ms_sum[p] = 0.0;
    for (size_t it = 0; it < c->timed_iters; ++it)
        for (int p = 0; p < 4; ++p) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, c->events[it * 8 + pairs[p][0]],
                                     c->events[it * 8 + pairs[p][1]]) != cudaSuccess)
                return DECO_ERR_CUDA;
            ms_sum[p] += ms;
        }
    *iterations = c->timed_iters;
    c->timed_iters = 0;
    return DECO_OK;
}

extern "C" deco_status deco_step(deco_ctx *c, const void *grads, void *stream)
{
    if (!c || !grads) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    if (c->n_total != c->n) return DECO_ERR_STATE;      // the exchange sits between the parts
    if (c->tau == 0 || !c->side_stream) {
        // the update of this iteration needs this iteration's aggregate: strictly in order
        deco_status st = deco_ef_compress(c, grads, stream);
        if (st == DECO_OK) st = deco_aggregate_stale(c, stream);
        if (st == DECO_OK) st = deco_apply_update(c, stream);
        return st;
    }
    if (reinterpret_cast<uintptr_t>(grads) & (c->g_stride != c->d ? 1u : 15u)) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    cudaStream_t s = as_stream(stream);
    // Where the server side of an iteration runs.  The streaming pass keeps the whole register
    // file busy, and a kernel beside it only displaces its CTAs; the selection that follows it
    // is a chain of short launches.  When that chain is separate launches, the server side
    // goes behind the pass: the aggregation of the previous iteration's messages (booked then,
    // launched now; this iteration's emit, which rewrites the messages, waits for it) and the
    // update with the aggregates that are due (cached in earlier iterations; it touches neither
    // e nor the messages).  When the chain is one cooperative launch (short vectors), which
    // would wait for every other kernel to leave the device, the update is forked off at the
    // start and the aggregation is launched right behind the emit, next to the following pass.
    // Either way the update is joined back into the caller's stream inside this call: e, the
    // messages and the parameters are complete, in stream order, when the caller's stream
    // passes the call.
    const bool behind_pass = selection_is_separate_launches(c);
    c->k_of_msg = c->k;
    set_message_layout(c, c->k);
    deco_status st = DECO_OK;
    if (!behind_pass) {
        if (cudaEventRecord(c->ev_fork, s) != cudaSuccess) return DECO_ERR_CUDA;
        if (cudaStreamWaitEvent(c->side_stream, c->ev_fork, 0) != cudaSuccess) return DECO_ERR_CUDA;
        // the only aggregation that can still be outstanding is that of iteration t - 1,
        // which is due now only if tau = 1
        if (c->tau <= 1) {
            if (launch_deferred_aggregate(c) != cudaSuccess) return DECO_ERR_CUDA;
            if (c->agg_pending && cudaStreamWaitEvent(c->side_stream, c->ev_agg, 0) != cudaSuccess)
                return DECO_ERR_CUDA;
        }
        mark(c, 5, c->side_stream);
        st = apply_due(c, c->side_stream);
        mark(c, 6, c->side_stream);
        if (cudaEventRecord(c->ev_join, c->side_stream) != cudaSuccess) return DECO_ERR_CUDA;
        if (st != DECO_OK) return st;
    }
    cudaError_t err = launch_begin_step(c, grads, s);
    mark(c, 0, s);
    if (err == cudaSuccess) err = launch_accumulate(c, grads, s);
    mark(c, 1, s);
    if (err == cudaSuccess) err = cudaEventRecord(c->ev_pass, s);
    if (err != cudaSuccess) return DECO_ERR_CUDA;
    if (c->agg_deferred) {
        if (cudaStreamWaitEvent(c->agg_stream, c->ev_pass, 0) != cudaSuccess) return DECO_ERR_CUDA;
        if (launch_deferred_aggregate(c) != cudaSuccess) return DECO_ERR_CUDA;
    } else if (behind_pass) {
        mark(c, 3, c->agg_stream);          // nothing to aggregate: an empty interval
        mark(c, 4, c->agg_stream);
    }
    if (behind_pass) {
        if (cudaStreamWaitEvent(c->side_stream, c->ev_pass, 0) != cudaSuccess) return DECO_ERR_CUDA;
        if (c->tau <= 1 && c->agg_pending && cudaStreamWaitEvent(c->side_stream, c->ev_agg, 0) != cudaSuccess)
            return DECO_ERR_CUDA;
        mark(c, 5, c->side_stream);
        st = apply_due(c, c->side_stream);
        mark(c, 6, c->side_stream);
        if (cudaEventRecord(c->ev_join, c->side_stream) != cudaSuccess) return DECO_ERR_CUDA;
        if (st != DECO_OK) return st;
    }
    err = launch_selection(c, s);
    mark(c, 2, s);
    if (err != cudaSuccess) return DECO_ERR_CUDA;
    // This iteration's aggregate is not needed before iteration t + tau: the ring slot is booked
    // now, the launch goes onto a second internal stream and is not joined.  Every later launch
    // that rewrites the messages or reads the cache orders itself after it (wait_for_aggregate).
    const uint32_t si = static_cast<uint32_t>(c->t % c->ring);
    Slot &sl = c->slot_info[si];
    if (sl.valid) return DECO_ERR_STATE;    // cannot happen while tau <= tau_max
    const bool dense = aggregate_as_vector(c, c->k_of_msg);
    sl.step = c->t;
    sl.positions = dense ? c->d : static_cast<uint64_t>(c->n_total) * c->k_of_msg;
    sl.dense = dense;
    sl.valid = true;
    if (cudaEventRecord(c->ev_emit, s) != cudaSuccess) return DECO_ERR_CUDA;
    c->agg_deferred = true;
    c->agg_slot = si;
    c->agg_dense = dense;
    if (!behind_pass && launch_deferred_aggregate(c) != cudaSuccess) return DECO_ERR_CUDA;
    if (cudaStreamWaitEvent(s, c->ev_join, 0) != cudaSuccess) return DECO_ERR_CUDA;
    finish_iteration(c);
    return DECO_OK;
}

extern "C" deco_status deco_join(deco_ctx *c, void *stream)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    return wait_for_aggregate(c, as_stream(stream)) == cudaSuccess ? DECO_OK : DECO_ERR_CUDA;
}

extern "C" deco_status deco_step_host(deco_ctx *c, const void *grads_host, deco_pair *msg_out,
                                      float *params_out, void *stream)
{
    if (!c || !grads_host) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    cudaStream_t s = as_stream(stream);
    const uint64_t gbytes = static_cast<uint64_t>(c->n) * c->d * (c->grad_dtype == DECO_BF16 ? 2 : 4);
    const int b = static_cast<int>(c->host_calls & 1);
    if (!c->copy_stream && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess)
        return DECO_ERR_CUDA;
    if (!c->grads_staging[b]) {
        void *q = nullptr;
        cudaError_t err = cudaMalloc(&q, gbytes);
        if (err == cudaSuccess) err = cudaEventCreateWithFlags(&c->ev_copied[b], cudaEventDisableTiming);
        if (err == cudaSuccess) err = cudaEventCreateWithFlags(&c->ev_consumed[b], cudaEventDisableTiming);
        if (err != cudaSuccess) {
            cudaGetLastError();
            cudaFree(q);
            return err == cudaErrorMemoryAllocation ? DECO_ERR_OOM : DECO_ERR_CUDA;
        }
        c->grads_staging[b] = q;
        c->device_bytes += gbytes;
    } else if (cudaStreamWaitEvent(c->copy_stream, c->ev_consumed[b], 0) != cudaSuccess) {
        return DECO_ERR_CUDA;              // the step of two calls ago still reads this buffer
    }
    if (cudaMemcpyAsync(c->grads_staging[b], grads_host, gbytes, cudaMemcpyHostToDevice, c->copy_stream) !=
            cudaSuccess ||
        cudaEventRecord(c->ev_copied[b], c->copy_stream) != cudaSuccess ||
        cudaStreamWaitEvent(s, c->ev_copied[b], 0) != cudaSuccess)
        return DECO_ERR_CUDA;
    c->launches += 1;
    c->host_calls += 1;
    deco_status st = deco_step(c, c->grads_staging[b], stream);
    // (recorded also after a step that failed to enqueue: the buffer is free either way)
    if (cudaEventRecord(c->ev_consumed[b], s) != cudaSuccess) return DECO_ERR_CUDA;
    if (st != DECO_OK) return st;
    if (msg_out) {
        // rows of k pairs, packed: [n][k]
        if (cudaMemcpy2DAsync(msg_out, c->k_of_msg * sizeof(deco_pair),
                              c->msg_rows + static_cast<uint64_t>(c->worker_base) * c->msg_stride,
                              c->msg_stride * sizeof(deco_pair), c->k_of_msg * sizeof(deco_pair), c->n,
                              cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return DECO_ERR_CUDA;
        c->launches += 1;
    }
    if (params_out) {
        if (cudaMemcpyAsync(params_out, c->params, sizeof(float) * c->d, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return DECO_ERR_CUDA;
        c->launches += 1;
    }
    return DECO_OK;
}

extern "C" deco_status deco_set_policy(deco_ctx *c, double delta, uint32_t tau)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    if (!(delta > 0.0) || !(delta <= 1.0)) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    const uint64_t k = deco_k_from_delta(delta, c->d);
    if (tau > c->tau_max || k > c->k_cap) return DECO_ERR_CAPACITY;
    if (c->agg_deferred) {
        // the launch takes the length of the messages from the policy they were made under
        DeviceGuard guard(c->device);
        if (!guard.ok || launch_deferred_aggregate(c) != cudaSuccess) return DECO_ERR_CUDA;
    }
    c->delta = delta;
    c->tau = tau;
    c->k = k;
    return DECO_OK;
}

extern "C" deco_status deco_set_lr(deco_ctx *c, float lr)
{
    if (!c || !(lr == lr)) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    c->lr = lr;
    return DECO_OK;
}

extern "C" deco_status deco_get_k(const deco_ctx *c, uint64_t *k)
{
    if (!c || !k) return DECO_ERR_INVALID_ARG;
    *k = c->k;
    return DECO_OK;
}

extern "C" deco_status deco_get_buffers(deco_ctx *c, float **e, uint64_t *e_stride,
                                        deco_pair **msg, uint64_t *k_cap, float **params)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    if (e) *e = c->e;
    if (e_stride) *e_stride = c->e_stride;
    if (msg) *msg = c->msg_rows + static_cast<uint64_t>(c->worker_base) * c->msg_stride;   // the local rows
    if (k_cap) *k_cap = c->msg_stride;
    if (params) *params = c->params;
    return DECO_OK;
}

extern "C" deco_status deco_get_aggregate(deco_ctx *c, uint64_t step, const deco_pair **entries,
                                          uint64_t *positions)
{
    if (!c || !entries || !positions) return DECO_ERR_INVALID_ARG;
    const Slot &sl = c->slot_info[step % c->ring];
    if (!sl.valid || sl.step != step || sl.dense) return DECO_ERR_STATE;
    {
        DeviceGuard guard(c->device);
        if (!guard.ok || drain_internal(c) != cudaSuccess) return DECO_ERR_CUDA;
    }
    *entries = c->slots + (step % c->ring) * c->slot_pairs;
    *positions = sl.positions;
    return DECO_OK;
}

extern "C" deco_status deco_get_aggregate_vector(deco_ctx *c, uint64_t step, const float **values)
{
    if (!c || !values) return DECO_ERR_INVALID_ARG;
    const Slot &sl = c->slot_info[step % c->ring];
    if (!sl.valid || sl.step != step || !sl.dense) return DECO_ERR_STATE;
    {
        DeviceGuard guard(c->device);
        if (!guard.ok || drain_internal(c) != cudaSuccess) return DECO_ERR_CUDA;
    }
    *values = reinterpret_cast<const float *>(c->slots + (step % c->ring) * c->slot_pairs);
    return DECO_OK;
}

extern "C" deco_status deco_get_select_info(deco_ctx *c, void *stream, uint32_t *threshold_key,
                                            uint32_t *n_greater, uint32_t *exact_passes)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    std::vector<SelectState> h;
    try {
        h.resize(c->n);
    } catch (...) {
        return DECO_ERR_OOM;
    }
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return DECO_ERR_CUDA;
    if (cudaMemcpy(h.data(), c->sel, sizeof(SelectState) * c->n, cudaMemcpyDeviceToHost) != cudaSuccess)
        return DECO_ERR_CUDA;
    for (uint32_t i = 0; i < c->n; ++i) {
        if (threshold_key) threshold_key[i] = h[i].threshold;
        if (n_greater) n_greater[i] = h[i].n_greater;
        if (exact_passes) exact_passes[i] = h[i].exact;
    }
    return DECO_OK;
}

extern "C" deco_status deco_get_stats(deco_ctx *c, void *stream, deco_stats *out)
{
    if (!c || !out) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return DECO_ERR_CUDA;
    if (drain_internal(c) != cudaSuccess) return DECO_ERR_CUDA;
    uint32_t st[4] = {0, 0, 0, 0};
    if (cudaMemcpy(st, c->dev_status, sizeof st, cudaMemcpyDeviceToHost) != cudaSuccess)
        return DECO_ERR_CUDA;
    std::vector<SelectState> h;
    try {
        h.resize(c->n);
    } catch (...) {
        return DECO_ERR_OOM;
    }
    if (cudaMemcpy(h.data(), c->sel, sizeof(SelectState) * c->n, cudaMemcpyDeviceToHost) != cudaSuccess)
        return DECO_ERR_CUDA;
    std::memset(out, 0, sizeof *out);
    out->step = c->t;
    out->k = c->k;
    out->delta = c->delta;
    out->tau = c->tau;
    out->device_status = st[0];
    for (uint32_t i = 0; i < c->n; ++i) out->exact_pass_workers += h[i].exact_total;
    for (const Slot &sl : c->slot_info) out->cached_aggregates += sl.valid ? 1 : 0;
    out->device_bytes = c->device_bytes;
    if (st[0] != 0) {
        std::fprintf(stderr, "libdeco: device check %u (site 0x%x, detail %u)\n", st[0], st[1], st[2]);
        return DECO_ERR_DEVICE_CHECK;
    }
    return DECO_OK;
}

extern "C" deco_status deco_get_exchange(deco_ctx *c, uint32_t **rows, uint64_t *row_words, uint32_t *row0,
                                         uint32_t *rows_local, uint32_t *rows_total)
{
    if (!c) return DECO_ERR_INVALID_ARG;
    if (!c->packed) return DECO_ERR_STATE;
    if (rows) *rows = c->xchg;
    if (row_words) *row_words = exchange_row_words(c, c->phase == 0 ? c->k : c->k_of_msg);
    if (row0) *row0 = c->worker_base;
    if (rows_local) *rows_local = c->n;
    if (rows_total) *rows_total = c->n_total;
    return DECO_OK;
}

extern "C" uint64_t deco_launch_count(const deco_ctx *c) { return c ? c->launches : 0; }

// ------------------------------------------------------------------ checkpoint / resume
namespace {

struct StateHeader {
    uint64_t magic, version;
    uint64_t d, n, k_cap, ring, t, k;
    double delta;
    uint32_t tau, grad_dtype, lr_at_server, compressor;
    float lr;
    uint32_t sharding;          // n_total << 16 | worker_base (both below 65536)
    uint64_t seed;
};
constexpr uint64_t STATE_MAGIC = 0x4F434544534F4345ull;   // "ECOSDECO"

struct SlotRecord {
    uint64_t step, positions, valid;
};

// bytes a cached aggregate takes in the blob: its pairs, or the d values of a dense one
uint64_t slot_bytes(const Slot &sl)
{
    return sl.dense ? sizeof(float) * sl.positions : sizeof(deco_pair) * sl.positions;
}

uint64_t state_size(const deco_ctx *c)
{
    uint64_t bytes = sizeof(StateHeader) + sizeof(SlotRecord) * c->ring;
    bytes += sizeof(float) * c->n * c->d + sizeof(float) * c->d;
    for (const Slot &sl : c->slot_info)
        if (sl.valid) bytes += slot_bytes(sl);
    return bytes;
}

}  // namespace

extern "C" deco_status deco_state_bytes(const deco_ctx *c, uint64_t *bytes)
{
    if (!c || !bytes) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    *bytes = state_size(c);
    return DECO_OK;
}

extern "C" deco_status deco_export_state(deco_ctx *c, void *buf, uint64_t bytes, void *stream)
{
    if (!c || !buf) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    if (bytes < state_size(c)) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    if (drain_internal(c) != cudaSuccess) return DECO_ERR_CUDA;
    cudaStream_t s = as_stream(stream);
    char *out = static_cast<char *>(buf);
    StateHeader h;
    std::memset(&h, 0, sizeof h);
    h.magic = STATE_MAGIC;
    h.version = 1;
    h.d = c->d; h.n = c->n; h.k_cap = c->k_cap; h.ring = c->ring; h.t = c->t; h.k = c->k;
    h.delta = c->delta; h.tau = c->tau; h.grad_dtype = c->grad_dtype;
    h.lr_at_server = c->lr_at_server; h.lr = c->lr;
    h.compressor = c->compressor; h.seed = c->seed;
    h.sharding = (c->n_total << 16) | c->worker_base;
    std::memcpy(out, &h, sizeof h);
    out += sizeof h;
    for (const Slot &sl : c->slot_info) {
        SlotRecord r = {sl.step, sl.positions, sl.valid ? (sl.dense ? 2ull : 1ull) : 0ull};
        std::memcpy(out, &r, sizeof r);
        out += sizeof r;
    }
    // e without its padding, then the parameters, then the cached aggregates
    if (cudaMemcpy2DAsync(out, sizeof(float) * c->d, c->e, sizeof(float) * c->e_stride,
                          sizeof(float) * c->d, c->n, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return DECO_ERR_CUDA;
    out += sizeof(float) * c->n * c->d;
    if (cudaMemcpyAsync(out, c->params, sizeof(float) * c->d, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return DECO_ERR_CUDA;
    out += sizeof(float) * c->d;
    for (uint32_t q = 0; q < c->ring; ++q) {
        const Slot &sl = c->slot_info[q];
        if (!sl.valid) continue;
        if (cudaMemcpyAsync(out, c->slots + static_cast<uint64_t>(q) * c->slot_pairs, slot_bytes(sl),
                            cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return DECO_ERR_CUDA;
        out += slot_bytes(sl);
    }
    c->launches += 2 + c->ring;
    return cudaStreamSynchronize(s) == cudaSuccess ? DECO_OK : DECO_ERR_CUDA;
}

extern "C" deco_status deco_import_state(deco_ctx *c, const void *buf, uint64_t bytes, void *stream)
{
    if (!c || !buf || bytes < sizeof(StateHeader)) return DECO_ERR_INVALID_ARG;
    if (c->phase != 0) return DECO_ERR_STATE;
    const char *in = static_cast<const char *>(buf);
    StateHeader h;
    std::memcpy(&h, in, sizeof h);
    in += sizeof h;
    if (h.magic != STATE_MAGIC || h.version != 1 || h.d != c->d || h.n != c->n ||
        h.k_cap != c->k_cap || h.ring != c->ring || h.grad_dtype != static_cast<uint32_t>(c->grad_dtype) ||
        h.lr_at_server != static_cast<uint32_t>(c->lr_at_server) || h.tau > c->tau_max || h.k > c->k_cap ||
        h.compressor != static_cast<uint32_t>(c->compressor) || h.seed != c->seed ||
        h.sharding != ((c->n_total << 16) | c->worker_base))
        return DECO_ERR_INVALID_ARG;
    // a blob that was cut, edited or damaged: the policy must be one deco_set_policy accepts
    if (!(h.delta > 0.0) || !(h.delta <= 1.0) || h.k < 1 || h.k != deco_k_from_delta(h.delta, c->d) ||
        !(h.lr == h.lr))
        return DECO_ERR_INVALID_ARG;
    if (bytes < sizeof(StateHeader) + sizeof(SlotRecord) * c->ring) return DECO_ERR_INVALID_ARG;
    std::vector<Slot> slots(c->ring);
    uint64_t need = sizeof(StateHeader) + sizeof(SlotRecord) * c->ring +
                    sizeof(float) * c->n * c->d + sizeof(float) * c->d;
    for (uint32_t q = 0; q < c->ring; ++q) {
        SlotRecord r;
        std::memcpy(&r, in, sizeof r);
        in += sizeof r;
        // a cached aggregate was sent in one of the last `ring` iterations before t and holds
        // the same number of positions for every worker
        if (r.valid > 2) return DECO_ERR_INVALID_ARG;
        if (r.valid && (r.step % c->ring != q || r.step >= h.t || r.step + c->ring < h.t))
            return DECO_ERR_INVALID_ARG;
        if (r.valid == 1 && (r.positions > static_cast<uint64_t>(c->n_total) * c->k_cap ||
                             r.positions < c->n_total || r.positions % c->n_total != 0))
            return DECO_ERR_INVALID_ARG;
        if (r.valid == 2 && (!c->dense_capable || r.positions != c->d)) return DECO_ERR_INVALID_ARG;
        slots[q].step = r.step;
        slots[q].positions = r.positions;
        slots[q].valid = r.valid != 0;
        slots[q].dense = r.valid == 2;
        if (slots[q].valid) need += slot_bytes(slots[q]);
    }
    if (bytes < need) return DECO_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return DECO_ERR_CUDA;
    if (drain_internal(c) != cudaSuccess) return DECO_ERR_CUDA;
    cudaStream_t s = as_stream(stream);
    deco_status st = zero_state(c, s);                       // padding of e, status, counters
    if (st != DECO_OK) return st;
    if (cudaMemcpy2DAsync(c->e, sizeof(float) * c->e_stride, in, sizeof(float) * c->d,
                          sizeof(float) * c->d, c->n, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return DECO_ERR_CUDA;
    in += sizeof(float) * c->n * c->d;
    if (cudaMemcpyAsync(c->params, in, sizeof(float) * c->d, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return DECO_ERR_CUDA;
    in += sizeof(float) * c->d;
    for (uint32_t q = 0; q < c->ring; ++q) {
        if (!slots[q].valid) continue;
        if (cudaMemcpyAsync(c->slots + static_cast<uint64_t>(q) * c->slot_pairs, in, slot_bytes(slots[q]),
                            cudaMemcpyHostToDevice, s) != cudaSuccess)
            return DECO_ERR_CUDA;
        in += slot_bytes(slots[q]);
        // the padding of a dense vector (entries d .. e_stride) is never read
    }
    c->slot_info = slots;
    c->t = h.t;
    c->k = h.k;
    set_message_layout(c, c->k);
    c->delta = h.delta;
    c->tau = h.tau;
    c->lr = h.lr;
    c->launches += 2 + c->ring;
    return cudaStreamSynchronize(s) == cudaSuccess ? DECO_OK : DECO_ERR_CUDA;
}
