// Internal declarations shared by the host API and the kernel translation units of libdeco.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "deco.h"

namespace deco {

// Geometry of one streaming tile.  A tile is TILE consecutive entries of one worker's
// vector, processed by one CTA of BLOCK threads; warp w owns the WARP_ELEMS consecutive
// entries [w*WARP_ELEMS, (w+1)*WARP_ELEMS) of the tile, so that every warp-level load
// instruction is one contiguous 512-byte request and entry order is (warp, round, lane,
// component).  Tiles are also the index blocks of the message directory.
constexpr int TILE = 8192;
constexpr int BLOCK = 256;
constexpr int WARPS = BLOCK / 32;
constexpr int WARP_ELEMS = TILE / WARPS;   // 1024

// Radix levels over the 31-bit magnitude key: 12 + 12 + 7 bits, most significant first.
constexpr int RADIX_BINS = 4096;
constexpr int RADIX_LEVELS = 3;

// Counters per worker: CTA arrivals at level A, level B, classification, sampling (resets
// itself) and chunk sums; the length of the emit work list.
constexpr int DONE_SLOTS = 6;

// Per-worker selection record (device).  One 64-byte line per worker.
struct SelectState {
    uint32_t prefix;        // key bits resolved so far (right-aligned)
    uint32_t k_rem;         // entries still to take among keys matching `prefix`
    uint32_t n_greater;     // entries known to be strictly above the threshold
    uint32_t threshold;     // final: key of the k-th largest magnitude
    uint32_t ties_take;     // final: how many entries equal to `threshold` are taken (by index)
    uint32_t exact;         // 1: this worker runs the multi-pass selection over e this step
    uint32_t spec_key;      // speculative lower bound used by the streaming pass (or DISABLED)
    uint32_t cert_key;      // staged entries with key >= cert_key are taken to be above the
                            // threshold (checked by count); the others form the band
    // what the streaming pass staged, updated with one 64-bit atomic per tile: low word =
    // candidates (key >= spec_key), high word = those of them inside the band (key < cert_key)
    unsigned long long staged_band;
    uint32_t exact_total;   // cumulative count of steps that took the multi-pass path
    uint32_t rel_shift;     // log2 width of a coarse bin of the band-key histogram (10..12)
    uint32_t thr_prev;      // thresholds of the two iterations before the last one, newest first
    uint32_t thr_prev2;     // (for a carried bound)
    uint32_t swing;         // decaying maximum of the threshold's change of step, in key units
    uint32_t hint_key;      // the last iteration's speculative bound: where the sample's fine histogram is centred
};
static_assert(sizeof(SelectState) == 64, "one line per worker");
static_assert(offsetof(SelectState, staged_band) % 8 == 0, "64-bit atomic target");

constexpr uint32_t SPEC_DISABLED = 0x80000000u;   // above every 31-bit key

// Tiles are grouped into chunks of one warp's width; message positions are first fixed per
// chunk (one CTA walks the chunks) and then per tile inside each chunk (one warp scan).
constexpr uint32_t CHUNK_TILES = 32;

// Keys of the per-iteration sample kept per worker (8192 groups of 4 entries).
constexpr uint32_t SAMPLE_KEYS = 131072;
constexpr uint32_t SAMPLE_BINS = 4096;                  // bins of the sample histogram
// Fine histogram of the sample around the previous bound: WINDOW_BINS coarse bins, each cut into
// 64, one counter each; one more word counts the sample keys above the window.
constexpr uint32_t WINDOW_BINS = 16;
constexpr uint32_t WINDOW_SUB_BITS = 6;
constexpr uint32_t WINDOW_WORDS = (WINDOW_BINS << WINDOW_SUB_BITS) + 1;

struct Slot {
    uint64_t step = 0;
    uint64_t positions = 0;     // pairs of a sparse aggregate; d for a dense one
    bool valid = false;
    bool dense = false;         // the slot holds the plain vector S[d] instead of pairs
};

}  // namespace deco

struct deco_ctx {
    // problem
    uint64_t d = 0;
    uint32_t n = 0;
    // worker-sharded context: n local workers with global ids worker_base .. worker_base+n-1
    // of n_total; message buffer, directory, cache and update cover all n_total
    uint32_t n_total = 0, worker_base = 0;
    double delta = 0, delta_max = 0;
    uint32_t tau = 0, tau_max = 0;
    float lr = 0;
    int grad_dtype = DECO_F32;
    int lr_at_server = 0;
    int select_mode = DECO_SELECT_AUTO;
    int compressor = DECO_COMPRESSOR_TOPK;
    uint64_t seed = 0;                  // Random-k: key of the priority stream
    int device = 0;
    // entries between consecutive gradient rows: d, or the full vector length when the context
    // works on one layer of a longer vector (then the rows need not be 16-byte aligned)
    uint64_t g_stride = 0;
    // derived
    uint64_t k = 0, k_cap = 0;
    uint64_t e_stride = 0;      // floats per worker row of e (multiple of TILE)
    uint32_t ntiles = 0;
    uint32_t ring = 0;          // tau_max + 1 slots
    uint64_t stage_cap = 0;     // staged candidates per worker
    // device memory
    float *e = nullptr;
    float *params = nullptr;
    bool own_params = false;
    deco_pair *msg = nullptr;           // [n][k_cap] (not allocated with the exchange layout)
    // Exchange layout (context created with n_total): one buffer of n_total rows, row w = the k
    // pairs of global worker w's message followed by its tile directory (ntiles + 1 words),
    // padded to an even number of words, so that what the ranks of a job all-gather is one
    // contiguous range that holds k, not k_cap, pairs per worker.
    bool packed = false;
    uint32_t *xchg = nullptr;           // [n_total][xrow_cap] words
    uint64_t xrow_cap = 0;              // words of a row at k = k_cap
    // where the messages and their directory lie for the k of the current iteration
    deco_pair *msg_rows = nullptr;      // row of global worker 0
    uint64_t msg_stride = 0;            // pairs between rows
    uint32_t *dir_rows = nullptr;
    uint64_t dir_stride = 0;            // words between rows
    deco_pair *slots = nullptr;         // [ring][slot_pairs]
    uint64_t slot_pairs = 0;            // pairs per cache slot: n_total * k_cap, or room for a dense vector
    bool dense_capable = false;         // a slot can hold S as a plain fp32 vector of e_stride entries
    deco_pair *stage = nullptr;         // [n][stage_cap] candidates, tile by tile in index order
    deco_pair *band = nullptr;          // [n][stage_cap] the candidates below cert_key once more, unordered
    uint2 *work = nullptr;              // [n][work_cap] emit work list: (tile, slice)
    uint64_t work_cap = 0;
    uint32_t *hist = nullptr;           // [n][2 routes][RADIX_LEVELS][RADIX_BINS]
    uint32_t *done = nullptr;           // [n][DONE_SLOTS] CTA arrival counters
    uint32_t *sample_keys = nullptr;    // [n][SAMPLE_KEYS] keys of the per-iteration sample
    uint32_t *sample_hist = nullptr;    // [n][SAMPLE_BINS] sample keys per bin of their top bits (self-clearing)
    uint32_t *sample_win = nullptr;     // [n][WINDOW_WORDS] fine histogram around the previous bound (self-clearing)
    uint32_t fallback_grid = 0;         // CTAs of the cooperative fallback launch
    uint32_t chain_grid = 0;            // most CTAs the cooperative selection launch may have
    deco::SelectState *sel = nullptr;   // [n]
    uint32_t *tile_gt = nullptr;        // [n][ntiles]  entries above the threshold per tile
    uint32_t *tile_eq = nullptr;        // [n][ntiles]  entries equal to it per tile
    uint32_t *tile_take = nullptr;      // [n][ntiles]  ties taken per tile
    uint32_t *tile_start = nullptr;     // [n][ntiles + 1] message position of each tile (not with the exchange layout)
    uint32_t *tile_off = nullptr;       // [n][ntiles]  staging offset of each tile's candidates
    uint32_t *tile_cnt = nullptr;       // [n][ntiles]  staged candidates per tile
    uint32_t *tile_rej = nullptr;       // [n][ntiles]  staged candidates below the threshold
    uint32_t nchunks = 0;               // ceil(ntiles / CHUNK_TILES)
    uint32_t *chunk_cnt = nullptr;      // [n][nchunks] staged candidates per chunk
    uint32_t *chunk_rej = nullptr;      // [n][nchunks] rejected candidates per chunk
    uint32_t *chunk_eq = nullptr;       // [n][nchunks] ties per chunk
    uint32_t *chunk_eqb = nullptr;      // [n][nchunks] ties in earlier chunks
    uint32_t *chunk_start = nullptr;    // [n][nchunks + 1] message position of each chunk
    uint32_t *dev_status = nullptr;     // [4]: status, two detail words, fallback flag
    // deco_step_host: two device copies of host gradients, filled in turn on a stream of their
    // own, so that the copy for one call runs while the previous call's kernels do
    void *grads_staging[2] = {nullptr, nullptr};
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr};      // the buffer holds the call's gradients
    cudaEvent_t ev_consumed[2] = {nullptr, nullptr};    // the step that read the buffer is through
    uint64_t host_calls = 0;
    uint64_t device_bytes = 0;
    // host bookkeeping
    uint64_t t = 0;
    int phase = 0;                      // 0: expect compress, 1: aggregate, 2: apply
    std::vector<deco::Slot> slot_info;
    uint64_t launches = 0;
    uint64_t k_of_msg = 0;              // k used by the last compress
    // internal stream of deco_step: the stale update runs next to the streaming pass
    cudaStream_t side_stream = nullptr;      // stale update next to the worker side
    cudaStream_t agg_stream = nullptr;       // aggregation left running past the end of deco_step
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // deco_step leaves the aggregation of its iteration running on agg_stream: ev_emit marks
    // the messages complete, ev_agg the aggregation done; agg_pending says that a later launch
    // which rewrites the messages or reads the cache has to wait for ev_agg first
    cudaEvent_t ev_emit = nullptr, ev_agg = nullptr;
    bool agg_pending = false;
    // deco_step does not launch the aggregation of its iteration at once: the slot is booked
    // and the launch waits for the end of the next streaming pass (ev_pass), so that it runs
    // beside the selection kernels, which leave most of the device idle, and not beside the
    // pass, which does not.  Whatever needs the aggregate or rewrites the messages earlier
    // launches it first (launch_deferred_aggregate).
    cudaEvent_t ev_pass = nullptr;
    bool agg_deferred = false;
    uint32_t agg_slot = 0;              // ring slot the deferred aggregation fills
    bool agg_dense = false;             // ... as a plain vector
    // optional event timing: 8 events per recorded iteration
    bool timing = false;
    std::vector<cudaEvent_t> events;
    size_t timed_iters = 0;
};

namespace deco {

// --- kernel launchers (deco_compress.cu) -------------------------------------------------
cudaError_t query_fallback_grid(deco_ctx *c);
cudaError_t launch_begin_step(deco_ctx *c, const void *grads, cudaStream_t s);
cudaError_t launch_accumulate(deco_ctx *c, const void *grads, cudaStream_t s);
cudaError_t launch_selection(deco_ctx *c, cudaStream_t s);
// streaming route with the staged-pair chain as a row of ordinary launches (not the multi-pass
// route, not the single cooperative launch of short vectors)
bool selection_is_separate_launches(const deco_ctx *c);

// deco_init with the distance between gradient rows given (0: d)
deco_status init_context(deco_ctx **out, uint64_t d, uint32_t n, double delta, uint32_t tau, float lr,
                         const deco_options *opt, uint64_t g_stride);

// Words of an exchange row at k pairs per message.
inline uint64_t exchange_row_words(const deco_ctx *c, uint64_t k)
{
    return (2 * k + c->ntiles + 1 + 1) & ~1ull;
}

// Point msg_rows / dir_rows at the layout for messages of k pairs.
inline void set_message_layout(deco_ctx *c, uint64_t k)
{
    if (c->packed) {
        const uint64_t rw = exchange_row_words(c, k);
        c->msg_rows = reinterpret_cast<deco_pair *>(c->xchg);
        c->msg_stride = rw / 2;
        c->dir_rows = c->xchg + 2 * k;
        c->dir_stride = rw;
    } else {
        c->msg_rows = c->msg;
        c->msg_stride = c->k_cap;
        c->dir_rows = c->tile_start;
        c->dir_stride = static_cast<uint64_t>(c->ntiles) + 1;
    }
}

// Launch the aggregation that deco_step booked but has not launched yet, if there is one, on
// the internal stream behind the messages it reads (deco_api.cu).
cudaError_t launch_deferred_aggregate(deco_ctx *c);

// Order stream s after the aggregation that deco_step left to the internal stream.
inline cudaError_t wait_for_aggregate(deco_ctx *c, cudaStream_t s)
{
    if (c->agg_deferred) {
        const cudaError_t err = launch_deferred_aggregate(c);
        if (err != cudaSuccess) return err;
    }
    if (!c->agg_pending) return cudaSuccess;
    c->agg_pending = false;
    return cudaStreamWaitEvent(s, c->ev_agg, 0);
}
// --- worker side of many contexts in a fixed number of launches (deco_compress.cu) ----------
// All contexts have n workers, Top-k on the streaming route, and read their gradients from one
// buffer of rows of g_stride entries, context l at entry g_off[l] of every row.
struct MultiPlan;
MultiPlan *multi_plan_create(const std::vector<deco_ctx *> &layers, const std::vector<uint64_t> &g_off,
                             uint32_t n, int grad_dtype);
void multi_plan_destroy(MultiPlan *mp);
void multi_plan_mark_dirty(MultiPlan *mp);       // some context's k changed
// begin_step .. fallback of every context on stream s; the contexts' host state is untouched
cudaError_t multi_compress(MultiPlan *mp, const void *grads, float alpha, cudaStream_t s);
// host state of c after its worker side was run by multi_compress: ready for deco_aggregate_stale
deco_status mark_compressed_external(deco_ctx *c);

// --- server side of many contexts in a fixed number of launches (deco_server.cu) ------------
struct ServerLayer {
    const deco_pair *msg;    // [n][k_cap]
    uint64_t k_cap;
    const uint32_t *tile_start;
    deco_pair *slots;        // [ring][n * k_cap]
    float *params;
    uint32_t *status;
    uint32_t *slot_pos;      // [ring] positions held by each cache slot (written on the device)
    uint64_t d;
    uint32_t ntiles, first_tile;
    uint32_t k;              // entries kept per worker at the current delta
    uint32_t dense;          // aggregate with the CTA-wide accumulator (many entries per tile)
};
bool aggregate_prefers_dense(const deco_ctx *c);
// all layers' messages into cache slot slot_write of each (tiles numbered across the layers)
cudaError_t launch_multi_aggregate(const ServerLayer *table, const uint32_t *tile_layer, uint32_t total_tiles,
                                   uint32_t n, uint32_t slot_write, bool any_dense, bool any_sparse,
                                   cudaStream_t s);
// cache slot slot_read of every layer onto its parameters
cudaError_t launch_multi_apply(const ServerLayer *table, uint32_t layers, uint32_t n, uint32_t ctas_per_layer,
                               uint32_t slot_read, float neg_scale, cudaStream_t s);

// --- batch of short layers (per-layer Top-k): deco_small.cu, deco_server.cu ---------------
// One entry per layer of at most TILE entries; the table lives in device memory.  All pointers
// are the buffers of that layer's own context, in their usual layouts.
struct SmallLayer {
    float *e;                // [n][e_stride]
    uint64_t e_stride;
    uint64_t g_off;          // entries from the start of a gradient row to the layer
    deco_pair *msg;          // [n][k_cap]
    uint64_t k_cap;
    deco_pair *slots;        // [ring][n * k_cap]
    uint32_t *tile_start;    // [n][2]
    SelectState *sel;        // [n]
    float *params;           // the layer's slice of the parameter vector
    uint32_t *status;        // the context's device status words
    uint32_t *slot_pos;      // [ring] positions held by each cache slot (written on the device)
    uint32_t d;              // entries of the layer
    uint32_t k;              // entries kept per worker at the current delta
};

constexpr int SMALL_DUE_MAX = 16;        // cache slots one server launch can apply
struct SmallDue {
    uint32_t count;
    uint32_t slot[SMALL_DUE_MAX];        // slot numbers, oldest aggregate first
};

// worker side of every listed layer for all n workers: one CTA per (layer, worker)
cudaError_t launch_small_workers(const SmallLayer *table, uint32_t layers, uint32_t n, const void *grads,
                                 uint64_t g_stride, int grad_dtype, float alpha, cudaStream_t s);
// server side of every listed layer: aggregate the n messages into cache slot `slot_write`
// (unless aggregate is false), then apply the listed slots, oldest first; one CTA per layer
cudaError_t launch_small_server(const SmallLayer *table, uint32_t layers, uint32_t n, bool aggregate,
                                uint32_t slot_write, const SmallDue &due, float neg_scale, cudaStream_t s);

// Host bookkeeping of one whole iteration of c whose device work is done by the batch kernels:
// the cache slot of iteration t becomes valid, the slots due at t are appended to `due` (slot
// numbers, oldest first) and marked applied, t advances.  Returns the slot written.
uint32_t advance_iteration_external(deco_ctx *c, std::vector<uint32_t> *due);

// --- kernel launchers (deco_server.cu) ---------------------------------------------------
cudaError_t launch_aggregate(deco_ctx *c, deco_pair *slot, cudaStream_t s);
// the same with the aggregate kept as a plain vector of ntiles * TILE entries (dense messages)
cudaError_t launch_aggregate_dense(deco_ctx *c, float *slot, cudaStream_t s);
cudaError_t launch_apply_dense(deco_ctx *c, const float *slot, float neg_scale, cudaStream_t s);
// dense when the messages of an iteration hold at least d / 8 entries in all
inline bool aggregate_as_vector(const deco_ctx *c, uint64_t k)
{
    return c->dense_capable && static_cast<uint64_t>(c->n_total) * k * 8 >= c->d;
}
cudaError_t launch_apply(deco_ctx *c, const deco_pair *slot, uint64_t positions, float neg_scale,
                         cudaStream_t s);

}  // namespace deco
