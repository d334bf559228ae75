/*
 * libdeco — the data-parallel hot path of DD-EF-SGD / DeCo-SGD on one NVIDIA B200 (sm_100a).
 *
 * For n workers simulated on one GPU the library runs, per training iteration t
 * (Algorithm 1 of the paper, "DD-EF-SGD"):
 *
 *   worker i :  a       = e_i + gamma * g_i
 *               Delta_i = C_delta(a)        Top-k: the k largest-|a| entries, as (index, value)
 *               e_i     = a - Delta_i
 *   server   :  S_t     = sum_i Delta_i     kept in a cache (ring) of stale aggregates
 *               x       = x - (1/n) * S_{t - tau}
 *
 * and, on the host, the DeCo decision (Algorithm 3) that picks (tau, delta) from the
 * measured bandwidth and latency, with the iteration-time model of Theorem 3.
 *
 * Conventions
 *   - Plain C ABI.  Pointers are marked HOST or DEVICE.  No allocation is visible to the
 *     caller except through deco_init / deco_destroy.
 *   - Every device operation is enqueued on the CUDA stream the caller passes
 *     (a cudaStream_t cast to void*; NULL = the default stream) and returns without
 *     waiting.  Argument and state errors are found on the host before anything is
 *     launched and leave the context unchanged.
 *   - Every function returns a deco_status; nothing throws, aborts or traps.  Anomalies seen
 *     by a kernel (an index out of range, a count that does not add up) are latched in a
 *     device status word and reported by deco_get_stats.
 *   - One context is used from one host thread at a time, on one stream at a time.
 *   - There is no CPU fallback: without a CUDA device deco_init fails with DECO_ERR_CUDA.
 *
 * Fixed readings where the paper is silent
 *   - "largest" compares |a| through the IEEE-754 bit pattern with the sign cleared
 *     (so +0 == -0, and NaN > Inf > finite, deterministically); equal magnitudes are
 *     taken in order of increasing index.
 *   - k = ceil(delta * d) clamped to [1, d] (delta*d within 1e-6 of an integer is that
 *     integer); Top-k is over the whole flat vector, not per layer.
 *   - iterations count from 0; update t applies S_{t-tau} iff t - tau >= 0.  If tau changes
 *     at run time the cache is drained exactly once, oldest first: update t applies every
 *     cached aggregate whose step is <= t - tau.
 *   - state is fp32; each arithmetic statement is one fused multiply-add (round to nearest
 *     even, no flush to zero); the n messages are summed in fp32 in worker order 0..n-1.
 */
#ifndef DECO_H_
#define DECO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct deco_ctx deco_ctx;            /* opaque, owned by the library */

typedef enum {
    DECO_OK = 0,
    DECO_ERR_INVALID_ARG = 1,   /* NULL pointer, d == 0, delta outside (0,1], misaligned buffer ... */
    DECO_ERR_OOM = 2,           /* device or host allocation failed */
    DECO_ERR_CUDA = 3,          /* a CUDA runtime call failed (no device, launch error ...) */
    DECO_ERR_STATE = 4,         /* calls out of order (compress -> aggregate -> apply) */
    DECO_ERR_CAPACITY = 5,      /* tau > tau_max, or k(delta) > k(delta_max) */
    DECO_ERR_TIMEOUT = 6,       /* reserved: a bounded device-side wait ran out */
    DECO_ERR_DEVICE_CHECK = 7   /* a kernel's self-check latched an anomaly */
} deco_status;

typedef enum { DECO_F32 = 0, DECO_BF16 = 1 } deco_dtype;

/* One element of a compressed update Delta (what a worker would send): 8 bytes. */
typedef struct { uint32_t idx; float val; } deco_pair;

/* idx value of an unused position inside a cached aggregate (see deco_get_aggregate). */
#define DECO_NO_INDEX 0xFFFFFFFFu

typedef enum {
    DECO_SELECT_AUTO = 0,       /* sampled threshold + one streaming pass; exact multi-pass
                                   selection only for the workers where the sample fails */
    DECO_SELECT_EXACT_PASSES = 1 /* always the multi-pass radix selection (no sampling) */
} deco_select_mode;

/*
 * The sparsifier C_delta.  Top-k is the paper's default; Random-k ("random k% of entries",
 * the appendix on other compressors) keeps k entries chosen uniformly at random, independently
 * per worker and iteration: entry j gets the priority  Philox4x32-10(key = seed,
 * counter = (j / 4, t_lo, worker, t_hi ^ 0x52414E44))[j % 4] >> 9  and the k largest
 * priorities are kept, equal ones by increasing index.  Error feedback, messages, aggregation
 * and update are the same for both.
 */
typedef enum { DECO_COMPRESSOR_TOPK = 0, DECO_COMPRESSOR_RANDK = 1 } deco_compressor;

/* Options of deco_init.  A zero-filled struct selects every default. */
typedef struct {
    int32_t  grad_dtype;     /* deco_dtype of the gradients handed to deco_ef_compress; default F32 */
    uint32_t tau_max;        /* largest staleness deco_set_policy may ask for; 0 -> the initial tau */
    double   delta_max;      /* largest ratio deco_set_policy may ask for; 0 -> the initial delta */
    int32_t  lr_at_server;   /* 0: paper form, a = e + gamma*g and update scale 1/n;
                                1: a = e + g and update scale gamma/n */
    float   *params;         /* DEVICE, [d] fp32, 16-byte aligned, caller-owned; NULL -> the library
                                allocates a zero-filled vector and frees it in deco_destroy */
    int32_t  device;         /* CUDA device ordinal */
    int32_t  select_mode;    /* deco_select_mode */
    int32_t  compressor;     /* deco_compressor; default Top-k */
    uint32_t seed_lo;        /* Random-k: 64-bit seed of the priority stream, low word */
    uint32_t seed_hi;        /*           high word */
    uint32_t n_total;        /* worker-sharded context: workers of the whole job (0: n, no exchange buffer) */
    uint32_t worker_base;    /* ... and the global id of this context's first worker */
    uint32_t reserved[3];    /* must be zero */
} deco_options;

typedef struct {
    uint64_t step;                 /* iterations completed (t of the next compress) */
    uint64_t k;                    /* entries kept per worker at the current delta */
    double   delta;
    uint32_t tau;
    uint32_t device_status;        /* 0, or a deco_status latched by a kernel */
    uint64_t exact_pass_workers;   /* worker-iterations that needed the multi-pass selection */
    uint64_t cached_aggregates;    /* aggregates sent but not yet applied */
    uint64_t device_bytes;         /* device memory held by the context */
} deco_stats;

/* ------------------------------------------------------------------ life cycle */

/*
 * Create the state of Algorithm 1 ("Initialize x_0, e_0^i = 0"): error terms e[n][d] = 0, an
 * empty cache of stale aggregates, iteration counter 0, and the inputs n, gamma (lr), delta,
 * tau.  d < 2^32 - 1, n >= 1, 0 < delta <= 1.  Allocates all device memory the context will
 * ever use (sized by delta_max and tau_max).  *out is set only on success.
 */
deco_status deco_init(deco_ctx **out, uint64_t d, uint32_t n, double delta, uint32_t tau,
                      float lr, const deco_options *opt /* HOST, may be NULL */);

/* Free the context and everything it owns (waits for the device first).  NULL is allowed. */
void deco_destroy(deco_ctx *ctx);

/* Back to the state right after deco_init (e = 0, cache empty, t = 0; library-owned
 * parameters are zeroed, caller-owned ones are left alone).  Enqueued on `stream`. */
deco_status deco_reset(deco_ctx *ctx, void *stream);

/* ------------------------------------------------------- the iteration (hot path) */

/*
 * Worker side of iteration t for all n workers (Algorithm 1: "Delta = C_delta(e + gamma g)",
 * "e = e + gamma g - Delta").
 *   grads  DEVICE, [n][d] row-major without padding, dtype = grad_dtype, read-only; the base
 *          must be 16-byte aligned.  Rows that are not 16-byte aligned (d*sizeof(g) % 16 != 0)
 *          are accepted and read with narrower loads.  May be reused once the stream has
 *          passed this call.
 * Afterwards (in stream order) the message buffer holds, per worker, exactly k pairs sorted
 * by increasing index, val being the selected entry of a verbatim, and e holds a with +0
 * at the selected positions.
 */
deco_status deco_ef_compress(deco_ctx *ctx, const void *grads, void *stream);

/*
 * Server side, arrival of iteration t's messages (Algorithm 1: the sum inside
 * "x = x - (1/n) sum_i Delta_{t-tau}^i", kept in the server's cache of stale updates):
 * S_t[j] = sum over workers, in worker order, of the values sent for index j, stored in cache
 * slot t mod (tau_max + 1): as (index, sum) pairs, or, when the n messages together hold at
 * least d / 8 entries, as the plain vector S_t[0 .. d) (see deco_get_aggregate_vector).  Must
 * follow deco_ef_compress of the same iteration.
 */
deco_status deco_aggregate_stale(deco_ctx *ctx, void *stream);

/*
 * Server update of iteration t (Algorithm 1: "x_{t+1} = x_t - (1/n) sum_i Delta_{t-tau}^i"):
 * x[j] = fma(-scale, S_s[j], x[j]) for every cached aggregate with s <= t - tau, oldest
 * first (normally exactly one; none while t < tau), scale = 1/n (or gamma/n with
 * lr_at_server).  Then t advances.  Must follow deco_aggregate_stale.
 */
deco_status deco_apply_update(deco_ctx *ctx, void *stream);

/*
 * The three calls above for callers that do not interleave other work.  With tau >= 1 the
 * server side runs on internal streams:
 *   - the update of the aggregates that are due (it depends on neither e nor the messages) is
 *     forked from `stream` inside the call and joined back at its end, so e, the messages and
 *     the parameters are complete, in stream order, when `stream` passes the call;
 *   - the aggregation S_t of this iteration's messages, which Algorithm 1 needs only tau
 *     iterations later, is left to the internal stream: it runs either right behind this call
 *     or behind the streaming pass of the next one (the library picks by the size of the
 *     problem).  It reads the messages and writes a cache slot only the library sees; every
 *     later library call orders itself after it (calls without a stream argument wait on the
 *     host), and deco_join does so explicitly.  The messages must not be overwritten by the
 *     caller before deco_join or the next library call on this context.
 * With tau = 0 the three steps run strictly in order on `stream`.  Results are bit-identical
 * to the three calls in every case.
 */
deco_status deco_step(deco_ctx *ctx, const void *grads /* DEVICE */, void *stream);

/* Launch the aggregation a previous deco_step left to the internal stream, if it has not been
 * launched yet, and make `stream` wait for it (no-op if there is none).  After it, all device work of the library is ordered before
 * whatever is enqueued on `stream` next. */
deco_status deco_join(deco_ctx *ctx, void *stream);

/*
 * One iteration with HOST buffers: copies grads_host ([n][d], grad_dtype) to the device,
 * runs deco_step, and copies back what a deployment would move: the n messages
 * (msg_host_out, [n][k] pairs, may be NULL) and the parameters (params_host_out, [d] fp32,
 * may be NULL).  Use pinned host memory.  The copy of grads_host runs on a stream of the
 * library's own into one of two device buffers, so that it overlaps the kernels of the previous
 * call: grads_host must hold the gradients when the call is made (the copy does not wait for
 * earlier work on `stream`) and must stay unchanged until `stream` has passed the call.  The
 * step and the copies back are ordered on `stream`; synchronise it before reading the outputs.
 */
deco_status deco_step_host(deco_ctx *ctx, const void *grads_host, deco_pair *msg_host_out,
                           float *params_host_out, void *stream);

/* ------------------------------------------------------------- policy (Algorithms 2, 3) */

/*
 * Algorithm 2: "Broadcast new tau and delta".  Takes effect from the next deco_ef_compress;
 * may only be called between iterations.  tau > tau_max or k(delta) > k(delta_max) gives
 * DECO_ERR_CAPACITY and changes nothing.
 */
deco_status deco_set_policy(deco_ctx *ctx, double delta, uint32_t tau);

/* New stepsize gamma from the next iteration on. */
deco_status deco_set_lr(deco_ctx *ctx, float lr);

/*
 * Algorithm 3 (DeCo), pure host arithmetic in double: walk tau from
 * ceil((b + V_g/a_bar)/T_comp) down to ceil(b/T_comp), delta = delta*(tau) =
 * min{(tau T_comp - b) a_bar / V_g, T_comp a_bar / V_g, 1}, keep the pair with the smallest
 * phi = (1-delta)/(delta (1-delta/2)^tau) (phi' = phi/delta when non_iid != 0); equal phi
 * goes to the smaller tau; candidates with delta <= 0 are skipped; if none is feasible
 * tau = ceil(b/T_comp) + 1.  Finally tau is clamped to tau_cap (delta recomputed for the
 * clamped tau) when tau_cap != 0.
 *   V_g_bits > 0, a_bar_bps > 0, b_s >= 0, T_comp_s > 0;  tau_out, delta_out HOST.
 */
deco_status deco_policy_select(double V_g_bits, double a_bar_bps, double b_s, double T_comp_s,
                               uint32_t tau_cap, int32_t non_iid,
                               uint32_t *tau_out, double *delta_out);

/*
 * Look-up table of the implementation section ("Efficient Implementation of DeCo"): the
 * bandwidth range [a_min, a_max] profiled during warm-up is cut into `points` linearly spaced
 * sample bandwidths (the paper uses about 20) and DeCo is run once per sample for the measured
 * latency b.  deco_lut_lookup returns the entry of the sample nearest to a_bar (the lower one
 * on a tie) when a_min <= a_bar <= a_max, and falls back to deco_policy_select outside the
 * range.  Both are pure host arithmetic; `lut` is a HOST array of `points` entries owned by
 * the caller.  points >= 1, a_min <= a_max.
 */
typedef struct { double a_bps; double delta; uint32_t tau; uint32_t reserved; } deco_lut_entry;
deco_status deco_lut_build(double V_g_bits, double a_min_bps, double a_max_bps, double b_s,
                           double T_comp_s, uint32_t points, uint32_t tau_cap, int32_t non_iid,
                           deco_lut_entry *lut);
deco_status deco_lut_lookup(const deco_lut_entry *lut, uint32_t points, double a_bar_bps,
                            double V_g_bits, double b_s, double T_comp_s, uint32_t tau_cap,
                            int32_t non_iid, uint32_t *tau_out, double *delta_out);

/* Theorem 3: T_avg ~ max{(T_comp + b + delta V_g/a_bar)/(tau+1), delta V_g/a_bar, T_comp}.
 * Returns a negative value for invalid arguments. */
double deco_t_avg(double delta, uint32_t tau, double V_g_bits, double a_bar_bps, double b_s,
                  double T_comp_s);

/* k kept for ratio delta on a length-d vector (0 for invalid arguments). */
uint64_t deco_k_from_delta(double delta, uint64_t d);

/* --------------------------------------------------------------------- inspection */

deco_status deco_get_k(const deco_ctx *ctx, uint64_t *k /* HOST */);

/*
 * Device pointers of the library-owned state (any out-pointer may be NULL):
 *   e       [n][e_stride] fp32, error terms; columns >= d are padding
 *   msg     [n][k_cap] pairs, the messages of the last deco_ef_compress (first k valid); *k_cap is
 *           the distance between rows in pairs: k(delta_max), or, in a context created with
 *           n_total, half the current exchange row (see deco_get_exchange)
 *   params  [d] fp32
 */
deco_status deco_get_buffers(deco_ctx *ctx, float **e, uint64_t *e_stride, deco_pair **msg,
                             uint64_t *k_cap, float **params);

/*
 * The cached aggregate of iteration `step` (must still be in the cache), in the layout the
 * library chose when it was formed (Algorithm 1 only fixes its value, S_step = sum_i Delta^i):
 *   deco_get_aggregate         pair layout: DEVICE pointer to `positions` pairs; positions with
 *                              idx == DECO_NO_INDEX are unused, the others hold each touched
 *                              index once (increasing) with its fp32 sum
 *   deco_get_aggregate_vector  vector layout (messages of at least d / 8 entries in all):
 *                              DEVICE pointer to d fp32 values, S_step[j] at j, +0 where no
 *                              worker sent j
 * Each returns DECO_ERR_STATE when the aggregate is kept in the other layout (or is not cached).
 */
deco_status deco_get_aggregate(deco_ctx *ctx, uint64_t step, const deco_pair **entries,
                               uint64_t *positions);
deco_status deco_get_aggregate_vector(deco_ctx *ctx, uint64_t step, const float **values);

/*
 * Per-worker facts about the last deco_ef_compress (waits for `stream`); each HOST array has
 * n entries and may be NULL:
 *   threshold_key  magnitude key (bit pattern, sign cleared) of the k-th largest |a|
 *   n_greater      entries strictly above it
 *   exact_passes   1 if the worker went through the multi-pass selection in that call
 */
deco_status deco_get_select_info(deco_ctx *ctx, void *stream, uint32_t *threshold_key,
                                 uint32_t *n_greater, uint32_t *exact_passes);

/*
 * Checkpoint / resume (no counterpart in the paper's algorithms; the state is exactly what
 * Algorithm 1 carries between iterations): the iteration counter, gamma, (delta, tau), the
 * error terms e, the parameters x and every cached aggregate with its step id.
 *   deco_state_bytes   size of the blob for the current state
 *   deco_export_state  waits for `stream`, then writes the blob to buf (HOST, `bytes` long)
 *   deco_import_state  loads a blob into a context created with the same d, n, capacities
 *                      and options (else DECO_ERR_INVALID_ARG); waits for `stream` before it
 *                      returns.  Continuing from an imported state gives the same bits as
 *                      continuing the run that exported it.
 * All three may only be called between iterations.
 */
deco_status deco_state_bytes(const deco_ctx *ctx, uint64_t *bytes);
deco_status deco_export_state(deco_ctx *ctx, void *buf, uint64_t bytes, void *stream);
deco_status deco_import_state(deco_ctx *ctx, const void *buf, uint64_t bytes, void *stream);

/* Waits for `stream`, then fills *out (HOST); returns DECO_ERR_DEVICE_CHECK if a kernel
 * latched an anomaly since the context was created or reset. */
deco_status deco_get_stats(deco_ctx *ctx, void *stream, deco_stats *out);

/*
 * Optional device timing with CUDA events recorded on the caller's stream around the parts of
 * an iteration.  While enabled (up to 4096 iterations are kept) every iteration records
 * events around: [0] the streaming accumulate kernel, [1] the rest of deco_ef_compress
 * (selection and message build), [2] deco_aggregate_stale, [3] deco_apply_update.
 * deco_get_kernel_timing waits for `stream`, returns the summed milliseconds per part in
 * ms_sum[4] (HOST) and the number of iterations they cover, and clears the record.
 */
deco_status deco_set_kernel_timing(deco_ctx *ctx, int32_t enabled);
deco_status deco_get_kernel_timing(deco_ctx *ctx, void *stream, double *ms_sum /* [4] */,
                                   uint64_t *iterations);

/* Number of kernels and memset/memcpy nodes the library has enqueued so far. */
uint64_t deco_launch_count(const deco_ctx *ctx);

/* ------------------------------------------------- workers sharded over several contexts */

/*
 * Algorithm 1's workers are separate machines that exchange only the sparse messages.  A
 * context created with opt->n_total >= n holds n of the job's n_total workers (global ids
 * worker_base ... worker_base + n - 1: e, gradients and the worker side are local) and a full
 * replica of the server side.  Its messages live in one exchange buffer of n_total rows:
 *
 *   row w = | k pairs: the message of global worker w | tiles + 1 words: message position of
 *           | every 8192-entry index block of worker w | padding to an even number of words |
 *
 * with k the current number of kept entries (not the capacity k(delta_max)), rows back to back.
 * deco_ef_compress fills the context's own rows; the CALLER brings the other rows in with ONE
 * all-gather of rows_total * row_words 32-bit words among the contexts of the job (NCCL over
 * NVLink between GPUs: the rows land in local memory; plain copies between contexts on one
 * GPU); then deco_aggregate_stale sums all n_total messages in global worker order and
 * deco_apply_update scales by 1/n_total, so every replica of x stays bit-identical to the
 * single-context run.  Random-k draws with the global id.  deco_step is not available while
 * n_total > n (the exchange sits between its parts): DECO_ERR_STATE.
 *
 *   rows        DEVICE, the exchange buffer, valid for the context's lifetime
 *   row_words   words per row for the current k; changes when deco_set_policy changes k
 *   row0 / rows_local   the rows this context writes;  rows_total = n_total
 * Every out pointer may be NULL.  DECO_ERR_STATE for a context created without n_total.
 */
deco_status deco_get_exchange(deco_ctx *ctx, uint32_t **rows, uint64_t *row_words, uint32_t *row0,
                              uint32_t *rows_local, uint32_t *rows_total);

/* ------------------------------------------------------------- per-layer Top-k (variant) */

/*
 * The paper applies "Top-k ... to gradients" (Section 5, implementation) without saying whether
 * k counts over the whole model or per tensor; the contexts above take the whole flat vector.
 * This variant takes it per layer: the vector is cut into n_layers ranges
 * [layer_offsets[l], layer_offsets[l+1]) and C_delta keeps, for every worker, the
 * k_l = k(delta, d_l) largest entries of each range (ties by increasing index).  Nothing else in
 * Algorithm 1 couples entries of different layers, so a layered context is a batch of ordinary
 * contexts, one per layer, sharing policy, stepsize, gradient buffer and parameter vector.
 * With Top-k on the streaming route the layers are not stepped one by one: every kernel of the
 * path runs once for all layers (a table of the layers' buffers in device memory, grid rows
 * = layer x worker), and layers of at most 8192 entries are done by one CTA per (layer, worker).
 * With Random-k or DECO_SELECT_EXACT_PASSES each layer's context is stepped on its own.
 *   layer_offsets  HOST, [n_layers + 1], strictly increasing, first 0, last d
 *   opt            as for deco_init; opt->params (DEVICE, [d], 16-byte aligned) or NULL;
 *                  tau_max and delta_max apply to every layer
 * Random-k: layer l uses seed + l.
 */
typedef struct deco_layered deco_layered;
deco_status deco_layered_init(deco_layered **out, uint64_t d, uint32_t n,
                              const uint64_t *layer_offsets, uint32_t n_layers, double delta,
                              uint32_t tau, float lr, const deco_options *opt);

/* Frees the layered context and every layer's context (waits for the device first). */
void deco_layered_destroy(deco_layered *ctx);

/*
 * One iteration of every layer.  grads: DEVICE, [n][d] row-major, dtype = grad_dtype, 16-byte
 * aligned base.  The work runs on internal streams forked from `stream` at the start of the
 * call and joined back at its end; where layers are stepped one by one (deco_step per layer),
 * each may leave its aggregation running (deco_layered_join orders `stream` after them).
 * The first error of a layer is returned; layers after it are not stepped.
 */
deco_status deco_layered_step(deco_layered *ctx, const void *grads, void *stream);
deco_status deco_layered_join(deco_layered *ctx, void *stream);

/* deco_set_policy / deco_set_lr for all layers; the policy changes all layers or none
 * (DECO_ERR_CAPACITY if any layer lacks the capacity). */
deco_status deco_layered_set_policy(deco_layered *ctx, double delta, uint32_t tau);
deco_status deco_layered_set_lr(deco_layered *ctx, float lr);

/*
 * The context of one layer, for the getters above (deco_get_k, deco_get_buffers,
 * deco_get_aggregate, deco_get_stats, ...): its indices are relative to the layer's offset.
 * It stays owned by the layered context: do not destroy it and do not step it on its own.
 * Every out pointer may be NULL.
 */
deco_status deco_layered_layer(deco_layered *ctx, uint32_t layer, deco_ctx **layer_ctx,
                               uint64_t *offset, uint64_t *length);

/* Number of layers, sum of the layers' k, the parameter vector (DEVICE, [d]) and the number of
 * completed iterations.  Every out pointer may be NULL. */
deco_status deco_layered_info(deco_layered *ctx, uint32_t *n_layers, uint64_t *k_total,
                              float **params, uint64_t *step);

/*
 * Top-k compression of one vector without any allocation.  (The paper has no counterpart:
 * this entry point exists for callers that cannot allocate device memory at the moment they
 * need C_delta — code running while a stream is being captured, plugins inside a host
 * program that owns the memory pool, loops that cannot afford cudaMalloc's implicit
 * synchronisation.)  Same selection rule as the context-based path: the k largest |a[j]|,
 * equal magnitudes by increasing index, written as k pairs sorted by index.
 *   a        DEVICE, [d] fp32, read-only, any alignment
 *   msg_out  DEVICE, [k] pairs, 8-byte aligned
 *   1 <= k <= d <= DECO_STATIC_MAX_D; longer vectors return DECO_ERR_CAPACITY (and print
 *   the limit to stderr) — use a context for those.
 * Works on the CURRENT device; a and msg_out must live there.  Calls no cudaMalloc, cudaFree
 * or other allocating routine: the working memory (histograms, selection record, per-tile
 * counters, 82 KB) is a fixed device array inside the library that every GPU loading the
 * library holds until the process exits.  The first call on each device looks up that
 * array's device address (cudaGetSymbolAddress) — make that first call before any stream
 * capture begins.  All calls share the array and it keeps the previous call's contents; each
 * call clears what it needs first, so calls in one stream are safe, but two calls that
 * overlap on the GPU (different streams, different host threads) race on it.
 */
#define DECO_STATIC_MAX_D 16777216ull
deco_status deco_topk_compress_static(const float *a, uint64_t d, uint64_t k,
                                      deco_pair *msg_out, void *stream);

const char *deco_status_string(deco_status s);

#ifdef __cplusplus
}
#endif
#endif /* DECO_H_ */
