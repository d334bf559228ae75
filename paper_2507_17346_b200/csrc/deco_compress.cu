// Worker side of Algorithm 1 on the device: a = e + gamma*g, exact Top-k of |a| with ties to
// the lower index, messages as packed (index, value) pairs sorted by index, residual in e.
//
// Two routes give the same bits.
//
// Streaming route (DECO_SELECT_AUTO): a small sample of a fixes, per worker, a lower bound
// `spec_key` that is below the k-th largest magnitude with overwhelming probability.  One pass
// reads e and g, writes a into e and stages every entry whose key reaches the bound (a few
// times k pairs, each tile's entries in index order); staged entries are written to e as +0
// on the guess that they will be selected.  The exact threshold is then found by a two-level
// radix selection over the staged pairs only (on key - spec_key), a classification pass counts
// the rejected entries and the ties per tile and per chunk of tiles, the message is an ordered
// filter of the staged pairs, and the staged entries that are not selected get their value back
// as the filter passes over them.  The count of staged pairs proves the bound was valid (>= k of
// them); if it was not, or the staging area overflowed, that worker takes the second route in
// the same call.  For dense messages (delta >= 1/32) the sample also fixes an upper bound
// `cert_key` of the threshold: staged entries above it are selected for certain (again proved by
// a count), and the selection and classification read only the band between the two bounds.
//
// Multi-pass route (DECO_SELECT_EXACT_PASSES, and the fallback of the first): three radix
// histogram passes over e fix the threshold key, one pass counts per tile, one pass emits.
// It handles any input (all entries equal, all zero, k = d ...).
//
// Entry order inside a tile is (warp, round, lane, component): warp w owns WARP_ELEMS
// consecutive entries, and in round u lane l owns V consecutive ones, so each warp-level
// load is one contiguous 512-byte request.
#include <cooperative_groups.h>

#include <algorithm>
#include <new>
#include <cuda_bf16.h>

#include "deco_internal.h"

namespace cg = cooperative_groups;

namespace deco {

namespace {

constexpr uint32_t FULL = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
// as 1, 2, 3", SC'11), written from the published definition: per round the two counter words
// 0 and 2 are multiplied by fixed constants, the high halves are xored with the other two
// words and the key, and the key is bumped by the Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c;
}

// Random-k: the priority of entry j of worker i at iteration t is a 23-bit word of the
// Philox stream keyed by the context's seed with counter (j / 4, t_lo, i, t_hi ^ "RAND");
// the k largest priorities (equal ones by increasing index) are the selected entries.
struct RandParams {
    uint32_t on;                 // 0: Top-k on |a|, 1: Random-k
    uint32_t seed_lo, seed_hi, step_lo, step_hi;
    uint32_t worker_base;        // global id of the context's first worker
};

__device__ __forceinline__ uint4 rand_keys4(const RandParams &rk, uint32_t worker, uint64_t j4)
{
    // priorities of the four entries 4*j4 .. 4*j4 + 3
    uint4 o = philox4x32_10(make_uint4(static_cast<uint32_t>(j4), rk.step_lo, rk.worker_base + worker,
                                       rk.step_hi ^ 0x52414E44u), rk.seed_lo, rk.seed_hi);
    return make_uint4(o.x >> 9, o.y >> 9, o.z >> 9, o.w >> 9);
}

__device__ __forceinline__ uint32_t rand_key(const RandParams &rk, uint32_t worker, uint32_t j)
{
    const uint4 o = rand_keys4(rk, worker, j >> 2);
    const uint32_t w = j & 3u;
    return w == 0 ? o.x : (w == 1 ? o.y : (w == 2 ? o.z : o.w));
}

// Everything the selection kernels need, passed by value.
struct Sel {
    float *e;
    uint64_t e_stride;
    uint64_t d;
    uint64_t g_stride;       // entries between gradient rows
    uint32_t n;
    uint32_t ntiles;
    uint32_t k;
    SelectState *sel;
    uint32_t *hist;          // [n][2][RADIX_LEVELS][RADIX_BINS]: 0 = staged route, 1 = multi-pass
    uint32_t *done;          // [n][DONE_SLOTS] CTA arrival counters
    uint32_t *sample_keys;   // [n][4 * SAMPLE_CHUNKS] keys of the sample
    uint32_t *sample_hist;   // [n][SAMPLE_BINS] sample keys per bin of their top bits; cleared by its reader
    uint32_t *sample_win;    // [n][WINDOW_WORDS] fine histogram around the previous bound; cleared by its reader
    uint32_t *tile_gt, *tile_eq, *tile_take, *tile_start, *tile_off, *tile_cnt, *tile_rej;
    uint32_t nchunks;        // chunks of CHUNK_TILES tiles
    uint32_t *chunk_cnt, *chunk_rej, *chunk_eq;   // [n][nchunks] staged / rejected / ties
    uint32_t *chunk_eqb;     // [n][nchunks] ties in earlier chunks
    uint32_t *chunk_start;   // [n][nchunks + 1] message position of each chunk
    deco_pair *msg;          // first local worker's message; rows k_cap pairs apart
    uint64_t k_cap;
    uint64_t dir_stride;     // words between the workers' rows of tile_start
    deco_pair *stage;        // [n][stage_cap] candidates, each tile's in index order
    deco_pair *band;         // [n][stage_cap] the candidates below cert_key, unordered
    uint64_t stage_cap;
    uint2 *work;             // [n][work_cap] (tile, slice) entries of the emit work list
    uint64_t work_cap;
    uint32_t *status;        // [0] latched status, [1..2] detail, [3] "some worker needs the multi-pass route"
    RandParams rk;
    uint32_t use_band;       // the streaming pass writes the band list (dense messages only)
    uint32_t sample_shift;   // sample histogram bin = key >> sample_shift
    uint32_t bound_low_bit;  // lowest key bit the bound is refined to
};

// selection key of a staged pair
__device__ __forceinline__ uint32_t key_of(const Sel &p, uint32_t i, const deco_pair &pr)
{
    return p.rk.on ? rand_key(p.rk, i, pr.idx) : mag_key(pr.val);
}


__device__ __forceinline__ void latch(uint32_t *status, uint32_t code, uint32_t a, uint32_t b)
{
    if (atomicCAS(status, 0u, code) == 0u) {
        status[1] = a;
        status[2] = b;
    }
}

// Loads of what earlier kernels, or earlier phases of the same cooperative launch, left behind.
// As launches of their own the selection bodies use plain loads: every CTA of a grid reads the
// same 64-byte selection record, which the L1 caches then serve once per SM (read through L2
// by every warp, that one line becomes the bottleneck of a grid of a thousand CTAs).  Inside the
// cooperative launch (COH), whose grids are small, they read through L2.
template <bool COH, typename T>
__device__ __forceinline__ T ldq(const T *p)
{
    return COH ? __ldcg(p) : *p;
}

// What the streaming pass staged for a worker: candidates in all, and those inside the band.
template <bool COH>
__device__ __forceinline__ void staged_counts(const SelectState &s, uint32_t &n_staged, uint32_t &n_band)
{
    const unsigned long long v = ldq<COH>(&s.staged_band);
    n_staged = static_cast<uint32_t>(v);
    n_band = static_cast<uint32_t>(v >> 32);
}

// The list the selection kernels read for worker i and its length: the band list, or (when the
// streaming pass does not write one) all staged candidates.
__device__ __forceinline__ const deco_pair *select_list(const Sel &p, uint32_t i, uint32_t n_staged,
                                                        uint32_t &n_band)
{
    if (!p.use_band) n_band = n_staged;
    return (p.use_band ? p.band : p.stage) + static_cast<size_t>(i) * p.stage_cap;
}

__device__ __forceinline__ uint32_t *hist_of(const Sel &p, uint32_t i, int route, int level)
{
    return p.hist + ((static_cast<size_t>(i) * 2 + route) * RADIX_LEVELS + level) * RADIX_BINS;
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(FULL, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Exclusive prefix of per-thread counts in the order (warp, round u, lane).  Every thread of
// the CTA must call it; s_w is WARPS words of shared memory.
template <int U>
__device__ __forceinline__ void ordered_prefix(const uint32_t (&cnt)[U], uint32_t (&pos)[U],
                                               uint32_t *s_w, uint32_t &block_total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t run = 0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t incl = warp_incl_scan(cnt[u]);
        pos[u] = run + incl - cnt[u];
        run += __shfl_sync(FULL, incl, 31);
    }
    if (lane == 0) s_w[w] = run;
    __syncthreads();
    uint32_t before = 0, total = 0;
#pragma unroll
    for (int ww = 0; ww < WARPS; ++ww) {
        const uint32_t v = s_w[ww];
        before += (ww < w) ? v : 0u;
        total += v;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) pos[u] += before;
    block_total = total;
    __syncthreads();
}

// ordered_prefix plus, for a second per-thread count nb, positions that are unique inside the
// CTA (in thread order) and the CTA's total.  s_w and s_b are WARPS words each.
template <int U>
__device__ __forceinline__ void ordered_prefix2(const uint32_t (&m)[U], uint32_t (&pos)[U], uint32_t nb,
                                                uint32_t &bpos, uint32_t *s_w, uint32_t *s_b,
                                                uint32_t &block_total, uint32_t &band_total)
{
    // m[u]: the low byte marks the thread's entries of round u that count
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t run = 0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t c = __popc(m[u] & 0xFFu);
        const uint32_t incl = warp_incl_scan(c);
        pos[u] = run + incl - c;
        run += __shfl_sync(FULL, incl, 31);
    }
    const uint32_t bincl = warp_incl_scan(nb);
    if (lane == 0) s_w[w] = run;
    if (lane == 31) s_b[w] = bincl;
    __syncthreads();
    uint32_t before = 0, total = 0, bbefore = 0, btotal = 0;
#pragma unroll
    for (int ww = 0; ww < WARPS; ++ww) {
        const uint32_t v = s_w[ww], vb = s_b[ww];
        before += (ww < w) ? v : 0u;
        total += v;
        bbefore += (ww < w) ? vb : 0u;
        btotal += vb;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) pos[u] += before;
    bpos = bbefore + bincl - nb;
    block_total = total;
    band_total = btotal;
    __syncthreads();
}

// Exclusive scan over the CTA (any multiple of 32 threads up to 1024); s_w has 33 words.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t *s_w, uint32_t &total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int nw = blockDim.x >> 5;
    const uint32_t incl = warp_incl_scan(v);
    if (lane == 31) s_w[w] = incl;
    __syncthreads();
    if (w == 0) {
        const uint32_t x = lane < nw ? s_w[lane] : 0u;
        const uint32_t xi = warp_incl_scan(x);
        s_w[lane] = xi - x;
        if (lane == 31) s_w[32] = xi;
    }
    __syncthreads();
    const uint32_t out = s_w[w] + incl - v;
    total = s_w[32];
    __syncthreads();
    return out;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

template <int GT>
struct Geo {
    static constexpr int V = GT ? 8 : 4;                 // entries per thread and round
    static constexpr int U = WARP_ELEMS / (32 * V);      // rounds
};

template <int GT>
__device__ __forceinline__ float load_g(const void *grow, uint64_t j)
{
    if (GT) {
        const uint16_t h = reinterpret_cast<const uint16_t *>(grow)[j];
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
    return reinterpret_cast<const float *>(grow)[j];
}

// ------------------------------------------------------------------------------------------
// Radix helpers.  Multi-pass route: 31-bit key = 12 + 12 + 7 bits, most significant first.
// ------------------------------------------------------------------------------------------
template <int LEVEL>
__device__ __forceinline__ void radix_bin(uint32_t key, uint32_t prefix, uint32_t *h)
{
    if (LEVEL == 0) {
        atomicAdd(&h[key >> 19], 1u);
    } else if (LEVEL == 1) {
        if ((key >> 19) == prefix) atomicAdd(&h[(key >> 7) & 0xFFFu], 1u);
    } else {
        if ((key >> 7) == prefix) atomicAdd(&h[key & 0x7Fu], 1u);
    }
}

// One CTA of BLOCK threads: the bin b with  count(bins > b) < want <= count(bins >= b)  of
// histogram h (RADIX_BINS bins, read through L2) and the count above it.  s_scan: 33 words,
// s_out: 2 words.  All threads get the result; bin 0xFFFFFFFF means the histogram holds fewer
// than `want` entries.
__device__ __forceinline__ void pick_bin(const uint32_t *h, uint32_t want, uint32_t *s_scan,
                                         uint32_t *s_out, uint32_t &bin_out, uint32_t &above_out)
{
    constexpr int PER = RADIX_BINS / BLOCK;   // 16 bins per thread
    // thread t owns the bins of the mirrored position, so the exclusive prefix over threads
    // is the number of entries in higher bins
    const int rt = BLOCK - 1 - static_cast<int>(threadIdx.x);
    uint32_t loc[PER], sum = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) {
        loc[b] = __ldcg(&h[rt * PER + b]);
        sum += loc[b];
    }
    if (threadIdx.x == 0) {
        s_out[0] = 0xFFFFFFFFu;
        s_out[1] = 0;
    }
    uint32_t total;
    const uint32_t s_above = block_excl_scan(sum, s_scan, total);
    if (s_above < want && s_above + sum >= want) {
        uint32_t acc = s_above;
        int bin = rt * PER;
#pragma unroll
        for (int b = PER - 1; b >= 0; --b) {
            if (acc + loc[b] >= want) {
                bin = rt * PER + b;
                break;
            }
            acc += loc[b];
        }
        s_out[0] = static_cast<uint32_t>(bin);
        s_out[1] = acc;
    }
    __syncthreads();
    bin_out = s_out[0];
    above_out = s_out[1];
    __syncthreads();
}

// Multi-pass route: one CTA appends the picked bin of level LEVEL to the key prefix of s.
template <int LEVEL>
__device__ __forceinline__ void pick_body(SelectState &s, const uint32_t *h, uint32_t *s_scan,
                                          uint32_t *s_out, uint32_t *status, uint32_t i)
{
    constexpr int BITS = (LEVEL == 2) ? 7 : 12;
    const uint32_t k_rem = s.k_rem;
    uint32_t bin, above;
    pick_bin(h, k_rem, s_scan, s_out, bin, above);
    if (threadIdx.x == 0) {
        if (bin == 0xFFFFFFFFu) {
            latch(status, DECO_ERR_DEVICE_CHECK, 0x100u + LEVEL, i);
        } else {
            s.n_greater += above;
            s.k_rem = k_rem - above;
            const uint32_t prefix = (s.prefix << BITS) | bin;
            s.prefix = prefix;
            if (LEVEL == 2) {
                s.threshold = prefix;
                s.ties_take = k_rem - above;
            }
        }
    }
    __syncthreads();
}

// true for exactly one CTA per counter: the last of `ctas` to get here (nothing waits)
__device__ __forceinline__ bool last_cta_to_arrive(uint32_t *counter, uint32_t *s_flag, uint32_t ctas)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *s_flag = (atomicAdd(counter, 1u) == ctas - 1) ? 1u : 0u;
    __syncthreads();
    const bool last = *s_flag != 0;
    if (last) __threadfence();
    return last;
}

// ------------------------------------------------------------------------------------------
// Start of an iteration.  Up to SAMPLE_CTAS CTAs per worker: together they clear the histograms and,
// on the streaming route, draw the sample (each thread one group of 4 consecutive entries,
// groups evenly spread over [0, d)) and leave its keys in global memory; CTA 0 re-arms the
// selection record; the last CTA of a worker to arrive fixes spec_key from the sample.
// ------------------------------------------------------------------------------------------
constexpr int BEGIN_BLOCK = 1024;
constexpr int SAMPLE_CTAS = 32;
constexpr int SAMPLE_CHUNKS = SAMPLE_CTAS * BEGIN_BLOCK;   // at most 32768 groups of 4 entries
constexpr int SAMPLE_HIST_BITS = 12;                       // top key bits the histogram resolves
constexpr uint32_t SAMPLE_HIST_BINS = 1u << SAMPLE_HIST_BITS;
constexpr int SAMPLE_BINS_PER_THREAD = SAMPLE_HIST_BINS / BEGIN_BLOCK;
constexpr int SAMPLE_WARP_LIST = 256;                      // list slots per warp in the search
static_assert(4 * SAMPLE_CHUNKS == SAMPLE_KEYS, "sample buffer size");
static_assert(SAMPLE_HIST_BINS == SAMPLE_BINS, "sample histogram size");
static_assert(SAMPLE_HIST_BINS + WINDOW_WORDS <= (BEGIN_BLOCK / 32) * SAMPLE_WARP_LIST,
              "both histograms share the list storage");
static_assert((WINDOW_BINS << WINDOW_SUB_BITS) == BEGIN_BLOCK, "one fine bin per thread of the last CTA");

// Number of sample groups S.  A group costs two random line fetches (e and g); a candidate
// that is staged and then rejected costs about as much (its +0 guess is undone), and their
// number falls like 5 k / sqrt(4 S k / d).  The sum is smallest near S = (k d)^(1/3); the
// factor is fitted to measurements.  Between a quarter of the maximum and the maximum, never
// more than the vector has.
static uint32_t sample_groups(uint64_t d, uint64_t k)
{
    const uint64_t nchunks = (d + 3) >> 2;
    uint64_t want = static_cast<uint64_t>(0.6 * cbrt(static_cast<double>(d) * static_cast<double>(k)));
    // at least a quarter of the maximum, but for short vectors (layers of the per-layer variant)
    // no more than one group in 16, down to one CTA's worth
    uint64_t least = nchunks / 16;
    if (least > SAMPLE_CHUNKS / 4) least = SAMPLE_CHUNKS / 4;
    if (least < BEGIN_BLOCK) least = BEGIN_BLOCK;
    if (want < least) want = least;
    if (want > SAMPLE_CHUNKS) want = SAMPLE_CHUNKS;
    return static_cast<uint32_t>(nchunks < want ? nchunks : want);
}

// nparts: the CTAs (blockIdx.x = 0 .. nparts - 1) that work on worker i; others leave at once.
// G: sample groups per thread (nparts * G * BEGIN_BLOCK >= S).
template <int GT, int G>
__device__ __forceinline__ void begin_step_body(const Sel &p, const uint32_t i, const void *__restrict__ grads,
                                                float alpha, uint32_t exact_all, uint32_t S, const uint32_t nparts)
{
    const uint32_t part = blockIdx.x;
    if (part >= nparts) return;
    const int t = threadIdx.x;
    SelectState &s = p.sel[i];
    uint32_t *hz = hist_of(p, i, 0, 0);
    for (int q = part * BEGIN_BLOCK + t; q < 2 * RADIX_LEVELS * RADIX_BINS;
         q += nparts * BEGIN_BLOCK)
        hz[q] = 0;
    if (part == 0) {
        if (t < 3) p.done[i * DONE_SLOTS + t] = 0;          // levels A, B, classification
        if (t == 4) p.done[i * DONE_SLOTS + 4] = 0;         // chunk sums
        if (t == 5) p.done[i * DONE_SLOTS + 5] = 0;         // length of the emit work list
        if (i == 0 && t == 0) p.status[3] = exact_all;
        if (t == 0) {
            s.thr_prev2 = s.thr_prev;          // the last iterations' exact thresholds
            s.thr_prev = s.threshold;
            s.swing = 0;
            s.prefix = 0;
            s.k_rem = p.k;
            s.n_greater = 0;
            s.threshold = 0;
            s.ties_take = 0;
            s.exact = exact_all;
            s.spec_key = SPEC_DISABLED;
            s.cert_key = SPEC_DISABLED;
            s.staged_band = 0;
            s.rel_shift = 12;
            if (exact_all) s.exact_total += 1;
        }
    }
    if (exact_all) return;

    constexpr int NW = BEGIN_BLOCK / 32;
    __shared__ uint32_t s_buf[NW * SAMPLE_WARP_LIST];        // histogram, later the warp lists
    __shared__ uint32_t s_cnt[NW];
    __shared__ uint32_t s_w[33];
    __shared__ uint32_t s_flag;
    __shared__ uint32_t s_hi;
    const float *erow = p.e + static_cast<size_t>(i) * p.e_stride;
    const char *grow = reinterpret_cast<const char *>(grads) +
                       static_cast<size_t>(i) * p.g_stride * (GT ? 2 : 4);
    const uint64_t nchunks = (p.d + 3) >> 2;
    uint4 *skeys = reinterpret_cast<uint4 *>(p.sample_keys) + static_cast<size_t>(i) * SAMPLE_CHUNKS;
    // Window of WINDOW_BINS coarse bins (one octave) around the previous iteration's bound, each
    // bin cut into 64: when the sampled ranks fall inside it (they do unless the gradients'
    // scale jumps) the last CTA reads the bounds off this histogram and never looks at the
    // sample keys again.  hint_key was written by the previous launch; nothing writes it here
    // before the last CTA does.
    const uint32_t hint_bin = min(s.hint_key >> p.sample_shift, SAMPLE_HIST_BINS - 1);
    const uint32_t win_lo = min(hint_bin > WINDOW_BINS / 2 ? hint_bin - WINDOW_BINS / 2 : 0u,
                                SAMPLE_HIST_BINS - WINDOW_BINS);
    uint32_t *s_win = s_buf + SAMPLE_HIST_BINS;               // WINDOW_WORDS words behind the coarse histogram
    {
        // G sample groups per thread, all loads issued before the first use
        uint32_t kk[G][4];
#pragma unroll
        for (int gq = 0; gq < G; ++gq) {
            const uint32_t sidx = (part * G + gq) * BEGIN_BLOCK + t;
#pragma unroll
            for (int c = 0; c < 4; ++c) kk[gq][c] = 0;           // 0 = "not a sample"
            if (sidx < S) {
                const uint64_t j = ((static_cast<uint64_t>(sidx) * nchunks) / S) << 2;
                if (p.rk.on) {
                    const uint4 r4 = rand_keys4(p.rk, i, j >> 2);
                    const uint32_t rs[4] = {r4.x, r4.y, r4.z, r4.w};
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (j + c < p.d) kk[gq][c] = rs[c];
                } else {
                    const float4 ev = *reinterpret_cast<const float4 *>(erow + j);
                    const float es[4] = {ev.x, ev.y, ev.z, ev.w};
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (j + c < p.d)
                            kk[gq][c] = mag_key(__fmaf_rn(alpha, load_g<GT>(grow, j + c), es[c]));
                }
            }
        }
#pragma unroll
        for (int gq = 0; gq < G; ++gq)
            skeys[(part * G + gq) * BEGIN_BLOCK + t] = make_uint4(kk[gq][0], kk[gq][1], kk[gq][2], kk[gq][3]);
        // histogram of the top SAMPLE_HIST_BITS key bits of this CTA's nonzero keys: lanes
        // with the same bin elect one of them to add the group's size
#pragma unroll
        for (int c = 0; c < SAMPLE_BINS_PER_THREAD; ++c) s_buf[c * BEGIN_BLOCK + t] = 0;
        for (uint32_t q = t; q < WINDOW_WORDS; q += BEGIN_BLOCK) s_win[q] = 0;
        __syncthreads();
        uint32_t above_window = 0;
#pragma unroll
        for (int gq = 0; gq < G; ++gq) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t key = kk[gq][c];
                const uint32_t hb = key ? min(key >> p.sample_shift, SAMPLE_HIST_BINS - 1) : SAMPLE_HIST_BINS;
                const uint32_t grp = __match_any_sync(FULL, hb);
                if (hb < SAMPLE_HIST_BINS && (t & 31) == __ffs(grp) - 1) atomicAdd(&s_buf[hb], __popc(grp));
                if (hb < SAMPLE_HIST_BINS && hb >= win_lo) {
                    if (hb >= win_lo + WINDOW_BINS) {
                        above_window += 1;
                    } else {
                        const uint32_t sub = (key >> (p.sample_shift - WINDOW_SUB_BITS)) & ((1u << WINDOW_SUB_BITS) - 1u);
                        atomicAdd(&s_win[((hb - win_lo) << WINDOW_SUB_BITS) + sub], 1u);
                    }
                }
            }
        }
        above_window = __reduce_add_sync(FULL, above_window);
        if ((t & 31) == 0 && above_window) atomicAdd(&s_win[WINDOW_WORDS - 1], above_window);
        __syncthreads();
#pragma unroll
        for (int c = 0; c < SAMPLE_BINS_PER_THREAD; ++c) {
            const uint32_t v = s_buf[c * BEGIN_BLOCK + t];
            if (v) atomicAdd(&p.sample_hist[i * SAMPLE_HIST_BINS + c * BEGIN_BLOCK + t], v);
        }
        for (uint32_t q = t; q < WINDOW_WORDS; q += BEGIN_BLOCK) {
            const uint32_t v = s_win[q];
            if (v) atomicAdd(&p.sample_win[i * WINDOW_WORDS + q], v);
        }
    }
    // the arrival counter resets itself: only the last CTA touches it afterwards
    uint32_t *arrive = &p.done[i * DONE_SLOTS + 3];
    if (!last_cta_to_arrive(arrive, &s_flag, nparts)) return;
    if (t == 0) *arrive = 0;

    // every sampled group is complete unless the sample is the whole vector
    const uint32_t m_total = (S == nchunks) ? static_cast<uint32_t>(p.d) : 4u * S;
    // rank inside the sample: mean + 5 sigma + 2 of a binomial with p = k/d (exact when the
    // sample is the whole vector)
    uint32_t R;
    uint32_t R_hi = 0;          // sample rank of the certainty bound: mean - 5 sigma - 2, if there is one
    uint32_t rel_shift = 10;
    if (m_total >= p.d) {
        R = p.k;
    } else {
        const double mean = static_cast<double>(p.k) * m_total / static_cast<double>(p.d);
        const double r = mean + 5.0 * sqrt(mean) + 2.0;
        R = r >= static_cast<double>(m_total) ? m_total + 1u : static_cast<uint32_t>(r) + 1u;
        const double rh = mean - 5.0 * sqrt(mean) - 2.0;
        R_hi = (p.use_band && rh >= 1.0) ? static_cast<uint32_t>(rh) : 0u;
        // how far the sampled rank sits above k/d decides how far above the bound the
        // threshold may lie (in value: that ratio to the power 1/tail-index)
        const double rho = static_cast<double>(R) / (mean > 1e-9 ? mean : 1e-9);
        rel_shift = rho <= 1.7 ? 10u : 12u;
        if (p.rk.on) rel_shift = 10u;          // uniform 23-bit priorities: 4095 << 10 is half the range
    }
    uint32_t *gh = p.sample_hist + i * SAMPLE_HIST_BINS;
    uint32_t *gw = p.sample_win + i * WINDOW_WORDS;
    // fine bin WINDOW-1-t of the window belongs to thread t, so that the prefix over threads
    // counts the sample keys in higher fine bins; both histograms are left cleared
    const uint32_t fine = (WINDOW_BINS << WINDOW_SUB_BITS) - 1u - t;
    const uint32_t in_fine = __ldcg(&gw[fine]);
    const uint32_t above_window = __ldcg(&gw[WINDOW_WORDS - 1]);
    gw[fine] = 0;
    if (R > m_total) {                         // the sample cannot bound the threshold
        if (t == 0) {
            s.spec_key = 0;                    // stage everything: the count check decides
            s.hint_key = 0;
            gw[WINDOW_WORDS - 1] = 0;
        }
#pragma unroll
        for (int c = 0; c < SAMPLE_BINS_PER_THREAD; ++c) gh[c * BEGIN_BLOCK + t] = 0;
        return;
    }
    {
        // Both sampled ranks inside the window: the bounds are edges of its fine bins (1/1024 of
        // an octave wide), and the sample keys are not looked at again.
        uint32_t tot;
        const uint32_t higher = above_window + block_excl_scan(in_fine, s_w, tot);
        if (t == 0) {
            s_flag = 0xFFFFFFFFu;
            s_hi = R_hi ? 0xFFFFFFFFu : SPEC_DISABLED;
            gw[WINDOW_WORDS - 1] = 0;
        }
        __syncthreads();
        const uint32_t sub_shift = p.sample_shift - WINDOW_SUB_BITS;
        const uint32_t edge = ((win_lo << WINDOW_SUB_BITS) + fine) << sub_shift;     // lower edge of my fine bin
        if (higher < R && higher + in_fine >= R) s_flag = edge;
        if (R_hi && higher < R_hi && higher + in_fine >= R_hi) s_hi = edge + (1u << sub_shift);
        __syncthreads();
        const uint32_t w_bound = s_flag, w_cert = s_hi;
        __syncthreads();
        if (w_bound != 0xFFFFFFFFu && w_cert != 0xFFFFFFFFu) {
#pragma unroll
            for (int c = 0; c < SAMPLE_BINS_PER_THREAD; ++c) gh[c * BEGIN_BLOCK + t] = 0;
            if (t == 0) {
                s.spec_key = w_bound;
                s.cert_key = w_cert;
                s.rel_shift = rel_shift;
                s.hint_key = w_bound;
            }
            return;
        }
    }
    // Largest key prefix v (a multiple of 2^bound_low_bit) with  #(sample keys >= v) >= R.
    // The top bits come from the histogram the sampling CTAs filled: thread t looks at bins
    // BINS-1-4t .. BINS-4-4t, so that the prefix over threads counts the higher bins.
    uint32_t bound = 0, above = 0;                           // above = #(keys in higher bins)
    {
        uint32_t cnt[SAMPLE_BINS_PER_THREAD];
        uint32_t mine = 0;
#pragma unroll
        for (int c = 0; c < SAMPLE_BINS_PER_THREAD; ++c) {
            const uint32_t hb = SAMPLE_HIST_BINS - 1 - (t * SAMPLE_BINS_PER_THREAD + c);
            cnt[c] = __ldcg(&gh[hb]);
            gh[hb] = 0;                                       // ready for the next iteration
            mine += cnt[c];
        }
        uint32_t tot;
        uint32_t higher = block_excl_scan(mine, s_w, tot);
        if (t == 0) {
            s_flag = 0;
            s_cnt[0] = 0;
            s_hi = SPEC_DISABLED;
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < SAMPLE_BINS_PER_THREAD; ++c) {
            const uint32_t hb = SAMPLE_HIST_BINS - 1 - (t * SAMPLE_BINS_PER_THREAD + c);
            if (higher < R && higher + cnt[c] >= R) {
                s_flag = hb << p.sample_shift;
                s_cnt[0] = higher;
            }
            // certainty bound: upper edge of the bin that holds the sample key of rank R_hi, so
            // that fewer than R_hi sample keys reach it (the edge above the top bin is beyond
            // every key: nothing is certain then)
            if (R_hi && higher < R_hi && higher + cnt[c] >= R_hi) s_hi = (hb + 1u) << p.sample_shift;
            higher += cnt[c];
        }
        __syncthreads();
        bound = s_flag;
        above = s_cnt[0];
        __syncthreads();
    }
    // The sample keys of that bin go onto per-warp lists in shared memory and the remaining
    // bits are settled on those.  Zero keys never count: every candidate is positive.
    const int lane = t & 31, w = t >> 5;
    const uint32_t bin_end = bound + (1u << p.sample_shift);    // no overflow: keys have 31 bits
    const int parts = static_cast<int>((S + BEGIN_BLOCK - 1) / BEGIN_BLOCK);
    uint32_t mine = 0;                                       // warp-uniform running count
    for (int q0 = 0; q0 < parts; q0 += 4) {
        uint4 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
            v[q] = q0 + q < parts ? __ldcg(skeys + (q0 + q) * BEGIN_BLOCK + t) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t ks[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const bool keep = ks[c] >= bound && ks[c] < bin_end && ks[c] != 0;
                const uint32_t m = __ballot_sync(FULL, keep);
                if (m == 0) continue;
                const uint32_t at = mine + __popc(m & ((1u << lane) - 1u));
                if (keep && at < SAMPLE_WARP_LIST) s_buf[w * SAMPLE_WARP_LIST + at] = ks[c];
                mine += __popc(m);
            }
        }
    }
    if (lane == 0) s_cnt[w] = mine;
    __syncthreads();
    uint32_t longest = 0;
#pragma unroll
    for (int ww = 0; ww < NW; ++ww) longest = max(longest, s_cnt[ww]);
    __syncthreads();
    const int nbits = static_cast<int>(p.sample_shift) - static_cast<int>(p.bound_low_bit);
    if (longest <= SAMPLE_WARP_LIST) {
        // two rounds of a 64-bin histogram over the listed keys settle the remaining bits
        __shared__ uint32_t s_h[64];
        const uint32_t listed = min(mine, static_cast<uint32_t>(SAMPLE_WARP_LIST));
        uint32_t settled = 0;                                // bits below sample_shift, settled so far
        int done_bits = 0;
        for (int round = 0; round < 2; ++round) {
            const int take = round == 0 ? nbits - 6 : 6;      // nbits is 11 or 12
            const int low = static_cast<int>(p.sample_shift) - done_bits - take;
            if (t < 64) s_h[t] = 0;
            __syncthreads();
            for (uint32_t slot = lane; slot < listed; slot += 32) {
                const uint32_t sub = s_buf[w * SAMPLE_WARP_LIST + slot] - bound;
                // keys that agree with the bits settled so far
                if (done_bits == 0 || (sub >> (low + take)) == (settled >> (low + take)))
                    atomicAdd(&s_h[(sub >> low) & ((1u << take) - 1u)], 1u);
            }
            __syncthreads();
            if (t == 0) {
                uint32_t acc = above;
                int pick = 0;
                for (int bnum = (1 << take) - 1; bnum >= 0; --bnum) {
                    if (acc + s_h[bnum] >= R) {
                        pick = bnum;
                        break;
                    }
                    acc += s_h[bnum];
                }
                s_w[0] = static_cast<uint32_t>(pick);
                s_w[1] = acc;
            }
            __syncthreads();
            settled |= s_w[0] << low;
            above = s_w[1];
            done_bits += take;
            __syncthreads();
        }
        bound += settled;
    } else {
        // a list overflowed (very many sample keys in one bin): settle the bits one by one with
        // counts over the whole sample
#pragma unroll 1
        for (int bit = static_cast<int>(p.sample_shift) - 1; bit >= static_cast<int>(p.bound_low_bit); --bit) {
            const uint32_t cand = bound | (1u << bit);
            uint32_t c = 0;
            for (int q = 0; q < parts; ++q) {
                const uint4 v = __ldcg(skeys + q * BEGIN_BLOCK + t);
                c += (v.x >= cand) + (v.y >= cand) + (v.z >= cand) + (v.w >= cand);
            }
            uint32_t all;
            (void)block_excl_scan(c, s_w, all);
            if (all >= R) bound = cand;
        }
    }
    if (t == 0) {
        s.spec_key = bound;                    // lower edge of a 2^bound_low_bit-wide key bin
        s.cert_key = s_hi;                     // above the bound's own histogram bin
        s.rel_shift = rel_shift;
        s.hint_key = bound;                    // centre of the next iteration's window
    }
}

template <int GT>
__global__ void __launch_bounds__(BEGIN_BLOCK, 2)
begin_step_kernel(Sel p, const void *__restrict__ grads, float alpha, uint32_t exact_all, uint32_t S)
{
    begin_step_body<GT, 1>(p, blockIdx.y, grads, alpha, exact_all, S, gridDim.x);
}

// ------------------------------------------------------------------------------------------
// Streaming pass.  GT = 0: fp32 gradients; GT = 1: bfloat16 gradients.  ALIGNED: every
// gradient row starts on a 16-byte boundary, so whole tiles are read with 128-bit loads;
// otherwise (and in the tile that holds the end of the vector) gradients are read entry by
// entry.  SPEC: stage the entries whose key reaches sel[i].spec_key.
// ------------------------------------------------------------------------------------------
template <int GT, bool ALIGNED, bool SPEC, bool RANDK, bool BAND>
__device__ __forceinline__ void
ef_accumulate_body(const uint32_t tile, const uint32_t i, const bool rows_aligned,
                   float *__restrict__ e, uint64_t e_stride, const void *__restrict__ grads,
                   uint64_t d, uint64_t g_stride, float alpha, const RandParams &rk, SelectState *__restrict__ sel,
                   deco_pair *__restrict__ stage, deco_pair *__restrict__ band, uint64_t stage_cap,
                   uint32_t *__restrict__ tile_off, uint32_t *__restrict__ tile_cnt,
                   uint32_t *__restrict__ tile_rej, uint32_t *__restrict__ tile_eq,
                   uint32_t ntiles)
{
    constexpr int V = Geo<GT>::V, U = Geo<GT>::U;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    float *erow = e + static_cast<size_t>(i) * e_stride;
    const char *grow = reinterpret_cast<const char *>(grads) +
                       static_cast<size_t>(i) * g_stride * (GT ? 2 : 4);
    const uint64_t tile_base = static_cast<uint64_t>(tile) * TILE;
    const uint64_t wbase = tile_base + static_cast<uint64_t>(w) * WARP_ELEMS;
    const bool full = ALIGNED && rows_aligned && (tile_base + TILE <= d);

    float x[U][V];
    if (full) {
        if (GT == 0) {
            float4 ev[U], gv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint64_t j = wbase + u * 128 + lane * 4;
                ev[u] = *reinterpret_cast<const float4 *>(erow + j);
                gv[u] = __ldcs(reinterpret_cast<const float4 *>(grow) + (j >> 2));
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                x[u][0] = __fmaf_rn(alpha, gv[u].x, ev[u].x);
                x[u][1] = __fmaf_rn(alpha, gv[u].y, ev[u].y);
                x[u][2] = __fmaf_rn(alpha, gv[u].z, ev[u].z);
                x[u][3] = __fmaf_rn(alpha, gv[u].w, ev[u].w);
            }
        } else {
            float4 ev[U][2];
            uint4 gv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint64_t j = wbase + u * 256 + lane * 8;
                ev[u][0] = *reinterpret_cast<const float4 *>(erow + j);
                ev[u][1] = *reinterpret_cast<const float4 *>(erow + j + 4);
                gv[u] = __ldcs(reinterpret_cast<const uint4 *>(grow) + (j >> 3));
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                x[u][0] = __fmaf_rn(alpha, bf16_lo(gv[u].x), ev[u][0].x);
                x[u][1] = __fmaf_rn(alpha, bf16_hi(gv[u].x), ev[u][0].y);
                x[u][2] = __fmaf_rn(alpha, bf16_lo(gv[u].y), ev[u][0].z);
                x[u][3] = __fmaf_rn(alpha, bf16_hi(gv[u].y), ev[u][0].w);
                x[u][4] = __fmaf_rn(alpha, bf16_lo(gv[u].z), ev[u][1].x);
                x[u][5] = __fmaf_rn(alpha, bf16_hi(gv[u].z), ev[u][1].y);
                x[u][6] = __fmaf_rn(alpha, bf16_lo(gv[u].w), ev[u][1].z);
                x[u][7] = __fmaf_rn(alpha, bf16_hi(gv[u].w), ev[u][1].w);
            }
        }
    } else {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint64_t j = wbase + u * (32 * V) + lane * V;
#pragma unroll
            for (int c = 0; c < V; ++c) {
                const float ej = erow[j + c];                     // padding of e is in bounds
                x[u][c] = (j + c < d) ? __fmaf_rn(alpha, load_g<GT>(grow, j + c), ej) : ej;
            }
        }
    }
    // zero_mask: per round, the entries to write as +0 instead of their value
    auto store_tile = [&](const uint32_t *zero_mask) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint64_t j = wbase + u * (32 * V) + lane * V;
            float y[V];
#pragma unroll
            for (int c = 0; c < V; ++c)
                y[c] = (zero_mask && (zero_mask[u] & (1u << c))) ? 0.0f : x[u][c];
#pragma unroll
            for (int q = 0; q < V / 4; ++q)
                *reinterpret_cast<float4 *>(erow + j + 4 * q) =
                    make_float4(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
        }
    };
    if (!SPEC) {
        store_tile(nullptr);
        return;
    }

    // Stage every entry whose key reaches the speculative bound, in index order, into a
    // segment reserved with one atomic per tile.  Staged entries are written to e as +0 (the
    // guess is that they are selected); the selection kernels write the value back for the
    // few that are not.  The store is issued before any barrier; a tile whose segment turns
    // out not to fit stores its values again.  With BAND the staged entries below the
    // certainty bound (the band: only among them can the threshold lie) are written once more,
    // in any order, to the band list, which is then all the selection kernels have to read.
    __shared__ uint32_t s_w[WARPS], s_b[WARPS];
    __shared__ uint32_t s_off, s_boff;
    const uint32_t bound = sel[i].spec_key;
    const uint32_t cert = BAND ? sel[i].cert_key : SPEC_DISABLED;
    // m[u]: bit c = entry c of round u is staged, bit 8 + c = and lies in the band
    uint32_t m[U], pos[U], any = 0, nb = 0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint64_t j = wbase + u * (32 * V) + lane * V;
        m[u] = 0;
        uint32_t keys[V];
        if (RANDK) {
#pragma unroll
            for (int q = 0; q < V / 4; ++q) {
                const uint4 r4 = rand_keys4(rk, i, (j >> 2) + q);
                keys[4 * q] = r4.x; keys[4 * q + 1] = r4.y; keys[4 * q + 2] = r4.z; keys[4 * q + 3] = r4.w;
            }
        } else {
#pragma unroll
            for (int c = 0; c < V; ++c) keys[c] = mag_key(x[u][c]);
        }
#pragma unroll
        for (int c = 0; c < V; ++c)
            if (keys[c] >= bound && (full || j + c < d))
                m[u] |= ((BAND && keys[c] < cert) ? 0x101u : 0x1u) << c;
        if (BAND) nb += __popc(m[u] >> 8);
        any |= m[u];
    }
    store_tile(m);
    uint32_t total = 0, band_total = 0, bpos = 0;
    if (__syncthreads_or(any != 0)) {
        if (BAND) {
            ordered_prefix2<U>(m, pos, nb, bpos, s_w, s_b, total, band_total);
        } else {
            uint32_t cnt[U];
#pragma unroll
            for (int u = 0; u < U; ++u) cnt[u] = __popc(m[u]);
            ordered_prefix<U>(cnt, pos, s_w, total);
        }
    }
    if (threadIdx.x == 0) {
        uint32_t off = 0, boff = 0;
        if (total) {
            if (BAND) {
                const unsigned long long old = atomicAdd(
                    &sel[i].staged_band, static_cast<unsigned long long>(total) |
                                             (static_cast<unsigned long long>(band_total) << 32));
                off = static_cast<uint32_t>(old);
                boff = static_cast<uint32_t>(old >> 32);
            } else {
                // the low word alone (little-endian): the candidate count
                off = atomicAdd(reinterpret_cast<uint32_t *>(&sel[i].staged_band), total);
            }
        }
        tile_off[static_cast<size_t>(i) * ntiles + tile] = off;
        tile_cnt[static_cast<size_t>(i) * ntiles + tile] = total;
        tile_rej[static_cast<size_t>(i) * ntiles + tile] = 0;
        tile_eq[static_cast<size_t>(i) * ntiles + tile] = 0;
        s_off = off;
        if (BAND) s_boff = boff;
    }
    if (total == 0) return;
    __syncthreads();
    const uint64_t off = s_off;
    if (off + total > stage_cap) {                   // overflow: the counts tell the selector,
        store_tile(nullptr);                         // and this tile takes its values back
        return;
    }
    // band entries are a subset of the staged ones and both offsets grow in the same atomic,
    // so the band segment fits whenever the staged segment does
    deco_pair *out = stage + static_cast<size_t>(i) * stage_cap + off;
    deco_pair *bout = BAND ? band + static_cast<size_t>(i) * stage_cap + s_boff + bpos : nullptr;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint64_t j = wbase + u * (32 * V) + lane * V;
        uint32_t q = pos[u];
#pragma unroll
        for (int c = 0; c < V; ++c)
            if (m[u] & (1u << c)) {
                deco_pair pr;
                pr.idx = static_cast<uint32_t>(j + c);
                pr.val = x[u][c];
                out[q++] = pr;
                if (BAND && (m[u] & (0x100u << c))) *bout++ = pr;
            }
    }
}

template <int GT, bool ALIGNED, bool SPEC, bool RANDK>
__global__ void __launch_bounds__(BLOCK)
ef_accumulate_kernel(float *__restrict__ e, uint64_t e_stride, const void *__restrict__ grads,
                     uint64_t d, uint64_t g_stride, float alpha, RandParams rk, SelectState *__restrict__ sel,
                     deco_pair *__restrict__ stage, uint64_t stage_cap,
                     uint32_t *__restrict__ tile_off, uint32_t *__restrict__ tile_cnt,
                     uint32_t *__restrict__ tile_rej, uint32_t *__restrict__ tile_eq,
                     uint32_t ntiles)
{
    ef_accumulate_body<GT, ALIGNED, SPEC, RANDK, false>(blockIdx.x, blockIdx.y, true, e, e_stride, grads, d,
                                                        g_stride, alpha, rk, sel, stage, nullptr, stage_cap, tile_off,
                                                        tile_cnt, tile_rej, tile_eq, ntiles);
}

// The same with the band list.  Left to itself the compiler takes more than 85 registers for
// it, which would cost the third CTA per SM: the limit is forced here (and only here: forcing
// it on the kernel above, which needs 80 by itself, makes that one slower).
template <int GT, bool ALIGNED, bool RANDK>
__global__ void __launch_bounds__(BLOCK, 3)
ef_accumulate_band_kernel(float *__restrict__ e, uint64_t e_stride, const void *__restrict__ grads,
                          uint64_t d, uint64_t g_stride, float alpha, RandParams rk, SelectState *__restrict__ sel,
                          deco_pair *__restrict__ stage, deco_pair *__restrict__ band, uint64_t stage_cap,
                          uint32_t *__restrict__ tile_off, uint32_t *__restrict__ tile_cnt,
                          uint32_t *__restrict__ tile_rej, uint32_t *__restrict__ tile_eq,
                          uint32_t ntiles)
{
    ef_accumulate_body<GT, ALIGNED, true, RANDK, true>(blockIdx.x, blockIdx.y, true, e, e_stride, grads, d,
                                                       g_stride, alpha, rk, sel, stage, band, stage_cap, tile_off,
                                                       tile_cnt, tile_rej, tile_eq, ntiles);
}

// ------------------------------------------------------------------------------------------
// Streaming route: exact selection among the staged pairs.
// ------------------------------------------------------------------------------------------
// Staged keys are at or above spec_key, and the threshold sits just above it, so the two
// radix levels work on  rel = key - spec_key : level A bins rel >> shift (everything from
// 4095 << shift up, i.e. half an octave to two octaves above the bound, shares the top bin),
// level B bins the low `shift` bits inside the chosen A bin.
constexpr uint32_t REL_TOP = RADIX_BINS - 1;

// The width of a level-A bin is 2^shift key units with shift = sel[i].rel_shift in 10..12,
// chosen with the bound: the further the sampled rank had to be pushed above k/d (small k),
// the further above the bound the threshold may lie, and the wider the bins.
__device__ __forceinline__ uint32_t rel_bin_a(uint32_t key, uint32_t spec, uint32_t shift)
{
    const uint32_t b = (key - spec) >> shift;
    return b < REL_TOP ? b : REL_TOP;
}

__device__ void scan_tiles_body(const Sel &p, uint32_t i, uint32_t *s_w, bool streaming);

// Emit works on slices: EMIT_SLICE consecutive staged entries of one tile.  A tile with at most
// EMIT_LANE_MAX staged entries is walked by a single lane; every other tile is cut into slices
// that are listed (in no particular order) in a per-worker work list, so that a layer whose
// tiles hold thousands of candidates is spread over as many warps as it has slices.
constexpr uint32_t EMIT_SLICE = 256;
constexpr uint32_t EMIT_LANE_MAX = 16;

// whole_tiles: with dense messages every tile holds hundreds of staged entries and there are
// tiles enough to fill the machine: one warp walks the whole tile (no slice is read twice).
__device__ __forceinline__ uint32_t emit_items_of(uint32_t cnt, bool whole_tiles)
{
    return cnt > EMIT_LANE_MAX ? (whole_tiles ? 1u : (cnt + EMIT_SLICE - 1) / EMIT_SLICE) : 0u;
}

// Work list of a worker: one (tile, slice) entry per slice; every thread looks at one tile, a
// warp reserves its entries with one atomic.  Called by all threads of the `nctas` CTAs that a
// kernel between the streaming pass and emit has for the worker.
__device__ __forceinline__ void build_emit_work(const Sel &p, uint32_t i, const uint32_t cta, const uint32_t nctas)
{
    const int lane = threadIdx.x & 31;
    uint32_t *count = &p.done[i * DONE_SLOTS + 5];
    uint2 *work = p.work + static_cast<size_t>(i) * p.work_cap;
    const uint32_t tiles_up = (p.ntiles + 31u) & ~31u;       // whole warps stay together
    for (uint32_t tile = cta * BLOCK + threadIdx.x; tile < tiles_up; tile += nctas * BLOCK) {
        const uint32_t items =
            tile < p.ntiles ? emit_items_of(p.tile_cnt[static_cast<size_t>(i) * p.ntiles + tile], p.use_band != 0) : 0u;
        const uint32_t incl = warp_incl_scan(items);
        const uint32_t total = __shfl_sync(FULL, incl, 31);
        if (total == 0) continue;
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(count, total);
        base = __shfl_sync(FULL, base, 0) + incl - items;
        if (base + items > p.work_cap) {
            if (items) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x320u, tile);
            continue;
        }
        for (uint32_t j = 0; j < items; ++j) work[base + j] = make_uint2(tile, j);
    }
}


// Shared memory of the selection bodies: one radix histogram and a few words.
struct SelectShared {
    uint32_t h[RADIX_BINS];
    uint32_t scan[33];
    uint32_t misc[3];
    uint32_t warp[WARPS];
    uint32_t out[2];
};
// One instance per kernel that runs any of the bodies (a variable of namespace scope, so that
// every access is known to be a shared-memory access).
__shared__ SelectShared sm;

// Level A: histogram of the coarse bins of the band keys.  The last CTA of a worker to
// arrive takes the decision: is the staged set usable (at least k candidates, so it contains
// the k largest; no overflow of the staging area; fewer than k of them at or above the
// certainty bound, so the threshold lies in the band), and which coarse bin holds the entry of
// rank k - (candidates above the band).  If the set is not usable, or the threshold falls into
// the shared top bin, the worker is handed to the multi-pass route.
template <bool COH>
__device__ __forceinline__ void stage_hist_a_body(const Sel &p, const uint32_t i, const uint32_t cta,
                                                  const uint32_t nctas)
{
    SelectState &s = p.sel[i];
    if (ldq<COH>(&s.exact)) return;
    uint32_t n_staged, n_band;
    staged_counts<COH>(s, n_staged, n_band);
    const deco_pair *src = select_list(p, i, n_staged, n_band);
    const uint32_t n_cert = n_staged - n_band;
    const uint32_t spec = ldq<COH>(&s.spec_key), shift = ldq<COH>(&s.rel_shift);
    const bool valid = n_staged >= p.k && n_staged <= p.stage_cap && n_cert < p.k;
    uint32_t *h = sm.h;
    if (valid) {
        for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK) h[b] = 0;
        __syncthreads();
        for (uint32_t base = cta * (4 * BLOCK); base < n_band;
             base += nctas * (4 * BLOCK)) {
            deco_pair v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint32_t q = base + r * BLOCK + threadIdx.x;
                v[r].idx = 0;
                v[r].val = 0.0f;
                if (q < n_band) v[r] = src[q];
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
                if (base + r * BLOCK + threadIdx.x < n_band)
                    atomicAdd(&h[rel_bin_a(key_of(p, i, v[r]), spec, shift)], 1u);
        }
        __syncthreads();
        uint32_t *out = hist_of(p, i, 0, 0);
        for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK)
            if (h[b]) atomicAdd(&out[b], h[b]);
    }
    if (!last_cta_to_arrive(&p.done[i * DONE_SLOTS + 0], &sm.misc[2], nctas)) return;
    uint32_t a_sel = REL_TOP, above_a = 0;
    if (valid) pick_bin(hist_of(p, i, 0, 0), p.k - n_cert, sm.scan, sm.misc, a_sel, above_a);
    if (threadIdx.x == 0) {
        if (!valid || a_sel >= REL_TOP) {
            s.exact = 1;
            s.exact_total += 1;
            p.status[3] = 1;
        } else {
            s.prefix = a_sel;
            s.n_greater = n_cert + above_a;
            s.k_rem = p.k - n_cert - above_a;
        }
    }
}

__global__ void __launch_bounds__(BLOCK) stage_hist_a_kernel(Sel p)
{
    stage_hist_a_body<false>(p, blockIdx.y, blockIdx.x, gridDim.x);
}

// Level B: histogram of the low bits of the band keys that fell into the chosen A bin; the
// last CTA of a worker to arrive fixes the threshold key and the number of ties to take.
template <bool COH>
__device__ __forceinline__ void stage_hist_b_body(const Sel &p, const uint32_t i, const uint32_t cta,
                                                  const uint32_t nctas)
{
    SelectState &s = p.sel[i];
    if (ldq<COH>(&s.exact)) return;
    uint32_t *h = sm.h;
    uint32_t n_staged, n_band;
    staged_counts<COH>(s, n_staged, n_band);
    const uint32_t spec = ldq<COH>(&s.spec_key), shift = ldq<COH>(&s.rel_shift);
    const uint32_t a_sel = ldq<COH>(&s.prefix), above_a = ldq<COH>(&s.n_greater),
                   k_rem = ldq<COH>(&s.k_rem);                         // from level A
    const uint32_t low_mask = (1u << shift) - 1u;
    const deco_pair *src = select_list(p, i, n_staged, n_band);
    for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK) h[b] = 0;
    build_emit_work(p, i, cta, nctas);                  // independent of the histogram
    __syncthreads();
    for (uint32_t base = cta * (4 * BLOCK); base < n_band;
         base += nctas * (4 * BLOCK)) {
        deco_pair v[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint32_t q = base + r * BLOCK + threadIdx.x;
            v[r].idx = 0;
            v[r].val = 0.0f;
            if (q < n_band) v[r] = src[q];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            if (base + r * BLOCK + threadIdx.x >= n_band) continue;
            const uint32_t key = key_of(p, i, v[r]);
            if (rel_bin_a(key, spec, shift) == a_sel) atomicAdd(&h[(key - spec) & low_mask], 1u);
        }
    }
    __syncthreads();
    uint32_t *out = hist_of(p, i, 0, 1);
    for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK)
        if (h[b]) atomicAdd(&out[b], h[b]);
    if (!last_cta_to_arrive(&p.done[i * DONE_SLOTS + 1], &sm.misc[2], nctas)) return;
    uint32_t bin, above;
    pick_bin(hist_of(p, i, 0, 1), k_rem, sm.scan, sm.misc, bin, above);
    if (threadIdx.x == 0) {
        if (bin == 0xFFFFFFFFu) {                   // counts do not add up: report, stay safe
            latch(p.status, DECO_ERR_DEVICE_CHECK, 0x120u, i);
            s.threshold = 0x7FFFFFFFu;
            s.ties_take = 0;
        } else {
            s.prefix = (a_sel << shift) | bin;
            s.k_rem = k_rem - above;
            s.threshold = spec + (a_sel << shift) + bin;
            s.n_greater = above_a + above;
            s.ties_take = k_rem - above;
        }
    }
}

__global__ void __launch_bounds__(BLOCK) stage_hist_b_kernel(Sel p)
{
    stage_hist_b_body<false>(p, blockIdx.y, blockIdx.x, gridDim.x);
}

// One CTA: ties are granted to chunks in index order until ties_take are used up, then every
// chunk gets its position in the message.  Per thread a contiguous range of chunks.  The sums
// of a chunk are taken here from its CHUNK_TILES tile counters (few chunks).
__device__ void chunk_walk(const Sel &p, uint32_t i, uint32_t *s_scan /*[33]*/)
{
    uint32_t *ccnt = p.chunk_cnt + static_cast<size_t>(i) * p.nchunks;
    uint32_t *crej = p.chunk_rej + static_cast<size_t>(i) * p.nchunks;
    uint32_t *ceq = p.chunk_eq + static_cast<size_t>(i) * p.nchunks;
    uint32_t *cstart = p.chunk_start + static_cast<size_t>(i) * (p.nchunks + 1);
    uint32_t *ceqb = p.chunk_eqb + static_cast<size_t>(i) * p.nchunks;
    const uint32_t *tcnt = p.tile_cnt + static_cast<size_t>(i) * p.ntiles;
    const uint32_t *rej = p.tile_rej + static_cast<size_t>(i) * p.ntiles;
    const uint32_t *eqc = p.tile_eq + static_cast<size_t>(i) * p.ntiles;
    const uint32_t ties = p.sel[i].ties_take;
    const uint32_t per = (p.nchunks + blockDim.x - 1) / blockDim.x;
    const uint32_t lo = min(p.nchunks, threadIdx.x * per), hi = min(p.nchunks, lo + per);
    uint32_t eq_sum = 0;
    for (uint32_t c = lo; c < hi; ++c) {
        uint32_t a = 0, b = 0, q = 0;
        const uint32_t t0 = c * CHUNK_TILES, t1 = min(p.ntiles, t0 + CHUNK_TILES);
        for (uint32_t t = t0; t < t1; ++t) {
            a += tcnt[t];
            b += __ldcg(&rej[t]);
            q += __ldcg(&eqc[t]);
        }
        ccnt[c] = a;
        crej[c] = b;
        ceq[c] = q;
        eq_sum += q;
    }
    uint32_t eq_total;
    uint32_t eq_before = block_excl_scan(eq_sum, s_scan, eq_total);
    uint32_t sel_sum = 0;
    for (uint32_t c = lo; c < hi; ++c) {
        const uint32_t q = __ldcg(&ceq[c]);
        const uint32_t left = ties > eq_before ? ties - eq_before : 0u;
        ceqb[c] = eq_before;
        sel_sum += __ldcg(&ccnt[c]) - __ldcg(&crej[c]) - q + min(q, left);
        eq_before += q;
    }
    uint32_t sel_total;
    uint32_t pos = block_excl_scan(sel_sum, s_scan, sel_total);
    for (uint32_t c = lo; c < hi; ++c) {
        const uint32_t q = __ldcg(&ceq[c]);
        const uint32_t eb = ceqb[c];
        const uint32_t left = ties > eb ? ties - eb : 0u;
        cstart[c] = pos;
        pos += __ldcg(&ccnt[c]) - __ldcg(&crej[c]) - q + min(q, left);
    }
    if (threadIdx.x == 0) {
        cstart[p.nchunks] = sel_total;
        if (sel_total != p.k) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x200u, i);
    }
    __syncthreads();
}

// The same walk over many chunks whose sums chunk_sums_kernel left in chunk_cnt/rej/eq: the
// sums go through shared memory (sm.h, free in that kernel) in segments of WALK_SEG chunks,
// fetched with coalesced loads in one round trip; a thread then owns WALK_PER consecutive
// chunks of the segment, and the two running totals carry over from segment to segment.
constexpr uint32_t WALK_PER = 8;
constexpr uint32_t WALK_SEG = WALK_PER * BLOCK;
static_assert(2 * WALK_SEG <= RADIX_BINS, "two words per chunk of a segment in sm.h");

__device__ void chunk_walk_sums(const Sel &p, uint32_t i, uint32_t *s_scan /*[33]*/)
{
    const uint32_t *ccnt = p.chunk_cnt + static_cast<size_t>(i) * p.nchunks;
    const uint32_t *crej = p.chunk_rej + static_cast<size_t>(i) * p.nchunks;
    const uint32_t *ceq = p.chunk_eq + static_cast<size_t>(i) * p.nchunks;
    uint32_t *cstart = p.chunk_start + static_cast<size_t>(i) * (p.nchunks + 1);
    uint32_t *ceqb = p.chunk_eqb + static_cast<size_t>(i) * p.nchunks;
    const uint32_t ties = p.sel[i].ties_take;
    uint32_t *s_q = sm.h, *s_sel = sm.h + WALK_SEG;          // ties / entries surely selected, per chunk
    uint32_t eq_carry = 0, pos_carry = 0;
    for (uint32_t seg = 0; seg < p.nchunks; seg += WALK_SEG) {
        const uint32_t m = min(WALK_SEG, p.nchunks - seg);
        for (uint32_t c = threadIdx.x; c < WALK_SEG; c += BLOCK) {
            uint32_t q = 0, surely = 0;
            if (c < m) {
                q = __ldcg(&ceq[seg + c]);
                surely = __ldcg(&ccnt[seg + c]) - __ldcg(&crej[seg + c]) - q;
            }
            s_q[c] = q;
            s_sel[c] = surely;
        }
        __syncthreads();
        const uint32_t lo = threadIdx.x * WALK_PER;
        uint32_t eq_sum = 0;
#pragma unroll
        for (uint32_t j = 0; j < WALK_PER; ++j) eq_sum += s_q[lo + j];
        uint32_t eq_total;
        uint32_t eq_before = eq_carry + block_excl_scan(eq_sum, s_scan, eq_total);
        uint32_t sel_sum = 0;
#pragma unroll
        for (uint32_t j = 0; j < WALK_PER; ++j) {
            const uint32_t q = s_q[lo + j];
            const uint32_t left = ties > eq_before ? ties - eq_before : 0u;
            if (lo + j < m) ceqb[seg + lo + j] = eq_before;
            const uint32_t take = s_sel[lo + j] + min(q, left);
            s_sel[lo + j] = take;                            // own words only
            sel_sum += take;
            eq_before += q;
        }
        uint32_t sel_total;
        uint32_t pos = pos_carry + block_excl_scan(sel_sum, s_scan, sel_total);
#pragma unroll
        for (uint32_t j = 0; j < WALK_PER; ++j) {
            if (lo + j < m) cstart[seg + lo + j] = pos;
            pos += s_sel[lo + j];
        }
        eq_carry += eq_total;
        pos_carry += sel_total;
        __syncthreads();                                     // sm.h is refilled by the next segment
    }
    if (threadIdx.x == 0) {
        cstart[p.nchunks] = pos_carry;
        if (pos_carry != p.k) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x200u, i);
    }
    __syncthreads();
}

// Many chunks: their sums are taken in parallel, one warp per chunk (three coalesced loads
// and a warp reduction; the CTAs stride over the chunks), and the last CTA of a worker to
// arrive walks the chunks.
__device__ __forceinline__ void chunk_sums_body(const Sel &p, const uint32_t i, const uint32_t cta,
                                                const uint32_t nctas)
{
    if (p.sel[i].exact) return;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (uint32_t chunk = cta * WARPS + w; chunk < p.nchunks; chunk += nctas * WARPS) {
        const uint32_t tile = chunk * CHUNK_TILES + lane;
        const size_t ti = static_cast<size_t>(i) * p.ntiles + tile;
        uint32_t a = 0, b = 0, q = 0;
        if (tile < p.ntiles) {
            a = p.tile_cnt[ti];
            b = p.tile_rej[ti];
            q = p.tile_eq[ti];
        }
        for (int o = 16; o > 0; o >>= 1) {
            a += __shfl_down_sync(FULL, a, o);
            b += __shfl_down_sync(FULL, b, o);
            q += __shfl_down_sync(FULL, q, o);
        }
        if (lane == 0) {
            p.chunk_cnt[static_cast<size_t>(i) * p.nchunks + chunk] = a;
            p.chunk_rej[static_cast<size_t>(i) * p.nchunks + chunk] = b;
            p.chunk_eq[static_cast<size_t>(i) * p.nchunks + chunk] = q;
        }
    }
    if (!last_cta_to_arrive(&p.done[i * DONE_SLOTS + 4], &sm.misc[2], nctas)) return;
    chunk_walk_sums(p, i, sm.scan);
}

__global__ void __launch_bounds__(BLOCK) chunk_sums_kernel(Sel p)
{
    chunk_sums_body(p, blockIdx.y, blockIdx.x, gridDim.x);
}

// Classification.  With the threshold known every band entry below it is rejected: counted
// for its tile; entries equal to it are counted as ties.  (The
// candidates above the band are above the threshold.)  With few chunks (walk_here) the last
// CTA of a worker to arrive then walks the chunks once; with many, the chunk sums follow.
// (The per-tile positions follow from these inside the emit step, so nothing here is serial
// in the number of tiles.)
template <bool COH>
__device__ __forceinline__ void stage_classify_body(const Sel &p, const uint32_t i, uint32_t walk_here,
                                                    const uint32_t cta, const uint32_t nctas)
{
    const SelectState &s = p.sel[i];
    if (ldq<COH>(&s.exact)) return;
    uint32_t n_staged, n_band;
    staged_counts<COH>(s, n_staged, n_band);
    const uint32_t T = ldq<COH>(&s.threshold);
    const deco_pair *src = select_list(p, i, n_staged, n_band);
    uint32_t *rej = p.tile_rej + static_cast<size_t>(i) * p.ntiles;
    uint32_t *eqc = p.tile_eq + static_cast<size_t>(i) * p.ntiles;
    const int lane = threadIdx.x & 31;
    for (uint32_t base = cta * (4 * BLOCK); base < n_band;
         base += nctas * (4 * BLOCK)) {
        deco_pair prs[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint32_t q = base + r * BLOCK + threadIdx.x;
            prs[r].idx = 0;
            prs[r].val = __uint_as_float(0x7FFFFFFFu);       // above any threshold: no action
            if (q < n_band) prs[r] = src[q];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            // neighbours in the band list mostly belong to the same tile: lanes with the
            // same (tile, class) elect one of them to add the group's size
            const bool in = base + r * BLOCK + threadIdx.x < n_band;
            const uint32_t key = in ? key_of(p, i, prs[r]) : 0x7FFFFFFFu;
            const uint32_t tile = prs[r].idx / TILE;
            const uint32_t cls = !in ? 0u : (key < T ? 1u : (key == T ? 2u : 0u));
            const uint32_t grp = __match_any_sync(FULL, cls ? (tile * 2 + cls - 1) : 0xFFFFFFFFu);
            if (cls && lane == __ffs(grp) - 1)
                atomicAdd(cls == 1 ? &rej[tile] : &eqc[tile], static_cast<uint32_t>(__popc(grp)));
        }
    }
    // (the rejected entries get their value back in e from emit, which reads every staged pair anyway)
    if (!last_cta_to_arrive(&p.done[i * DONE_SLOTS + 2], &sm.misc[2], nctas)) return;
    if (walk_here) chunk_walk(p, i, sm.scan);
}

__global__ void __launch_bounds__(BLOCK) stage_classify_kernel(Sel p, uint32_t walk_here)
{
    stage_classify_body<false>(p, blockIdx.y, walk_here, blockIdx.x, gridDim.x);
}

// What a warp learns about the CHUNK_TILES tiles of one chunk from three coalesced loads and
// two warp scans: lane l holds tile chunk*32 + l.
struct TileInfo {
    uint32_t cnt;     // staged entries of the tile
    uint32_t take;    // ties of the tile that are taken
    uint32_t sel;     // entries of the tile that go into the message
    uint32_t start;   // message position of the tile's first entry
};

template <bool WRITE_DIR, bool COH>
__device__ __forceinline__ TileInfo chunk_header(const Sel &p, uint32_t i, uint32_t chunk)
{
    const int lane = threadIdx.x & 31;
    const uint32_t tile = chunk * CHUNK_TILES + lane;
    const size_t ti = static_cast<size_t>(i) * p.ntiles + tile;
    uint32_t cnt = 0, rej = 0, eq = 0;
    if (tile < p.ntiles) {
        cnt = p.tile_cnt[ti];
        rej = ldq<COH>(&p.tile_rej[ti]);
        eq = ldq<COH>(&p.tile_eq[ti]);
    }
    const size_t cb = static_cast<size_t>(i) * p.nchunks + chunk, cs = static_cast<size_t>(i) * (p.nchunks + 1) + chunk;
    const uint32_t ties = ldq<COH>(&p.sel[i].ties_take);
    const uint32_t eqb0 = ldq<COH>(&p.chunk_eqb[cb]);
    const uint32_t start0 = ldq<COH>(&p.chunk_start[cs]);
    const uint32_t eq_before = eqb0 + warp_incl_scan(eq) - eq;
    const uint32_t left = ties > eq_before ? ties - eq_before : 0u;
    TileInfo t;
    t.cnt = cnt;
    t.take = min(eq, left);
    t.sel = cnt - rej - eq + t.take;
    t.start = start0 + warp_incl_scan(t.sel) - t.sel;
    if (WRITE_DIR) {
        // the directory the aggregation reads: message position of every tile
        if (tile < p.ntiles) p.tile_start[static_cast<size_t>(i) * p.dir_stride + tile] = t.start;
        if (tile == p.ntiles - 1)
            p.tile_start[static_cast<size_t>(i) * p.dir_stride + p.ntiles] = t.start + t.sel;
    }
    return t;
}

// The whole warp filters staged entries [begin, end) of one tile's segment, in order, into the
// message; `written` entries of the tile were emitted and `ties_seen` ties met before `begin`.
// The selected entries are already +0 in e; the others (below the threshold, or ties that are not
// taken) get their value back: the +0 guess of the streaming pass is undone here.
// Returns the number of entries written.
__device__ __forceinline__ uint32_t emit_segment_warp(const Sel &p, uint32_t i, uint32_t tile,
                                                      uint32_t off, uint32_t begin, uint32_t end,
                                                      uint32_t start, uint32_t written,
                                                      uint32_t ties_seen, uint32_t take, uint32_t T)
{
    const int lane = threadIdx.x & 31;
    const deco_pair *src = p.stage + static_cast<size_t>(i) * p.stage_cap + off;
    deco_pair *out = p.msg + static_cast<size_t>(i) * p.k_cap;
    float *erow = p.e + static_cast<size_t>(i) * p.e_stride;
    for (uint32_t base = begin; base < end; base += 128) {     // four loads in flight per lane
        deco_pair prs[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint32_t q = base + r * 32 + lane;
            prs[r].idx = 0;
            prs[r].val = 0.f;
            if (q < end) prs[r] = src[q];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const deco_pair pr = prs[r];
            bool gt = false, eq = false;
            const bool in = base + r * 32 + lane < end;
            if (in) {
                const uint32_t key = key_of(p, i, pr);
                gt = key > T;
                eq = key == T;
            }
            const uint32_t eq_mask = __ballot_sync(FULL, eq);
            const uint32_t rank = ties_seen + __popc(eq_mask & ((1u << lane) - 1u));
            const bool pick = gt || (eq && rank < take);
            const uint32_t pick_mask = __ballot_sync(FULL, pick);
            if (pick) {
                const uint32_t pos = start + written + __popc(pick_mask & ((1u << lane) - 1u));
                if (pos < p.k && pr.idx < p.d) {
                    out[pos] = pr;                           // e already holds +0 there
                } else {
                    latch(p.status, DECO_ERR_DEVICE_CHECK, 0x310u, tile);
                }
            }
            if (in && !pick && pr.idx < p.d) erow[pr.idx] = pr.val;   // not selected: undo the guess
            written += __popc(pick_mask);
            ties_seen += __popc(eq_mask);
        }
    }
    return written;
}

// Emit, directory part: CTA `cta` of `nctas`; a warp per chunk of CHUNK_TILES tiles (the CTAs
// stride over the chunks) writes the directory and each lane walks its own tile if that holds
// at most EMIT_LANE_MAX staged entries.
template <bool COH>
__device__ __forceinline__ void emit_directory_part(const Sel &p, const uint32_t i, uint32_t cta, uint32_t nctas)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t T = ldq<COH>(&p.sel[i].threshold);
    for (uint32_t chunk = cta * WARPS + w; chunk < p.nchunks; chunk += nctas * WARPS) {
        const TileInfo t = chunk_header<true, COH>(p, i, chunk);
        const uint32_t tile = chunk * CHUNK_TILES + lane;
        if (t.cnt == 0 || t.cnt > EMIT_LANE_MAX) continue;
        const uint32_t off = p.tile_off[static_cast<size_t>(i) * p.ntiles + tile];
        const deco_pair *src = p.stage + static_cast<size_t>(i) * p.stage_cap + off;
        deco_pair *out = p.msg + static_cast<size_t>(i) * p.k_cap;
        float *erow = p.e + static_cast<size_t>(i) * p.e_stride;
        uint32_t written = 0, ties_seen = 0;
        for (uint32_t q = 0; q < t.cnt; ++q) {
            const deco_pair pr = src[q];
            const uint32_t key = key_of(p, i, pr);
            const bool eq = key == T;
            const bool pick = key > T || (eq && ties_seen < t.take);
            ties_seen += eq ? 1u : 0u;
            if (pick) {
                const uint32_t pos = t.start + written++;
                if (pos < p.k && pr.idx < p.d) out[pos] = pr;
                else latch(p.status, DECO_ERR_DEVICE_CHECK, 0x312u, tile);
            } else if (pr.idx < p.d) {
                erow[pr.idx] = pr.val;                       // not selected: undo the guess
            }
        }
        if (written != t.sel) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x313u, tile);
    }
}

// Emit, work-list part: the warps of CTA `cta` of `nctas` stride over the work list; a warp
// that gets slice j > 0 of a tile first counts, with independent loads, what the slices before
// it emit.
template <bool COH>
__device__ __forceinline__ void emit_items_part(const Sel &p, const uint32_t i, uint32_t cta, uint32_t nctas)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t T = ldq<COH>(&p.sel[i].threshold);
    const uint32_t n_items = min(ldq<COH>(&p.done[i * DONE_SLOTS + 5]), static_cast<uint32_t>(p.work_cap));
    const uint2 *work = p.work + static_cast<size_t>(i) * p.work_cap;
    const uint32_t warps = nctas * WARPS;
    for (uint32_t q = cta * WARPS + w; q < n_items; q += warps) {
        const uint2 item = work[q];
        const uint32_t tile = item.x, slice = item.y;
        if (tile >= p.ntiles) {
            if (lane == 0) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x321u, q);
            continue;
        }
        const TileInfo t = chunk_header<false, COH>(p, i, tile / CHUNK_TILES);
        const uint32_t my = tile % CHUNK_TILES;
        const uint32_t cnt = __shfl_sync(FULL, t.cnt, my), start = __shfl_sync(FULL, t.start, my);
        const uint32_t want = __shfl_sync(FULL, t.sel, my), take = __shfl_sync(FULL, t.take, my);
        const uint32_t off = p.tile_off[static_cast<size_t>(i) * p.ntiles + tile];
        const uint32_t slice_len = p.use_band ? static_cast<uint32_t>(TILE) : EMIT_SLICE;
        const uint32_t begin = slice * slice_len;
        if (begin >= cnt) {
            if (lane == 0) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x322u, tile);
            continue;
        }
        const uint32_t end = min(cnt, begin + slice_len);
        uint32_t written = 0, ties_seen = 0;
        if (begin) {
            // what slices 0..slice-1 emit: the entries above the threshold plus the ties
            // that are still granted; whole slices, so every load is in range
            const deco_pair *src = p.stage + static_cast<size_t>(i) * p.stage_cap + off;
            uint32_t g = 0, e = 0;
            for (uint32_t base = 0; base < begin; base += EMIT_SLICE) {
                deco_pair prs[EMIT_SLICE / 32];
#pragma unroll
                for (uint32_t r = 0; r < EMIT_SLICE / 32; ++r) prs[r] = src[base + r * 32 + lane];
#pragma unroll
                for (uint32_t r = 0; r < EMIT_SLICE / 32; ++r) {
                    const uint32_t key = key_of(p, i, prs[r]);
                    g += key > T ? 1u : 0u;
                    e += key == T ? 1u : 0u;
                }
            }
            for (int o = 16; o > 0; o >>= 1) {
                g += __shfl_xor_sync(FULL, g, o);
                e += __shfl_xor_sync(FULL, e, o);
            }
            written = g + min(e, take);
            ties_seen = e;
        }
        written = emit_segment_warp(p, i, tile, off, begin, end, start, written, ties_seen, take, T);
        if (end == cnt && lane == 0 && written != want)
            latch(p.status, DECO_ERR_DEVICE_CHECK, 0x311u, tile);
    }
}

// Emit as a launch of its own: CTAs [0, dir_ctas) of a worker do the directory part, the
// remaining CTAs the work list.
__device__ __forceinline__ void emit_stage_body(const Sel &p, const uint32_t i, const uint32_t cta,
                                                const uint32_t nctas, uint32_t dir_ctas)
{
    if (p.sel[i].exact) return;
    if (cta < dir_ctas) emit_directory_part<false>(p, i, cta, dir_ctas);
    else emit_items_part<false>(p, i, cta - dir_ctas, nctas - dir_ctas);
}

__global__ void __launch_bounds__(BLOCK) emit_stage_kernel(Sel p, uint32_t dir_ctas)
{
    emit_stage_body(p, blockIdx.y, blockIdx.x, gridDim.x, dir_ctas);
}

// ------------------------------------------------------------------------------------------
// Multi-pass route: bodies written for one CTA of BLOCK threads working on (worker, part).
// ------------------------------------------------------------------------------------------
template <int LEVEL>
__device__ __forceinline__ void hist_e_body(const Sel &p, uint32_t i, uint32_t part,
                                            uint32_t nparts, uint32_t *h)
{
    for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK) h[b] = 0;
    __syncthreads();
    const uint32_t prefix = p.sel[i].prefix;
    const float4 *row = reinterpret_cast<const float4 *>(p.e + static_cast<size_t>(i) * p.e_stride);
    const uint64_t nvec = (p.d + 3) >> 2;
    for (uint64_t v = static_cast<uint64_t>(part) * BLOCK + threadIdx.x; v < nvec;
         v += static_cast<uint64_t>(nparts) * BLOCK) {
        const uint64_t j = v << 2;
        uint4 kq;
        if (p.rk.on) {
            kq = rand_keys4(p.rk, i, v);
        } else {
            const float4 q = row[v];
            kq = make_uint4(mag_key(q.x), mag_key(q.y), mag_key(q.z), mag_key(q.w));
        }
        radix_bin<LEVEL>(kq.x, prefix, h);
        if (j + 1 < p.d) radix_bin<LEVEL>(kq.y, prefix, h);
        if (j + 2 < p.d) radix_bin<LEVEL>(kq.z, prefix, h);
        if (j + 3 < p.d) radix_bin<LEVEL>(kq.w, prefix, h);
    }
    __syncthreads();
    uint32_t *out = hist_of(p, i, 1, LEVEL);
    for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK)
        if (h[b]) atomicAdd(&out[b], h[b]);
    __syncthreads();
}

__device__ __forceinline__ void count_e_tile(const Sel &p, uint32_t i, uint32_t tile,
                                             uint32_t *s_a /*[WARPS]*/, uint32_t *s_b /*[WARPS]*/)
{
    const uint32_t T = p.sel[i].threshold;
    const float *row = p.e + static_cast<size_t>(i) * p.e_stride;
    const uint64_t base = static_cast<uint64_t>(tile) * TILE;
    uint32_t gt = 0, eq = 0;
#pragma unroll
    for (int r = 0; r < TILE / (4 * BLOCK); ++r) {
        const uint64_t j = base + (static_cast<uint64_t>(r) * BLOCK + threadIdx.x) * 4;
        uint4 kq;
        if (p.rk.on) {
            kq = rand_keys4(p.rk, i, j >> 2);
        } else {
            const float4 q = *reinterpret_cast<const float4 *>(row + j);
            kq = make_uint4(mag_key(q.x), mag_key(q.y), mag_key(q.z), mag_key(q.w));
        }
        const uint32_t ks[4] = {kq.x, kq.y, kq.z, kq.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t key = ks[c];
            const bool in = j + c < p.d;
            gt += (in && key > T);
            eq += (in && key == T);
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        gt += __shfl_down_sync(FULL, gt, o);
        eq += __shfl_down_sync(FULL, eq, o);
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) {
        s_a[w] = gt;
        s_b[w] = eq;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t a = 0, b = 0;
        for (int ww = 0; ww < WARPS; ++ww) {
            a += s_a[ww];
            b += s_b[ww];
        }
        p.tile_gt[static_cast<size_t>(i) * p.ntiles + tile] = a;
        p.tile_eq[static_cast<size_t>(i) * p.ntiles + tile] = b;
    }
    __syncthreads();
}

// One CTA per worker (any block size): ties are granted to tiles in index order until
// ties_take are used up, then every tile gets its position in the message.  On the streaming
// route the entries above the threshold of a tile are its staged entries minus the rejected
// ones and the ties; on the multi-pass route they were counted directly.
__device__ void scan_tiles_body(const Sel &p, uint32_t i, uint32_t *s_w /*[33]*/, bool streaming)
{
    const uint32_t nt = blockDim.x;
    const uint32_t *gtp = p.tile_gt + static_cast<size_t>(i) * p.ntiles;
    const uint32_t *cnt = p.tile_cnt + static_cast<size_t>(i) * p.ntiles;
    const uint32_t *rej = p.tile_rej + static_cast<size_t>(i) * p.ntiles;
    const uint32_t *eq = p.tile_eq + static_cast<size_t>(i) * p.ntiles;
    auto gt = [&](uint32_t t) { return streaming ? cnt[t] - rej[t] - eq[t] : gtp[t]; };
    uint32_t *take = p.tile_take + static_cast<size_t>(i) * p.ntiles;
    uint32_t *start = p.tile_start + static_cast<size_t>(i) * p.dir_stride;
    const uint32_t ties = p.sel[i].ties_take;
    const uint32_t per = (p.ntiles + nt - 1) / nt;
    const uint32_t lo = min(p.ntiles, threadIdx.x * per), hi = min(p.ntiles, lo + per);
    uint32_t sel_total;
    constexpr uint32_t REG = 8;
    if (per <= REG) {
        // short ranges: every load is issued once, up front
        uint32_t g[REG], q[REG];
#pragma unroll
        for (uint32_t r = 0; r < REG; ++r) {
            const uint32_t t = lo + r;
            g[r] = q[r] = 0;
            if (t < hi) {
                q[r] = eq[t];
                g[r] = gt(t);
            }
        }
        uint32_t eq_sum = 0;
#pragma unroll
        for (uint32_t r = 0; r < REG; ++r) eq_sum += q[r];
        uint32_t eq_total;
        uint32_t eq_before = block_excl_scan(eq_sum, s_w, eq_total);
        uint32_t sel_sum = 0;
#pragma unroll
        for (uint32_t r = 0; r < REG; ++r) {
            const uint32_t left = ties > eq_before ? ties - eq_before : 0u;
            const uint32_t tk = min(q[r], left);
            eq_before += q[r];
            q[r] = tk;
            sel_sum += g[r] + tk;
        }
        uint32_t pos = block_excl_scan(sel_sum, s_w, sel_total);
#pragma unroll
        for (uint32_t r = 0; r < REG; ++r) {
            const uint32_t t = lo + r;
            if (t < hi) {
                take[t] = q[r];
                start[t] = pos;
            }
            pos += g[r] + q[r];
        }
    } else {
        uint32_t eq_sum = 0;
        for (uint32_t t = lo; t < hi; ++t) eq_sum += eq[t];
        uint32_t eq_total;
        uint32_t eq_before = block_excl_scan(eq_sum, s_w, eq_total);
        uint32_t sel_sum = 0;
        for (uint32_t t = lo; t < hi; ++t) {
            const uint32_t q = eq[t];
            const uint32_t left = ties > eq_before ? ties - eq_before : 0u;
            const uint32_t tk = min(q, left);
            take[t] = tk;
            sel_sum += gt(t) + tk;
            eq_before += q;
        }
        uint32_t pos = block_excl_scan(sel_sum, s_w, sel_total);
        for (uint32_t t = lo; t < hi; ++t) {
            start[t] = pos;
            pos += gt(t) + take[t];
        }
    }
    if (threadIdx.x == 0) {
        start[p.ntiles] = sel_total;
        if (sel_total != p.k) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x200u, i);
    }
    __syncthreads();
}

__device__ __forceinline__ void emit_e_tile(const Sel &p, uint32_t i, uint32_t tile,
                                            uint32_t *s_w /*[WARPS]*/)
{
    constexpr int V = 4, U = WARP_ELEMS / (32 * V);
    const uint32_t start = p.tile_start[static_cast<size_t>(i) * p.dir_stride + tile];
    const uint32_t count = p.tile_start[static_cast<size_t>(i) * p.dir_stride + tile + 1] - start;
    if (count == 0) return;
    const uint32_t T = p.sel[i].threshold;
    const uint32_t take = p.tile_take[static_cast<size_t>(i) * p.ntiles + tile];
    const uint32_t n_eq = p.tile_eq[static_cast<size_t>(i) * p.ntiles + tile];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    float *erow = p.e + static_cast<size_t>(i) * p.e_stride;
    const uint64_t wbase = static_cast<uint64_t>(tile) * TILE + static_cast<uint64_t>(w) * WARP_ELEMS;

    float x[U][V];
    uint32_t gt[U], eq[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint64_t j = wbase + u * 128 + lane * 4;
        const float4 q = *reinterpret_cast<const float4 *>(erow + j);
        x[u][0] = q.x; x[u][1] = q.y; x[u][2] = q.z; x[u][3] = q.w;
        gt[u] = eq[u] = 0;
        uint4 kq = make_uint4(mag_key(q.x), mag_key(q.y), mag_key(q.z), mag_key(q.w));
        if (p.rk.on) kq = rand_keys4(p.rk, i, j >> 2);
        const uint32_t ks[4] = {kq.x, kq.y, kq.z, kq.w};
#pragma unroll
        for (int c = 0; c < V; ++c) {
            const uint32_t key = ks[c];
            if (j + c < p.d) {
                gt[u] |= (key > T) ? (1u << c) : 0u;
                eq[u] |= (key == T) ? (1u << c) : 0u;
            }
        }
    }
    uint32_t m[U], cnt[U], pos[U], total;
    if (take == 0 || take == n_eq) {
#pragma unroll
        for (int u = 0; u < U; ++u) m[u] = gt[u] | (take ? eq[u] : 0u);
    } else {
        // the one tile per worker where the tie class is cut: rank the ties by index
#pragma unroll
        for (int u = 0; u < U; ++u) cnt[u] = __popc(eq[u]);
        ordered_prefix<U>(cnt, pos, s_w, total);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            uint32_t rank = pos[u];
            m[u] = gt[u];
#pragma unroll
            for (int c = 0; c < V; ++c)
                if (eq[u] & (1u << c)) {
                    if (rank < take) m[u] |= 1u << c;
                    ++rank;
                }
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) cnt[u] = __popc(m[u]);
    ordered_prefix<U>(cnt, pos, s_w, total);
    if (total != count) {
        if (threadIdx.x == 0) latch(p.status, DECO_ERR_DEVICE_CHECK, 0x300u, tile);
        return;
    }
    deco_pair *out = p.msg + static_cast<size_t>(i) * p.k_cap;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!m[u]) continue;
        const uint64_t j = wbase + u * 128 + lane * 4;
        uint32_t q = start + pos[u];
#pragma unroll
        for (int c = 0; c < V; ++c)
            if (m[u] & (1u << c)) {
                if (q < p.k) {
                    deco_pair pr;
                    pr.idx = static_cast<uint32_t>(j + c);
                    pr.val = x[u][c];
                    out[q] = pr;
                }
                ++q;
                x[u][c] = 0.0f;
            }
        *reinterpret_cast<float4 *>(erow + j) = make_float4(x[u][0], x[u][1], x[u][2], x[u][3]);
    }
}

// ---- dedicated kernels of the multi-pass route (every worker takes it) --------------------
template <int LEVEL>
__global__ void __launch_bounds__(BLOCK) radix_hist_e_kernel(Sel p)
{
    const uint32_t i = blockIdx.y;
    if (!p.sel[i].exact) return;
    __shared__ uint32_t h[RADIX_BINS];
    hist_e_body<LEVEL>(p, i, blockIdx.x, gridDim.x, h);
}

template <int LEVEL>
__global__ void __launch_bounds__(BLOCK) radix_pick_kernel(Sel p)
{
    const uint32_t i = blockIdx.x;
    if (!p.sel[i].exact) return;
    __shared__ uint32_t s_scan[33];
    __shared__ uint32_t s_out[2];
    pick_body<LEVEL>(p.sel[i], hist_of(p, i, 1, LEVEL), s_scan, s_out, p.status, i);
}

__global__ void __launch_bounds__(BLOCK) tile_count_e_kernel(Sel p)
{
    const uint32_t i = blockIdx.y;
    if (!p.sel[i].exact) return;
    __shared__ uint32_t s_a[WARPS], s_b[WARPS];
    count_e_tile(p, i, blockIdx.x, s_a, s_b);
}

constexpr int SCAN_BLOCK = 1024;
__global__ void __launch_bounds__(SCAN_BLOCK) tile_scan_kernel(Sel p)
{
    const uint32_t i = blockIdx.x;
    if (!p.sel[i].exact) return;
    __shared__ uint32_t s_w[33];
    scan_tiles_body(p, i, s_w, false);
}

__global__ void __launch_bounds__(BLOCK) emit_e_kernel(Sel p)
{
    const uint32_t i = blockIdx.y;
    if (!p.sel[i].exact) return;
    __shared__ uint32_t s_w[WARPS];
    emit_e_tile(p, i, blockIdx.x, s_w);
}

// ---- fallback of the streaming route: the whole multi-pass route in one cooperative launch.
// Leaves at once unless some worker's staged set was rejected.  All CTAs take every
// grid-wide barrier: the decision to leave is the same for the whole grid.
__device__ __forceinline__ void exact_fallback_body(const Sel &p, cg::grid_group &grid, uint32_t *h,
                                                    uint32_t *s_a, uint32_t *s_b, uint32_t *s_out)
{
    // CTAs numbered in a row, whatever the shape of the grid
    const uint32_t cta = blockIdx.y * gridDim.x + blockIdx.x, ncta = gridDim.x * gridDim.y;
    // The streaming pass wrote +0 over the staged entries of every tile whose segment fitted;
    // the passes below need the values back.
    for (uint32_t i = 0; i < p.n; ++i) {
        if (!p.sel[i].exact) continue;
        float *erow = p.e + static_cast<size_t>(i) * p.e_stride;
        for (uint32_t tile = cta; tile < p.ntiles; tile += ncta) {
            const size_t ti = static_cast<size_t>(i) * p.ntiles + tile;
            const uint32_t cnt = p.tile_cnt[ti];
            const uint64_t off = p.tile_off[ti];
            if (cnt == 0 || off + cnt > p.stage_cap) continue;
            const deco_pair *src = p.stage + static_cast<size_t>(i) * p.stage_cap + off;
            for (uint32_t q = threadIdx.x; q < cnt; q += BLOCK) {
                const deco_pair pr = src[q];
                if (pr.idx < p.d) erow[pr.idx] = pr.val;
            }
        }
    }
    __threadfence();
    grid.sync();
    for (int level = 0; level < RADIX_LEVELS; ++level) {
        for (uint32_t i = 0; i < p.n; ++i) {
            if (!p.sel[i].exact) continue;
            if (level == 0) hist_e_body<0>(p, i, cta, ncta, h);
            else if (level == 1) hist_e_body<1>(p, i, cta, ncta, h);
            else hist_e_body<2>(p, i, cta, ncta, h);
        }
        __threadfence();
        grid.sync();
        for (uint32_t i = cta; i < p.n; i += ncta) {
            if (!p.sel[i].exact) continue;
            if (level == 0) pick_body<0>(p.sel[i], hist_of(p, i, 1, 0), s_a, s_out, p.status, i);
            else if (level == 1) pick_body<1>(p.sel[i], hist_of(p, i, 1, 1), s_a, s_out, p.status, i);
            else pick_body<2>(p.sel[i], hist_of(p, i, 1, 2), s_a, s_out, p.status, i);
        }
        __threadfence();
        grid.sync();
    }
    for (uint32_t i = 0; i < p.n; ++i) {
        if (!p.sel[i].exact) continue;
        for (uint32_t tile = cta; tile < p.ntiles; tile += ncta) count_e_tile(p, i, tile, s_a, s_b);
    }
    __threadfence();
    grid.sync();
    for (uint32_t i = cta; i < p.n; i += ncta) {
        if (!p.sel[i].exact) continue;
        scan_tiles_body(p, i, s_a, false);
    }
    __threadfence();
    grid.sync();
    for (uint32_t i = 0; i < p.n; ++i) {
        if (!p.sel[i].exact) continue;
        for (uint32_t tile = cta; tile < p.ntiles; tile += ncta) {
            emit_e_tile(p, i, tile, s_b);
            __syncthreads();
        }
    }
}

__global__ void __launch_bounds__(BLOCK) exact_fallback_kernel(Sel p)
{
    if (__ldcg(&p.status[3]) == 0) return;
    cg::grid_group grid = cg::this_grid();
    __shared__ uint32_t h[RADIX_BINS];
    __shared__ uint32_t s_a[33], s_b[WARPS], s_out[2];
    exact_fallback_body(p, grid, h, s_a, s_b, s_out);
}

// ---- small problems: the whole selection of the streaming route in one cooperative launch —
// level A, level B, classification with the chunk walk, emit — each separated from the next by
// a grid-wide barrier where the separate kernels have a launch boundary, then the multi-pass
// route for the workers whose staged set was rejected, if there are any.  Grid: x = CTAs of a
// worker, y = worker; every body strides over its work by gridDim.x.  Only for vectors of few
// chunks (the classification's last CTA walks them itself).  Which barriers a CTA takes depends
// on a flag that is final after the first barrier, so the whole grid takes the same ones.
__global__ void __launch_bounds__(BLOCK, 3) select_chain_kernel(Sel p)
{
    cg::grid_group grid = cg::this_grid();
    const uint32_t i = blockIdx.y;
    stage_hist_a_body<true>(p, i, blockIdx.x, gridDim.x);
    grid.sync();
    stage_hist_b_body<true>(p, i, blockIdx.x, gridDim.x);
    grid.sync();
    stage_classify_body<true>(p, i, 1u, blockIdx.x, gridDim.x);
    grid.sync();
    if (!__ldcg(&p.sel[i].exact)) {
        emit_directory_part<true>(p, i, blockIdx.x, gridDim.x);
        emit_items_part<true>(p, i, blockIdx.x, gridDim.x);
    }
    if (__ldcg(&p.status[3]) == 0) return;
    __syncthreads();
    exact_fallback_body(p, grid, sm.h, sm.scan, sm.warp, sm.out);
}

// ------------------------------------------------------------------------------------------
// Many contexts in one launch (per-layer Top-k: one context per layer, all with n workers).
// The layer's parameters come from a table in device memory.  The sampling and carry kernels
// have grid row y = worker y % n of layer y / n.  The kernels that work on the staged pairs give
// every layer a number of CTAs in proportion to its work (a layer of half a million entries next
// to one of sixty-five million): grid row y is the worker, and a map in device memory says which
// layer CTA x belongs to; the layer's record says where its CTAs start and how many they are,
// and the bodies stride over their work and count arrivals by that number.  The streaming pass,
// which has one CTA per tile, finds its layer from the tile number.
// ------------------------------------------------------------------------------------------
struct MultiLayer {
    Sel p;
    uint64_t g_off;          // entries from the start of a gradient row to the layer
    uint32_t S;              // sample groups of begin_step
    uint32_t walk_here;      // classification walks the chunks itself (few chunks)
    uint32_t rows_aligned;   // the layer's gradient rows start on 16-byte boundaries
    uint32_t carry;          // the layer's bound is carried over between iterations (short layers)
    // first CTA and number of CTAs per worker: levels A, B and classification / chunk sums
    // (0 CTAs where the classification walks the chunks) / emit, of which emit_dir do the
    // directory part
    uint32_t sel_first, sel_ctas, cs_first, cs_ctas, emit_first, emit_ctas, emit_dir;
};
constexpr uint32_t MULTI_MAP_CAP = 8192;        // CTAs per worker and kernel that the maps hold at least

// With hundreds of (layer, worker) rows the sampling kernel is bound by the number of CTAs it
// has to get through, so each thread takes several sample groups.
constexpr int MULTI_BEGIN_GROUPS = 4;

template <int GT>
__global__ void __launch_bounds__(BEGIN_BLOCK, 2)
begin_step_multi_kernel(const MultiLayer *__restrict__ table, uint32_t n, const void *__restrict__ grads,
                        float alpha, uint32_t carrying)
{
    const MultiLayer &m = table[blockIdx.y / n];
    constexpr uint32_t PER_CTA = MULTI_BEGIN_GROUPS * BEGIN_BLOCK;
    if (carrying && m.carry) return;                         // carry_step_multi_kernel's row
    if (blockIdx.x * PER_CTA >= m.S) return;
    const Sel p = m.p;
    const char *g = static_cast<const char *>(grads) + m.g_off * (GT ? 2 : 4);
    begin_step_body<GT, MULTI_BEGIN_GROUPS>(p, blockIdx.y % n, g, alpha, 0u, m.S, (m.S + PER_CTA - 1) / PER_CTA);
}

// Start of an iteration without a sample: the speculative bound of every (layer, worker) row is
// carried over from the exact thresholds T1, T2, T3 of the three previous iterations (newest
// first).  With the steps r1 = T1 - T2 and r2 = T2 - T3 (in key units, 2^23 to the octave):
//   trend   while error feedback still raises the threshold (both steps up) three quarters of
//           the smaller step is added: the rises shrink from iteration to iteration, and the
//           entries that error feedback piles up just below the threshold make a bound that
//           lags behind it stage many times k candidates; a fall is followed in full;
//   swing   |r1 - r2|, the amplitude where the threshold moves back and forth, is subtracted
//           (kept as a maximum that decays by a quarter per iteration: a row whose threshold
//           has swung keeps a wider berth for some iterations);
//   margin  0.04 + 1.5 / sqrt(k) octaves for the fluctuation of the k-th largest magnitude.
// The bound only has to be below the new threshold and not too far below: the count of staged
// candidates checks both, and a row where it fails takes the multi-pass route for this
// iteration, whose cost is in proportion to the layer.  A quantile estimate from a sample needs
// about 35 / delta keys per row however short the layer is, which for hundreds of rows costs
// more than all the selection kernels together.
// One CTA per row: clears the row's histograms and counters and re-arms its selection record.
__global__ void __launch_bounds__(BEGIN_BLOCK)
carry_step_multi_kernel(const MultiLayer *__restrict__ table, uint32_t n)
{
    if (!table[blockIdx.x / n].carry) return;                // begin_step_multi_kernel's row
    const Sel p = table[blockIdx.x / n].p;
    const uint32_t i = blockIdx.x % n;
    const int t = threadIdx.x;
    uint32_t *hz = hist_of(p, i, 0, 0);
    for (int q = t; q < 2 * RADIX_LEVELS * RADIX_BINS; q += BEGIN_BLOCK) hz[q] = 0;
    if (t < DONE_SLOTS && t != 3) p.done[i * DONE_SLOTS + t] = 0;
    if (t != 0) return;
    if (i == 0) p.status[3] = 0;
    SelectState &s = p.sel[i];
    // (the multi-pass route, when a row takes it, leaves its thresholds on record as well)
    const long long T1 = s.threshold, T2 = s.thr_prev, T3 = s.thr_prev2;
    const double margin_oct = fmin(1.0, 0.04 + 1.5 / sqrt(static_cast<double>(p.k)));
    const long long margin = static_cast<long long>(margin_oct * 8388608.0);     // key units per octave: 2^23
    const long long r1 = T1 - T2, r2 = T2 - T3;
    const long long trend = (r1 > 0 && r2 > 0) ? 3 * (r1 < r2 ? r1 : r2) / 4 : (r1 < 0 ? r1 : 0);
    long long swing = r1 > r2 ? r1 - r2 : r2 - r1;
    const long long remembered = 3 * static_cast<long long>(s.swing) / 4;
    if (swing < remembered) swing = remembered;
    if (swing > (1ll << 24)) swing = 1ll << 24;
    s.swing = static_cast<uint32_t>(swing);
    long long bound = T1 + trend - swing - margin;
    if (bound < 0) bound = 0;
    if (bound > 0x7F000000ll) bound = 0x7F000000ll;
    // level A resolves 4095 coarse bins above the bound: half an octave of 2^10-wide ones
    const bool narrow = margin + swing + (trend < 0 ? -trend : trend) <= (1ll << 23) / 5;
    s.thr_prev2 = static_cast<uint32_t>(T2);
    s.thr_prev = static_cast<uint32_t>(T1);
    s.prefix = 0;
    s.k_rem = p.k;
    s.n_greater = 0;
    s.threshold = 0;
    s.ties_take = 0;
    s.exact = 0;
    s.spec_key = static_cast<uint32_t>(bound) & ~((1u << p.bound_low_bit) - 1u);
    s.cert_key = SPEC_DISABLED;
    s.staged_band = 0;
    s.rel_shift = narrow ? 10u : 12u;
}

// The streaming pass of many layers.  Its per-layer arguments travel as a kernel parameter
// (constant bank: no dependent global load before the tile's own loads can be issued); the
// layer of a tile is found by bisection over the layers' first tiles.  ALIGNED: the launch for
// the layers whose gradient rows start on 16-byte boundaries (tiles of the other layers leave
// at once); !ALIGNED: the launch for the others, if there are any.
constexpr int ACC_LAYERS_MAX = 256;
struct AccLayer {
    float *e;
    deco_pair *stage, *band;
    SelectState *sel;
    uint32_t *tile_off, *tile_cnt, *tile_rej, *tile_eq;
    uint64_t e_stride, stage_cap, d, g_off;
    uint32_t ntiles, rows_aligned;
};
struct AccTable {
    // first tile of every layer, relative to the table's first layer: one kilobyte that the
    // bisection of every CTA walks, so it stays in the constant cache
    uint32_t first_tile[ACC_LAYERS_MAX];
    uint32_t count, pad;
    AccLayer L[ACC_LAYERS_MAX];
};
static_assert(sizeof(AccTable) < 32000, "kernel parameters are limited to 32764 bytes");

template <int GT, bool ALIGNED>
__global__ void __launch_bounds__(BLOCK, 3)
ef_accumulate_multi_kernel(const __grid_constant__ AccTable tab, const void *__restrict__ grads,
                           uint64_t g_stride, float alpha)
{
    uint32_t lo = 0, hi = tab.count;                         // the layer lies in [lo, hi)
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (tab.first_tile[mid] <= blockIdx.x) lo = mid;
        else hi = mid;
    }
    const AccLayer &m = tab.L[lo];
    const uint32_t tile = blockIdx.x - tab.first_tile[lo];
    if ((m.rows_aligned != 0) != ALIGNED) return;
    const char *g = static_cast<const char *>(grads) + m.g_off * (GT ? 2 : 4);
    RandParams rk;
    rk.on = 0;
    rk.seed_lo = rk.seed_hi = rk.step_lo = rk.step_hi = rk.worker_base = 0;
    ef_accumulate_body<GT, ALIGNED, true, false, false>(tile, blockIdx.y, true, m.e, m.e_stride, g,
                                                 m.d, g_stride, alpha, rk, m.sel, m.stage, m.band, m.stage_cap,
                                                 m.tile_off, m.tile_cnt, m.tile_rej, m.tile_eq, m.ntiles);
}

__global__ void __launch_bounds__(BLOCK)
stage_hist_a_multi_kernel(const MultiLayer *__restrict__ table, const uint32_t *__restrict__ map)
{
    const MultiLayer &m = table[map[blockIdx.x]];
    const Sel p = m.p;
    stage_hist_a_body<false>(p, blockIdx.y, blockIdx.x - m.sel_first, m.sel_ctas);
}

__global__ void __launch_bounds__(BLOCK)
stage_hist_b_multi_kernel(const MultiLayer *__restrict__ table, const uint32_t *__restrict__ map)
{
    const MultiLayer &m = table[map[blockIdx.x]];
    const Sel p = m.p;
    stage_hist_b_body<false>(p, blockIdx.y, blockIdx.x - m.sel_first, m.sel_ctas);
}

__global__ void __launch_bounds__(BLOCK)
stage_classify_multi_kernel(const MultiLayer *__restrict__ table, const uint32_t *__restrict__ map)
{
    const MultiLayer &m = table[map[blockIdx.x]];
    const Sel p = m.p;
    stage_classify_body<false>(p, blockIdx.y, m.walk_here, blockIdx.x - m.sel_first, m.sel_ctas);
}

// (only the layers whose classification does not walk the chunks itself are on this map)
__global__ void __launch_bounds__(BLOCK)
chunk_sums_multi_kernel(const MultiLayer *__restrict__ table, const uint32_t *__restrict__ map)
{
    const MultiLayer &m = table[map[blockIdx.x]];
    const Sel p = m.p;
    chunk_sums_body(p, blockIdx.y, blockIdx.x - m.cs_first, m.cs_ctas);
}

__global__ void __launch_bounds__(BLOCK)
emit_stage_multi_kernel(const MultiLayer *__restrict__ table, const uint32_t *__restrict__ map)
{
    const MultiLayer &m = table[map[blockIdx.x]];
    const Sel p = m.p;
    emit_stage_body(p, blockIdx.y, blockIdx.x - m.emit_first, m.emit_ctas, m.emit_dir);
}

// Cooperative: the layers with a rejected staged set, one after the other.  Which layers those
// are is read from memory that no CTA of this kernel writes, so every CTA takes the same
// barriers.
__global__ void __launch_bounds__(BLOCK) exact_fallback_multi_kernel(const MultiLayer *__restrict__ table, uint32_t layers)
{
    // nothing to do (the usual case): every thread looks at one layer's flag
    int any = 0;
    for (uint32_t l = threadIdx.x; l < layers; l += BLOCK) any |= __ldcg(&table[l].p.status[3]) != 0;
    if (!__syncthreads_or(any)) return;
    cg::grid_group grid = cg::this_grid();
    __shared__ uint32_t h[RADIX_BINS];
    __shared__ uint32_t s_a[33], s_b[WARPS], s_out[2];
    for (uint32_t l = 0; l < layers; ++l) {
        if (__ldcg(&table[l].p.status[3]) == 0) continue;
        const Sel p = table[l].p;
        exact_fallback_body(p, grid, h, s_a, s_b, s_out);
        __syncthreads();
    }
}

// The band list costs the streaming pass a second, unordered write of some candidates and a
// few instructions per entry, and saves the selection kernels the candidates that are certain to
// be selected.  That pays when the messages are dense (many candidates, most of them certain).
bool band_route(const deco_ctx *c) { return c->band != nullptr && c->k * 32 >= c->d; }

RandParams make_rand(const deco_ctx *c)
{
    RandParams rk;
    rk.on = c->compressor == DECO_COMPRESSOR_RANDK ? 1u : 0u;
    rk.seed_lo = static_cast<uint32_t>(c->seed);
    rk.seed_hi = static_cast<uint32_t>(c->seed >> 32);
    rk.step_lo = static_cast<uint32_t>(c->t);
    rk.step_hi = static_cast<uint32_t>(c->t >> 32);
    rk.worker_base = c->worker_base;
    return rk;
}

Sel make_sel(const deco_ctx *c)
{
    Sel p;
    p.e = c->e;
    p.e_stride = c->e_stride;
    p.d = c->d;
    p.g_stride = c->g_stride;
    p.n = c->n;
    p.ntiles = c->ntiles;
    p.k = static_cast<uint32_t>(c->k);
    p.sel = c->sel;
    p.hist = c->hist;
    p.done = c->done;
    p.sample_keys = c->sample_keys;
    p.sample_hist = c->sample_hist;
    p.sample_win = c->sample_win;
    p.tile_gt = c->tile_gt;
    p.tile_eq = c->tile_eq;
    p.tile_take = c->tile_take;
    // the context's own rows of the job-wide directory and message buffer
    p.tile_start = c->dir_rows + static_cast<size_t>(c->worker_base) * c->dir_stride;
    p.dir_stride = c->dir_stride;
    p.tile_off = c->tile_off;
    p.tile_cnt = c->tile_cnt;
    p.tile_rej = c->tile_rej;
    p.nchunks = c->nchunks;
    p.chunk_cnt = c->chunk_cnt;
    p.chunk_rej = c->chunk_rej;
    p.chunk_eq = c->chunk_eq;
    p.chunk_eqb = c->chunk_eqb;
    p.chunk_start = c->chunk_start;
    p.msg = c->msg_rows + static_cast<size_t>(c->worker_base) * c->msg_stride;
    p.k_cap = c->msg_stride;
    p.stage = c->stage;
    p.band = c->band;
    p.stage_cap = c->stage_cap;
    p.work = c->work;
    p.work_cap = c->work_cap;
    p.status = c->dev_status;
    p.rk = make_rand(c);
    p.use_band = band_route(c) ? 1u : 0u;
    // Top-k keys have 31 bits, Random-k priorities 23
    p.sample_shift = (p.rk.on ? 23u : 31u) - SAMPLE_HIST_BITS;
    p.bound_low_bit = p.rk.on ? 0u : 7u;
    return p;
}

uint32_t part_blocks(const deco_ctx *c, uint64_t items_per_worker, uint32_t items_per_cta)
{
    // enough CTAs per worker to fill the machine, never more than there is work for
    const uint64_t want = (items_per_worker + items_per_cta - 1) / items_per_cta;
    const uint64_t cap = (148ull * 8 + c->n - 1) / c->n;
    return static_cast<uint32_t>(want < 1 ? 1 : (want < cap ? want : cap));
}

}  // namespace

// ------------------------------------------------------------------------------------------
// Launchers
// ------------------------------------------------------------------------------------------
bool streaming_route(const deco_ctx *c) { return c->select_mode == DECO_SELECT_AUTO; }

// Up to this many staged pairs (estimated, all workers), and with few enough chunks for the
// classification to walk them itself, the selection runs as one cooperative launch; beyond
// that the separate kernels' higher occupancy outweighs their launch boundaries.
constexpr uint64_t FUSED_CHAIN_MAX_PAIRS = 4ull << 20;

cudaError_t launch_begin_step(deco_ctx *c, const void *grads, cudaStream_t s)
{
    const float alpha = c->lr_at_server ? 1.0f : c->lr;
    const uint32_t exact_all = streaming_route(c) ? 0u : 1u;
    // one CTA per BEGIN_BLOCK sample groups
    const uint32_t S = sample_groups(c->d, c->k);
    const dim3 grid((S + BEGIN_BLOCK - 1) / BEGIN_BLOCK, c->n);
    if (c->grad_dtype == DECO_BF16)
        begin_step_kernel<1><<<grid, BEGIN_BLOCK, 0, s>>>(make_sel(c), grads, alpha, exact_all, S);
    else
        begin_step_kernel<0><<<grid, BEGIN_BLOCK, 0, s>>>(make_sel(c), grads, alpha, exact_all, S);
    c->launches += 1;
    return cudaGetLastError();
}

template <int GT, bool ALIGNED, bool SPEC, bool RANDK, bool BAND>
static void launch_acc_variant(deco_ctx *c, const void *grads, float alpha, cudaStream_t s)
{
    dim3 grid(c->ntiles, c->n);
    if (BAND)
        ef_accumulate_band_kernel<GT, ALIGNED, RANDK><<<grid, BLOCK, 0, s>>>(
            c->e, c->e_stride, grads, c->d, c->g_stride, alpha, make_rand(c), c->sel, c->stage, c->band,
            c->stage_cap, c->tile_off, c->tile_cnt, c->tile_rej, c->tile_eq, c->ntiles);
    else
        ef_accumulate_kernel<GT, ALIGNED, SPEC, RANDK><<<grid, BLOCK, 0, s>>>(
            c->e, c->e_stride, grads, c->d, c->g_stride, alpha, make_rand(c), c->sel, c->stage, c->stage_cap,
            c->tile_off, c->tile_cnt, c->tile_rej, c->tile_eq, c->ntiles);
}

template <int GT, bool ALIGNED>
static void launch_acc(deco_ctx *c, const void *grads, float alpha, cudaStream_t s)
{
    const bool randk = c->compressor == DECO_COMPRESSOR_RANDK;
    if (streaming_route(c)) {
        if (band_route(c)) {
            if (randk) launch_acc_variant<GT, ALIGNED, true, true, true>(c, grads, alpha, s);
            else launch_acc_variant<GT, ALIGNED, true, false, true>(c, grads, alpha, s);
        } else {
            if (randk) launch_acc_variant<GT, ALIGNED, true, true, false>(c, grads, alpha, s);
            else launch_acc_variant<GT, ALIGNED, true, false, false>(c, grads, alpha, s);
        }
    } else {
        // the multi-pass route derives the keys itself: nothing is staged here
        launch_acc_variant<GT, ALIGNED, false, false, false>(c, grads, alpha, s);
    }
}

cudaError_t launch_accumulate(deco_ctx *c, const void *grads, cudaStream_t s)
{
    const float alpha = c->lr_at_server ? 1.0f : c->lr;
    const uint64_t row_bytes = c->g_stride * (c->grad_dtype == DECO_BF16 ? 2 : 4);
    const bool aligned = (reinterpret_cast<uintptr_t>(grads) % 16 == 0) &&
                         ((c->n == 1) || (row_bytes % 16 == 0));
    if (c->grad_dtype == DECO_BF16) {
        if (aligned) launch_acc<1, true>(c, grads, alpha, s);
        else launch_acc<1, false>(c, grads, alpha, s);
    } else {
        if (aligned) launch_acc<0, true>(c, grads, alpha, s);
        else launch_acc<0, false>(c, grads, alpha, s);
    }
    c->launches += 1;
    return cudaGetLastError();
}

cudaError_t query_fallback_grid(deco_ctx *c)
{
    int per_sm = 0, sms = 0;
    cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, exact_fallback_kernel,
                                                                    BLOCK, 0);
    if (err != cudaSuccess) return err;
    err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    if (per_sm > 4) per_sm = 4;
    c->fallback_grid = static_cast<uint32_t>(per_sm * sms);
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_chain_kernel, BLOCK, 0);
    if (err != cudaSuccess) return err;
    c->chain_grid = per_sm < 1 ? 0u : static_cast<uint32_t>((per_sm > 8 ? 8 : per_sm) * sms);
    return cudaSuccess;
}

// The staged-pair chain as one cooperative launch: short vectors only (one CTA walks the
// chunks, all CTAs resident at once, few staged pairs).
static bool chain_is_one_launch(const deco_ctx *c)
{
    return c->nchunks <= 256 && c->chain_grid >= c->n &&
           static_cast<uint64_t>(c->n) * (2 * c->k + 65536) <= FUSED_CHAIN_MAX_PAIRS;
}

bool selection_is_separate_launches(const deco_ctx *c)
{
    return streaming_route(c) && !chain_is_one_launch(c);
}

cudaError_t launch_selection(deco_ctx *c, cudaStream_t s)
{
    Sel p = make_sel(c);
    dim3 tgrid(c->ntiles, c->n);
    if (!streaming_route(c)) {
        if (wait_for_aggregate(c, s) != cudaSuccess) return cudaGetLastError();
        dim3 hgrid(part_blocks(c, (c->d + 3) / 4, BLOCK * 8), c->n);
        radix_hist_e_kernel<0><<<hgrid, BLOCK, 0, s>>>(p);
        radix_pick_kernel<0><<<c->n, BLOCK, 0, s>>>(p);
        radix_hist_e_kernel<1><<<hgrid, BLOCK, 0, s>>>(p);
        radix_pick_kernel<1><<<c->n, BLOCK, 0, s>>>(p);
        radix_hist_e_kernel<2><<<hgrid, BLOCK, 0, s>>>(p);
        radix_pick_kernel<2><<<c->n, BLOCK, 0, s>>>(p);
        tile_count_e_kernel<<<tgrid, BLOCK, 0, s>>>(p);
        tile_scan_kernel<<<c->n, SCAN_BLOCK, 0, s>>>(p);
        emit_e_kernel<<<tgrid, BLOCK, 0, s>>>(p);
        c->launches += 9;
        return cudaGetLastError();
    }
    // staged pairs per worker are a few times k: size the grids for that
    dim3 sgrid(part_blocks(c, 2 * c->k + 65536, BLOCK * 4), c->n);
    // the chunk walk is done by one CTA: with many chunks their sums are taken in parallel first
    const bool walk_here = c->nchunks <= 256;
    // the kernels from here on rewrite the messages and their directory, which the previous
    // iteration's aggregation may still be reading on the internal stream
    if (chain_is_one_launch(c)) {
        // one cooperative launch for the whole chain: as many CTAs per worker as the separate
        // kernels would use, as far as they can all be resident at once
        if (wait_for_aggregate(c, s) != cudaSuccess) return cudaGetLastError();
        uint32_t gx = sgrid.x;
        if (gx > c->chain_grid / c->n) gx = c->chain_grid / c->n;
        void *args[] = {&p};
        c->launches += 1;
        return cudaLaunchCooperativeKernel(reinterpret_cast<void *>(select_chain_kernel), dim3(gx, c->n),
                                           dim3(BLOCK), args, 0, s);
    }
    // more workers than CTAs that can be resident together: one launch per step of the chain
    stage_hist_a_kernel<<<sgrid, BLOCK, 0, s>>>(p);
    stage_hist_b_kernel<<<sgrid, BLOCK, 0, s>>>(p);
    stage_classify_kernel<<<sgrid, BLOCK, 0, s>>>(p, walk_here ? 1u : 0u);
    if (!walk_here) {
        chunk_sums_kernel<<<dim3((c->nchunks + WARPS - 1) / WARPS, c->n), BLOCK, 0, s>>>(p);
        c->launches += 1;
    }
    if (wait_for_aggregate(c, s) != cudaSuccess) return cudaGetLastError();
    {
        // directory CTAs (a warp per chunk), then the CTAs whose warps stride over the work list:
        // enough of them for one slice per warp at about 1.3 k staged entries, capped at a few
        // waves of the device
        const uint32_t dir_ctas = (c->nchunks + WARPS - 1) / WARPS;
        const uint64_t staged = 13 * c->k / 10, many = staged / (EMIT_LANE_MAX + 1);
        const uint64_t est_items = staged / EMIT_SLICE + (many < c->ntiles ? many : c->ntiles);
        uint64_t item_ctas = (est_items + WARPS - 1) / WARPS + 1;
        const uint64_t cap = (148ull * 8 * 8 + c->n - 1) / c->n;
        if (item_ctas > cap) item_ctas = cap;
        emit_stage_kernel<<<dim3(dir_ctas + static_cast<uint32_t>(item_ctas), c->n), BLOCK, 0, s>>>(p, dir_ctas);
    }
    c->launches += 4;
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    void *args[] = {&p};
    err = cudaLaunchCooperativeKernel(reinterpret_cast<void *>(exact_fallback_kernel),
                                      dim3(c->fallback_grid), dim3(BLOCK), args, 0, s);
    c->launches += 1;
    return err;
}

// ------------------------------------------------------------------------------------------
// Worker side of many contexts (the layers of the per-layer variant) in a fixed number of
// launches.
// ------------------------------------------------------------------------------------------
// The first iterations under a policy take their bound from a sample: the thresholds on record
// are those of another k, and right after the start they rise too fast to extrapolate.
constexpr uint32_t CARRY_AFTER = 4;
// Layers up to this length carry their bound; longer ones keep the sample: there the sample is a
// small part of the layer's work, and a bound that fails costs five passes over the layer.
constexpr uint64_t CARRY_MAX_ENTRIES = 3ull << 20;

struct MultiPlan {
    std::vector<deco_ctx *> layers;
    std::vector<uint64_t> g_off;
    std::vector<MultiLayer> host;
    MultiLayer *dev = nullptr;
    uint32_t n = 0;
    int grad_dtype = DECO_F32;
    uint32_t fallback_grid = 0;
    bool dirty = true;
    // iterations run since the table was last rebuilt (a policy change): the bound is carried
    // over once the thresholds of enough iterations under the current policy are on record
    uint32_t age = 0;
    bool any_carry = false, any_sampled = false;     // layers on either side of CARRY_MAX_ENTRIES
    // streaming pass: the layers in groups of at most ACC_LAYERS_MAX, one launch (or two) each
    struct AccGroup {
        AccTable tab;
        uint32_t tiles = 0;
        bool any_aligned = false, any_unaligned = false;
    };
    std::vector<AccGroup> acc;
    // grid width of the sampling kernel (shared by all layers); CTAs per worker of the kernels
    // on the staged pairs, and their maps CTA -> layer in device memory (map_cap words each)
    uint32_t begin_ctas = 1, sel_total = 1, cs_total = 0, emit_total = 1;
    uint32_t *maps = nullptr;
    uint32_t map_cap = 0;
    std::vector<uint32_t> maps_host;
};

MultiPlan *multi_plan_create(const std::vector<deco_ctx *> &layers, const std::vector<uint64_t> &g_off,
                             uint32_t n, int grad_dtype)
{
    if (layers.empty()) return nullptr;
    MultiPlan *mp = new (std::nothrow) MultiPlan();
    if (!mp) return nullptr;
    try {
        mp->layers = layers;
        mp->g_off = g_off;
        mp->host.resize(layers.size());
        mp->n = n;
        mp->grad_dtype = grad_dtype;
        int per_sm = 0, sms = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, exact_fallback_multi_kernel, BLOCK, 0) !=
                cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, layers[0]->device) != cudaSuccess ||
            per_sm < 1)
            throw 1;
        mp->fallback_grid = static_cast<uint32_t>((per_sm > 4 ? 4 : per_sm) * sms);
        if (cudaMalloc(reinterpret_cast<void **>(&mp->dev), sizeof(MultiLayer) * layers.size()) != cudaSuccess)
            throw 2;
        // a map holds a share of the budget (at most 1.5 times 148 * 8 * 2 CTAs: emit's two parts)
        // plus the one CTA that every layer gets in any case (two on emit's map)
        mp->map_cap = std::max<uint32_t>(MULTI_MAP_CAP, 4096u + 4u * static_cast<uint32_t>(layers.size()));
        if (cudaMalloc(reinterpret_cast<void **>(&mp->maps), sizeof(uint32_t) * 3 * mp->map_cap) != cudaSuccess)
            throw 2;
        mp->maps_host.resize(3 * static_cast<size_t>(mp->map_cap));
    } catch (...) {
        cudaGetLastError();
        multi_plan_destroy(mp);
        return nullptr;
    }
    return mp;
}

void multi_plan_destroy(MultiPlan *mp)
{
    if (!mp) return;
    cudaFree(mp->dev);
    cudaFree(mp->maps);
    delete mp;
}

void multi_plan_mark_dirty(MultiPlan *mp)
{
    if (mp) mp->dirty = true;
}

// Table and grid widths for the layers' current k (after a policy change).
static cudaError_t multi_plan_refresh(MultiPlan *mp, const void *grads, cudaStream_t s)
{
    const uint32_t L = static_cast<uint32_t>(mp->layers.size());
    const uint64_t esz = mp->grad_dtype == DECO_BF16 ? 2 : 4;
    uint64_t begin_max = 1;
    std::vector<uint64_t> want_sel(L), want_cs(L), want_dir(L), want_items(L);
    for (uint32_t l = 0; l < L; ++l) {
        const deco_ctx *c = mp->layers[l];
        MultiLayer &m = mp->host[l];
        m.p = make_sel(c);
        m.p.use_band = 0;                // the streaming pass of many layers writes no band list
        m.g_off = mp->g_off[l];
        m.S = sample_groups(c->d, c->k);
        m.walk_here = c->nchunks <= 256 ? 1u : 0u;
        m.carry = c->d <= CARRY_MAX_ENTRIES ? 1u : 0u;
        m.rows_aligned = ((mp->g_off[l] * esz) % 16 == 0 && (c->g_stride * esz) % 16 == 0) ? 1u : 0u;
        begin_max = std::max<uint64_t>(begin_max, (m.S + MULTI_BEGIN_GROUPS * BEGIN_BLOCK - 1) /
                                                      (MULTI_BEGIN_GROUPS * BEGIN_BLOCK));
        // what the layer would use by itself: a CTA per trip over about 2 k staged pairs, a warp
        // per chunk, a warp per expected emit work item
        want_sel[l] = (2 * c->k + 1024 + BLOCK * 4 - 1) / (BLOCK * 4);
        want_cs[l] = m.walk_here ? 0 : (c->nchunks + WARPS - 1) / WARPS;
        want_dir[l] = (c->nchunks + WARPS - 1) / WARPS;
        const uint64_t staged = 13 * c->k / 10, many = staged / (EMIT_LANE_MAX + 1);
        const uint64_t est_items = staged / EMIT_SLICE + (many < c->ntiles ? many : c->ntiles);
        want_items[l] = (est_items + WARPS - 1) / WARPS + 1;
    }
    // Shares of a budget of CTAs per worker (two waves of the device over all workers; the maps'
    // capacity at most): in proportion to what the layers want, at least one each where they
    // want any.  The bodies stride over their work, so fewer CTAs than wanted only means trips.
    const uint64_t budget = std::min<uint64_t>(mp->map_cap / 2, std::max<uint64_t>(1, 148ull * 8 * 2 / mp->n));
    auto share = [&](const std::vector<uint64_t> &want, std::vector<uint32_t> &got, uint64_t room) {
        uint64_t sum = 0;
        for (uint64_t w : want) sum += w;
        got.assign(L, 0);
        for (uint32_t l = 0; l < L; ++l) {
            if (want[l] == 0) continue;
            const uint64_t g = sum <= room ? want[l] : want[l] * room / sum;
            got[l] = static_cast<uint32_t>(g < 1 ? 1 : g);
        }
    };
    std::vector<uint32_t> got_sel, got_cs, got_dir, got_items;
    share(want_sel, got_sel, budget);
    share(want_cs, got_cs, budget);
    share(want_dir, got_dir, budget / 2);
    share(want_items, got_items, budget);
    uint32_t *map_sel = mp->maps_host.data(), *map_cs = map_sel + mp->map_cap, *map_emit = map_cs + mp->map_cap;
    mp->sel_total = mp->cs_total = mp->emit_total = 0;
    for (uint32_t l = 0; l < L; ++l) {
        MultiLayer &m = mp->host[l];
        m.sel_first = mp->sel_total;
        m.sel_ctas = got_sel[l];
        m.cs_first = mp->cs_total;
        m.cs_ctas = got_cs[l];
        m.emit_first = mp->emit_total;
        m.emit_dir = got_dir[l];
        m.emit_ctas = got_dir[l] + got_items[l];
        if (mp->sel_total + m.sel_ctas > mp->map_cap || mp->cs_total + m.cs_ctas > mp->map_cap ||
            mp->emit_total + m.emit_ctas > mp->map_cap)
            return cudaErrorInvalidValue;          // cannot happen: the shares fit the budget
        for (uint32_t q = 0; q < m.sel_ctas; ++q) map_sel[mp->sel_total++] = l;
        for (uint32_t q = 0; q < m.cs_ctas; ++q) map_cs[mp->cs_total++] = l;
        for (uint32_t q = 0; q < m.emit_ctas; ++q) map_emit[mp->emit_total++] = l;
    }
    mp->acc.assign((L + ACC_LAYERS_MAX - 1) / ACC_LAYERS_MAX, MultiPlan::AccGroup());
    for (uint32_t l = 0; l < L; ++l) {
        const MultiLayer &m = mp->host[l];
        MultiPlan::AccGroup &grp = mp->acc[l / ACC_LAYERS_MAX];
        AccLayer &a = grp.tab.L[l % ACC_LAYERS_MAX];
        a.e = m.p.e;
        a.stage = m.p.stage;
        a.band = m.p.band;
        a.sel = m.p.sel;
        a.tile_off = m.p.tile_off;
        a.tile_cnt = m.p.tile_cnt;
        a.tile_rej = m.p.tile_rej;
        a.tile_eq = m.p.tile_eq;
        a.e_stride = m.p.e_stride;
        a.stage_cap = m.p.stage_cap;
        a.d = m.p.d;
        a.g_off = m.g_off;
        a.ntiles = m.p.ntiles;
        grp.tab.first_tile[l % ACC_LAYERS_MAX] = grp.tiles;
        a.rows_aligned = m.rows_aligned;
        grp.tiles += m.p.ntiles;
        grp.tab.count = l % ACC_LAYERS_MAX + 1;
        grp.tab.pad = 0;
        (m.rows_aligned ? grp.any_aligned : grp.any_unaligned) = true;
    }
    mp->begin_ctas = static_cast<uint32_t>(begin_max);
    (void)grads;
    // the host tables are pageable: the copies have left them when the calls return
    cudaError_t err = cudaMemcpyAsync(mp->dev, mp->host.data(), sizeof(MultiLayer) * L,
                                      cudaMemcpyHostToDevice, s);
    if (err == cudaSuccess)
        err = cudaMemcpyAsync(mp->maps, mp->maps_host.data(), sizeof(uint32_t) * 3 * mp->map_cap,
                              cudaMemcpyHostToDevice, s);
    if (err == cudaSuccess) {
        mp->dirty = false;
        mp->age = 0;
        mp->any_carry = mp->any_sampled = false;
        for (const MultiLayer &m : mp->host) (m.carry ? mp->any_carry : mp->any_sampled) = true;
    }
    return err;
}

cudaError_t multi_compress(MultiPlan *mp, const void *grads, float alpha, cudaStream_t s)
{
    if (mp->dirty) {
        const cudaError_t err = multi_plan_refresh(mp, grads, s);
        if (err != cudaSuccess) return err;
    }
    const uint32_t L = static_cast<uint32_t>(mp->layers.size()), n = mp->n, rows = L * n;
    const bool bf16 = mp->grad_dtype == DECO_BF16;
    const uint32_t carrying = (mp->age >= CARRY_AFTER && mp->any_carry) ? 1u : 0u;
    if (carrying) carry_step_multi_kernel<<<rows, BEGIN_BLOCK, 0, s>>>(mp->dev, n);
    if (!carrying || mp->any_sampled) {
        if (bf16)
            begin_step_multi_kernel<1><<<dim3(mp->begin_ctas, rows), BEGIN_BLOCK, 0, s>>>(mp->dev, n, grads, alpha,
                                                                                       carrying);
        else
            begin_step_multi_kernel<0><<<dim3(mp->begin_ctas, rows), BEGIN_BLOCK, 0, s>>>(mp->dev, n, grads, alpha,
                                                                                       carrying);
    }
    mp->age += 1;
    const uint64_t g_stride = mp->layers[0]->g_stride;
    for (const MultiPlan::AccGroup &grp : mp->acc) {
        const dim3 agrid(grp.tiles, n);
        if (grp.any_aligned) {
            if (bf16) ef_accumulate_multi_kernel<1, true><<<agrid, BLOCK, 0, s>>>(grp.tab, grads, g_stride, alpha);
            else ef_accumulate_multi_kernel<0, true><<<agrid, BLOCK, 0, s>>>(grp.tab, grads, g_stride, alpha);
        }
        if (grp.any_unaligned) {
            if (bf16) ef_accumulate_multi_kernel<1, false><<<agrid, BLOCK, 0, s>>>(grp.tab, grads, g_stride, alpha);
            else ef_accumulate_multi_kernel<0, false><<<agrid, BLOCK, 0, s>>>(grp.tab, grads, g_stride, alpha);
        }
    }
    const uint32_t *map_sel = mp->maps, *map_cs = map_sel + mp->map_cap, *map_emit = map_cs + mp->map_cap;
    const dim3 sgrid(mp->sel_total, n);
    stage_hist_a_multi_kernel<<<sgrid, BLOCK, 0, s>>>(mp->dev, map_sel);
    stage_hist_b_multi_kernel<<<sgrid, BLOCK, 0, s>>>(mp->dev, map_sel);
    stage_classify_multi_kernel<<<sgrid, BLOCK, 0, s>>>(mp->dev, map_sel);
    if (mp->cs_total) chunk_sums_multi_kernel<<<dim3(mp->cs_total, n), BLOCK, 0, s>>>(mp->dev, map_cs);
    emit_stage_multi_kernel<<<dim3(mp->emit_total, n), BLOCK, 0, s>>>(mp->dev, map_emit);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    const MultiLayer *tab = mp->dev;
    uint32_t layers = L;
    void *args[] = {&tab, &layers};
    err = cudaLaunchCooperativeKernel(reinterpret_cast<void *>(exact_fallback_multi_kernel),
                                      dim3(mp->fallback_grid), dim3(BLOCK), args, 0, s);
    mp->layers[0]->launches += mp->cs_total ? 9 : 8;
    return err;
}

}  // namespace deco
