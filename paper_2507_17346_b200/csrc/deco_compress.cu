// Worker side of Algorithm 1 on the device: a = e + gamma*g, exact Top-k of |a| with ties to
// the lower index, messages as packed (index, value) pairs sorted by index, residual in e.
//
// Kernels in this file
//   ef_accumulate_kernel   streaming pass: reads e and g once, writes a into e
//   radix_hist_e_kernel    histogram of one radix level of the magnitude keys of a
//   radix_pick_kernel      walks a histogram from the top and fixes the next key bits
//   tile_count_e_kernel    per tile: entries above / equal to the threshold
//   tile_scan_kernel       per worker: prefix sums over tiles -> message position of each tile
//   emit_e_kernel          ordered compaction of the selected entries, zeroing them in e
#include <cuda_bf16.h>

#include "deco_internal.h"

namespace deco {

namespace {

constexpr uint32_t FULL = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

__device__ __forceinline__ void latch(uint32_t *status, uint32_t code, uint32_t a, uint32_t b)
{
    if (atomicCAS(status, 0u, code) == 0u) {
        status[1] = a;
        status[2] = b;
    }
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

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// ------------------------------------------------------------------------------------------
// Streaming pass.  GT = 0: fp32 gradients, 4 entries per thread and round; GT = 1: bfloat16
// gradients, 8 entries per thread and round.  ALIGNED: every gradient row starts on a
// 16-byte boundary, so whole tiles are read with 128-bit loads; otherwise (and in the tile
// that contains the end of the vector) gradients are read entry by entry.
// ------------------------------------------------------------------------------------------
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

template <int GT, bool ALIGNED, bool SPEC>
__global__ void __launch_bounds__(BLOCK)
ef_accumulate_kernel(float *__restrict__ e, uint64_t e_stride, const void *__restrict__ grads,
                     uint64_t d, float alpha, SelectState *__restrict__ sel,
                     deco_pair *__restrict__ stage, uint64_t stage_cap,
                     uint32_t *__restrict__ tile_off, uint32_t *__restrict__ tile_cnt,
                     uint32_t ntiles)
{
    constexpr int V = Geo<GT>::V, U = Geo<GT>::U;
    const uint32_t tile = blockIdx.x, i = blockIdx.y;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    float *erow = e + static_cast<size_t>(i) * e_stride;
    const char *grow = reinterpret_cast<const char *>(grads) +
                       static_cast<size_t>(i) * d * (GT ? 2 : 4);
    const uint64_t tile_base = static_cast<uint64_t>(tile) * TILE;
    const uint64_t wbase = tile_base + static_cast<uint64_t>(w) * WARP_ELEMS;
    const bool full = ALIGNED && (tile_base + TILE <= d);

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
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint64_t j = wbase + u * (32 * V) + lane * V;
#pragma unroll
        for (int q = 0; q < V / 4; ++q)
            *reinterpret_cast<float4 *>(erow + j + 4 * q) =
                make_float4(x[u][4 * q], x[u][4 * q + 1], x[u][4 * q + 2], x[u][4 * q + 3]);
    }

    if (SPEC) {
        // Stage every entry whose key reaches the speculative bound, in index order, into a
        // segment reserved with one atomic per tile.
        __shared__ uint32_t s_w[WARPS];
        __shared__ uint32_t s_off;
        const uint32_t bound = sel[i].spec_key;
        uint32_t m[U], cnt[U], pos[U], any = 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint64_t j = wbase + u * (32 * V) + lane * V;
            m[u] = 0;
#pragma unroll
            for (int c = 0; c < V; ++c)
                if (mag_key(x[u][c]) >= bound && (full || j + c < d)) m[u] |= 1u << c;
            cnt[u] = __popc(m[u]);
            any |= m[u];
        }
        uint32_t total = 0;
        if (__syncthreads_or(any != 0)) {
            ordered_prefix<U>(cnt, pos, s_w, total);
        }
        if (threadIdx.x == 0) {
            uint32_t off = 0;
            if (total) off = atomicAdd(&sel[i].n_staged, total);
            tile_off[static_cast<size_t>(i) * ntiles + tile] = off;
            tile_cnt[static_cast<size_t>(i) * ntiles + tile] = total;
            s_off = off;
        }
        if (total == 0) return;
        __syncthreads();
        const uint64_t off = s_off;
        if (off + total > stage_cap) return;         // overflow: n_staged tells the selector
        deco_pair *out = stage + static_cast<size_t>(i) * stage_cap + off;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint64_t j = wbase + u * (32 * V) + lane * V;
            uint32_t p = pos[u];
#pragma unroll
            for (int c = 0; c < V; ++c)
                if (m[u] & (1u << c)) {
                    deco_pair pr;
                    pr.idx = static_cast<uint32_t>(j + c);
                    pr.val = x[u][c];
                    out[p++] = pr;
                }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Multi-pass exact selection over e (workers with sel[i].exact != 0).
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

template <int LEVEL>
__global__ void __launch_bounds__(BLOCK)
radix_hist_e_kernel(const float *__restrict__ e, uint64_t e_stride, uint64_t d,
                    const SelectState *__restrict__ sel, uint32_t *__restrict__ hist)
{
    const uint32_t i = blockIdx.y;
    if (!sel[i].exact) return;
    __shared__ uint32_t h[RADIX_BINS];
    for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK) h[b] = 0;
    __syncthreads();
    const uint32_t prefix = sel[i].prefix;
    const float4 *row = reinterpret_cast<const float4 *>(e + static_cast<size_t>(i) * e_stride);
    const uint64_t nvec = (d + 3) >> 2;
    for (uint64_t v = static_cast<uint64_t>(blockIdx.x) * BLOCK + threadIdx.x; v < nvec;
         v += static_cast<uint64_t>(gridDim.x) * BLOCK) {
        const float4 q = row[v];
        const uint64_t j = v << 2;
        radix_bin<LEVEL>(mag_key(q.x), prefix, h);
        if (j + 1 < d) radix_bin<LEVEL>(mag_key(q.y), prefix, h);
        if (j + 2 < d) radix_bin<LEVEL>(mag_key(q.z), prefix, h);
        if (j + 3 < d) radix_bin<LEVEL>(mag_key(q.w), prefix, h);
    }
    __syncthreads();
    uint32_t *out = hist + (static_cast<size_t>(i) * RADIX_LEVELS + LEVEL) * RADIX_BINS;
    for (int b = threadIdx.x; b < RADIX_BINS; b += BLOCK)
        if (h[b]) atomicAdd(&out[b], h[b]);
}

// One CTA per worker.  Finds the bin b with  count(bins > b) < k_rem <= count(bins >= b)
// and appends it to the key prefix.  After the last level the prefix is the threshold key.
template <int LEVEL>
__global__ void __launch_bounds__(BLOCK)
radix_pick_kernel(SelectState *__restrict__ sel, const uint32_t *__restrict__ hist,
                  uint32_t want_exact, uint32_t *__restrict__ status)
{
    constexpr int BITS = (LEVEL == 2) ? 7 : 12;
    constexpr int PER = RADIX_BINS / BLOCK;   // 16 bins per thread
    const uint32_t i = blockIdx.x;
    if (sel[i].exact != want_exact) return;
    const uint32_t k_rem = sel[i].k_rem;
    const uint32_t *h = hist + (static_cast<size_t>(i) * RADIX_LEVELS + LEVEL) * RADIX_BINS;
    __shared__ uint32_t suf[BLOCK + 1];
    const int t = threadIdx.x;
    uint32_t loc[PER], sum = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) {
        loc[b] = h[t * PER + b];
        sum += loc[b];
    }
    suf[t] = sum;
    if (t == 0) suf[BLOCK] = 0;
    __syncthreads();
    for (int o = 1; o < BLOCK; o <<= 1) {      // inclusive suffix sums over threads
        const uint32_t v = (t + o < BLOCK) ? suf[t + o] : 0u;
        __syncthreads();
        suf[t] += v;
        __syncthreads();
    }
    const uint32_t s_here = suf[t], s_above = suf[t + 1];
    if (t == 0 && s_here < k_rem) latch(status, DECO_ERR_DEVICE_CHECK, 0x100u + LEVEL, i);
    if (s_here >= k_rem && s_above < k_rem) {
        uint32_t acc = s_above;
        int bin = t * PER;
#pragma unroll
        for (int b = PER - 1; b >= 0; --b) {
            if (acc + loc[b] >= k_rem) {
                bin = t * PER + b;
                break;
            }
            acc += loc[b];
        }
        SelectState &s = sel[i];
        s.n_greater += acc;
        s.k_rem = k_rem - acc;
        const uint32_t prefix = (s.prefix << BITS) | static_cast<uint32_t>(bin);
        s.prefix = prefix;
        if (LEVEL == 2) {
            s.threshold = prefix;
            s.ties_take = k_rem - acc;
        }
    }
}

__global__ void __launch_bounds__(BLOCK)
tile_count_e_kernel(const float *__restrict__ e, uint64_t e_stride, uint64_t d,
                    const SelectState *__restrict__ sel, uint32_t *__restrict__ tile_gt,
                    uint32_t *__restrict__ tile_eq, uint32_t ntiles)
{
    const uint32_t tile = blockIdx.x, i = blockIdx.y;
    if (!sel[i].exact) return;
    const uint32_t T = sel[i].threshold;
    const float *row = e + static_cast<size_t>(i) * e_stride;
    const uint64_t base = static_cast<uint64_t>(tile) * TILE;
    uint32_t gt = 0, eq = 0;
#pragma unroll
    for (int r = 0; r < TILE / (4 * BLOCK); ++r) {
        const uint64_t j = base + (static_cast<uint64_t>(r) * BLOCK + threadIdx.x) * 4;
        const float4 q = *reinterpret_cast<const float4 *>(row + j);
        const float xs[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t key = mag_key(xs[c]);
            const bool in = j + c < d;
            gt += (in && key > T);
            eq += (in && key == T);
        }
    }
    __shared__ uint32_t s_gt[WARPS], s_eq[WARPS];
    for (int o = 16; o > 0; o >>= 1) {
        gt += __shfl_down_sync(FULL, gt, o);
        eq += __shfl_down_sync(FULL, eq, o);
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) {
        s_gt[w] = gt;
        s_eq[w] = eq;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t a = 0, b = 0;
        for (int ww = 0; ww < WARPS; ++ww) {
            a += s_gt[ww];
            b += s_eq[ww];
        }
        tile_gt[static_cast<size_t>(i) * ntiles + tile] = a;
        tile_eq[static_cast<size_t>(i) * ntiles + tile] = b;
    }
}

// Exclusive scan over SCAN_BLOCK threads; returns the prefix of `v`, total in `total`.
constexpr int SCAN_BLOCK = 1024;
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t *s_w /*[33]*/,
                                                    uint32_t &total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t incl = warp_incl_scan(v);
    if (lane == 31) s_w[w] = incl;
    __syncthreads();
    if (w == 0) {
        const uint32_t x = s_w[lane];
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

// One CTA per worker: ties are granted to tiles in index order until ties_take are used up,
// then every tile gets its position in the message.
__global__ void __launch_bounds__(SCAN_BLOCK)
tile_scan_kernel(const SelectState *__restrict__ sel, const uint32_t *__restrict__ tile_gt,
                 const uint32_t *__restrict__ tile_eq, uint32_t *__restrict__ tile_take,
                 uint32_t *__restrict__ tile_start, uint32_t ntiles, uint32_t k,
                 uint32_t *__restrict__ status)
{
    const uint32_t i = blockIdx.x;
    __shared__ uint32_t s_w[33];
    const uint32_t *gt = tile_gt + static_cast<size_t>(i) * ntiles;
    const uint32_t *eq = tile_eq + static_cast<size_t>(i) * ntiles;
    uint32_t *take = tile_take + static_cast<size_t>(i) * ntiles;
    uint32_t *start = tile_start + static_cast<size_t>(i) * (ntiles + 1);
    const uint32_t ties = sel[i].ties_take;
    const uint32_t per = (ntiles + SCAN_BLOCK - 1) / SCAN_BLOCK;
    const uint32_t lo = min(ntiles, threadIdx.x * per), hi = min(ntiles, lo + per);
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
        sel_sum += gt[t] + tk;
        eq_before += q;
    }
    uint32_t sel_total;
    uint32_t pos = block_excl_scan(sel_sum, s_w, sel_total);
    for (uint32_t t = lo; t < hi; ++t) {
        start[t] = pos;
        pos += gt[t] + take[t];
    }
    if (threadIdx.x == 0) {
        start[ntiles] = sel_total;
        if (sel_total != k) latch(status, DECO_ERR_DEVICE_CHECK, 0x200u, i);
    }
}

__global__ void __launch_bounds__(BLOCK)
emit_e_kernel(float *__restrict__ e, uint64_t e_stride, uint64_t d,
              const SelectState *__restrict__ sel, const uint32_t *__restrict__ tile_eq,
              const uint32_t *__restrict__ tile_take, const uint32_t *__restrict__ tile_start,
              deco_pair *__restrict__ msg, uint64_t k_cap, uint32_t k, uint32_t ntiles,
              uint32_t *__restrict__ status)
{
    constexpr int V = 4, U = WARP_ELEMS / (32 * V);
    const uint32_t tile = blockIdx.x, i = blockIdx.y;
    if (!sel[i].exact) return;
    const uint32_t start = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile];
    const uint32_t count = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile + 1] - start;
    if (count == 0) return;
    const uint32_t T = sel[i].threshold;
    const uint32_t take = tile_take[static_cast<size_t>(i) * ntiles + tile];
    const uint32_t n_eq = tile_eq[static_cast<size_t>(i) * ntiles + tile];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    float *erow = e + static_cast<size_t>(i) * e_stride;
    const uint64_t wbase = static_cast<uint64_t>(tile) * TILE + static_cast<uint64_t>(w) * WARP_ELEMS;
    __shared__ uint32_t s_w[WARPS];

    float x[U][V];
    uint32_t gt[U], eq[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint64_t j = wbase + u * 128 + lane * 4;
        const float4 q = *reinterpret_cast<const float4 *>(erow + j);
        x[u][0] = q.x; x[u][1] = q.y; x[u][2] = q.z; x[u][3] = q.w;
        gt[u] = eq[u] = 0;
#pragma unroll
        for (int c = 0; c < V; ++c) {
            const uint32_t key = mag_key(x[u][c]);
            if (j + c < d) {
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
        if (threadIdx.x == 0) latch(status, DECO_ERR_DEVICE_CHECK, 0x300u, tile);
        return;
    }
    deco_pair *out = msg + static_cast<size_t>(i) * k_cap;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!m[u]) continue;
        const uint64_t j = wbase + u * 128 + lane * 4;
        uint32_t p = start + pos[u];
#pragma unroll
        for (int c = 0; c < V; ++c)
            if (m[u] & (1u << c)) {
                if (p < k) {
                    deco_pair pr;
                    pr.idx = static_cast<uint32_t>(j + c);
                    pr.val = x[u][c];
                    out[p] = pr;
                }
                ++p;
                x[u][c] = 0.0f;
            }
        *reinterpret_cast<float4 *>(erow + j) = make_float4(x[u][0], x[u][1], x[u][2], x[u][3]);
    }
}

// Per step: clear the histograms and (re)arm the per-worker selection records.
__global__ void begin_step_kernel(SelectState *sel, uint32_t n, uint32_t k, uint32_t exact_all)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    SelectState &s = sel[i];
    s.prefix = 0;
    s.k_rem = k;
    s.n_greater = 0;
    s.threshold = 0;
    s.ties_take = 0;
    s.exact = exact_all;
    s.spec_key = SPEC_DISABLED;
    s.n_staged = 0;
    if (exact_all) s.exact_total += 1;
}

}  // namespace

// ------------------------------------------------------------------------------------------
// Launchers
// ------------------------------------------------------------------------------------------
cudaError_t launch_begin_step(deco_ctx *c, cudaStream_t s)
{
    cudaError_t err = cudaMemsetAsync(
        c->hist, 0, sizeof(uint32_t) * c->n * RADIX_LEVELS * RADIX_BINS, s);
    if (err != cudaSuccess) return err;
    const uint32_t exact_all = 1;   // speculative path not wired yet
    begin_step_kernel<<<(c->n + 127) / 128, 128, 0, s>>>(c->sel, c->n,
                                                          static_cast<uint32_t>(c->k), exact_all);
    c->launches += 2;
    return cudaGetLastError();
}

template <int GT, bool ALIGNED>
static void launch_acc(deco_ctx *c, const void *grads, float alpha, cudaStream_t s)
{
    dim3 grid(c->ntiles, c->n);
    ef_accumulate_kernel<GT, ALIGNED, false><<<grid, BLOCK, 0, s>>>(
        c->e, c->e_stride, grads, c->d, alpha, c->sel, c->stage, c->stage_cap, c->tile_off,
        c->tile_cnt, c->ntiles);
}

cudaError_t launch_accumulate(deco_ctx *c, const void *grads, cudaStream_t s)
{
    const float alpha = c->lr_at_server ? 1.0f : c->lr;
    const uint64_t row_bytes = c->d * (c->grad_dtype == DECO_BF16 ? 2 : 4);
    const bool aligned = (c->n == 1) || (row_bytes % 16 == 0);
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

static uint32_t hist_blocks(const deco_ctx *c)
{
    // enough CTAs to fill the machine, never more than there are 128-bit words per CTA round
    const uint64_t nvec = (c->d + 3) / 4;
    const uint64_t want = (nvec + BLOCK * 8 - 1) / (BLOCK * 8);
    const uint64_t cap = (148ull * 8 + c->n - 1) / c->n;
    return static_cast<uint32_t>(want < 1 ? 1 : (want < cap ? want : cap));
}

cudaError_t launch_exact_selection(deco_ctx *c, cudaStream_t s)
{
    dim3 hgrid(hist_blocks(c), c->n);
    dim3 tgrid(c->ntiles, c->n);
    const uint32_t k = static_cast<uint32_t>(c->k);
    radix_hist_e_kernel<0><<<hgrid, BLOCK, 0, s>>>(c->e, c->e_stride, c->d, c->sel, c->hist);
    radix_pick_kernel<0><<<c->n, BLOCK, 0, s>>>(c->sel, c->hist, 1u, c->dev_status);
    radix_hist_e_kernel<1><<<hgrid, BLOCK, 0, s>>>(c->e, c->e_stride, c->d, c->sel, c->hist);
    radix_pick_kernel<1><<<c->n, BLOCK, 0, s>>>(c->sel, c->hist, 1u, c->dev_status);
    radix_hist_e_kernel<2><<<hgrid, BLOCK, 0, s>>>(c->e, c->e_stride, c->d, c->sel, c->hist);
    radix_pick_kernel<2><<<c->n, BLOCK, 0, s>>>(c->sel, c->hist, 1u, c->dev_status);
    tile_count_e_kernel<<<tgrid, BLOCK, 0, s>>>(c->e, c->e_stride, c->d, c->sel, c->tile_gt,
                                                c->tile_eq, c->ntiles);
    tile_scan_kernel<<<c->n, SCAN_BLOCK, 0, s>>>(c->sel, c->tile_gt, c->tile_eq, c->tile_take,
                                                 c->tile_start, c->ntiles, k, c->dev_status);
    emit_e_kernel<<<tgrid, BLOCK, 0, s>>>(c->e, c->e_stride, c->d, c->sel, c->tile_eq,
                                          c->tile_take, c->tile_start, c->msg, c->k_cap, k,
                                          c->ntiles, c->dev_status);
    c->launches += 9;
    return cudaGetLastError();
}

}  // namespace deco
