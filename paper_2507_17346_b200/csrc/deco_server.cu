// Server side of Algorithm 1 on the device: S_t = sum_i Delta_t^i into a cache slot, and the
// stale update x = x - scale * S_{t-tau}.
//
//   aggregate_kernel  merges the n index-sorted messages tile by tile: a dense fp32
//                     accumulator of one tile lives in shared memory, workers are added in
//                     order 0..n-1 (so the fp32 sum is the sequential one), and the touched
//                     entries are written out in index order.  The output segment of a tile
//                     starts at the sum of the workers' message positions for that tile, which
//                     needs no communication between CTAs; positions a tile does not use (an
//                     index sent by several workers is stored once) are filled with
//                     DECO_NO_INDEX.
//   apply_kernel      one fused multiply-add per stored entry.
#include "deco_internal.h"

namespace deco {

namespace {

constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr uint32_t PREFETCH_WORKERS = 16;   // workers whose entries one thread holds at once

__device__ __forceinline__ void latch(uint32_t *status, uint32_t code, uint32_t a, uint32_t b)
{
    if (atomicCAS(status, 0u, code) == 0u) {
        status[1] = a;
        status[2] = b;
    }
}

// One tile by the whole CTA: dense fp32 accumulator and touched-bit mask in shared memory (both
// all-zero on entry and on exit), workers added in order, output in index order.  NW: how many
// workers' ranges and entries a thread holds in registers at once (the code is unrolled NW
// times, so callers pick the smallest NW >= n they have).
template <uint32_t NW>
__device__ __forceinline__ void dense_tile(const deco_pair *__restrict__ msg, uint64_t k_cap,
                                           const uint32_t *__restrict__ tile_start, uint64_t dir_stride,
                                           uint32_t ntiles,
                                           uint32_t n, deco_pair *__restrict__ slot,
                                           uint64_t positions, uint32_t *__restrict__ status,
                                           uint32_t tile, float *acc, uint32_t *mask, uint32_t *s_w)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint64_t out_off = 0;
    uint32_t cap = 0, longest = 0;
    constexpr bool KEEP = NW <= 8;                         // ranges stay in registers for the loads below
    constexpr uint32_t NR = KEEP ? NW : 1;
    uint32_t ra[NR], rb[NR];
    if (KEEP) {
#pragma unroll
        for (uint32_t i = 0; i < NR; ++i) {
            ra[i] = rb[i] = 0;
            if (i < n) {
                ra[i] = tile_start[static_cast<size_t>(i) * dir_stride + tile];
                rb[i] = tile_start[static_cast<size_t>(i) * dir_stride + tile + 1];
            }
            out_off += ra[i];
            cap += rb[i] - ra[i];
            longest = max(longest, rb[i] - ra[i]);
        }
    }
    for (uint32_t i = KEEP ? NW : 0; i < n; ++i) {
        const uint32_t a = tile_start[static_cast<size_t>(i) * dir_stride + tile];
        const uint32_t b = tile_start[static_cast<size_t>(i) * dir_stride + tile + 1];
        out_off += a;
        cap += b - a;
        longest = max(longest, b - a);
    }
    if (cap == 0) return;
    if (out_off + cap > positions) {
        if (threadIdx.x == 0) latch(status, DECO_ERR_DEVICE_CHECK, 0x400u, tile);
        return;
    }
    const uint32_t first = tile * static_cast<uint32_t>(TILE);
    if (n <= NW && longest <= static_cast<uint32_t>(BLOCK)) {
        // At most one entry per thread and worker.  All loads are issued before the first
        // barrier, then the workers are added in order from registers.
        deco_pair pre[NW];
#pragma unroll
        for (uint32_t i = 0; i < NW; ++i) {
            pre[i].idx = DECO_NO_INDEX;
            pre[i].val = 0.0f;
            uint32_t a, b;
            if (KEEP) {
                a = ra[i < NR ? i : 0];
                b = rb[i < NR ? i : 0];
            } else {
                a = b = 0;
                if (i < n) {
                    a = tile_start[static_cast<size_t>(i) * dir_stride + tile];
                    b = tile_start[static_cast<size_t>(i) * dir_stride + tile + 1];
                }
            }
            if (a + threadIdx.x < b) pre[i] = msg[static_cast<size_t>(i) * k_cap + a + threadIdx.x];
        }
#pragma unroll
        for (uint32_t i = 0; i < NW; ++i) {
            if (i >= n) break;
            if (pre[i].idx != DECO_NO_INDEX) {
                const uint32_t loc = pre[i].idx - first;
                if (loc >= static_cast<uint32_t>(TILE)) {
                    latch(status, DECO_ERR_DEVICE_CHECK, 0x401u, pre[i].idx);
                } else {
                    acc[loc] = acc[loc] + pre[i].val;      // indices are unique per worker
                    atomicOr(&mask[loc >> 5], 1u << (loc & 31));
                }
            }
            __syncthreads();
        }
    } else {
        for (uint32_t i = 0; i < n; ++i) {                 // worker order 0..n-1
            const uint32_t a = tile_start[static_cast<size_t>(i) * dir_stride + tile];
            const uint32_t b = tile_start[static_cast<size_t>(i) * dir_stride + tile + 1];
            if (b == a) continue;
            const deco_pair *src = msg + static_cast<size_t>(i) * k_cap;
            for (uint32_t p0 = a; p0 < b; p0 += 4 * BLOCK) {   // four loads in flight
                deco_pair prs[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const uint32_t p = p0 + r * BLOCK + threadIdx.x;
                    prs[r].idx = DECO_NO_INDEX;
                    prs[r].val = 0.0f;
                    if (p < b) prs[r] = src[p];
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (prs[r].idx == DECO_NO_INDEX) continue;
                    const uint32_t loc = prs[r].idx - first;
                    if (loc >= static_cast<uint32_t>(TILE)) {
                        latch(status, DECO_ERR_DEVICE_CHECK, 0x401u, prs[r].idx);
                        continue;
                    }
                    acc[loc] = acc[loc] + prs[r].val;      // indices are unique per worker
                    atomicOr(&mask[loc >> 5], 1u << (loc & 31));
                }
            }
            __syncthreads();
        }
    }
    uint32_t word = mask[threadIdx.x];
    const uint32_t c = __popc(word);
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_w[w] = incl;
    __syncthreads();
    uint32_t before = 0, uniq = 0;
#pragma unroll
    for (int ww = 0; ww < WARPS; ++ww) {
        const uint32_t v = s_w[ww];
        before += (ww < w) ? v : 0u;
        uniq += v;
    }
    deco_pair *out = slot + out_off;
    uint32_t p = before + incl - c;
    while (word) {
        const uint32_t b = __ffs(word) - 1;
        word &= word - 1;
        const uint32_t loc = threadIdx.x * 32 + b;
        deco_pair pr;
        pr.idx = first + loc;
        pr.val = acc[loc];
        out[p++] = pr;
        acc[loc] = 0.0f;
    }
    mask[threadIdx.x] = 0;
    for (uint32_t q = uniq + threadIdx.x; q < cap; q += BLOCK) {
        deco_pair pr;
        pr.idx = DECO_NO_INDEX;
        pr.val = 0.0f;
        out[q] = pr;
    }
    __syncthreads();
}

// dense_tile with the smallest unrolling that holds all n workers (the branch is CTA-uniform)
__device__ __forceinline__ void dense_tile_n(const deco_pair *__restrict__ msg, uint64_t k_cap,
                                             const uint32_t *__restrict__ tile_start, uint64_t dir_stride,
                                             uint32_t ntiles, uint32_t n, deco_pair *__restrict__ slot,
                                             uint64_t positions, uint32_t *__restrict__ status,
                                             uint32_t tile, float *acc, uint32_t *mask, uint32_t *s_w)
{
    if (n <= 4)
        dense_tile<4>(msg, k_cap, tile_start, dir_stride, ntiles, n, slot, positions, status, tile, acc, mask, s_w);
    else if (n <= 8)
        dense_tile<8>(msg, k_cap, tile_start, dir_stride, ntiles, n, slot, positions, status, tile, acc, mask, s_w);
    else
        dense_tile<PREFETCH_WORKERS>(msg, k_cap, tile_start, dir_stride, ntiles, n, slot, positions, status, tile,
                                     acc, mask, s_w);
}

// Persistent CTAs, every tile by the whole CTA: for messages with many entries per tile.
__global__ void __launch_bounds__(BLOCK)
aggregate_kernel(const deco_pair *__restrict__ msg, uint64_t k_cap,
                 const uint32_t *__restrict__ tile_start, uint64_t dir_stride, uint32_t ntiles, uint32_t n,
                 deco_pair *__restrict__ slot, uint64_t positions, uint32_t *__restrict__ status)
{
    static_assert(TILE / 32 == BLOCK, "one mask word per thread");
    __shared__ float acc[TILE];
    __shared__ uint32_t mask[TILE / 32];
    __shared__ uint32_t s_w[WARPS];
    for (int q = threadIdx.x; q < TILE; q += BLOCK) acc[q] = 0.0f;
    mask[threadIdx.x] = 0;
    __syncthreads();
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x)
        dense_tile_n(msg, k_cap, tile_start, dir_stride, ntiles, n, slot, positions, status, tile, acc, mask, s_w);
}

// Dense messages (n k entries in all comparable with d): the aggregate is kept as the plain
// vector S[0 .. tiles * TILE) with +0 where no worker sent the index.  Same accumulator, same
// worker order; the tile is then written out whole, with no mask and no compaction.
constexpr int DENSE_BATCH = 4;      // workers whose entries of a tile are fetched together
constexpr int DENSE_ROUNDS = 4;     // entries per thread and worker held at once

__global__ void __launch_bounds__(BLOCK)
aggregate_dense_kernel(const deco_pair *__restrict__ msg, uint64_t k_cap,
                       const uint32_t *__restrict__ tile_start, uint64_t dir_stride, uint32_t ntiles, uint32_t n,
                       float *__restrict__ slot, uint32_t *__restrict__ status)
{
    __shared__ __align__(16) float acc[TILE];
    for (int q = threadIdx.x; q < TILE; q += BLOCK) acc[q] = 0.0f;
    __syncthreads();
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const uint32_t first = tile * static_cast<uint32_t>(TILE);
        for (uint32_t i0 = 0; i0 < n; i0 += DENSE_BATCH) {
            // the ranges of a batch of workers, then all their entries, are fetched before the
            // first use; the additions follow in worker order with a barrier between workers
            uint32_t a[DENSE_BATCH], b[DENSE_BATCH];
            bool fits = true;
#pragma unroll
            for (int w = 0; w < DENSE_BATCH; ++w) {
                a[w] = b[w] = 0;
                if (i0 + w < n) {
                    a[w] = tile_start[static_cast<size_t>(i0 + w) * dir_stride + tile];
                    b[w] = tile_start[static_cast<size_t>(i0 + w) * dir_stride + tile + 1];
                }
                fits = fits && b[w] - a[w] <= static_cast<uint32_t>(DENSE_ROUNDS * BLOCK);
            }
            if (fits) {
                deco_pair pre[DENSE_BATCH][DENSE_ROUNDS];
#pragma unroll
                for (int w = 0; w < DENSE_BATCH; ++w)
#pragma unroll
                    for (int r = 0; r < DENSE_ROUNDS; ++r) {
                        const uint32_t p = a[w] + r * BLOCK + threadIdx.x;
                        pre[w][r].idx = DECO_NO_INDEX;
                        pre[w][r].val = 0.0f;
                        if (p < b[w]) pre[w][r] = msg[static_cast<size_t>(i0 + w) * k_cap + p];
                    }
#pragma unroll
                for (int w = 0; w < DENSE_BATCH; ++w) {
                    if (b[w] <= a[w]) continue;                    // the same for the whole CTA
#pragma unroll
                    for (int r = 0; r < DENSE_ROUNDS; ++r) {
                        if (pre[w][r].idx == DECO_NO_INDEX) continue;
                        const uint32_t loc = pre[w][r].idx - first;
                        if (loc >= static_cast<uint32_t>(TILE)) {
                            latch(status, DECO_ERR_DEVICE_CHECK, 0x401u, pre[w][r].idx);
                            continue;
                        }
                        acc[loc] = acc[loc] + pre[w][r].val;       // indices are unique per worker
                    }
                    __syncthreads();
                }
                continue;
            }
            for (int w = 0; w < DENSE_BATCH; ++w) {                // a worker with more entries in the tile
                if (b[w] <= a[w]) continue;
                const deco_pair *src = msg + static_cast<size_t>(i0 + w) * k_cap;
                for (uint32_t p0 = a[w]; p0 < b[w]; p0 += 4 * BLOCK) {   // four loads in flight
                    deco_pair prs[4];
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const uint32_t p = p0 + r * BLOCK + threadIdx.x;
                        prs[r].idx = DECO_NO_INDEX;
                        prs[r].val = 0.0f;
                        if (p < b[w]) prs[r] = src[p];
                    }
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        if (prs[r].idx == DECO_NO_INDEX) continue;
                        const uint32_t loc = prs[r].idx - first;
                        if (loc >= static_cast<uint32_t>(TILE)) {
                            latch(status, DECO_ERR_DEVICE_CHECK, 0x401u, prs[r].idx);
                            continue;
                        }
                        acc[loc] = acc[loc] + prs[r].val;
                    }
                }
                __syncthreads();
            }
        }
        float4 *out = reinterpret_cast<float4 *>(slot + static_cast<size_t>(tile) * TILE);
        float4 *acc4 = reinterpret_cast<float4 *>(acc);
#pragma unroll
        for (int q = threadIdx.x; q < TILE / 4; q += BLOCK) {
            out[q] = acc4[q];
            acc4[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
        __syncthreads();
    }
}

// x[j] = fma(neg_scale, S[j], x[j]) for every j < d, S being a dense aggregate.  Where S is +0
// the result is x[j] itself, bit for bit (also for x = -0), so groups of four untouched entries
// are not written back.
__global__ void __launch_bounds__(256)
apply_dense_kernel(const float *__restrict__ S, float neg_scale, float *__restrict__ params, uint64_t d)
{
    const uint64_t nvec = d >> 2;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    const float4 *S4 = reinterpret_cast<const float4 *>(S);
    float4 *x4 = reinterpret_cast<float4 *>(params);
    for (uint64_t v0 = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; v0 < nvec; v0 += 4 * stride) {
        float4 sv[4], xv[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint64_t v = v0 + r * stride;
            sv[r] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            xv[r] = sv[r];
            if (v < nvec) {
                sv[r] = __ldcs(S4 + v);
                xv[r] = x4[v];
            }
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint64_t v = v0 + r * stride;
            if (v >= nvec) continue;
            if (sv[r].x == 0.0f && sv[r].y == 0.0f && sv[r].z == 0.0f && sv[r].w == 0.0f) continue;
            x4[v] = make_float4(__fmaf_rn(neg_scale, sv[r].x, xv[r].x), __fmaf_rn(neg_scale, sv[r].y, xv[r].y),
                                __fmaf_rn(neg_scale, sv[r].z, xv[r].z), __fmaf_rn(neg_scale, sv[r].w, xv[r].w));
        }
    }
    // the last d % 4 entries
    if (blockIdx.x == 0 && threadIdx.x < (d & 3)) {
        const uint64_t j = (nvec << 2) + threadIdx.x;
        params[j] = __fmaf_rn(neg_scale, S[j], params[j]);
    }
}

// The entries a warp holds (one per lane, at most 32, worker-major and index-sorted within a
// worker; lanes without one pass valid = false) merged into out[0 .. uniq): entries with the
// same index are summed in worker order starting from +0, the sums are written in index order.
// Returns uniq.
__device__ __forceinline__ uint32_t warp_merge(bool valid, uint32_t idx, float val,
                                               deco_pair *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    // lanes without an entry get keys of their own, so that they match nobody
    const uint32_t grp = __match_any_sync(FULL, valid ? idx : (0xFFFFFF00u | lane));
    const bool head = valid && lane == __ffs(grp) - 1;
    float sum = 0.0f;
    uint32_t rest = valid ? grp : 0u;
    while (__any_sync(FULL, rest != 0)) {                     // ascending lanes = worker order
        const int src = rest ? __ffs(rest) - 1 : 0;
        const float v = __shfl_sync(FULL, val, src);
        if (rest) {
            sum = sum + v;
            rest &= rest - 1;
        }
    }
    const uint32_t heads = __ballot_sync(FULL, head);
    uint32_t rank = 0;
    for (uint32_t h = heads; h; h &= h - 1) {
        const uint32_t other = __shfl_sync(FULL, idx, __ffs(h) - 1);
        rank += other < idx ? 1u : 0u;
    }
    if (head) {
        deco_pair pr;
        pr.idx = idx;
        pr.val = sum;
        out[rank] = pr;
    }
    return __popc(heads);
}

// Sparse messages (a few entries per tile): one warp per tile, no accumulator.  Lane i first
// holds worker i's range of the tile.  At most 32 entries in all are merged in one go;
// otherwise the tile's index range is cut into windows that are merged one after the other,
// each with at most 32 entries: halves where that is enough (up to 64 entries), else
// SPARSE_WINDOWS quarters.  A tile that does not fit is left to the whole CTA afterwards
// (dense_tile).
constexpr int SPARSE_WINDOWS = 4;

// The entries of one tile, cut into windows of STEP quarters of its index range, merged window
// after window (lane i holds worker i's range [a, a + len) and, in below[q], how many of its
// entries lie below the end of quarter q - 1).  Returns false, with nothing written, if some
// window holds more than 32 entries.
template <int STEP>
__device__ __forceinline__ bool merge_windows(const deco_pair *__restrict__ msg, uint64_t k_cap, uint32_t n,
                                              uint32_t a, const uint32_t (&below)[SPARSE_WINDOWS + 1],
                                              uint32_t first, deco_pair *__restrict__ out, uint32_t cap,
                                              uint32_t *__restrict__ status)
{
    constexpr int NWIN = SPARSE_WINDOWS / STEP;
    const int lane = threadIdx.x & 31;
    // per window: entries of the workers before lane's own, and in all
    uint32_t before[NWIN], total[NWIN];
    bool fits = true;
#pragma unroll
    for (int q = 0; q < NWIN; ++q) {
        const uint32_t mine = below[(q + 1) * STEP] - below[q * STEP];
        uint32_t incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(FULL, incl, o);
            if (lane >= o) incl += t;
        }
        before[q] = incl - mine;
        total[q] = __shfl_sync(FULL, incl, 31);
        fits = fits && total[q] <= 32;
    }
    if (!fits) return false;
    uint32_t uniq = 0;
#pragma unroll
    for (int q = 0; q < NWIN; ++q) {
        if (total[q] == 0) continue;
        const uint32_t part_a = a + below[q * STEP], part_len = below[(q + 1) * STEP] - below[q * STEP];
        deco_pair pr;
        pr.idx = DECO_NO_INDEX;
        pr.val = 0.0f;
        bool valid = false;
        for (uint32_t i = 0; i < n; ++i) {
            const uint32_t pb = __shfl_sync(FULL, before[q], i);
            const uint32_t pl = __shfl_sync(FULL, part_len, i);
            const uint32_t pa = __shfl_sync(FULL, part_a, i);
            if (static_cast<uint32_t>(lane) >= pb && static_cast<uint32_t>(lane) < pb + pl) {
                pr = msg[static_cast<size_t>(i) * k_cap + pa + (lane - pb)];
                valid = true;
            }
        }
        if (valid && pr.idx - first >= static_cast<uint32_t>(TILE)) {
            latch(status, DECO_ERR_DEVICE_CHECK, 0x401u, pr.idx);
            valid = false;
        }
        uniq += warp_merge(valid, pr.idx, pr.val, out + uniq);
    }
    for (uint32_t q = uniq + lane; q < cap; q += 32) {
        deco_pair pr;
        pr.idx = DECO_NO_INDEX;
        pr.val = 0.0f;
        out[q] = pr;
    }
    return true;
}

// One tile by one warp.  Returns true (to every lane) if the tile does not fit and has to be
// done by the whole CTA with the dense accumulator.
__device__ __forceinline__ bool sparse_tile_warp(const deco_pair *__restrict__ msg, uint64_t k_cap,
                                                 const uint32_t *__restrict__ tile_start, uint64_t dir_stride,
                                                 uint32_t ntiles,
                                                 uint32_t n, deco_pair *__restrict__ slot, uint64_t positions,
                                                 uint32_t *__restrict__ status, uint32_t tile)
{
    const int lane = threadIdx.x & 31;
    uint32_t a = 0, b = 0;
    if (static_cast<uint32_t>(lane) < n) {
        a = tile_start[static_cast<size_t>(lane) * dir_stride + tile];
        b = tile_start[static_cast<size_t>(lane) * dir_stride + tile + 1];
    }
    const uint32_t len = b - a;
    uint32_t cap = len, longest = len;
    uint64_t out_off = a;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        cap += __shfl_xor_sync(FULL, cap, o);
        longest = max(longest, __shfl_xor_sync(FULL, longest, o));
        out_off += __shfl_xor_sync(FULL, out_off, o);
    }
    const uint32_t first = tile * static_cast<uint32_t>(TILE);
    if (cap == 0) return false;
    if (out_off + cap > positions) {
        if (lane == 0) latch(status, DECO_ERR_DEVICE_CHECK, 0x400u, tile);
        return false;
    }
    if (cap > 32u * SPARSE_WINDOWS || longest > 32) return true;
    deco_pair *out = slot + out_off;
    uint32_t below[SPARSE_WINDOWS + 1];
    below[0] = 0;
#pragma unroll
    for (int q = 1; q <= SPARSE_WINDOWS; ++q) below[q] = len;
    // at most 32 entries in all: one window
    if (cap <= 32) return !merge_windows<SPARSE_WINDOWS>(msg, k_cap, n, a, below, first, out, cap, status);
    // lane i: how many of worker i's entries lie below the end of each quarter
    // (every lane looks at one entry of each worker in turn: ranges are at most 32 long)
    for (uint32_t i = 0; i < n; ++i) {
        const uint32_t ai = __shfl_sync(FULL, a, i), li = __shfl_sync(FULL, len, i);
        uint32_t loc = DECO_NO_INDEX;
        if (static_cast<uint32_t>(lane) < li)
            loc = msg[static_cast<size_t>(i) * k_cap + ai + lane].idx - first;
#pragma unroll
        for (int q = 1; q < SPARSE_WINDOWS; ++q) {
            const uint32_t cnt = __popc(__ballot_sync(FULL, loc < q * (TILE / SPARSE_WINDOWS)));
            if (static_cast<uint32_t>(lane) == i) below[q] = cnt;
        }
    }
    // halves if they hold at most 32 entries each, else quarters
    if (cap <= 64 && merge_windows<2>(msg, k_cap, n, a, below, first, out, cap, status)) return false;
    return !merge_windows<1>(msg, k_cap, n, a, below, first, out, cap, status);
}

__global__ void __launch_bounds__(BLOCK)
aggregate_sparse_kernel(const deco_pair *__restrict__ msg, uint64_t k_cap,
                        const uint32_t *__restrict__ tile_start, uint64_t dir_stride, uint32_t ntiles, uint32_t n,
                        deco_pair *__restrict__ slot, uint64_t positions,
                        uint32_t *__restrict__ status)
{
    __shared__ float acc[TILE];
    __shared__ uint32_t mask[TILE / 32];
    __shared__ uint32_t s_w[WARPS];
    __shared__ uint32_t s_heavy;
    if (threadIdx.x == 0) s_heavy = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t tile = blockIdx.x * WARPS + w;
    if (tile < ntiles &&
        sparse_tile_warp(msg, k_cap, tile_start, dir_stride, ntiles, n, slot, positions, status, tile) &&
        lane == 0)
        atomicOr(&s_heavy, 1u << w);
    __syncthreads();
    uint32_t heavy = s_heavy;
    if (heavy == 0) return;
    for (int q = threadIdx.x; q < TILE; q += BLOCK) acc[q] = 0.0f;
    mask[threadIdx.x] = 0;
    __syncthreads();
    for (; heavy; heavy &= heavy - 1)
        dense_tile_n(msg, k_cap, tile_start, dir_stride, ntiles, n, slot, positions, status,
                   blockIdx.x * WARPS + __ffs(heavy) - 1, acc, mask, s_w);
}

// ---- the server side of many contexts (layers of the per-layer variant) in one launch each.
// Tiles of all layers are numbered in a row; tile_layer gives the layer of each.
__global__ void __launch_bounds__(BLOCK)
aggregate_multi_kernel(const ServerLayer *__restrict__ table, const uint32_t *__restrict__ tile_layer,
                       uint32_t total_tiles, uint32_t n, uint32_t slot_write)
{
    __shared__ float acc[TILE];
    __shared__ uint32_t mask[TILE / 32];
    __shared__ uint32_t s_w[WARPS];
    for (int q = threadIdx.x; q < TILE; q += BLOCK) acc[q] = 0.0f;
    mask[threadIdx.x] = 0;
    __syncthreads();
    for (uint32_t g = blockIdx.x; g < total_tiles; g += gridDim.x) {
        const ServerLayer &L = table[tile_layer[g]];
        if (!L.dense) continue;
        const uint32_t tile = g - L.first_tile;
        const uint64_t positions = static_cast<uint64_t>(n) * L.k;
        if (tile == 0 && threadIdx.x == 0) L.slot_pos[slot_write] = static_cast<uint32_t>(positions);
        dense_tile_n(L.msg, L.k_cap, L.tile_start, L.ntiles + 1, L.ntiles, n, L.slots + slot_write * (n * L.k_cap),
                   positions, L.status, tile, acc, mask, s_w);
    }
}

__global__ void __launch_bounds__(BLOCK)
aggregate_sparse_multi_kernel(const ServerLayer *__restrict__ table, const uint32_t *__restrict__ tile_layer,
                              uint32_t total_tiles, uint32_t n, uint32_t slot_write)
{
    __shared__ float acc[TILE];
    __shared__ uint32_t mask[TILE / 32];
    __shared__ uint32_t s_w[WARPS];
    __shared__ uint32_t s_heavy;
    if (threadIdx.x == 0) s_heavy = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t g = blockIdx.x * WARPS + w;
    if (g < total_tiles) {
        const ServerLayer &L = table[tile_layer[g]];
        if (!L.dense) {
            const uint32_t tile = g - L.first_tile;
            const uint64_t positions = static_cast<uint64_t>(n) * L.k;
            if (tile == 0 && lane == 0) L.slot_pos[slot_write] = static_cast<uint32_t>(positions);
            if (sparse_tile_warp(L.msg, L.k_cap, L.tile_start, L.ntiles + 1, L.ntiles, n,
                                 L.slots + slot_write * (n * L.k_cap), positions, L.status, tile) && lane == 0)
                atomicOr(&s_heavy, 1u << w);
        }
    }
    __syncthreads();
    uint32_t heavy = s_heavy;
    if (heavy == 0) return;
    for (int q = threadIdx.x; q < TILE; q += BLOCK) acc[q] = 0.0f;
    mask[threadIdx.x] = 0;
    __syncthreads();
    for (; heavy; heavy &= heavy - 1) {
        const uint32_t gh = blockIdx.x * WARPS + __ffs(heavy) - 1;
        const ServerLayer &L = table[tile_layer[gh]];
        dense_tile_n(L.msg, L.k_cap, L.tile_start, L.ntiles + 1, L.ntiles, n, L.slots + slot_write * (n * L.k_cap),
                   static_cast<uint64_t>(n) * L.k, L.status, gh - L.first_tile, acc, mask, s_w);
    }
}

// Row y of the grid applies cache slot `slot_read` of layer y to the layer's parameters.
__global__ void __launch_bounds__(256)
apply_multi_kernel(const ServerLayer *__restrict__ table, uint32_t n, uint32_t slot_read, float neg_scale)
{
    const ServerLayer &L = table[blockIdx.y];
    const deco_pair *slot = L.slots + slot_read * (static_cast<uint64_t>(n) * L.k_cap);
    const uint64_t positions = L.slot_pos[slot_read];
    if (positions > static_cast<uint64_t>(n) * L.k_cap) {
        if (threadIdx.x == 0 && blockIdx.x == 0) latch(L.status, DECO_ERR_DEVICE_CHECK, 0x520u, slot_read);
        return;
    }
    float *params = L.params;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    // four independent entries per thread and trip (entries of a slot are distinct)
    for (uint64_t p0 = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; p0 < positions;
         p0 += 4 * stride) {
        deco_pair pr[4];
        float x[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint64_t p = p0 + r * stride;
            pr[r].idx = DECO_NO_INDEX;
            pr[r].val = 0.0f;
            if (p < positions) pr[r] = slot[p];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            x[r] = 0.0f;
            if (pr[r].idx == DECO_NO_INDEX) continue;
            if (pr[r].idx >= L.d) {
                latch(L.status, DECO_ERR_DEVICE_CHECK, 0x500u, pr[r].idx);
                pr[r].idx = DECO_NO_INDEX;
                continue;
            }
            x[r] = params[pr[r].idx];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
            if (pr[r].idx != DECO_NO_INDEX) params[pr[r].idx] = __fmaf_rn(neg_scale, pr[r].val, x[r]);
    }
}

__global__ void __launch_bounds__(256)
apply_kernel(const deco_pair *__restrict__ slot, uint64_t positions, float neg_scale,
             float *__restrict__ params, uint64_t d, uint32_t *__restrict__ status)
{
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    // four independent entries per thread and trip (the entries of a slot are distinct), so that
    // the dependent pair -> parameter loads of four entries overlap
    for (uint64_t p0 = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; p0 < positions;
         p0 += 4 * stride) {
        deco_pair pr[4];
        float x[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint64_t p = p0 + r * stride;
            pr[r].idx = DECO_NO_INDEX;
            pr[r].val = 0.0f;
            if (p < positions) pr[r] = slot[p];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            x[r] = 0.0f;
            if (pr[r].idx == DECO_NO_INDEX) continue;
            if (pr[r].idx >= d) {
                latch(status, DECO_ERR_DEVICE_CHECK, 0x500u, pr[r].idx);
                pr[r].idx = DECO_NO_INDEX;
                continue;
            }
            x[r] = params[pr[r].idx];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
            if (pr[r].idx != DECO_NO_INDEX) params[pr[r].idx] = __fmaf_rn(neg_scale, pr[r].val, x[r]);
    }
}

// Short layers of the per-layer variant, one CTA per layer: the n messages are merged into the
// layer's cache slot (the layer is one tile), then the listed slots are applied to the layer's
// slice of the parameters, oldest first, one fused multiply-add per stored entry.
__global__ void __launch_bounds__(BLOCK)
small_server_kernel(const SmallLayer *__restrict__ table, uint32_t n, uint32_t aggregate,
                    uint32_t slot_write, SmallDue due, float neg_scale)
{
    __shared__ float acc[TILE];
    __shared__ uint32_t mask[TILE / 32];
    __shared__ uint32_t s_w[WARPS];
    const SmallLayer L = table[blockIdx.x];
    const uint64_t slot_len = static_cast<uint64_t>(n) * L.k_cap;
    if (aggregate) {
        for (int q = threadIdx.x; q < TILE; q += BLOCK) acc[q] = 0.0f;
        mask[threadIdx.x] = 0;
        __syncthreads();
        const uint64_t positions = static_cast<uint64_t>(n) * L.k;
        dense_tile_n(L.msg, L.k_cap, L.tile_start, 2, 1, n, L.slots + slot_write * slot_len, positions,
                   L.status, 0, acc, mask, s_w);
        if (threadIdx.x == 0) L.slot_pos[slot_write] = static_cast<uint32_t>(positions);
        __syncthreads();
    }
    for (uint32_t q = 0; q < due.count; ++q) {
        const deco_pair *slot = L.slots + due.slot[q] * slot_len;
        const uint32_t positions = L.slot_pos[due.slot[q]];
        if (positions > slot_len) {
            if (threadIdx.x == 0) latch(L.status, DECO_ERR_DEVICE_CHECK, 0x520u, positions);
            return;
        }
        for (uint32_t p = threadIdx.x; p < positions; p += BLOCK) {
            const deco_pair pr = slot[p];
            if (pr.idx == DECO_NO_INDEX) continue;
            if (pr.idx >= L.d) {
                latch(L.status, DECO_ERR_DEVICE_CHECK, 0x500u, pr.idx);
                continue;
            }
            L.params[pr.idx] = __fmaf_rn(neg_scale, pr.val, L.params[pr.idx]);
        }
        __syncthreads();          // an entry may be held by several slots: one pass after the other
    }
}

}  // namespace

cudaError_t launch_small_server(const SmallLayer *table, uint32_t layers, uint32_t n, bool aggregate,
                                uint32_t slot_write, const SmallDue &due, float neg_scale, cudaStream_t s)
{
    if (layers == 0) return cudaSuccess;
    small_server_kernel<<<layers, BLOCK, 0, s>>>(table, n, aggregate ? 1u : 0u, slot_write, due, neg_scale);
    return cudaGetLastError();
}

cudaError_t launch_multi_aggregate(const ServerLayer *table, const uint32_t *tile_layer, uint32_t total_tiles,
                                   uint32_t n, uint32_t slot_write, bool any_dense, bool any_sparse,
                                   cudaStream_t s)
{
    if (any_sparse)
        aggregate_sparse_multi_kernel<<<(total_tiles + WARPS - 1) / WARPS, BLOCK, 0, s>>>(table, tile_layer,
                                                                                       total_tiles, n, slot_write);
    if (any_dense) {
        const uint32_t blocks = total_tiles < 148u * 6 ? total_tiles : 148u * 6;
        aggregate_multi_kernel<<<blocks, BLOCK, 0, s>>>(table, tile_layer, total_tiles, n, slot_write);
    }
    return cudaGetLastError();
}

cudaError_t launch_multi_apply(const ServerLayer *table, uint32_t layers, uint32_t n, uint32_t ctas_per_layer,
                               uint32_t slot_read, float neg_scale, cudaStream_t s)
{
    apply_multi_kernel<<<dim3(ctas_per_layer, layers), 256, 0, s>>>(table, n, slot_read, neg_scale);
    return cudaGetLastError();
}

// the rule of launch_aggregate: a warp per tile up to 80 entries per tile on average
bool aggregate_prefers_dense(const deco_ctx *c)
{
    const uint64_t positions = static_cast<uint64_t>(c->n_total) * c->k;
    return !(c->n_total <= 32 && positions <= 80ull * c->ntiles);
}

cudaError_t launch_aggregate(deco_ctx *c, deco_pair *slot, cudaStream_t s)
{
    const uint64_t positions = static_cast<uint64_t>(c->n_total) * c->k_of_msg;
    c->launches += 1;
    if (c->n_total <= 32 && positions <= 80ull * c->ntiles) {
        // on average at most 80 entries per tile over all workers: a warp per tile
        aggregate_sparse_kernel<<<(c->ntiles + WARPS - 1) / WARPS, BLOCK, 0, s>>>(
            c->msg_rows, c->msg_stride, c->dir_rows, c->dir_stride, c->ntiles, c->n_total, slot, positions,
            c->dev_status);
        return cudaGetLastError();
    }
    // next to the streaming pass of the following iteration the aggregation takes half the
    // CTA slots it could hold, so that the pass keeps most of its loads in flight
    const uint32_t per_sm = (c->agg_stream && s == c->agg_stream) ? 3u : 6u;
    const uint32_t blocks = c->ntiles < 148u * per_sm ? c->ntiles : 148u * per_sm;
    aggregate_kernel<<<blocks, BLOCK, 0, s>>>(c->msg_rows, c->msg_stride, c->dir_rows, c->dir_stride, c->ntiles,
                                              c->n_total, slot, positions, c->dev_status);
    return cudaGetLastError();
}

cudaError_t launch_aggregate_dense(deco_ctx *c, float *slot, cudaStream_t s)
{
    c->launches += 1;
    const uint32_t per_sm = (c->agg_stream && s == c->agg_stream) ? 3u : 6u;
    const uint32_t blocks = c->ntiles < 148u * per_sm ? c->ntiles : 148u * per_sm;
    aggregate_dense_kernel<<<blocks, BLOCK, 0, s>>>(c->msg_rows, c->msg_stride, c->dir_rows, c->dir_stride,
                                                    c->ntiles, c->n_total, slot, c->dev_status);
    return cudaGetLastError();
}

cudaError_t launch_apply_dense(deco_ctx *c, const float *slot, float neg_scale, cudaStream_t s)
{
    uint64_t blocks = ((c->d >> 2) + 4 * 256 - 1) / (4 * 256);
    if (blocks < 1) blocks = 1;
    if (blocks > 148ull * 8) blocks = 148ull * 8;
    apply_dense_kernel<<<static_cast<uint32_t>(blocks), 256, 0, s>>>(slot, neg_scale, c->params, c->d);
    c->launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_apply(deco_ctx *c, const deco_pair *slot, uint64_t positions, float neg_scale,
                         cudaStream_t s)
{
    if (positions == 0) return cudaSuccess;
    uint64_t blocks = (positions + 4 * 256 - 1) / (4 * 256);
    if (blocks > 148ull * 16) blocks = 148ull * 16;
    apply_kernel<<<static_cast<uint32_t>(blocks), 256, 0, s>>>(slot, positions, neg_scale,
                                                               c->params, c->d, c->dev_status);
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace deco
