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

__global__ void __launch_bounds__(BLOCK)
aggregate_kernel(const deco_pair *__restrict__ msg, uint64_t k_cap,
                 const uint32_t *__restrict__ tile_start, uint32_t ntiles, uint32_t n,
                 deco_pair *__restrict__ slot, uint64_t positions, uint32_t *__restrict__ status)
{
    static_assert(TILE / 32 == BLOCK, "one mask word per thread");
    __shared__ float acc[TILE];
    __shared__ uint32_t mask[TILE / 32];
    __shared__ uint32_t s_w[WARPS];
    for (int q = threadIdx.x; q < TILE; q += BLOCK) acc[q] = 0.0f;
    mask[threadIdx.x] = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;

    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        uint64_t out_off = 0;
        uint32_t cap = 0, longest = 0;
        for (uint32_t i = 0; i < n; ++i) {
            const uint32_t a = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile];
            const uint32_t b = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile + 1];
            out_off += a;
            cap += b - a;
            longest = max(longest, b - a);
        }
        if (cap == 0) continue;
        if (out_off + cap > positions) {
            if (threadIdx.x == 0) latch(status, DECO_ERR_DEVICE_CHECK, 0x400u, tile);
            continue;
        }
        const uint32_t first = tile * static_cast<uint32_t>(TILE);
        if (n <= PREFETCH_WORKERS && longest <= static_cast<uint32_t>(BLOCK)) {
            // Sparse case: at most one entry per thread and worker.  All loads are issued
            // before the first barrier, then the workers are added in order from registers.
            deco_pair pre[PREFETCH_WORKERS];
#pragma unroll
            for (uint32_t i = 0; i < PREFETCH_WORKERS; ++i) {
                pre[i].idx = DECO_NO_INDEX;
                pre[i].val = 0.0f;
                if (i < n) {
                    const uint32_t a = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile];
                    const uint32_t b = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile + 1];
                    if (a + threadIdx.x < b) pre[i] = msg[static_cast<size_t>(i) * k_cap + a + threadIdx.x];
                }
            }
#pragma unroll
            for (uint32_t i = 0; i < PREFETCH_WORKERS; ++i) {
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
                const uint32_t a = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile];
                const uint32_t b = tile_start[static_cast<size_t>(i) * (ntiles + 1) + tile + 1];
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
}

__global__ void __launch_bounds__(256)
apply_kernel(const deco_pair *__restrict__ slot, uint64_t positions, float neg_scale,
             float *__restrict__ params, uint64_t d, uint32_t *__restrict__ status)
{
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t p = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
         p < positions; p += stride) {
        const deco_pair pr = slot[p];
        if (pr.idx == DECO_NO_INDEX) continue;
        if (pr.idx >= d) {
            latch(status, DECO_ERR_DEVICE_CHECK, 0x500u, pr.idx);
            continue;
        }
        params[pr.idx] = __fmaf_rn(neg_scale, pr.val, params[pr.idx]);
    }
}

}  // namespace

cudaError_t launch_aggregate(deco_ctx *c, deco_pair *slot, cudaStream_t s)
{
    // next to the streaming pass of the following iteration the aggregation takes half the
    // CTA slots it could hold, so that the pass keeps most of its loads in flight
    const uint32_t per_sm = (c->agg_stream && s == c->agg_stream) ? 3u : 6u;
    const uint32_t blocks = c->ntiles < 148u * per_sm ? c->ntiles : 148u * per_sm;
    aggregate_kernel<<<blocks, BLOCK, 0, s>>>(c->msg, c->k_cap, c->tile_start, c->ntiles, c->n,
                                              slot, static_cast<uint64_t>(c->n) * c->k_of_msg,
                                              c->dev_status);
    c->launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_apply(deco_ctx *c, const deco_pair *slot, uint64_t positions, float neg_scale,
                         cudaStream_t s)
{
    if (positions == 0) return cudaSuccess;
    uint64_t blocks = (positions + 255) / 256;
    if (blocks > 148ull * 16) blocks = 148ull * 16;
    apply_kernel<<<static_cast<uint32_t>(blocks), 256, 0, s>>>(slot, positions, neg_scale,
                                                               c->params, c->d, c->dev_status);
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace deco
