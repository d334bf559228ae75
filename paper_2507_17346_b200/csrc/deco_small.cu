// Per-layer Top-k, layers of at most one tile (normalisation vectors, biases, small kernels):
// the worker side of Algorithm 1 for one (layer, worker) pair by a single CTA, all such pairs
// of a model in one launch.  The whole layer sits in shared memory: a = e + gamma*g, an exact
// radix selection of the k-th largest |a| (8 + 8 + 8 + 7 key bits, ties to the lower index),
// the message in index order and the residual, in the layouts of the layer's own context.
#include "deco_internal.h"

namespace deco {

namespace {

constexpr uint32_t FULL = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t key_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

__device__ __forceinline__ void latch_small(uint32_t *status, uint32_t code, uint32_t a, uint32_t b)
{
    if (atomicCAS(status, 0u, code) == 0u) {
        status[1] = a;
        status[2] = b;
    }
}

template <int GT>
__device__ __forceinline__ float grad_at(const char *grow, uint32_t j)
{
    if (GT) return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t *>(grow)[j]) << 16);
    return reinterpret_cast<const float *>(grow)[j];
}

// Entry order inside the layer is (warp, round, lane): warp w owns the 1024 consecutive entries
// from w * 1024, lane l the entry r * 32 + l of them in round r, so that ballots walk the
// entries in index order and shared memory is read without bank conflicts.
template <int GT>
__global__ void __launch_bounds__(BLOCK)
small_worker_kernel(const SmallLayer *__restrict__ table, const void *__restrict__ grads,
                    uint64_t g_stride, float alpha)
{
    static_assert(BLOCK == 256 && TILE == 8192, "one bin per thread, 32 rounds per warp");
    const SmallLayer L = table[blockIdx.x];
    const uint32_t i = blockIdx.y;
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    __shared__ float a[TILE];
    __shared__ uint32_t h[BLOCK];
    __shared__ uint32_t s_w[WARPS];
    __shared__ uint32_t s_gt[WARPS], s_eq[WARPS];
    __shared__ uint32_t s_pick[2];
    float *erow = L.e + static_cast<size_t>(i) * L.e_stride;
    const char *grow = reinterpret_cast<const char *>(grads) +
                       (static_cast<size_t>(i) * g_stride + L.g_off) * (GT ? 2 : 4);
    const uint32_t d = L.d, k = L.k;
    if (d == 0 || d > static_cast<uint32_t>(TILE) || k == 0 || k > d) {
        if (t == 0) latch_small(L.status, DECO_ERR_DEVICE_CHECK, 0x600u, d);
        return;
    }
    for (uint32_t j = t; j < static_cast<uint32_t>(TILE); j += BLOCK)
        a[j] = j < d ? __fmaf_rn(alpha, grad_at<GT>(grow, j), erow[j]) : 0.0f;
    __syncthreads();

    // threshold key: the bin of the k-th largest key, eight bits at a time
    uint32_t prefix = 0, k_rem = k, n_greater = 0;
#pragma unroll 1
    for (int level = 0; level < 4; ++level) {
        const int bits = level == 3 ? 7 : 8;
        const int shift = level == 3 ? 0 : 23 - 8 * level;
        h[t] = 0;
        __syncthreads();
        for (uint32_t j = t; j < d; j += BLOCK) {
            const uint32_t key = key_bits(a[j]);
            if ((key >> (shift + bits)) == prefix) atomicAdd(&h[(key >> shift) & ((1u << bits) - 1u)], 1u);
        }
        __syncthreads();
        // thread t looks at bin 255 - t: the prefix over threads counts the higher bins
        const uint32_t cnt = h[BLOCK - 1 - t];
        uint32_t incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(FULL, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) s_w[w] = incl;
        if (t == 0) s_pick[0] = 0xFFFFFFFFu;
        __syncthreads();
        uint32_t above = incl - cnt;
#pragma unroll
        for (int ww = 0; ww < WARPS; ++ww) above += (ww < w) ? s_w[ww] : 0u;
        if (above < k_rem && above + cnt >= k_rem) {
            s_pick[0] = static_cast<uint32_t>(BLOCK - 1 - t);
            s_pick[1] = above;
        }
        __syncthreads();
        const uint32_t bin = s_pick[0];
        if (bin == 0xFFFFFFFFu) {                            // fewer than k_rem keys: cannot happen
            if (t == 0) latch_small(L.status, DECO_ERR_DEVICE_CHECK, 0x601u + level, i);
            return;
        }
        n_greater += s_pick[1];
        k_rem -= s_pick[1];
        prefix = (prefix << bits) | bin;
        __syncthreads();
    }
    const uint32_t T = prefix, take = k_rem;                 // ties taken, in index order

    // entries above the threshold and ties per warp
    const uint32_t wbase = static_cast<uint32_t>(w) * 1024u;
    uint32_t gt_w = 0, eq_w = 0;
#pragma unroll 4
    for (int r = 0; r < 32; ++r) {
        const uint32_t j = wbase + r * 32 + lane;
        const uint32_t key = key_bits(a[j]);
        gt_w += __popc(__ballot_sync(FULL, j < d && key > T));
        eq_w += __popc(__ballot_sync(FULL, j < d && key == T));
    }
    if (lane == 0) {
        s_gt[w] = gt_w;
        s_eq[w] = eq_w;
    }
    __syncthreads();
    uint32_t eq_run = 0, sel_run = 0;                        // ties / selected entries before this warp
    for (int ww = 0; ww < w; ++ww) {
        const uint32_t e_ = s_eq[ww];
        const uint32_t left = take > eq_run ? take - eq_run : 0u;
        sel_run += s_gt[ww] + (e_ < left ? e_ : left);
        eq_run += e_;
    }
    deco_pair *out = L.msg + static_cast<size_t>(i) * L.k_cap;
    const uint32_t below = (1u << lane) - 1u;
#pragma unroll 2
    for (int r = 0; r < 32; ++r) {
        const uint32_t j = wbase + r * 32 + lane;
        const float v = a[j];
        const uint32_t key = key_bits(v);
        const bool in = j < d;
        const uint32_t m_eq = __ballot_sync(FULL, in && key == T);
        const bool sel = in && (key > T || (key == T && eq_run + __popc(m_eq & below) < take));
        const uint32_t m_sel = __ballot_sync(FULL, sel);
        if (sel) {
            const uint32_t pos = sel_run + __popc(m_sel & below);
            if (pos < k) {
                deco_pair pr;
                pr.idx = j;
                pr.val = v;
                out[pos] = pr;
            } else {
                latch_small(L.status, DECO_ERR_DEVICE_CHECK, 0x610u, j);
            }
        }
        if (in) erow[j] = sel ? 0.0f : v;
        eq_run += __popc(m_eq);
        sel_run += __popc(m_sel);
    }
    if (w == WARPS - 1 && lane == 0) {
        if (sel_run != k) latch_small(L.status, DECO_ERR_DEVICE_CHECK, 0x611u, sel_run);
        L.tile_start[static_cast<size_t>(i) * 2] = 0;
        L.tile_start[static_cast<size_t>(i) * 2 + 1] = k;
        SelectState &s = L.sel[i];
        s.threshold = T;
        s.ties_take = take;
        s.n_greater = n_greater;
        s.k_rem = take;
        s.exact = 0;
        s.staged_band = 0;
        s.cert_key = SPEC_DISABLED;
        s.spec_key = SPEC_DISABLED;
    }
}

}  // namespace

cudaError_t launch_small_workers(const SmallLayer *table, uint32_t layers, uint32_t n, const void *grads,
                                 uint64_t g_stride, int grad_dtype, float alpha, cudaStream_t s)
{
    if (layers == 0) return cudaSuccess;
    const dim3 grid(layers, n);
    if (grad_dtype == DECO_BF16)
        small_worker_kernel<1><<<grid, BLOCK, 0, s>>>(table, grads, g_stride, alpha);
    else
        small_worker_kernel<0><<<grid, BLOCK, 0, s>>>(table, grads, g_stride, alpha);
    return cudaGetLastError();
}

}  // namespace deco
