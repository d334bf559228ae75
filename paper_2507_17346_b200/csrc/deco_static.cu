// deco_topk_compress_static: Top-k compression of one vector with no allocation anywhere.
//
// Some callers cannot allocate device memory when they need a compressed update: code that
// runs while a CUDA stream is being captured, plugins living inside a host program that owns
// the whole memory pool, and latency-critical loops where cudaMalloc's implicit
// synchronisation is not acceptable.  For them the working memory of the selection
// (histograms, the selection record and the per-tile counters) sits in one file-scope device
// array of fixed size, which every GPU that loads the library carries until the process
// exits.  The price is a hard limit on the vector length and no concurrency: all calls share
// the array.
//
// The kernels here are self-contained (nothing is shared with the context-based path): three
// radix-histogram passes over the magnitude keys fix the threshold, one pass counts per tile,
// one CTA turns the counts into message positions, one pass writes the pairs in index order.
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>
#include <mutex>

#include "deco.h"

namespace {

constexpr int ST_TILE = 8192;                    // entries per tile
constexpr int ST_BLOCK = 256;
constexpr int ST_PER_THREAD = ST_TILE / ST_BLOCK;   // 32 consecutive entries per thread
constexpr int ST_BINS = 4096;
constexpr uint32_t ST_MAX_TILES = DECO_STATIC_MAX_D / ST_TILE;   // 2048

// Layout of the scratch array, in 32-bit words.
constexpr uint32_t OFF_HIST = 0;                                 // [3][ST_BINS]
constexpr uint32_t OFF_STATE = OFF_HIST + 3 * ST_BINS;           // 16 words, see below
constexpr uint32_t OFF_TILE_GT = OFF_STATE + 16;                 // [ST_MAX_TILES]
constexpr uint32_t OFF_TILE_EQ = OFF_TILE_GT + ST_MAX_TILES;     // [ST_MAX_TILES]
constexpr uint32_t OFF_TILE_TAKE = OFF_TILE_EQ + ST_MAX_TILES;   // [ST_MAX_TILES]
constexpr uint32_t OFF_TILE_START = OFF_TILE_TAKE + ST_MAX_TILES;   // [ST_MAX_TILES + 1]
constexpr uint32_t SCRATCH_WORDS = OFF_TILE_START + ST_MAX_TILES + 1 + 15;
// state words: 0 prefix, 1 k_rem, 2 n_greater, 3 threshold, 4 ties_take

// The scratch memory itself: 82 KB per GPU, alive from library load to process exit.
static __device__ __align__(256) uint32_t deco_static_scratch[SCRATCH_WORDS];

__device__ __forceinline__ uint32_t st_key(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

__device__ __forceinline__ uint32_t st_warp_scan(uint32_t v)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Exclusive scan over a CTA of ST_BLOCK threads; s_w has 9 words.
__device__ __forceinline__ uint32_t st_block_scan(uint32_t v, uint32_t *s_w, uint32_t &total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t incl = st_warp_scan(v);
    if (lane == 31) s_w[w] = incl;
    __syncthreads();
    uint32_t before = 0, tot = 0;
#pragma unroll
    for (int ww = 0; ww < ST_BLOCK / 32; ++ww) {
        const uint32_t x = s_w[ww];
        before += (ww < w) ? x : 0u;
        tot += x;
    }
    total = tot;
    __syncthreads();
    return before + incl - v;
}

// Everything that must start from zero is cleared here: the array keeps the last call's data.
__global__ void st_clear_kernel(uint32_t *scratch, uint32_t k, uint32_t ntiles)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t stride = gridDim.x * blockDim.x;
    for (uint32_t q = t; q < 3 * ST_BINS; q += stride) scratch[OFF_HIST + q] = 0;
    for (uint32_t q = t; q < 16; q += stride) scratch[OFF_STATE + q] = (q == 1) ? k : 0u;
    for (uint32_t q = t; q < ntiles; q += stride) {
        scratch[OFF_TILE_GT + q] = 0;
        scratch[OFF_TILE_EQ + q] = 0;
        scratch[OFF_TILE_TAKE + q] = 0;
    }
    for (uint32_t q = t; q <= ntiles; q += stride) scratch[OFF_TILE_START + q] = 0;
}

template <int LEVEL>
__global__ void __launch_bounds__(ST_BLOCK)
st_hist_kernel(const float *__restrict__ a, uint64_t d, uint32_t *scratch)
{
    __shared__ uint32_t h[ST_BINS];
    for (int b = threadIdx.x; b < ST_BINS; b += ST_BLOCK) h[b] = 0;
    __syncthreads();
    const uint32_t prefix = scratch[OFF_STATE + 0];
    for (uint64_t j = static_cast<uint64_t>(blockIdx.x) * ST_BLOCK + threadIdx.x; j < d;
         j += static_cast<uint64_t>(gridDim.x) * ST_BLOCK) {
        const uint32_t key = st_key(a[j]);
        if (LEVEL == 0) atomicAdd(&h[key >> 19], 1u);
        else if (LEVEL == 1) { if ((key >> 19) == prefix) atomicAdd(&h[(key >> 7) & 0xFFFu], 1u); }
        else { if ((key >> 7) == prefix) atomicAdd(&h[key & 0x7Fu], 1u); }
    }
    __syncthreads();
    uint32_t *out = scratch + OFF_HIST + LEVEL * ST_BINS;
    for (int b = threadIdx.x; b < ST_BINS; b += ST_BLOCK)
        if (h[b]) atomicAdd(&out[b], h[b]);
}

// One CTA: walk the histogram from the top bin down until k_rem entries are covered.
template <int LEVEL>
__global__ void __launch_bounds__(ST_BLOCK) st_pick_kernel(uint32_t *scratch)
{
    constexpr int BITS = (LEVEL == 2) ? 7 : 12;
    constexpr int PER = ST_BINS / ST_BLOCK;
    __shared__ uint32_t s_w[9];
    const uint32_t *h = scratch + OFF_HIST + LEVEL * ST_BINS;
    uint32_t *st = scratch + OFF_STATE;
    const uint32_t k_rem = st[1];
    // thread t owns bins [t*PER, (t+1)*PER); scan from the top: reverse the thread order
    const int rt = ST_BLOCK - 1 - threadIdx.x;
    uint32_t loc[PER], sum = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) {
        loc[b] = h[rt * PER + b];
        sum += loc[b];
    }
    uint32_t total;
    const uint32_t above = st_block_scan(sum, s_w, total);     // entries in bins above mine
    if (above < k_rem && above + sum >= k_rem) {
        uint32_t acc = above;
        int bin = rt * PER;
#pragma unroll
        for (int b = PER - 1; b >= 0; --b) {
            if (acc + loc[b] >= k_rem) {
                bin = rt * PER + b;
                break;
            }
            acc += loc[b];
        }
        st[2] += acc;
        st[1] = k_rem - acc;
        const uint32_t prefix = (st[0] << BITS) | static_cast<uint32_t>(bin);
        st[0] = prefix;
        if (LEVEL == 2) {
            st[3] = prefix;
            st[4] = k_rem - acc;
        }
    }
}

__global__ void __launch_bounds__(ST_BLOCK)
st_count_kernel(const float *__restrict__ a, uint64_t d, uint32_t *scratch)
{
    __shared__ uint32_t s_gt, s_eq;
    if (threadIdx.x == 0) s_gt = s_eq = 0;
    __syncthreads();
    const uint32_t T = scratch[OFF_STATE + 3];
    const uint64_t base = static_cast<uint64_t>(blockIdx.x) * ST_TILE +
                          static_cast<uint64_t>(threadIdx.x) * ST_PER_THREAD;
    uint32_t gt = 0, eq = 0;
    for (int c = 0; c < ST_PER_THREAD; ++c)
        if (base + c < d) {
            const uint32_t key = st_key(a[base + c]);
            gt += key > T;
            eq += key == T;
        }
    if (gt) atomicAdd(&s_gt, gt);
    if (eq) atomicAdd(&s_eq, eq);
    __syncthreads();
    if (threadIdx.x == 0) {
        scratch[OFF_TILE_GT + blockIdx.x] = s_gt;
        scratch[OFF_TILE_EQ + blockIdx.x] = s_eq;
    }
}

// One CTA: ties go to tiles in index order, then every tile gets its message position.
__global__ void __launch_bounds__(ST_BLOCK) st_scan_kernel(uint32_t *scratch, uint32_t ntiles)
{
    __shared__ uint32_t s_w[9];
    const uint32_t *gt = scratch + OFF_TILE_GT, *eq = scratch + OFF_TILE_EQ;
    uint32_t *take = scratch + OFF_TILE_TAKE, *start = scratch + OFF_TILE_START;
    const uint32_t ties = scratch[OFF_STATE + 4];
    const uint32_t per = (ntiles + ST_BLOCK - 1) / ST_BLOCK;
    const uint32_t lo = min(ntiles, threadIdx.x * per), hi = min(ntiles, lo + per);
    uint32_t eq_sum = 0;
    for (uint32_t t = lo; t < hi; ++t) eq_sum += eq[t];
    uint32_t tot;
    uint32_t eq_before = st_block_scan(eq_sum, s_w, tot);
    uint32_t sel_sum = 0;
    for (uint32_t t = lo; t < hi; ++t) {
        const uint32_t left = ties > eq_before ? ties - eq_before : 0u;
        const uint32_t tk = min(eq[t], left);
        take[t] = tk;
        sel_sum += gt[t] + tk;
        eq_before += eq[t];
    }
    uint32_t pos = st_block_scan(sel_sum, s_w, tot);
    for (uint32_t t = lo; t < hi; ++t) {
        start[t] = pos;
        pos += gt[t] + take[t];
    }
    if (threadIdx.x == 0) start[ntiles] = tot;
}

__global__ void __launch_bounds__(ST_BLOCK)
st_emit_kernel(const float *__restrict__ a, uint64_t d, uint32_t k, const uint32_t *scratch,
               deco_pair *__restrict__ msg)
{
    __shared__ uint32_t s_w[9];
    const uint32_t tile = blockIdx.x;
    const uint32_t T = scratch[OFF_STATE + 3];
    const uint32_t take = scratch[OFF_TILE_TAKE + tile];
    const uint32_t start = scratch[OFF_TILE_START + tile];
    const uint64_t base = static_cast<uint64_t>(tile) * ST_TILE +
                          static_cast<uint64_t>(threadIdx.x) * ST_PER_THREAD;
    uint32_t gt = 0, eq = 0;                                    // one bit per owned entry
    for (int c = 0; c < ST_PER_THREAD; ++c)
        if (base + c < d) {
            const uint32_t key = st_key(a[base + c]);
            gt |= (key > T) ? (1u << c) : 0u;
            eq |= (key == T) ? (1u << c) : 0u;
        }
    uint32_t tot;
    uint32_t rank = st_block_scan(__popc(eq), s_w, tot);        // ties before mine, by index
    uint32_t pick = gt;
    for (int c = 0; c < ST_PER_THREAD; ++c)
        if (eq & (1u << c)) {
            if (rank < take) pick |= 1u << c;
            ++rank;
        }
    uint32_t pos = start + st_block_scan(__popc(pick), s_w, tot);
    for (int c = 0; c < ST_PER_THREAD; ++c)
        if (pick & (1u << c)) {
            if (pos < k) {
                deco_pair pr;
                pr.idx = static_cast<uint32_t>(base + c);
                pr.val = a[base + c];
                msg[pos] = pr;
            }
            ++pos;
        }
}

// Device address of the scratch array, looked up once per device.
constexpr int ST_MAX_DEVICES = 64;
uint32_t *g_scratch_addr[ST_MAX_DEVICES] = {};
std::mutex g_scratch_mutex;

deco_status scratch_for_current_device(uint32_t **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= ST_MAX_DEVICES) return DECO_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        // In host code the array's name is only a handle; the kernels need its device address.
        uint32_t *ptr = nullptr;
        const cudaError_t err = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr),
                                                     deco_static_scratch);
        if (err != cudaSuccess || !ptr) {
            cudaGetLastError();
            std::fprintf(stderr, "libdeco: cudaGetSymbolAddress failed: %s\n",
                         cudaGetErrorString(err));
            return DECO_ERR_CUDA;
        }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return DECO_OK;
}

}  // namespace

extern "C" deco_status deco_topk_compress_static(const float *a, uint64_t d, uint64_t k,
                                                 deco_pair *msg_out, void *stream)
{
    if (!a || !msg_out || d == 0 || k == 0 || k > d) return DECO_ERR_INVALID_ARG;
    if (d > DECO_STATIC_MAX_D) {
        std::fprintf(stderr,
                     "libdeco: deco_topk_compress_static handles at most %llu entries (got %llu); "
                     "use a context (deco_init) for longer vectors\n",
                     static_cast<unsigned long long>(DECO_STATIC_MAX_D),
                     static_cast<unsigned long long>(d));
        return DECO_ERR_CAPACITY;
    }
    uint32_t *scratch = nullptr;
    const deco_status st = scratch_for_current_device(&scratch);
    if (st != DECO_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t ntiles = static_cast<uint32_t>((d + ST_TILE - 1) / ST_TILE);
    const uint32_t k32 = static_cast<uint32_t>(k);
    uint32_t hblocks = static_cast<uint32_t>((d + ST_BLOCK * 16 - 1) / (ST_BLOCK * 16));
    if (hblocks > 148 * 8) hblocks = 148 * 8;
    // an error some earlier, unrelated launch of this thread left behind is not this call's
    (void)cudaGetLastError();
    st_clear_kernel<<<32, 256, 0, s>>>(scratch, k32, ntiles);
    st_hist_kernel<0><<<hblocks, ST_BLOCK, 0, s>>>(a, d, scratch);
    st_pick_kernel<0><<<1, ST_BLOCK, 0, s>>>(scratch);
    st_hist_kernel<1><<<hblocks, ST_BLOCK, 0, s>>>(a, d, scratch);
    st_pick_kernel<1><<<1, ST_BLOCK, 0, s>>>(scratch);
    st_hist_kernel<2><<<hblocks, ST_BLOCK, 0, s>>>(a, d, scratch);
    st_pick_kernel<2><<<1, ST_BLOCK, 0, s>>>(scratch);
    st_count_kernel<<<ntiles, ST_BLOCK, 0, s>>>(a, d, scratch);
    st_scan_kernel<<<1, ST_BLOCK, 0, s>>>(scratch, ntiles);
    st_emit_kernel<<<ntiles, ST_BLOCK, 0, s>>>(a, d, k32, scratch, msg_out);
    return cudaGetLastError() == cudaSuccess ? DECO_OK : DECO_ERR_CUDA;
}
