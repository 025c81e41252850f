// Exclusive prefix sums of int32 counts (row lengths -> CSR row pointers; Alg. 1 step 2 bookkeeping).
// Two levels, three launches, no inter-block waiting: block totals, scan of the totals, final write.
#include "grf_internal.cuh"

namespace {

constexpr int SCAN_THREADS = 1024;
constexpr int SCAN_ITEMS = 4;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

__device__ __forceinline__ int32_t warp_inclusive_scan(int32_t x, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    return x;
}

// Exclusive scan of one value per thread across the block; the block total goes to *total (shared).
__device__ __forceinline__ int32_t block_exclusive_scan(int32_t x, int32_t* total)
{
    __shared__ int32_t warp_sums[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t inc = warp_inclusive_scan(x, lane);
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int nw = blockDim.x >> 5;
        const int32_t ws = lane < nw ? warp_sums[lane] : 0;
        const int32_t wi = warp_inclusive_scan(ws, lane);
        warp_sums[lane] = wi - ws;
        if (lane == 31) *total = wi;
    }
    __syncthreads();
    const int32_t r = inc - x + warp_sums[warp];
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(SCAN_THREADS)
scan_block_totals_kernel(const int32_t* __restrict__ in, int32_t n, int32_t* __restrict__ block_totals)
{
    __shared__ int32_t total;
    const int32_t* src = in + (size_t)blockIdx.y * n;
    const int32_t base = blockIdx.x * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
    int32_t s = 0;
#pragma unroll
    for (int q = 0; q < SCAN_ITEMS; ++q)
        if (base + q < n) s += src[base + q];
    block_exclusive_scan(s, &total);
    if (threadIdx.x == 0) block_totals[(size_t)blockIdx.y * gridDim.x + blockIdx.x] = total;
}

__global__ void __launch_bounds__(SCAN_THREADS)
scan_totals_kernel(int32_t* __restrict__ block_totals, int32_t nblocks)
{
    __shared__ int32_t total;
    int32_t* t = block_totals + (size_t)blockIdx.x * nblocks;
    int32_t carry = 0;
    for (int32_t base = 0; base < nblocks; base += SCAN_THREADS) {
        const int32_t idx = base + threadIdx.x;
        const int32_t x = idx < nblocks ? t[idx] : 0;
        const int32_t ex = block_exclusive_scan(x, &total);
        if (idx < nblocks) t[idx] = carry + ex;
        carry += total;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(SCAN_THREADS)
scan_write_kernel(const int32_t* __restrict__ in, int32_t n, const int32_t* __restrict__ block_offsets,
                  int32_t* __restrict__ out)
{
    __shared__ int32_t total;
    const int32_t* src = in + (size_t)blockIdx.y * n;
    int32_t* dst = out + (size_t)blockIdx.y * ((size_t)n + 1);
    const int32_t base = blockIdx.x * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
    int32_t v[SCAN_ITEMS];
    int32_t s = 0;
#pragma unroll
    for (int q = 0; q < SCAN_ITEMS; ++q) {
        v[q] = base + q < n ? src[base + q] : 0;
        s += v[q];
    }
    int32_t run = block_exclusive_scan(s, &total) + block_offsets[(size_t)blockIdx.y * gridDim.x + blockIdx.x];
#pragma unroll
    for (int q = 0; q < SCAN_ITEMS; ++q) {
        if (base + q < n) dst[base + q] = run;
        run += v[q];
        if (base + q == n - 1) dst[n] = run;
    }
}

}  // namespace

int grf_exclusive_scan(grf_ctx* ctx, const int32_t* in, int32_t* out, int32_t n, int32_t segments)
{
    if (n <= 0 || segments <= 0) return GRF_ERR_INVALID;
    const int nblocks = grf_ceil_div(n, SCAN_TILE);
    GRF_TRY(grf_buf_reserve(&ctx->scan_blocks, sizeof(int32_t) * (size_t)nblocks * segments));
    int32_t* totals = (int32_t*)ctx->scan_blocks.ptr;
    const dim3 grid(nblocks, segments);
    {
        grf_launch_scope scope(ctx, 1, 3);
        scan_block_totals_kernel<<<grid, SCAN_THREADS, 0, ctx->stream>>>(in, n, totals);
        scan_totals_kernel<<<segments, SCAN_THREADS, 0, ctx->stream>>>(totals, nblocks);
        scan_write_kernel<<<grid, SCAN_THREADS, 0, ctx->stream>>>(in, n, totals, out);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    return GRF_OK;
}

// Same three launches with the block-total scratch supplied by the caller (needs ceil(n / 4096) * segments
// int32 entries) and no context: used where nothing may be allocated.
int grf_exclusive_scan_scratch(cudaStream_t stream, const int32_t* in, int32_t* out, int32_t n, int32_t segments,
                               int32_t* totals)
{
    if (n <= 0 || segments <= 0 || !totals) return GRF_ERR_INVALID;
    const int nblocks = grf_ceil_div(n, SCAN_TILE);
    const dim3 grid(nblocks, segments);
    scan_block_totals_kernel<<<grid, SCAN_THREADS, 0, stream>>>(in, n, totals);
    scan_totals_kernel<<<segments, SCAN_THREADS, 0, stream>>>(totals, nblocks);
    scan_write_kernel<<<grid, SCAN_THREADS, 0, stream>>>(in, n, totals, out);
    GRF_CUDA_TRY(cudaGetLastError());
    return GRF_OK;
}
