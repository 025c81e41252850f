// Psi -> Psi^T: regroup a CSR matrix by column (Alg. 1 step 5 needs, for every node l, the list of
// keys j with Psi_jl != 0, so that Phi_K^T V becomes a segmented reduction with a fixed order).
//
// Bucket sort keyed on the full column index: count per column (integer atomics, order-free), scan,
// scatter into the buckets in arrival order, then order every bucket by source row.  Source rows
// inside a bucket are distinct, so the result is unique whatever the arrival order was.
#include "grf_internal.cuh"

namespace {

__global__ void __launch_bounds__(256)
column_histogram_kernel(int64_t nnz, const int32_t* __restrict__ col, int32_t* __restrict__ counts)
{
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < nnz; p += (int64_t)gridDim.x * blockDim.x)
        atomicAdd(counts + col[p], 1);
}

__global__ void __launch_bounds__(256)
bucket_scatter_kernel(int32_t rows, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                      const float* __restrict__ val, int32_t* __restrict__ cursor,
                      int32_t* __restrict__ tmp_row, float* __restrict__ tmp_val)
{
    const int lane = threadIdx.x & 31;
    const int32_t r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= rows) return;
    for (int32_t p = rowptr[r] + lane; p < rowptr[r + 1]; p += 32) {
        const int32_t dst = atomicAdd(cursor + col[p], 1);
        tmp_row[dst] = r;
        tmp_val[dst] = val[p];
    }
}

constexpr int BUCKET_SMEM = 1024;  // entries of one bucket staged per warp
constexpr int BUCKET_RANKED = 192; // up to this length ranking (len^2 / 32 comparisons per lane) beats the sorting network

// A warp sorts n (row, value) pairs by row, ascending, in place (shared or global memory): a bitonic network whose
// comparators all point the same way (every merge starts by comparing i with its mirror image in the block), so
// that a length that is no power of two needs no padding: a comparator whose upper end lies beyond n is skipped.
__device__ __forceinline__ void warp_sort_pairs(int32_t* rows, float* vals, int32_t n, int lane)
{
    int32_t P = 1;
    while (P < n) P <<= 1;
    auto exchange = [&](int32_t a, int32_t b) {
        if (b < n) {
            const int32_t ra = rows[a], rb = rows[b];
            if (rb < ra) {
                rows[a] = rb; rows[b] = ra;
                const float va = vals[a]; vals[a] = vals[b]; vals[b] = va;
            }
        }
    };
    for (int32_t k = 2; k <= P; k <<= 1) {
        const int32_t h = k >> 1;
        for (int32_t i = lane; i < (P >> 1); i += 32) {
            const int32_t blk = i / h, off = i - blk * h;
            exchange(blk * k + off, blk * k + (k - 1 - off));
        }
        __syncwarp();
        for (int32_t j = h >> 1; j >= 1; j >>= 1) {
            for (int32_t i = lane; i < (P >> 1); i += 32) {
                const int32_t a = (i / j) * 2 * j + (i % j);
                exchange(a, a + j);
            }
            __syncwarp();
        }
    }
}

// One warp per bucket: its entries are ordered by source row (rows are distinct, so the result is unique).  This
// kernel takes the buckets of up to BUCKET_RANKED entries: each element's place is the number of smaller rows.
__global__ void __launch_bounds__(128)
bucket_order_kernel(int32_t cols, const int32_t* __restrict__ t_rowptr,
                    const int32_t* __restrict__ tmp_row, const float* __restrict__ tmp_val,
                    int32_t* __restrict__ t_col, float* __restrict__ t_val)
{
    __shared__ int32_t staged[4][BUCKET_RANKED];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t c = blockIdx.x * 4 + warp;
    if (c >= cols) return;
    const int32_t beg = t_rowptr[c], len = t_rowptr[c + 1] - beg;
    if (len > BUCKET_RANKED) return;
    for (int32_t x = lane; x < len; x += 32) staged[warp][x] = tmp_row[beg + x];
    __syncwarp();
    for (int32_t x = lane; x < len; x += 32) {
        const int32_t mine = staged[warp][x];
        int32_t rank = 0;
        for (int32_t y = 0; y < len; ++y) rank += staged[warp][y] < mine;
        t_col[beg + rank] = mine;
        t_val[beg + rank] = tmp_val[beg + x];
    }
}

// The longer buckets (hub columns): sorted by the network above, in shared memory when they fit, else in place in
// the scratch arrays.
__global__ void __launch_bounds__(128)
bucket_sort_long_kernel(int32_t cols, const int32_t* __restrict__ t_rowptr,
                        int32_t* __restrict__ tmp_row, float* __restrict__ tmp_val,
                        int32_t* __restrict__ t_col, float* __restrict__ t_val)
{
    __shared__ int32_t staged[4][BUCKET_SMEM];
    __shared__ float staged_val[4][BUCKET_SMEM];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t c = blockIdx.x * 4 + warp;
    if (c >= cols) return;
    const int32_t beg = t_rowptr[c], len = t_rowptr[c + 1] - beg;
    if (len <= BUCKET_RANKED) return;
    if (len <= BUCKET_SMEM) {
        for (int32_t x = lane; x < len; x += 32) { staged[warp][x] = tmp_row[beg + x]; staged_val[warp][x] = tmp_val[beg + x]; }
        __syncwarp();
        warp_sort_pairs(staged[warp], staged_val[warp], len, lane);
        for (int32_t x = lane; x < len; x += 32) { t_col[beg + x] = staged[warp][x]; t_val[beg + x] = staged_val[warp][x]; }
    } else {
        warp_sort_pairs(tmp_row + beg, tmp_val + beg, len, lane);
        for (int32_t x = lane; x < len; x += 32) { t_col[beg + x] = tmp_row[beg + x]; t_val[beg + x] = tmp_val[beg + x]; }
    }
}

__global__ void copy_i32_kernel(const int32_t* __restrict__ src, int32_t* __restrict__ dst, int32_t n)
{
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = src[i];
}

}  // namespace

int grf_transpose_launch(grf_ctx* ctx, int32_t rows, int32_t cols, int64_t nnz,
                         const int32_t* rowptr, const int32_t* col, const float* val,
                         int32_t* t_rowptr, int32_t* t_col, float* t_val)
{
    if (rows <= 0 || cols <= 0 || nnz < 0) return GRF_ERR_INVALID;
    if (nnz >= (1ll << 31)) return GRF_ERR_TOO_LARGE;
    // scratch: per-column counts, later the scatter cursors; and the unordered buckets
    GRF_TRY(grf_buf_reserve(&ctx->t_cursor, sizeof(int32_t) * ((size_t)cols + 1)));
    // grown with head-room: resampling changes nnz a little every time, and a reallocation stalls the stream
    if (ctx->t_tmp_col.bytes < sizeof(int32_t) * (size_t)nnz || ctx->t_tmp_val.bytes < sizeof(float) * (size_t)nnz) {
        const size_t cap = (size_t)nnz + (size_t)nnz / 8 + 64;
        GRF_TRY(grf_buf_reserve(&ctx->t_tmp_col, sizeof(int32_t) * cap));
        GRF_TRY(grf_buf_reserve(&ctx->t_tmp_val, sizeof(float) * cap));
    }
    int32_t* cursor = (int32_t*)ctx->t_cursor.ptr;
    GRF_CUDA_TRY(cudaMemsetAsync(cursor, 0, sizeof(int32_t) * ((size_t)cols + 1), ctx->stream));
    if (nnz > 0) {
        int blocks = grf_ceil_div(nnz, 256);
        if (blocks > 148 * 16) blocks = 148 * 16;
        grf_launch_scope scope(ctx, 3);
        column_histogram_kernel<<<blocks, 256, 0, ctx->stream>>>(nnz, col, cursor);
    }
    GRF_TRY(grf_exclusive_scan(ctx, cursor, t_rowptr, cols, 1));
    {
        grf_launch_scope scope(ctx, 3);
        copy_i32_kernel<<<grf_ceil_div(cols, 256), 256, 0, ctx->stream>>>(t_rowptr, cursor, cols);
    }
    if (nnz > 0) {
        grf_launch_scope scope(ctx, 3, 3);
        bucket_scatter_kernel<<<grf_ceil_div(rows, 8), 256, 0, ctx->stream>>>(
            rows, rowptr, col, val, cursor, (int32_t*)ctx->t_tmp_col.ptr, (float*)ctx->t_tmp_val.ptr);
        bucket_order_kernel<<<grf_ceil_div(cols, 4), 128, 0, ctx->stream>>>(
            cols, t_rowptr, (const int32_t*)ctx->t_tmp_col.ptr, (const float*)ctx->t_tmp_val.ptr, t_col, t_val);
        bucket_sort_long_kernel<<<grf_ceil_div(cols, 4), 128, 0, ctx->stream>>>(
            cols, t_rowptr, (int32_t*)ctx->t_tmp_col.ptr, (float*)ctx->t_tmp_val.ptr, t_col, t_val);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    return GRF_OK;
}

extern "C" int grf_csr_transpose(grf_ctx* ctx, int32_t rows, int32_t cols, int64_t nnz,
                                 const int32_t* rowptr, const int32_t* col, const float* val,
                                 int32_t* t_rowptr, int32_t* t_col, float* t_val)
{
    if (!ctx || !rowptr || !t_rowptr) return GRF_ERR_INVALID;
    if (nnz > 0 && (!col || !val || !t_col || !t_val)) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    return grf_transpose_launch(ctx, rows, cols, nnz, rowptr, col, val, t_rowptr, t_col, t_val);
}

// ---------------------------------------------------------------------------------------------------
// Variant that allocates nothing: its scratch is a fixed array that is part of the loaded module.

namespace {

constexpr int32_t NOALLOC_MAX_COLS = GRF_NOALLOC_MAX_COLS;
constexpr int64_t NOALLOC_MAX_NNZ = GRF_NOALLOC_MAX_NNZ;
constexpr size_t NOALLOC_CURSOR_WORDS = (size_t)NOALLOC_MAX_COLS + 64;          // counts / cursors, padded
constexpr size_t NOALLOC_TOTALS_WORDS = 64;                                     // scan block totals (<= 17 used)
constexpr size_t NOALLOC_WORDS = NOALLOC_CURSOR_WORDS + NOALLOC_TOTALS_WORDS + 2 * (size_t)NOALLOC_MAX_NNZ;

// Every GPU that loads this library holds one copy of this array until the process exits.
static __device__ __align__(256) uint32_t g_noalloc_scratch[NOALLOC_WORDS];

constexpr int NOALLOC_MAX_DEVICES = 64;
uint32_t* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};   // device address of the array, per device, once resolved

}  // namespace

extern "C" int grf_csr_transpose_noalloc(int device, void* cuda_stream, int32_t rows, int32_t cols, int64_t nnz,
                                         const int32_t* rowptr, const int32_t* col, const float* val,
                                         int32_t* t_rowptr, int32_t* t_col, float* t_val)
{
    if (device < 0 || device >= NOALLOC_MAX_DEVICES || rows <= 0 || cols <= 0 || nnz < 0 || !rowptr || !t_rowptr)
        return GRF_ERR_INVALID;
    if (nnz > 0 && (!col || !val || !t_col || !t_val)) return GRF_ERR_INVALID;
    if (cols > NOALLOC_MAX_COLS || nnz > NOALLOC_MAX_NNZ) return GRF_ERR_TOO_LARGE;
    GRF_CUDA_TRY(cudaSetDevice(device));
    if (!g_noalloc_ptr[device]) {
        // In host code the array's name only stands for the symbol; the address kernels can use has to be
        // asked for, with the owning device current.
        uint32_t* p = nullptr;
        GRF_CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_noalloc_scratch));
        if (!p) return GRF_ERR_CUDA;
        g_noalloc_ptr[device] = p;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int32_t* cursor = (int32_t*)g_noalloc_ptr[device];
    int32_t* totals = cursor + NOALLOC_CURSOR_WORDS;
    int32_t* tmp_row = totals + NOALLOC_TOTALS_WORDS;
    float* tmp_val = (float*)(tmp_row + NOALLOC_MAX_NNZ);
    // the array keeps whatever the previous call left: the per-column counts must start from zero
    GRF_CUDA_TRY(cudaMemsetAsync(cursor, 0, sizeof(int32_t) * ((size_t)cols + 1), stream));
    if (nnz > 0) {
        int blocks = grf_ceil_div(nnz, 256);
        if (blocks > 148 * 16) blocks = 148 * 16;
        column_histogram_kernel<<<blocks, 256, 0, stream>>>(nnz, col, cursor);
    }
    GRF_TRY(grf_exclusive_scan_scratch(stream, cursor, t_rowptr, cols, 1, totals));
    copy_i32_kernel<<<grf_ceil_div(cols, 256), 256, 0, stream>>>(t_rowptr, cursor, cols);
    if (nnz > 0) {
        bucket_scatter_kernel<<<grf_ceil_div(rows, 8), 256, 0, stream>>>(rows, rowptr, col, val, cursor, tmp_row, tmp_val);
        bucket_order_kernel<<<grf_ceil_div(cols, 4), 128, 0, stream>>>(cols, t_rowptr, tmp_row, tmp_val, t_col, t_val);
        bucket_sort_long_kernel<<<grf_ceil_div(cols, 4), 128, 0, stream>>>(cols, t_rowptr, tmp_row, tmp_val, t_col, t_val);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    return GRF_OK;
}
