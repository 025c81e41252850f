// C-ABI entry points that are not kernels themselves: contexts, buffers, feature objects, the
// attention driver (Alg. 1 step 5 in chunks of problems) and the host-buffer path.
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "grf_internal.cuh"

int grf_buf_reserve(grf_buf* b, size_t bytes)
{
    if (bytes == 0) bytes = 1;
    if (b->bytes >= bytes) return GRF_OK;
    if (b->ptr) { cudaFree(b->ptr); b->ptr = nullptr; b->bytes = 0; }
    void* p = nullptr;
    const cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { cudaGetLastError(); return GRF_ERR_NOMEM; }
    b->ptr = p; b->bytes = bytes;
    return GRF_OK;
}

void grf_buf_release(grf_buf* b)
{
    if (b->ptr) cudaFree(b->ptr);
    b->ptr = nullptr; b->bytes = 0;
}

int grf_csr_reserve(grf_csr_dev* m, int32_t rows, int32_t cols, int64_t nnz_cap)
{
    m->rows = rows; m->cols = cols;
    GRF_TRY(grf_buf_reserve(&m->rowptr, sizeof(int32_t) * ((size_t)rows + 1)));
    GRF_TRY(grf_buf_reserve(&m->col, sizeof(int32_t) * (size_t)(nnz_cap > 0 ? nnz_cap : 1)));
    GRF_TRY(grf_buf_reserve(&m->val, sizeof(float) * (size_t)(nnz_cap > 0 ? nnz_cap : 1)));
    return GRF_OK;
}

extern "C" int grf_ctx_create(grf_ctx** out, int device, void* cuda_stream)
{
    if (!out || device < 0) return GRF_ERR_INVALID;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device >= count) { cudaGetLastError(); return GRF_ERR_CUDA; }
    GRF_CUDA_TRY(cudaSetDevice(device));
    grf_ctx* c = new (std::nothrow) grf_ctx();
    if (!c) return GRF_ERR_NOMEM;
    c->device = device;
    c->stream = (cudaStream_t)cuda_stream;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaMallocHost((void**)&c->pinned, 64) != cudaSuccess ||
        cudaMalloc((void**)&c->error_word, 2 * sizeof(int)) != cudaSuccess ||
        cudaMemset(c->error_word, 0, 2 * sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return GRF_ERR_CUDA;
    }
    *out = c;
    return GRF_OK;
}

extern "C" int grf_ctx_destroy(grf_ctx* ctx)
{
    if (!ctx) return GRF_ERR_INVALID;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    grf_buf* bufs[] = {&ctx->stage_col, &ctx->stage_val, &ctx->counts, &ctx->rowptr2, &ctx->scan_blocks,
                       &ctx->stage_dep_start, &ctx->stage_dep_t, &ctx->stage_dep_load, &ctx->dep_counts, &ctx->dep_rowptr2,
                       &ctx->t_cursor, &ctx->t_tmp_col, &ctx->t_tmp_val, &ctx->den_scratch, &ctx->h_rowptr, &ctx->h_col, &ctx->h_w,
                       &ctx->h_q, &ctx->h_k, &ctx->h_v, &ctx->h_out, &ctx->h_ws};
    for (grf_buf* b : bufs) grf_buf_release(b);
    if (ctx->h_feat) grf_features_free(ctx->h_feat);
    if (ctx->pinned) cudaFreeHost(ctx->pinned);
    if (ctx->error_word) cudaFree(ctx->error_word);
    if (ctx->copy_stream) {
        cudaStreamSynchronize(ctx->copy_stream); cudaStreamSynchronize(ctx->down_stream);
        cudaStreamDestroy(ctx->copy_stream); cudaStreamDestroy(ctx->down_stream);
        for (int p = 0; p < grf_ctx::HOST_PARTS; ++p) { cudaEventDestroy(ctx->up_done[p]); cudaEventDestroy(ctx->part_done[p]); }
        cudaEventDestroy(ctx->down_done);
    }
    for (auto& t : ctx->timed) { cudaEventDestroy(t.beg); cudaEventDestroy(t.end); }
    for (cudaEvent_t e : ctx->free_events) cudaEventDestroy(e);
    delete ctx;
    return GRF_OK;
}

static cudaEvent_t take_event(grf_ctx* c)
{
    if (!c->free_events.empty()) { cudaEvent_t e = c->free_events.back(); c->free_events.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return e;
}

// names of the kernel classes, as ranges in a profiler's timeline
static const char* const kernel_class_names[GRF_KERNEL_CLASSES] = {
    "grf:walk_merge", "grf:scan", "grf:compact", "grf:regroup", "grf:build_states", "grf:gather_contract",
    "grf:row_denominators", "grf:block_plan", "grf:mask_build", "grf:mhat_attention"};

grf_launch_scope::grf_launch_scope(grf_ctx* c, int cls_, int n_launches) : ctx(c), cls(cls_), n(n_launches)
{
    nvtxRangePushA(kernel_class_names[cls]);     // costs nothing unless a tool is attached
    if (!ctx->timing) return;
    beg = take_event(ctx); end = take_event(ctx);
    if (beg && end) cudaEventRecord(beg, ctx->stream);
}

grf_launch_scope::~grf_launch_scope()
{
    nvtxRangePop();
    ctx->launches += n;
    if (!ctx->timing || !beg || !end) return;
    cudaEventRecord(end, ctx->stream);
    ctx->timed.push_back({cls, beg, end});
}

extern "C" int grf_ctx_use_tensor_cores(grf_ctx* ctx, int enable)
{
    if (!ctx) return GRF_ERR_INVALID;
    ctx->use_tensor_cores = enable != 0;
    return GRF_OK;
}

extern "C" int grf_ctx_prefer_mask_route(grf_ctx* ctx, int enable)
{
    if (!ctx) return GRF_ERR_INVALID;
    ctx->prefer_mask_route = enable != 0;
    return GRF_OK;
}

extern "C" int grf_ctx_check_graphs(grf_ctx* ctx, int enable)
{
    if (!ctx) return GRF_ERR_INVALID;
    ctx->check_graphs = enable != 0;
    return GRF_OK;
}

extern "C" int grf_ctx_check(grf_ctx* ctx)
{
    if (!ctx) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 8, ctx->error_word, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    GRF_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    if (ctx->pinned[8] != 0) {
        cudaMemsetAsync(ctx->error_word, 0, sizeof(int), ctx->stream);
        return GRF_ERR_TIMEOUT;
    }
    return GRF_OK;
}

extern "C" int grf_ctx_enable_timing(grf_ctx* ctx, int enable)
{
    if (!ctx) return GRF_ERR_INVALID;
    ctx->timing = enable != 0;
    return GRF_OK;
}

extern "C" int grf_ctx_kernel_times(grf_ctx* ctx, float* ms, int64_t* launches)
{
    if (!ctx || !ms || !launches) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    GRF_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    for (int k = 0; k < GRF_KERNEL_CLASSES; ++k) { ms[k] = 0.0f; launches[k] = 0; }
    for (auto& t : ctx->timed) {
        float x = 0.0f;
        if (cudaEventElapsedTime(&x, t.beg, t.end) == cudaSuccess) { ms[t.cls] += x; launches[t.cls] += 1; }
        ctx->free_events.push_back(t.beg);
        ctx->free_events.push_back(t.end);
    }
    ctx->timed.clear();
    cudaGetLastError();
    return GRF_OK;
}

extern "C" int64_t grf_ctx_launch_count(const grf_ctx* ctx) { return ctx ? ctx->launches : -1; }

extern "C" int grf_deconvolve(const double* alpha, int32_t len, double* f_out)
{
    if (!alpha || !f_out || len < 1 || !(alpha[0] > 0.0)) return GRF_ERR_INVALID;
    // sum_{p=0..k} f_p f_{k-p} = alpha_k  =>  f_0 = sqrt(alpha_0), then solve for f_k (Remark 3.1)
    f_out[0] = sqrt(alpha[0]);
    for (int32_t k = 1; k < len; ++k) {
        double cross = 0.0;
        for (int32_t p = 1; p < k; ++p) cross += f_out[p] * f_out[k - p];
        f_out[k] = (alpha[k] - cross) / (2.0 * f_out[0]);
    }
    return GRF_OK;
}

extern "C" int grf_attn_flops(const grf_features* feat, int32_t m, int32_t d, int64_t* masked,
                              int64_t* unmasked_linear, int64_t* softmax)
{
    if (!feat || m <= 0 || d <= 0) return GRF_ERR_INVALID;
    const int64_t N = feat->phi.rows;
    const int64_t per_nonzero = (int64_t)m + 2 * (int64_t)m * (d + 1);     // scale phi(.), then multiply-add into [S_l | z_l]
    if (masked) *masked = (feat->phi.nnz + feat->psit.nnz) * per_nonzero + N * d;
    if (unmasked_linear) *unmasked_linear = 4 * N * m * (d + 1) + N * d;
    if (softmax) *softmax = N * N * (2 * (int64_t)m + 2 + 2 * (int64_t)d) + N * d;
    return GRF_OK;
}

static void csr_release(grf_csr_dev* m)
{
    grf_buf_release(&m->rowptr); grf_buf_release(&m->col); grf_buf_release(&m->val);
}

extern "C" int grf_features_free(grf_features* feat)
{
    if (!feat) return GRF_ERR_INVALID;
    cudaSetDevice(feat->device);
    csr_release(&feat->phi); csr_release(&feat->psi); csr_release(&feat->psit);
    grf_buf_release(&feat->plan_off); grf_buf_release(&feat->plan_cnt);
    grf_buf_release(&feat->plan_col); grf_buf_release(&feat->plan_total); grf_buf_release(&feat->plan_coef);
    grf_mask_release(feat);
    for (int e = 0; e < 2; ++e) {
        grf_buf_release(&feat->kept.dep_ptr[e]); grf_buf_release(&feat->kept.dep_t[e]); grf_buf_release(&feat->kept.dep_load[e]);
    }
    grf_buf_release(&feat->kept.psit_perm);
    delete feat;
    return GRF_OK;
}

extern "C" int grf_features_view(const grf_features* feat, int which, int32_t* rows, int32_t* cols, int64_t* nnz,
                                 const int32_t** rowptr, const int32_t** col, const float** val)
{
    if (!feat || which < 0 || which > 2) return GRF_ERR_INVALID;
    const grf_csr_dev& m = which == 0 ? feat->phi : (which == 1 ? feat->psi : feat->psit);
    if (rows) *rows = m.rows;
    if (cols) *cols = m.cols;
    if (nnz) *nnz = m.nnz;
    if (rowptr) *rowptr = (const int32_t*)m.rowptr.ptr;
    if (col) *col = (const int32_t*)m.col.ptr;
    if (val) *val = (const float*)m.val.ptr;
    return GRF_OK;
}

extern "C" int grf_features_copy(grf_ctx* ctx, const grf_features* feat, int which, int32_t* rowptr, int32_t* col,
                                 float* val)
{
    if (!ctx || !feat || which < 0 || which > 2 || !rowptr) return GRF_ERR_INVALID;
    const grf_csr_dev& m = which == 0 ? feat->phi : (which == 1 ? feat->psi : feat->psit);
    if (m.nnz > 0 && (!col || !val)) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    GRF_CUDA_TRY(cudaMemcpyAsync(rowptr, m.rowptr.ptr, sizeof(int32_t) * ((size_t)m.rows + 1), cudaMemcpyDeviceToDevice,
                                 ctx->stream));
    if (m.nnz > 0) {
        GRF_CUDA_TRY(cudaMemcpyAsync(col, m.col.ptr, sizeof(int32_t) * (size_t)m.nnz, cudaMemcpyDeviceToDevice, ctx->stream));
        GRF_CUDA_TRY(cudaMemcpyAsync(val, m.val.ptr, sizeof(float) * (size_t)m.nnz, cudaMemcpyDeviceToDevice, ctx->stream));
    }
    return GRF_OK;
}

extern "C" int grf_features_from_csr(grf_ctx* ctx, int32_t N, int32_t R,
                                     const int32_t* phi_rowptr, const int32_t* phi_col, const float* phi_val,
                                     const int32_t* psi_rowptr, const int32_t* psi_col, const float* psi_val,
                                     grf_features** out)
{
    if (!ctx || !out || N <= 0 || R <= 0 || !phi_rowptr || !psi_rowptr) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 0, phi_rowptr + N, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 1, psi_rowptr + N, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    GRF_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    const int64_t nnz_phi = ctx->pinned[0], nnz_psi = ctx->pinned[1];
    if (nnz_phi < 0 || nnz_psi < 0) return GRF_ERR_INVALID;
    if ((nnz_phi > 0 && (!phi_col || !phi_val)) || (nnz_psi > 0 && (!psi_col || !psi_val))) return GRF_ERR_INVALID;
    grf_features* f = new (std::nothrow) grf_features();
    if (!f) return GRF_ERR_NOMEM;
    f->device = ctx->device;
    int rc = grf_csr_reserve(&f->phi, N, R, nnz_phi);
    if (rc == GRF_OK) rc = grf_csr_reserve(&f->psi, N, R, nnz_psi);
    if (rc == GRF_OK) rc = grf_csr_reserve(&f->psit, R, N, nnz_psi);
    if (rc != GRF_OK) { grf_features_free(f); return rc; }
    f->phi.nnz = nnz_phi; f->psi.nnz = nnz_psi; f->psit.nnz = nnz_psi;
    auto copy = [&](grf_csr_dev& m, const int32_t* rp, const int32_t* c, const float* v, int64_t nnz) {
        cudaMemcpyAsync(m.rowptr.ptr, rp, sizeof(int32_t) * ((size_t)N + 1), cudaMemcpyDeviceToDevice, ctx->stream);
        if (nnz > 0) {
            cudaMemcpyAsync(m.col.ptr, c, sizeof(int32_t) * (size_t)nnz, cudaMemcpyDeviceToDevice, ctx->stream);
            cudaMemcpyAsync(m.val.ptr, v, sizeof(float) * (size_t)nnz, cudaMemcpyDeviceToDevice, ctx->stream);
        }
    };
    copy(f->phi, phi_rowptr, phi_col, phi_val, nnz_phi);
    copy(f->psi, psi_rowptr, psi_col, psi_val, nnz_psi);
    rc = grf_transpose_launch(ctx, N, R, nnz_psi, (const int32_t*)f->psi.rowptr.ptr, (const int32_t*)f->psi.col.ptr,
                              (const float*)f->psi.val.ptr, (int32_t*)f->psit.rowptr.ptr,
                              (int32_t*)f->psit.col.ptr, (float*)f->psit.val.ptr);
    if (rc == GRF_OK) { f->plan_stale = true; f->plan_ready = false; }   // built at the first attention that needs it
    if (rc == GRF_OK && cudaGetLastError() != cudaSuccess) rc = GRF_ERR_CUDA;
    if (rc != GRF_OK) { grf_features_free(f); return rc; }
    *out = f;
    return GRF_OK;
}

static bool dim_ok(int32_t x) { return x == 8 || x == 16 || x == 32 || x == 64 || x == 128; }
static size_t elem_size(int dtype) { return dtype == GRF_DTYPE_F32 ? 4 : 2; }
static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// per-problem workspace: R records (state tile in the storage type, then z in fp32), 256-byte aligned
static size_t ws_per_problem(int32_t R, int32_t m, int32_t d, int dtype)
{
    // one record per node: the state tile, z (fp32) and, with bf16 storage, z once more in bf16
    return align256((size_t)R * ((size_t)m * d * elem_size(dtype) + (size_t)m * sizeof(float) +
                                 (dtype == GRF_DTYPE_BF16 ? (size_t)m * 2 : 0)));
}

extern "C" size_t grf_attn_workspace_bytes(int32_t G, int32_t R, int32_t m, int32_t d, int dtype)
{
    if (G <= 0 || R <= 0 || !dim_ok(m) || !dim_ok(d) || (dtype != GRF_DTYPE_F32 && dtype != GRF_DTYPE_BF16)) return 0;
    return ws_per_problem(R, m, d, dtype) * (size_t)G;
}

extern "C" int grf_masked_linear_attn(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m,
                                      int32_t d, int dtype, const void* phiQ, const void* phiK, const void* V,
                                      void* out, float* den_out, void* workspace, size_t workspace_bytes)
{
    if (!ctx || !feat || !phiQ || !phiK || !V || !out || !workspace) return GRF_ERR_INVALID;
    if (G <= 0 || N <= 0 || !dim_ok(m) || !dim_ok(d)) return GRF_ERR_INVALID;
    if (dtype != GRF_DTYPE_F32 && dtype != GRF_DTYPE_BF16) return GRF_ERR_INVALID;
    if (feat->phi.rows != N || feat->psit.cols != N || feat->phi.cols != feat->psit.rows) return GRF_ERR_INVALID;
    if (((uintptr_t)workspace & 255) != 0) return GRF_ERR_INVALID;
    const int32_t R = feat->phi.cols;
    const size_t per = ws_per_problem(R, m, d, dtype);
    if (workspace_bytes < per) return GRF_ERR_WORKSPACE;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    int64_t chunk = (int64_t)(workspace_bytes / per);
    if (chunk > G) chunk = G;
    if (chunk > 65535) chunk = 65535;
    const size_t es = elem_size(dtype);
    // the plan's build waits for the stream once: do it before the attention kernels are queued, not between them
    // (only for shapes the tensor-core gather covers: other shapes never read the plan)
    if (dtype == GRF_DTYPE_BF16 && ctx->use_tensor_cores && m % 16 == 0 && d % 16 == 0)
        GRF_TRY(grf_ensure_block_plan(ctx, feat));
    for (int64_t g0 = 0; g0 < G; g0 += chunk) {
        const int32_t gc = (int32_t)((G - g0) < chunk ? (G - g0) : chunk);
        // chunk layout: records [gc][R], contiguous
        const char* k_ptr = (const char*)phiK + (size_t)g0 * N * m * es;
        const char* v_ptr = (const char*)V + (size_t)g0 * N * d * es;
        const char* q_ptr = (const char*)phiQ + (size_t)g0 * N * m * es;
        char* o_ptr = (char*)out + (size_t)g0 * N * d * es;
        float* den_ptr = den_out ? den_out + (size_t)g0 * N : nullptr;
        int rs = 1;
        if (dtype == GRF_DTYPE_BF16 && ctx->use_tensor_cores)
            rs = grf_build_states_tc(ctx, feat->psit, gc, N, m, d, k_ptr, v_ptr, workspace);
        if (rs > 0) rs = grf_build_states(ctx, feat->psit, gc, N, m, d, dtype, k_ptr, v_ptr, workspace);
        GRF_TRY(rs);
        int rc = 1;
        if (dtype == GRF_DTYPE_BF16 && ctx->use_tensor_cores)
            rc = grf_gather_contract_tc(ctx, feat, gc, N, m, d, q_ptr, workspace, o_ptr, den_ptr);
        if (rc > 0) rc = grf_gather_contract_alu(ctx, feat->phi, gc, N, m, d, dtype, q_ptr, workspace, o_ptr, den_ptr);
        GRF_TRY(rc);
    }
    return GRF_OK;
}

static int check_graph_host(int32_t N, const int32_t* rowptr, const int32_t* col)
{
    if (rowptr[0] != 0) return GRF_ERR_BADGRAPH;
    for (int32_t i = 0; i < N; ++i)
        if (rowptr[i + 1] < rowptr[i]) return GRF_ERR_BADGRAPH;
    const int64_t E = rowptr[N];
    for (int64_t p = 0; p < E; ++p)
        if (col[p] < 0 || col[p] >= N) return GRF_ERR_BADGRAPH;
    return GRF_OK;
}

extern "C" int grf_step_host(grf_ctx* ctx, int32_t N, const int32_t* rowptr, const int32_t* col, const float* w,
                             uint64_t seed, int32_t n_walks, float p_halt, int32_t max_len,
                             const float* f_phi, const float* f_psi,
                             int32_t G, int32_t m, int32_t d, int dtype,
                             const void* phiQ, const void* phiK, const void* V, void* out)
{
    if (!ctx || !rowptr || !col || !w || !phiQ || !phiK || !V || !out || N <= 0 || G <= 0) return GRF_ERR_INVALID;
    if (!dim_ok(m) || !dim_ok(d) || (dtype != GRF_DTYPE_F32 && dtype != GRF_DTYPE_BF16)) return GRF_ERR_INVALID;
    GRF_TRY(check_graph_host(N, rowptr, col));
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    const size_t E = (size_t)rowptr[N], es = elem_size(dtype);
    const size_t qk_bytes = (size_t)G * N * m * es, v_bytes = (size_t)G * N * d * es;
    GRF_TRY(grf_buf_reserve(&ctx->h_rowptr, ((size_t)N + 1) * 4));
    GRF_TRY(grf_buf_reserve(&ctx->h_col, E * 4));
    GRF_TRY(grf_buf_reserve(&ctx->h_w, E * 4));
    GRF_TRY(grf_buf_reserve(&ctx->h_q, qk_bytes));
    GRF_TRY(grf_buf_reserve(&ctx->h_k, qk_bytes));
    GRF_TRY(grf_buf_reserve(&ctx->h_v, v_bytes));
    GRF_TRY(grf_buf_reserve(&ctx->h_out, v_bytes));
    cudaStream_t s = ctx->stream;
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->h_rowptr.ptr, rowptr, ((size_t)N + 1) * 4, cudaMemcpyHostToDevice, s));
    if (E > 0) {
        GRF_CUDA_TRY(cudaMemcpyAsync(ctx->h_col.ptr, col, E * 4, cudaMemcpyHostToDevice, s));
        GRF_CUDA_TRY(cudaMemcpyAsync(ctx->h_w.ptr, w, E * 4, cudaMemcpyHostToDevice, s));
    }
    // The problems are handled in parts: the inputs of part p travel on a second stream while the features are
    // sampled and the earlier parts are computed; its outputs leave on a third stream while the next part runs.
    if (!ctx->copy_stream) {
        GRF_CUDA_TRY(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
        GRF_CUDA_TRY(cudaStreamCreateWithFlags(&ctx->down_stream, cudaStreamNonBlocking));
        for (int p = 0; p < grf_ctx::HOST_PARTS; ++p) {
            GRF_CUDA_TRY(cudaEventCreateWithFlags(&ctx->up_done[p], cudaEventDisableTiming));
            GRF_CUDA_TRY(cudaEventCreateWithFlags(&ctx->part_done[p], cudaEventDisableTiming));
        }
        GRF_CUDA_TRY(cudaEventCreateWithFlags(&ctx->down_done, cudaEventDisableTiming));
    }
    // Two parts on the route through the per-node states, whose kernels lose more on small batches than the finer
    // overlap returns (four parts were measured slower there); four on the route over the mask, whose attention is
    // short, so that most of the outputs leave while later parts are computed.
    const bool mask_shape = ctx->prefer_mask_route && dtype == GRF_DTYPE_BF16 && d == 64 && (m == 16 || m == 32 || m == 64);
    const int want_parts = mask_shape ? grf_ctx::HOST_PARTS : 2;
    const int parts = G >= 2 * want_parts ? want_parts : (G >= 2 ? 2 : 1);
    const int32_t gp = (G + parts - 1) / parts;           // problems per part
    for (int p = 0; p < parts; ++p) {
        const int32_t g0 = p * gp, gc = g0 + gp <= G ? gp : G - g0;
        if (gc <= 0) break;
        const size_t qo = (size_t)g0 * N * m * es, vo = (size_t)g0 * N * d * es;
        const size_t qb = (size_t)gc * N * m * es, vb = (size_t)gc * N * d * es;
        GRF_CUDA_TRY(cudaMemcpyAsync((char*)ctx->h_q.ptr + qo, (const char*)phiQ + qo, qb, cudaMemcpyHostToDevice, ctx->copy_stream));
        GRF_CUDA_TRY(cudaMemcpyAsync((char*)ctx->h_k.ptr + qo, (const char*)phiK + qo, qb, cudaMemcpyHostToDevice, ctx->copy_stream));
        GRF_CUDA_TRY(cudaMemcpyAsync((char*)ctx->h_v.ptr + vo, (const char*)V + vo, vb, cudaMemcpyHostToDevice, ctx->copy_stream));
        GRF_CUDA_TRY(cudaEventRecord(ctx->up_done[p], ctx->copy_stream));
    }
    GRF_TRY(grf_sample(ctx, N, (const int32_t*)ctx->h_rowptr.ptr, (const int32_t*)ctx->h_col.ptr,
                       (const float*)ctx->h_w.ptr, seed, n_walks, p_halt, max_len, f_phi, f_psi, &ctx->h_feat));
    // route: over the materialised mask when the caller prefers it and the shape and the graph allow it
    bool by_mask = false;
    if (ctx->prefer_mask_route && dtype == GRF_DTYPE_BF16 && d == 64 && (m == 16 || m == 32 || m == 64)) {
        const int rc = grf_features_materialise(ctx, ctx->h_feat);
        if (rc == GRF_OK) by_mask = true;
        else if (rc != GRF_ERR_TOO_LARGE) return rc;          // too large = no locality: the S/z route serves it
    }
    // workspace: one part's records if that is modest, else chunks of about 1 GiB
    const size_t per = by_mask ? 256 : ws_per_problem(N, m, d, dtype);
    size_t want = per * (size_t)gp;
    const size_t cap = (size_t)1 << 31;
    if (want > cap) want = per * (cap / per > 0 ? cap / per : 1);
    GRF_TRY(grf_buf_reserve(&ctx->h_ws, want));
    for (int p = 0; p < parts; ++p) {
        const int32_t g0 = p * gp, gc = g0 + gp <= G ? gp : G - g0;
        if (gc <= 0) break;
        const size_t qo = (size_t)g0 * N * m * es, vo = (size_t)g0 * N * d * es;
        GRF_CUDA_TRY(cudaStreamWaitEvent(s, ctx->up_done[p], 0));
        if (by_mask)
            GRF_TRY(grf_masked_attn_mhat(ctx, ctx->h_feat, gc, N, m, d, dtype, (const char*)ctx->h_q.ptr + qo,
                                         (const char*)ctx->h_k.ptr + qo, (const char*)ctx->h_v.ptr + vo,
                                         (char*)ctx->h_out.ptr + vo, nullptr));
        else
            GRF_TRY(grf_masked_linear_attn(ctx, ctx->h_feat, gc, N, m, d, dtype, (const char*)ctx->h_q.ptr + qo,
                                           (const char*)ctx->h_k.ptr + qo, (const char*)ctx->h_v.ptr + vo,
                                           (char*)ctx->h_out.ptr + vo, nullptr, ctx->h_ws.ptr, ctx->h_ws.bytes));
        GRF_CUDA_TRY(cudaEventRecord(ctx->part_done[p], s));
        GRF_CUDA_TRY(cudaStreamWaitEvent(ctx->down_stream, ctx->part_done[p], 0));
        GRF_CUDA_TRY(cudaMemcpyAsync((char*)out + vo, (const char*)ctx->h_out.ptr + vo, (size_t)gc * N * d * es,
                                     cudaMemcpyDeviceToHost, ctx->down_stream));
    }
    GRF_CUDA_TRY(cudaEventRecord(ctx->down_done, ctx->down_stream));
    GRF_CUDA_TRY(cudaStreamWaitEvent(s, ctx->down_done, 0));
    return grf_ctx_check(ctx);
}

extern "C" const char* grf_strerror(int code)
{
    switch (code) {
        case GRF_OK: return "ok";
        case GRF_ERR_INVALID: return "invalid argument";
        case GRF_ERR_TOO_LARGE: return "size exceeds a documented limit";
        case GRF_ERR_WORKSPACE: return "workspace too small";
        case GRF_ERR_CUDA: return "CUDA runtime error";
        case GRF_ERR_NOMEM: return "out of memory";
        case GRF_ERR_BADGRAPH: return "inconsistent graph CSR";
        case GRF_ERR_TIMEOUT: return "a kernel gave up a bounded wait";
        default: return "unknown error";
    }
}
