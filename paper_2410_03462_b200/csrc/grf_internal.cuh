// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "grf.h"

#define GRF_CUDA_TRY(expr)                                  \
    do {                                                    \
        cudaError_t _e = (expr);                            \
        if (_e != cudaSuccess) return GRF_ERR_CUDA;         \
    } while (0)

#define GRF_TRY(expr)                                       \
    do {                                                    \
        int _rc = (expr);                                   \
        if (_rc != GRF_OK) return _rc;                      \
    } while (0)

// A device buffer that only ever grows; owned by a context or a feature object.
struct grf_buf {
    void* ptr = nullptr;
    size_t bytes = 0;
};

struct grf_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int sm_count = 0;
    int64_t launches = 0;
    // sampler scratch
    grf_buf stage_col, stage_val;   // merged rows at a fixed stride, before compaction
    grf_buf counts;                 // per-row nonzero counts (both matrices)
    grf_buf rowptr2;                // scanned counts, [2][N+1]
    grf_buf scan_blocks;            // block totals of the two-level scan
    // sampler scratch when the walks' deposits are kept (grf_ctx_keep_walks)
    bool keep_walks = false;
    grf_buf stage_dep_start, stage_dep_t, stage_dep_load, dep_counts, dep_rowptr2;
    // transpose scratch
    grf_buf t_cursor, t_tmp_col, t_tmp_val;
    grf_buf den_scratch;            // denominators of the tensor-core gather path when the caller wants none
    // host-buffer path
    grf_buf h_rowptr, h_col, h_w, h_q, h_k, h_v, h_out, h_ws;
    grf_features* h_feat = nullptr;
    // host-buffer path: phi(Q), phi(K), V are uploaded on one stream and the outputs downloaded on another, in
    // parts of a few problems each, beside the sampler and the attention of the other parts
    static constexpr int HOST_PARTS = 4;     // most parts grf_step_host splits a batch into
    cudaStream_t copy_stream = nullptr, down_stream = nullptr;
    cudaEvent_t up_done[HOST_PARTS] = {}, part_done[HOST_PARTS] = {}, down_done = nullptr;
    int32_t* pinned = nullptr;      // small pinned host block for read-backs
    int* error_word = nullptr;      // device word set by a kernel that gave up a bounded wait
    bool use_tensor_cores = true;
    bool prefer_mask_route = false; // grf_step_host evaluates the attention over the materialised mask where it can
    bool check_graphs = false;      // grf_sample validates the device-resident CSR first (debugging aid)
    // optional per-launch timing
    bool timing = false;
    struct timed_launch { int cls; cudaEvent_t beg, end; };
    std::vector<timed_launch> timed;
    std::vector<cudaEvent_t> free_events;
};

// Brackets one kernel launch (or a short run of launches of one class) with events when timing is on.
struct grf_launch_scope {
    grf_ctx* ctx;
    int cls;
    int n;
    cudaEvent_t beg = nullptr, end = nullptr;
    grf_launch_scope(grf_ctx* c, int cls_, int n_launches = 1);
    ~grf_launch_scope();
};

struct grf_csr_dev {
    int32_t rows = 0, cols = 0;
    int64_t nnz = 0;
    grf_buf rowptr, col, val;
};

#define GRF_PLAN_BLOCK 128   // queries per block of the tensor-core gather kernel

// The deposits behind every entry of Phi (index 0) and Psi (index 1), kept when the sampler was asked to: entry p
// of the matrix owns deposits dep_ptr[p] .. dep_ptr[p+1]-1, each a (step t, load of the prefix) pair, in the
// order in which the sampler adds them.
struct grf_kept_walks {
    bool valid = false;
    int32_t n_walks = 0, max_len = 0;
    int64_t deposits[2] = {0, 0};
    grf_buf dep_ptr[2], dep_t[2], dep_load[2];
    bool perm_valid = false;        // psit_perm[x] = the entry of Psi that entry x of Psi^T copies (built by the first re-modulation)
    grf_buf psit_perm;
};

// The mask estimate Mhat = Phi Psi^T held as dense blocks: for every block of GRF_PLAN_BLOCK consecutive rows the
// sorted list of the keys j that any of its rows reaches (padded to a multiple of GRF_MASK_TILE with the last key
// and zero values) and the block's values in bf16, laid out [group of 8 keys][row of the block][8 keys].
#define GRF_MASK_TILE 64
struct grf_mask_dev {
    bool ready = false;
    bool structure_ready = false;   // key lists (and positions) match the features' structure; values may be stale
    bool by_position = false;       // which of the two value kernels the structure serves
    int32_t blocks = 0;
    int64_t entries = 0;            // padded key entries over all blocks
    grf_buf off, cnt, key;          // cnt holds [blocks] padded counts, then [blocks] the blocks by decreasing count
    grf_buf bits;                   // per block one bit per key: the block's key set
    // build scratch: where each node's key positions start (within its block; the blocks' offsets), the positions,
    // and per non-zero of Phi the start of its node's positions
    grf_buf node_off, blk_pos, pos16, phi_pos;
    grf_buf val;
};

struct grf_features {
    int device = 0;
    grf_csr_dev phi, psi, psit;
    grf_kept_walks kept;
    grf_mask_dev mask;
    // block plan of Phi: per block of GRF_PLAN_BLOCK rows, the sorted distinct columns
    grf_buf plan_off, plan_cnt, plan_col, plan_total;
    grf_buf plan_coef;              // dense bf16 coefficients [quad of union entries][row of the block][4]
    int32_t plan_blocks = 0;
    int64_t plan_entries = 0;       // node-list entries over all blocks (padded to multiples of 4)
    bool plan_ready = false;
    bool plan_coef_ready = false;   // the gather kernel's coefficient table exists for the present plan
    bool plan_stale = true;         // Phi changed since the plan was built: the gather kernel's launcher rebuilds it
};

int grf_buf_reserve(grf_buf* b, size_t bytes);          // grows (contents not preserved)
void grf_buf_release(grf_buf* b);
int grf_csr_reserve(grf_csr_dev* m, int32_t rows, int32_t cols, int64_t nnz_cap);

// sample.cu
struct grf_walk_params {
    int32_t N, n_walks, max_len;
    uint32_t key0, key1, halt_threshold;
    float inv_keep, inv_n;
    int32_t cap;        // n_walks * (max_len + 1)
    int32_t seq_bits;   // ceil(log2(cap)), at least 1
    float f[2][GRF_MAX_WALK_LEN + 1];
};
int grf_walk_params_init(grf_walk_params* p, int32_t N, uint64_t seed, int32_t n_walks, float p_halt,
                         int32_t max_len, const float* f_phi, const float* f_psi);

// scan.cu: exclusive scan of `segments` independent int32 arrays of length n each (in[s*n + i]) into
// out[s*(n+1) + i], with out[s*(n+1) + n] = total.
int grf_exclusive_scan(grf_ctx* ctx, const int32_t* in, int32_t* out, int32_t n, int32_t segments);

int grf_exclusive_scan_scratch(cudaStream_t stream, const int32_t* in, int32_t* out, int32_t n, int32_t segments,
                               int32_t* totals);

// transpose.cu
int grf_transpose_launch(grf_ctx* ctx, int32_t rows, int32_t cols, int64_t nnz,
                         const int32_t* rowptr, const int32_t* col, const float* val,
                         int32_t* t_rowptr, int32_t* t_col, float* t_val);

// attn_state.cu / attn_gather.cu
int grf_build_states(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, int32_t m, int32_t d, int dtype,
                     const void* phiK, const void* V, void* records);
int grf_build_states_tc(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, int32_t m, int32_t d,
                        const void* phiK, const void* V, void* records);
int grf_gather_contract_alu(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t m, int32_t d,
                            int dtype, const void* phiQ, const void* records, void* out, float* den_out);
// attn_mhat.cu
void grf_mask_invalidate(grf_features* feat);
void grf_mask_values_stale(grf_features* feat);
void grf_mask_release(grf_features* feat);
// attn_gather_tc.cu
int grf_build_block_plan(grf_ctx* ctx, grf_features* feat, bool with_coef = true);
int grf_ensure_block_plan(grf_ctx* ctx, const grf_features* feat, bool with_coef = true);   // builds it if Phi changed since the last build
int grf_gather_contract_tc(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                           const void* phiQ, const void* records, void* out, float* den_out);

// Layout of one state tile S_l (m x d) inside the workspace: 16-byte chunks that hold CH consecutive feature
// rows a of one column b, ordered [a / CH][b][a % CH].  With bf16 (CH = 8) this is the K-major, unswizzled
// shared-memory operand layout of the tensor-core gather kernel (8-row core matrices of 128 contiguous
// bytes), so a tile is brought in with one contiguous bulk copy; the ALU kernels read the same chunks.
template <typename T> __host__ __device__ constexpr int grf_tile_chunk() { return 16 / (int)sizeof(T); }
template <typename T> __host__ __device__ constexpr size_t grf_tile_index(int a, int b, int D)
{
    return ((size_t)(a / grf_tile_chunk<T>()) * D + b) * grf_tile_chunk<T>() + (a % grf_tile_chunk<T>());
}

// The workspace holds one record per (problem, node): the state tile S_l, then z_l (m fp32 values) and, with
// bf16 storage, z_l once more rounded to bf16 (the denominators kernel of the tensor-core path reads that copy:
// half the bytes per (query, node) pair).
template <typename T> __host__ __device__ constexpr size_t grf_record_bytes(int M, int D)
{
    return (size_t)M * D * sizeof(T) + (size_t)M * sizeof(float) + (sizeof(T) == 2 ? (size_t)M * 2 : 0);
}

static inline int grf_ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }
