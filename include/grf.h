/*
 * grf.h — C ABI of the GRF-masked linear-attention library (CUDA, sm_100a).
 *
 * The library evaluates linear attention under the topological mask M_alpha = sum_k alpha_k W^k
 * (Eq. 4), replaced by its sparse Monte-Carlo factorisation Mhat = Phi Psi^T built from halting
 * random walks (graph random features, Eq. 10), following Alg. 1.
 *
 * Conventions for every call
 *   - returns 0 (GRF_OK) or a negative GRF_ERR_* code; nothing is thrown or printed;
 *   - "DEVICE" pointers are plain CUDA device addresses on the context's device, "HOST" pointers
 *     are ordinary host memory; the library never takes ownership of a caller's buffer;
 *   - all device work is enqueued on the context's stream; unless a call says otherwise it
 *     returns without waiting for that work;
 *   - a context is not thread-safe: one host thread at a time per context;
 *   - matrices are CSR with int32 row pointers/column indices (ascending inside a row) and fp32 values.
 */
#ifndef GRF_H
#define GRF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GRF_OK              0
#define GRF_ERR_INVALID    (-1)  /* NULL pointer, non-positive size, p_halt outside [0,1), unsupported m/d/dtype */
#define GRF_ERR_TOO_LARGE  (-2)  /* a size exceeds a documented limit                                            */
#define GRF_ERR_WORKSPACE  (-3)  /* caller's workspace too small                                                 */
#define GRF_ERR_CUDA       (-4)  /* a CUDA runtime call failed                                                   */
#define GRF_ERR_NOMEM      (-5)  /* device or host allocation failed                                             */
#define GRF_ERR_BADGRAPH   (-6)  /* CSR input inconsistent (grf_step_host always checks; grf_sample on request)   */
#define GRF_ERR_TIMEOUT    (-7)  /* a kernel gave up a bounded wait; its outputs are not valid                   */

#define GRF_DTYPE_F32  0
#define GRF_DTYPE_BF16 1

/* similarity A_ij of grf_masked_attn_asym */
#define GRF_KERNEL_LINEAR  0   /* A_ij = phi(q_i) . phi(k_j): the caller passes phi(Q), phi(K) */
#define GRF_KERNEL_SOFTMAX 1   /* A_ij = exp(q_i . k_j): the caller passes Q, K (scaled as it wishes) */

#define GRF_MAX_WALK_LEN 255     /* largest max_len accepted by the sampler */

typedef struct grf_ctx grf_ctx;            /* device id, stream, reusable scratch                         */
typedef struct grf_features grf_features;  /* device-resident Phi (N x R), Psi (N x R), Psi^T (R x N)     */

/* Context bound to `device` and to the CUDA stream `cuda_stream` (a cudaStream_t passed as void*;
 * NULL = the default stream).  Scratch buffers grow on demand and live until destroy. */
int grf_ctx_create(grf_ctx** out, int device, void* cuda_stream);
int grf_ctx_destroy(grf_ctx* ctx);   /* waits for the stream, frees scratch; features are freed separately */

/* Remark 3.1: f with sum_{p=0..k} f_p f_{k-p} = alpha_k, k < len (fp64 recurrence on the host).
 * HOST pointers.  GRF_ERR_INVALID unless alpha[0] > 0. */
int grf_deconvolve(const double* alpha, int32_t len, double* f_out);

/*
 * Alg. 1 steps 1-2 (Sec. 3.3, Eqs. 9-10): simulate n_walks halting random walks out of every node for
 * each of two independent ensembles and assemble the sparse feature matrices Phi (ensemble 0, modulation
 * f_phi) and Psi (ensemble 1, modulation f_psi), plus Psi^T grouped by visited node.
 *
 *   N, rowptr[N+1], col[E], w[E]   DEVICE  CSR of the weighted adjacency matrix W
 *   seed                                   64-bit key of the counter-based generator
 *   n_walks >= 1, 0 <= p_halt < 1, 0 <= max_len <= GRF_MAX_WALK_LEN
 *   f_phi[max_len+1], f_psi[max_len+1]  HOST  modulation coefficients; f_psi == NULL means f_phi
 *   *inout   NULL: a new feature object is created; otherwise that object's buffers are reused
 *            (regrown if needed) and its previous contents are overwritten.
 *
 * Walk rule: the walk from node i deposits f_t * load_t / n_walks at the node reached after t hops
 * (nothing when f_t == 0), load_0 = 1 and load_{t+1} = load_t * W_uv * deg(u) / (1 - p_halt) for the hop
 * u -> v; before every hop it halts with probability p_halt; it also stops after max_len hops or at a
 * node without neighbours.  Random words come from Philox4x32-10 keyed by `seed` with counter
 * (node, walk, t/2, ensemble): the result depends only on these, never on launch geometry.
 * Deposits of a row that hit the same column are added in ascending (walk, t) order.
 *
 * Limits: n_walks*(max_len+1) <= 16384 and N * 2^ceil(log2(n_walks*(max_len+1))) <= 2^32, else
 * GRF_ERR_TOO_LARGE.  The call waits once for the device (it reads back the two nonzero counts).
 */
int grf_sample(grf_ctx* ctx, int32_t N, const int32_t* rowptr, const int32_t* col, const float* w,
               uint64_t seed, int32_t n_walks, float p_halt, int32_t max_len,
               const float* f_phi, const float* f_psi, grf_features** inout);

/*
 * Re-modulation without re-walking (Alg. 1: the modulation coefficients (f_i) are learnable, the walks are not;
 * Sec. 4: walks "can be pre-computed and frozen").
 *
 * grf_ctx_keep_walks(ctx, 1): from now on grf_sample also keeps, inside the feature object, the deposits behind
 * every entry: for each prefix of each walk that ends at the entry's node, its length t and its load (Eq. 9's
 * weight over its probability).  In this mode a prefix deposits whatever its coefficient, so the index structure
 * of Phi and Psi is the set of visited nodes and does not depend on f; an entry all of whose coefficients are 0
 * holds the value 0.  Entries that plain sampling would also create get bit-identical values.  Extra device
 * memory: 5 bytes per deposit plus 4 per entry.
 *
 * grf_remodulate: gives a feature object sampled in that mode new coefficients (HOST arrays of max_len + 1
 * values, max_len as sampled; f_psi == NULL means f_phi).  Values become sum (f_t * load) * (1 / n_walks) over the
 * entry's deposits, same operations and order as the sampler's: the result is bit-identical to sampling again
 * with the same seed and the new coefficients, without any walk being taken.  Psi^T receives the new values through
 * the entry order recorded at the first call.  The index structure is unchanged, so what was derived from it stays:
 * the next attention call rebuilds only the coefficient table of its block plan, the next grf_features_materialise
 * only the mask's values.  Asynchronous.  GRF_ERR_INVALID if the object holds no deposits or max_len differs.
 */
int grf_ctx_keep_walks(grf_ctx* ctx, int enable);
int grf_remodulate(grf_ctx* ctx, grf_features* feat, int32_t max_len, const float* f_phi, const float* f_psi);

/*
 * Floating-point operation counts of one attention problem (Sec. 4 "Time complexity", the figure of FLOPs against
 * the number of nodes), from the feature object's non-zero counts; HOST outputs, any may be NULL:
 *   masked          Eq. 12: every non-zero of Psi and of Phi costs m products with phi(k_j) / phi(q_i) and m(d+1)
 *                   multiply-adds (2 operations each) into / against [S_l | z_l]; plus N*d divisions;
 *   unmasked_linear Eq. 3 right to left: 4 N m (d+1) + N d;
 *   softmax         N^2 (2m + 2 + 2d) + N d  (scores, exponentials, row sums, weighted values).
 */
int grf_attn_flops(const grf_features* feat, int32_t m, int32_t d, int64_t* masked, int64_t* unmasked_linear,
                   int64_t* softmax);

/* The walks themselves, for checking (Sec. 3.3): traj and load are DEVICE arrays
 * [2][N][n_walks][max_len+1]; traj holds the node at step t or -1 after the walk ended, load the
 * importance weight of that prefix (0 after the end).  Same arguments and limits as grf_sample. */
int grf_debug_walks(grf_ctx* ctx, int32_t N, const int32_t* rowptr, const int32_t* col, const float* w,
                    uint64_t seed, int32_t n_walks, float p_halt, int32_t max_len,
                    int32_t* traj, float* load);

/* Feature object from caller-made matrices (DEVICE CSR, N x R each); copies them and builds Psi^T.
 * Used for the special case Psi = I (asymmetric features, App. "Asymmetric graph random features")
 * and for tests.  nnz are read from the row pointers: waits for the device once. */
int grf_features_from_csr(grf_ctx* ctx, int32_t N, int32_t R,
                          const int32_t* phi_rowptr, const int32_t* phi_col, const float* phi_val,
                          const int32_t* psi_rowptr, const int32_t* psi_col, const float* psi_val,
                          grf_features** out);

/* Borrowed DEVICE pointers into a feature object: which = 0 Phi, 1 Psi, 2 Psi^T.  Valid until the
 * object is freed or resampled.  rows/cols/nnz are returned through HOST pointers (any may be NULL). */
int grf_features_view(const grf_features* feat, int which, int32_t* rows, int32_t* cols, int64_t* nnz,
                      const int32_t** rowptr, const int32_t** col, const float** val);
/* Copies one matrix of a feature object into caller DEVICE arrays rowptr[rows+1], col[nnz], val[nnz]
 * (sizes as reported by grf_features_view).  Asynchronous. */
int grf_features_copy(grf_ctx* ctx, const grf_features* feat, int which, int32_t* rowptr, int32_t* col, float* val);
int grf_features_free(grf_features* feat);

/* Regroups a DEVICE CSR matrix (rows x cols, nnz = rowptr[rows] passed by the caller) by column:
 * t_rowptr[cols+1], t_col[nnz], t_val[nnz] DEVICE outputs; inside an output row the source rows ascend
 * (Psi -> Psi^T, which turns Phi_K^T V of Alg. 1 step 5 into a segmented reduction).  Asynchronous. */
int grf_csr_transpose(grf_ctx* ctx, int32_t rows, int32_t cols, int64_t nnz,
                      const int32_t* rowptr, const int32_t* col, const float* val,
                      int32_t* t_rowptr, int32_t* t_col, float* t_val);

/*
 * grf_csr_transpose without any allocation.  (The paper has no counterpart: this entry point exists for
 * the sake of callers, not of the method.)
 *
 * Who needs it: a process whose device memory is already handed out in full to its own pool or to a
 * framework's caching allocator, where a cudaMalloc inside a library call can fail or fragment that budget;
 * and code that must not stall its other streams, since cudaMalloc and cudaFree wait for the whole device.
 * grf_csr_transpose grows scratch buffers through its context when a larger matrix arrives; this variant
 * never does.  It takes no context: its scratch (column counters, unordered buckets, scan totals, about
 * 4.5 MB) is a fixed array inside the library image, so every GPU that loads libgrf.so holds that much
 * until the process ends, whether or not this function is ever called.
 *
 * Same inputs, outputs and result as grf_csr_transpose, all DEVICE pointers on `device`; work is
 * enqueued on `cuda_stream` (a cudaStream_t as void*, NULL = default stream) and not waited for.
 * Limits: cols <= GRF_NOALLOC_MAX_COLS and nnz <= GRF_NOALLOC_MAX_NNZ, otherwise GRF_ERR_TOO_LARGE and
 * nothing is launched.  The function calls no cudaMalloc/cudaFree and no allocating library routine.
 * The first call on a device looks up the array's device address (once per device); make that first
 * call before any stream capture begins, and, in a process that hands the whole device memory to its own pool,
 * before the pool takes it: where the CUDA module is loaded lazily, the array is reserved only at that first call,
 * which then fails with GRF_ERR_CUDA if no memory is left.  All calls on one GPU share the array and it keeps the previous
 * call's contents (the function clears what has to start at zero): two calls whose device work overlaps in
 * time, on different streams or from different threads, race on it and give wrong results — order them.
 */
#define GRF_NOALLOC_MAX_COLS 65536
#define GRF_NOALLOC_MAX_NNZ  524288
int grf_csr_transpose_noalloc(int device, void* cuda_stream, int32_t rows, int32_t cols, int64_t nnz,
                              const int32_t* rowptr, const int32_t* col, const float* val,
                              int32_t* t_rowptr, int32_t* t_col, float* t_val);

/* Bytes of DEVICE workspace with which grf_masked_linear_attn processes all G problems in one pass
 * (per problem and node one record: the state S_l, m x d in the storage type, followed by z_l, m fp32 values,
 * and with bf16 storage by z_l once more in bf16).  A smaller workspace is accepted
 * as long as it holds one problem; the call then works through G in chunks.  0 on invalid arguments. */
size_t grf_attn_workspace_bytes(int32_t G, int32_t R, int32_t m, int32_t d, int dtype);

/*
 * Alg. 1 step 5 / Eq. 12 for G independent problems (batch x heads) sharing one feature object:
 *   S_l = sum_j Psi_jl phi(k_j) v_j^T,  z_l = sum_j Psi_jl phi(k_j)              (per problem, per node l)
 *   out_i = sum_l Phi_il phi(q_i)^T S_l / sum_l Phi_il phi(q_i)^T z_l
 * phiQ, phiK [G][N][m], V [G][N][d], out [G][N][d]: DEVICE, row-major, 16-byte aligned, dtype
 * GRF_DTYPE_F32 or _BF16 (bf16: S is stored in bf16, sums are carried in fp32).  den_out: optional
 * DEVICE fp32 [G][N] receiving the denominators.  A row whose denominator is exactly 0 yields out = 0.
 * m, d in {8, 16, 32, 64, 128}.  workspace: DEVICE, 256-byte aligned.  Summation order is fixed, so
 * results are run-to-run identical.  Asynchronous, except that the first bf16 call with m and d multiples of 16
 * after the features were created, resampled or re-modulated prepares a per-block plan of Phi inside the feature
 * object, which waits for the stream once (so a feature object must not be used by two threads at the same time).
 */
int grf_masked_linear_attn(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                           int dtype, const void* phiQ, const void* phiK, const void* V,
                           void* out, float* den_out, void* workspace, size_t workspace_bytes);

/*
 * Masked attention with ASYMMETRIC graph random features (App. "Asymmetric graph random features", Alg. 2):
 * when the key-side modulation is f^(2) = delta_0 the key features are the identity, the mask estimate is
 * Phi itself, and
 *   out_i = sum_l Phi_il A_il v_l / sum_l Phi_il A_il    over the non-zeros of row i of Phi,
 * with A_il = phi(q_i) . phi(k_l) (GRF_KERNEL_LINEAR) or exp(q_i . k_l) (GRF_KERNEL_SOFTMAX); m + d
 * multiply-adds per non-zero, no workspace.  Only feat's Phi is used (N x N; sample it with f_phi = alpha
 * and f_psi = delta_0, or pass any CSR through grf_features_from_csr).  Q, K [G][N][m], V, out [G][N][d]:
 * DEVICE, row-major, 16-byte aligned, dtype GRF_DTYPE_F32 or _BF16 (sums in fp32); m, d in
 * {8, 16, 32, 64, 128}; G <= 65535.  den_out: optional DEVICE fp32 [G][N] receiving the denominators (with
 * the softmax kernel relative to exp(largest score of the row), which cancels in out).  A row whose
 * denominator is exactly 0 yields out = 0.  Summation order is fixed; asynchronous.
 */
int grf_masked_attn_asym(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                         int dtype, int kernel, const void* Q, const void* K, const void* V, void* out,
                         float* den_out);

/*
 * Masked attention with the mask estimate materialised (Eqs. 1-2 with Mhat = Phi Psi^T, Sec. 3.3: Mhat_ij =
 * phi_hat(v_i)^T phi_hat(v_j)): the same outputs as grf_masked_linear_attn, computed over the non-zeros of Mhat
 * instead of through the per-node states of Eq. 12.  It pays where consecutive node ids are neighbours in the
 * graph (grids, spatially sorted point clouds): the rows of a block of 128 queries then reach few keys between them.
 *
 * grf_features_materialise: forms Mhat once for a feature object (N x N; Phi and Psi may be N x R) as dense bf16
 * blocks, one per 128 consecutive rows, over the sorted list of keys the block reaches (sums in fp32, fixed order).
 * Needs the node lists of Phi's block plan (built here if absent).  Waits for the stream twice.  The mask is dropped
 * when the object is resampled; after grf_remodulate its values are stale (grf_mask_stats, grf_mask_rows and
 * grf_masked_attn_mhat return GRF_ERR_INVALID) until this call forms them again, which then takes one kernel over
 * the key lists already in place and does not wait for the stream.  GRF_ERR_TOO_LARGE when N > 294912 or the blocks would exceed 8 GiB (no
 * locality: use grf_masked_linear_attn).
 * grf_mask_stats: HOST outputs (any may be NULL): number of blocks, key entries summed over the blocks (padded
 * to multiples of 64), device bytes held.  GRF_ERR_INVALID when the object holds no mask.
 * grf_mask_rows: writes n dense rows of Mhat, out[x][j] = Mhat[rows[x]][j], fp32, to DEVICE out [n][N];
 * rows: DEVICE int32 [n].  Asynchronous.
 * grf_masked_attn_mhat: out_i = sum_j Mhat_ij (phi(q_i).phi(k_j)) v_j / sum_j Mhat_ij (phi(q_i).phi(k_j)) for G
 * problems; arguments as grf_masked_linear_attn, no workspace.  dtype GRF_DTYPE_BF16, d = 64, m in {16, 32, 64}
 * (other shapes: GRF_ERR_INVALID); scores are fp32, the masked scores are added into the denominator in fp32 and
 * rounded to bf16 before they multiply V.  Summation order is fixed.  Asynchronous.
 */
int grf_features_materialise(grf_ctx* ctx, grf_features* feat);
int grf_mask_stats(const grf_features* feat, int32_t* blocks, int64_t* key_entries, int64_t* bytes);
int grf_mask_rows(grf_ctx* ctx, const grf_features* feat, int32_t n, const int32_t* rows, float* out);
int grf_masked_attn_mhat(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                         int dtype, const void* phiQ, const void* phiK, const void* V, void* out, float* den_out);

/*
 * The whole path of Alg. 1 from HOST buffers, for callers that keep nothing on the device:
 * copies the graph and phi(Q), phi(K), V to the device, samples features, evaluates the attention and
 * copies `out` ([G][N][d], dtype) back; returns after the result is in `out`.  Device buffers and the
 * feature object are owned by the context and reused by later calls.  Graph consistency (monotone
 * rowptr, indices in range) is checked on the host: GRF_ERR_BADGRAPH.
 */
int grf_step_host(grf_ctx* ctx, int32_t N, const int32_t* rowptr, const int32_t* col, const float* w,
                  uint64_t seed, int32_t n_walks, float p_halt, int32_t max_len,
                  const float* f_phi, const float* f_psi,
                  int32_t G, int32_t m, int32_t d, int dtype,
                  const void* phiQ, const void* phiK, const void* V, void* out);

/* Debugging aid: while enabled, grf_sample first validates the device-resident graph with a kernel (row pointers
 * start at 0 and never decrease, column indices in [0, N); col is only read inside [0, rowptr[N])) and waits for
 * the result: GRF_ERR_BADGRAPH, and no walk is taken, if it is inconsistent.  Off by default (one extra pass over
 * the graph and one wait per call).  Kernel launches are also named as NVTX ranges ("grf:walk_merge", ...) for
 * profilers' timelines; that costs nothing when no tool is attached. */
int grf_ctx_check_graphs(grf_ctx* ctx, int enable);

/* Self-test of the bounded waits inside the tensor-core kernels: launches one warp that waits, with the kernels' own
 * wait routine and a limit of `limit_cycles` GPU clock cycles (1 .. 2e9), for a barrier that nothing arrives at.  The
 * wait gives up and raises the context's error word, so the next grf_ctx_check returns GRF_ERR_TIMEOUT; the device
 * stays usable.  Asynchronous. */
int grf_debug_wait_timeout(grf_ctx* ctx, int64_t limit_cycles);

/* Route of grf_step_host: 0 (default) = through the per-node states (grf_masked_linear_attn); 1 = over the materialised
 * mask (grf_features_materialise + grf_masked_attn_mhat) whenever the shape allows it (bf16, d = 64, m in {16, 32, 64})
 * and the mask can be built; otherwise the call falls back to the default route.  Same outputs within the stated
 * tolerance. */
int grf_ctx_prefer_mask_route(grf_ctx* ctx, int enable);

/* Waits for the context's stream and reports whether any kernel since the previous check gave up one of its
 * bounded waits (GRF_ERR_TIMEOUT; the affected outputs are invalid), else GRF_OK. */
int grf_ctx_check(grf_ctx* ctx);

/* Chooses the attention kernels for bf16 problems: 1 (default) = tensor-core kernels where they apply (state
 * build: m a multiple of 16 and d <= 64; gather-contract: a block plan exists and m, d are multiples of 16);
 * 0 = plain-ALU kernels always.  Results agree within the stated tolerance. */
int grf_ctx_use_tensor_cores(grf_ctx* ctx, int enable);

/* The block plan of Phi that the tensor-core gather uses (built here if absent; waits for the stream then): HOST
 * outputs, any may be NULL: number of 128-row blocks, and the node-list entries summed over the blocks (each is one
 * state tile a block brings into shared memory per problem).  GRF_ERR_TOO_LARGE when the object has no plan (see
 * grf_masked_linear_attn). */
int grf_plan_stats(grf_ctx* ctx, const grf_features* feat, int32_t* blocks, int64_t* entries);

/* Number of kernels the context has launched since it was created (for accounting in benchmarks). */
int64_t grf_ctx_launch_count(const grf_ctx* ctx);

/* Per-kernel device timing for benchmarks.  While enabled, every kernel launch of the context is
 * bracketed by two CUDA events on the context's stream.  grf_ctx_kernel_times waits for the stream, adds
 * the elapsed times since the previous read to ms[GRF_KERNEL_CLASSES] / launches[GRF_KERNEL_CLASSES]
 * (HOST arrays, overwritten) and clears the record.  Classes: 0 walk+merge, 1 prefix scans, 2 row
 * compaction, 3 column regrouping (histogram, scatter, ordering), 4 state build (S, z), 5 gather-contract,
 * 6 denominators pass of the tensor-core gather, 7 block plan of the tensor-core gather, 8 building the
 * materialised mask, 9 attention over the materialised mask. */
#define GRF_KERNEL_CLASSES 10
int grf_ctx_enable_timing(grf_ctx* ctx, int enable);
int grf_ctx_kernel_times(grf_ctx* ctx, float* ms, int64_t* launches);

const char* grf_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* GRF_H */
