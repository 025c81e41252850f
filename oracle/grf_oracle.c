/*
 * CPU oracle for GRF-masked linear attention.  TEST INFRASTRUCTURE ONLY: plain, slow,
 * single-threaded C written from the paper's definitions.  It shares no code with the
 * CUDA library and must never be called from the product path.
 *
 * What each function follows:
 *   oracle_philox4x32_10   Philox4x32 with 10 rounds, the counter-based generator of
 *                          Salmon, Moraes, Dror & Shaw (SC'11), from its published definition.
 *   oracle_walks           Sec. 3.3 "Using GRFs": n halting random walks per node, the
 *                          importance weight of a prefix walk being the product of
 *                          traversed edge weights (Eq. 9) over its probability
 *                          p(omega) = prod_hops (1 - p_halt)/deg (simple random walk with
 *                          geometric length, Thm 3.2's setting), modulated by f_len.
 *   oracle_features        Eq. 10: phi_hat(v_i)_q = (1/n) sum_walks sum_prefixes ending at q.  Because it works from
 *                          stored walks, calling it again with other coefficients f IS re-modulation without
 *                          re-walking (the "learnable mask parameters (f_i)" of Alg. 1 change, the walks do not).
 *   oracle_transpose       regrouping of a CSR matrix by column (no arithmetic).
 *   oracle_attn_sparse     Eq. 12 / Alg. 1 step 5 evaluated through the per-node states
 *                          S_l = sum_j Psi_jl phi(k_j) v_j^T, z_l = sum_j Psi_jl phi(k_j).
 *
 * Precision: the sampler's decisions are integer; walk loads and feature values are fp32
 * with the operation order written below (the precision and order the method's sampler is
 * specified in, so that index structure can be compared bit for bit); a parallel fp64 value is
 * kept for error accounting.  Attention is fp64 throughout.
 *
 * Conventions fixed here where the paper is silent:
 *   - the halting coin is tossed before every hop, the first included: P(>= k hops) = (1-p)^k;
 *   - the next node is uniform over the neighbours of the node being left;
 *   - a walk also stops after max_len hops or at a node without neighbours;
 *   - a prefix of length t deposits f_t * load_t / n at its end node unless f_t == 0 exactly;
 *   - random words: block = Philox(key = seed, counter = (node, walk, t >> 1, ensemble));
 *     hop t takes words (0,1) of the block when t is even, (2,3) when odd; the first word is the
 *     halting coin (halt iff word < floor(p_halt * 2^32)), the second picks neighbour
 *     floor(word * deg / 2^32);
 *   - within a feature row, equal columns are summed in ascending (walk, t) order.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---------------------------------------------------------------- Philox4x32-10 */

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ---------------------------------------------------------------- walks */

static uint32_t halt_threshold(float p_halt)
{
    double x = floor((double)p_halt * 4294967296.0);
    if (x > 4294967295.0) x = 4294967295.0;
    if (x < 0.0) x = 0.0;
    return (uint32_t)x;
}

/*
 * traj  [2][N][n][L+1] int32, node at step t or -1 after the walk ended
 * load  [2][N][n][L+1] fp32 importance weight of the prefix ending at step t (0 after the end)
 * Returns the total number of visited (node, step) pairs.
 */
int64_t oracle_walks(int32_t N, const int32_t* rowptr, const int32_t* col, const float* w,
                     uint64_t seed, int32_t n, float p_halt, int32_t L,
                     int32_t* traj, float* load_out)
{
    const uint32_t T = halt_threshold(p_halt);
    const float inv_keep = 1.0f / (1.0f - p_halt);
    const uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    const int64_t stride = (int64_t)L + 1;
    int64_t visited = 0;
    for (int32_t e = 0; e < 2; ++e)
        for (int32_t i = 0; i < N; ++i)
            for (int32_t k = 0; k < n; ++k) {
                int32_t* tr = traj + (((int64_t)e * N + i) * n + k) * stride;
                float* ld = load_out + (((int64_t)e * N + i) * n + k) * stride;
                for (int32_t t = 0; t <= L; ++t) { tr[t] = -1; ld[t] = 0.0f; }
                int32_t v = i;
                float load = 1.0f;
                uint32_t words[4] = {0, 0, 0, 0};
                for (int32_t t = 0;; ++t) {
                    tr[t] = v; ld[t] = load; ++visited;
                    if (t == L) break;
                    if ((t & 1) == 0) {
                        const uint32_t ctr[4] = { (uint32_t)i, (uint32_t)k, (uint32_t)(t >> 1), (uint32_t)e };
                        oracle_philox4x32_10(ctr, key, words);
                    }
                    const uint32_t r_halt = words[(t & 1) * 2 + 0];
                    const uint32_t r_next = words[(t & 1) * 2 + 1];
                    if (r_halt < T) break;
                    const int32_t deg = rowptr[v + 1] - rowptr[v];
                    if (deg == 0) break;
                    const int32_t eidx = rowptr[v] + (int32_t)(((uint64_t)r_next * (uint64_t)(uint32_t)deg) >> 32);
                    float step = w[eidx] * (float)deg;   /* W_uv * deg(u): edge weight over 1/deg */
                    step = step * inv_keep;              /* ... over the survival probability      */
                    load = load * step;
                    v = col[eidx];
                }
            }
    return visited;
}

/* ---------------------------------------------------------------- features (Eq. 10) */

typedef struct { int32_t col; int32_t seq; float val; double val64; } deposit_t;

static int cmp_deposit(const void* a, const void* b)
{
    const deposit_t* x = (const deposit_t*)a;
    const deposit_t* y = (const deposit_t*)b;
    if (x->col != y->col) return x->col < y->col ? -1 : 1;
    return x->seq < y->seq ? -1 : (x->seq > y->seq ? 1 : 0);
}

/*
 * Builds one feature matrix (ensemble e) in CSR from the trajectories and loads.
 * rowptr_out [N+1]; col_out/val_out/val64_out sized for N*n*(L+1) entries.  Returns nnz.
 * val   = fp32 sum, in ascending (walk, t) order, of (f_t * load) * (1/n), each product in fp32
 * val64 = the same sum carried in fp64 (terms widened from the fp32 loads)
 * keep_zero != 0: prefixes whose coefficient f_t is exactly 0 are deposited as well (their terms are zeros),
 * so that the index structure is the set of visited nodes whatever f is: the structure a feature object
 * must have if its coefficients are to be changed later without new walks.
 */
int64_t oracle_features(int32_t N, int32_t n, int32_t L, int32_t e,
                        const int32_t* traj, const float* load, const float* f,
                        int32_t* rowptr_out, int32_t* col_out, float* val_out, double* val64_out,
                        int32_t keep_zero)
{
    const int64_t stride = (int64_t)L + 1;
    const float inv_n = 1.0f / (float)n;
    deposit_t* buf = (deposit_t*)malloc(sizeof(deposit_t) * (size_t)n * (size_t)stride);
    if (!buf) return -1;
    int64_t nnz = 0;
    rowptr_out[0] = 0;
    for (int32_t i = 0; i < N; ++i) {
        int32_t cnt = 0;
        for (int32_t k = 0; k < n; ++k) {
            const int32_t* tr = traj + (((int64_t)e * N + i) * n + k) * stride;
            const float* ld = load + (((int64_t)e * N + i) * n + k) * stride;
            for (int32_t t = 0; t <= L && tr[t] >= 0; ++t) {
                if (f[t] == 0.0f && !keep_zero) continue;
                float dep = f[t] * ld[t];
                dep = dep * inv_n;
                buf[cnt].col = tr[t];
                buf[cnt].seq = k * (int32_t)stride + t;
                buf[cnt].val = dep;
                buf[cnt].val64 = (double)f[t] * (double)ld[t] / (double)n;
                ++cnt;
            }
        }
        qsort(buf, (size_t)cnt, sizeof(deposit_t), cmp_deposit);
        for (int32_t a = 0; a < cnt;) {
            float s = buf[a].val;
            double s64 = buf[a].val64;
            int32_t b = a + 1;
            while (b < cnt && buf[b].col == buf[a].col) { s = s + buf[b].val; s64 += buf[b].val64; ++b; }
            col_out[nnz] = buf[a].col; val_out[nnz] = s; val64_out[nnz] = s64; ++nnz;
            a = b;
        }
        rowptr_out[i + 1] = (int32_t)nnz;
    }
    free(buf);
    return nnz;
}

/* CSR (rows x cols) -> CSR of the transpose; inside an output row the source rows ascend. */
void oracle_transpose(int32_t rows, int32_t cols, const int32_t* rowptr, const int32_t* col, const float* val,
                      int32_t* t_rowptr, int32_t* t_col, float* t_val)
{
    int64_t nnz = rowptr[rows];
    memset(t_rowptr, 0, sizeof(int32_t) * ((size_t)cols + 1));
    for (int64_t p = 0; p < nnz; ++p) t_rowptr[col[p] + 1]++;
    for (int32_t c = 0; c < cols; ++c) t_rowptr[c + 1] += t_rowptr[c];
    int32_t* cur = (int32_t*)malloc(sizeof(int32_t) * ((size_t)cols + 1));
    memcpy(cur, t_rowptr, sizeof(int32_t) * ((size_t)cols + 1));
    for (int32_t r = 0; r < rows; ++r)
        for (int32_t p = rowptr[r]; p < rowptr[r + 1]; ++p) {
            int32_t dst = cur[col[p]]++;
            t_col[dst] = r; t_val[dst] = val[p];
        }
    free(cur);
}

/* ---------------------------------------------------------------- attention, S/z route (Eq. 12) */

/*
 * One problem g at a time.  phiQ, phiK [G][N][m], V [G][N][d] are fp32 arrays holding exactly the
 * values of the storage type.  Phi: CSR N x R.  PsiT: CSR R x N (row l lists the j with Psi_jl != 0).
 * num [G][N][d], den [G][N], and the sums of absolute values of the terms num_abs, den_abs
 * (the scale on which a tolerance is meaningful when terms cancel); any output pointer may be NULL
 * except num and den.  Returns 0, or -1 when memory runs out.
 */
int oracle_attn_sparse(int32_t G, int32_t N, int32_t R, int32_t m, int32_t d,
                       const float* phiQ, const float* phiK, const float* V,
                       const int32_t* phi_rowptr, const int32_t* phi_col, const float* phi_val,
                       const int32_t* psit_rowptr, const int32_t* psit_col, const float* psit_val,
                       double* num, double* den, double* num_abs, double* den_abs)
{
    const size_t md = (size_t)m * (size_t)d;
    double* S = (double*)malloc(sizeof(double) * (size_t)R * md);
    double* z = (double*)malloc(sizeof(double) * (size_t)R * (size_t)m);
    double* Sa = num_abs ? (double*)malloc(sizeof(double) * (size_t)R * md) : NULL;
    double* za = den_abs ? (double*)malloc(sizeof(double) * (size_t)R * (size_t)m) : NULL;
    if (!S || !z || (num_abs && !Sa) || (den_abs && !za)) { free(S); free(z); free(Sa); free(za); return -1; }
    for (int32_t g = 0; g < G; ++g) {
        const float* Qg = phiQ + (size_t)g * N * m;
        const float* Kg = phiK + (size_t)g * N * m;
        const float* Vg = V + (size_t)g * N * d;
        /* S_l = sum_j Psi_jl phi(k_j) v_j^T ;  z_l = sum_j Psi_jl phi(k_j) */
        for (int32_t l = 0; l < R; ++l) {
            double* Sl = S + (size_t)l * md;
            double* zl = z + (size_t)l * m;
            for (size_t x = 0; x < md; ++x) Sl[x] = 0.0;
            for (int32_t a = 0; a < m; ++a) zl[a] = 0.0;
            if (Sa) for (size_t x = 0; x < md; ++x) Sa[(size_t)l * md + x] = 0.0;
            if (za) for (int32_t a = 0; a < m; ++a) za[(size_t)l * m + a] = 0.0;
            for (int32_t p = psit_rowptr[l]; p < psit_rowptr[l + 1]; ++p) {
                const int32_t j = psit_col[p];
                const double psi = (double)psit_val[p];
                for (int32_t a = 0; a < m; ++a) {
                    const double pk = psi * (double)Kg[(size_t)j * m + a];
                    zl[a] += pk;
                    if (za) za[(size_t)l * m + a] += fabs(pk);
                    for (int32_t b = 0; b < d; ++b) {
                        const double term = pk * (double)Vg[(size_t)j * d + b];
                        Sl[(size_t)a * d + b] += term;
                        if (Sa) Sa[(size_t)l * md + (size_t)a * d + b] += fabs(term);
                    }
                }
            }
        }
        /* num_i = sum_l Phi_il phi(q_i)^T S_l ;  den_i = sum_l Phi_il phi(q_i)^T z_l */
        for (int32_t i = 0; i < N; ++i) {
            double* ni = num + ((size_t)g * N + i) * d;
            double* nai = num_abs ? num_abs + ((size_t)g * N + i) * d : NULL;
            double di = 0.0, dai = 0.0;
            for (int32_t b = 0; b < d; ++b) { ni[b] = 0.0; if (nai) nai[b] = 0.0; }
            for (int32_t p = phi_rowptr[i]; p < phi_rowptr[i + 1]; ++p) {
                const int32_t l = phi_col[p];
                const double phi = (double)phi_val[p];
                for (int32_t a = 0; a < m; ++a) {
                    const double c = phi * (double)Qg[(size_t)i * m + a];
                    di += c * z[(size_t)l * m + a];
                    if (za) dai += fabs(c) * za[(size_t)l * m + a];
                    const double* Sla = S + (size_t)l * md + (size_t)a * d;
                    for (int32_t b = 0; b < d; ++b) ni[b] += c * Sla[b];
                    if (nai) {
                        const double* Saa = Sa + (size_t)l * md + (size_t)a * d;
                        for (int32_t b = 0; b < d; ++b) nai[b] += fabs(c) * Saa[b];
                    }
                }
            }
            den[(size_t)g * N + i] = di;
            if (den_abs) den_abs[(size_t)g * N + i] = dai;
        }
    }
    free(S); free(z); free(Sa); free(za);
    return 0;
}
