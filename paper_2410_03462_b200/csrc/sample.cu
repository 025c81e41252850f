// Walk sampler and feature assembly (Alg. 1 steps 1-2; Sec. 3.3, Eqs. 9-10).
//
// One warp owns one feature row (ensemble e, source node i); its lanes are walkers.  Every decision
// of a walk is integer (Philox words against a threshold, multiply-high neighbour pick), the load is
// fp32 with a fixed operation order, so the walks do not depend on the launch geometry.  Deposits
// stay in shared memory: the warp sorts their keys by (column, walk, step) with a bitonic network (in
// registers and shuffles for rows of up to 512 deposits), adds equal columns in that order and writes the
// merged row once.
#include <new>

#include "grf_internal.cuh"

namespace {

constexpr uint32_t PHILOX_M0 = 0xD2511F53u, PHILOX_M1 = 0xCD9E8D57u;
constexpr uint32_t PHILOX_W0 = 0x9E3779B9u, PHILOX_W1 = 0xBB67AE85u;

// Philox4x32 with 10 rounds (Salmon et al., SC'11).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1, uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(PHILOX_M0, c0), lo0 = PHILOX_M0 * c0;
        const uint32_t hi1 = __umulhi(PHILOX_M1, c2), lo1 = PHILOX_M1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += PHILOX_W0;
        k1 += PHILOX_W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// State of one walker; `advance` takes the hop after step t (halting coin first).
struct Walker {
    int32_t v;
    float load;
    uint32_t words[4];
    bool alive;

    __device__ __forceinline__ void advance(const grf_walk_params& P, const int32_t* __restrict__ rowptr,
                                            const int32_t* __restrict__ col, const float* __restrict__ w,
                                            int32_t e, int32_t i, int32_t k, int32_t t)
    {
        if ((t & 1) == 0)
            philox4x32_10((uint32_t)i, (uint32_t)k, (uint32_t)(t >> 1), (uint32_t)e, P.key0, P.key1, words);
        const uint32_t r_halt = (t & 1) ? words[2] : words[0];
        const uint32_t r_next = (t & 1) ? words[3] : words[1];
        if (r_halt < P.halt_threshold) { alive = false; return; }
        const int32_t beg = __ldg(rowptr + v);
        const int32_t deg = __ldg(rowptr + v + 1) - beg;
        if (deg == 0) { alive = false; return; }
        const int32_t eidx = beg + (int32_t)__umulhi(r_next, (uint32_t)deg);
        float step = __fmul_rn(__ldg(w + eidx), (float)deg);
        step = __fmul_rn(step, P.inv_keep);
        load = __fmul_rn(load, step);
        v = __ldg(col + eidx);
    }
};

// Bitonic sort of 32 * E keys held E per lane (key x = lane * E + r sits in register r of its lane): partners
// closer than E are registers of the same lane, the others are reached with one shuffle.  Same network as
// the shared-memory loop it replaces, so the result is the same sorted row.
template <int E>
__device__ __forceinline__ void sort_in_registers(uint32_t* keys, int lane)
{
    uint32_t v[E];
#pragma unroll
    for (int r = 0; r < E; ++r) v[r] = keys[lane * E + r];
#pragma unroll
    for (int k = 2; k <= 32 * E; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j >= E) {
                const int lj = j / E;
                const bool keep_min = ((lane & lj) == 0) == (((lane * E) & k) == 0);
#pragma unroll
                for (int r = 0; r < E; ++r) {
                    const uint32_t p = __shfl_xor_sync(0xffffffffu, v[r], lj);
                    v[r] = keep_min ? min(v[r], p) : max(v[r], p);
                }
            } else {
#pragma unroll
                for (int r = 0; r < E; ++r) {
                    if ((r & j) == 0) {
                        const bool up = k < E ? (r & k) == 0 : ((lane * E) & k) == 0;
                        const uint32_t mn = min(v[r], v[r | j]), mx = max(v[r], v[r | j]);
                        v[r] = up ? mn : mx;
                        v[r | j] = up ? mx : mn;
                    }
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < E; ++r) keys[lane * E + r] = v[r];
}

// KEEP: the row's deposits themselves are kept as well (for grf_remodulate): every prefix deposits whatever its
// coefficient, the sorted list of (step, load) pairs of the row goes to a staging area of stride P.cap, and every
// merged entry records where its deposits begin in that list.  The values are computed by the same operations in
// the same order as without KEEP.
template <bool KEEP>
__global__ void __launch_bounds__(256)
walk_merge_kernel(const __grid_constant__ grf_walk_params P,
                  const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col, const float* __restrict__ w,
                  int32_t stage_stride, int32_t* __restrict__ stage_col, float* __restrict__ stage_val,
                  int32_t* __restrict__ counts,
                  int32_t* __restrict__ stage_dep_start, unsigned char* __restrict__ stage_dep_t,
                  float* __restrict__ stage_dep_load, int32_t* __restrict__ dep_counts)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int warps = blockDim.x >> 5;
    const int32_t row = blockIdx.x * warps + warp;
    if (row >= 2 * P.N) return;
    const int32_t e = row >= P.N ? 1 : 0;
    const int32_t i = row - e * P.N;

    const int32_t key_slots = max(32, 1 << P.seq_bits);   // the sort pads a row to at least one key per lane
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw) + (size_t)warp * (key_slots + P.cap);
    float* vals = reinterpret_cast<float*>(keys + key_slots);
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int32_t Lp1 = P.max_len + 1;

    // ---- walks: lanes are walkers, all at the same step t
    int32_t cnt = 0;
    for (int32_t k0 = 0; k0 < P.n_walks; k0 += 32) {
        const int32_t k = k0 + lane;
        Walker wk;
        wk.v = i; wk.load = 1.0f; wk.alive = k < P.n_walks;
        wk.words[0] = wk.words[1] = wk.words[2] = wk.words[3] = 0;
        for (int32_t t = 0;; ++t) {
            const float ft = P.f[e][t];
            const bool dep = wk.alive && (KEEP || ft != 0.0f);
            const uint32_t dm = __ballot_sync(0xffffffffu, dep);
            if (dep) {
                const int32_t seq = k * Lp1 + t;
                keys[cnt + __popc(dm & lt_mask)] = ((uint32_t)wk.v << P.seq_bits) | (uint32_t)seq;
                vals[seq] = KEEP ? wk.load : __fmul_rn(__fmul_rn(ft, wk.load), P.inv_n);
            }
            cnt += __popc(dm);
            if (t == P.max_len) break;
            if (wk.alive) wk.advance(P, rowptr, col, w, e, i, k, t);
            if (__ballot_sync(0xffffffffu, wk.alive) == 0u) break;
        }
    }
    __syncwarp();

    // ---- sort the row's deposits by (column, walk, step)
    int32_t Psort = 32;
    while (Psort < cnt) Psort <<= 1;
    for (int32_t x = cnt + lane; x < Psort; x += 32) keys[x] = 0xffffffffu;
    __syncwarp();
    if (Psort <= 512) {
        switch (Psort) {
            case 32: sort_in_registers<1>(keys, lane); break;
            case 64: sort_in_registers<2>(keys, lane); break;
            case 128: sort_in_registers<4>(keys, lane); break;
            case 256: sort_in_registers<8>(keys, lane); break;
            default: sort_in_registers<16>(keys, lane); break;
        }
        __syncwarp();
    } else
    for (int32_t k = 2; k <= Psort; k <<= 1)
        for (int32_t j = k >> 1; j > 0; j >>= 1) {
            for (int32_t idx = lane; idx < (Psort >> 1); idx += 32) {
                const int32_t a = ((idx & ~(j - 1)) << 1) | (idx & (j - 1));
                const int32_t b = a | j;
                const uint32_t ka = keys[a], kb = keys[b];
                const bool up = (a & k) == 0;
                if ((ka > kb) == up) { keys[a] = kb; keys[b] = ka; }
            }
            __syncwarp();
        }

    // ---- add equal columns in sorted order; one lane per distinct column
    const uint32_t seq_mask = (1u << P.seq_bits) - 1u;
    int32_t r = 0;
    const size_t out_base = (size_t)row * stage_stride;
    const size_t dep_base = (size_t)row * P.cap;
    // value of the deposit with sequence number seq = walk * (max_len + 1) + t
    auto term = [&](uint32_t seq) {
        if (!KEEP) return vals[seq];
        const int32_t t = (int32_t)seq % Lp1;
        return __fmul_rn(__fmul_rn(P.f[e][t], vals[seq]), P.inv_n);
    };
    for (int32_t base = 0; base < cnt; base += 32) {
        const int32_t p = base + lane;
        const bool valid = p < cnt;
        const uint32_t key = valid ? keys[p] : 0u;
        const uint32_t c = key >> P.seq_bits;
        const bool head = valid && (p == 0 || (keys[p - 1] >> P.seq_bits) != c);
        const uint32_t hm = __ballot_sync(0xffffffffu, head);
        if (KEEP && valid) {
            stage_dep_t[dep_base + p] = (unsigned char)((int32_t)(key & seq_mask) % Lp1);
            stage_dep_load[dep_base + p] = vals[key & seq_mask];
        }
        if (head) {
            float s = term(key & seq_mask);
            for (int32_t q = p + 1; q < cnt; ++q) {
                const uint32_t kq = keys[q];
                if ((kq >> P.seq_bits) != c) break;
                s = __fadd_rn(s, term(kq & seq_mask));
            }
            const int32_t rank = r + __popc(hm & lt_mask);
            stage_col[out_base + rank] = (int32_t)c;
            stage_val[out_base + rank] = s;
            if (KEEP) stage_dep_start[out_base + rank] = p;
        }
        r += __popc(hm);
    }
    if (lane == 0) {
        counts[row] = r;
        if (KEEP) dep_counts[row] = cnt;
    }
}

// Kept deposits: moves every row's sorted (step, load) list from the staging area to its place and turns the
// entries' in-row start positions into absolute offsets (dep_ptr has one more element than the matrix has entries).
__global__ void __launch_bounds__(256)
compact_deposits_kernel(int32_t N, int32_t stage_stride, int32_t cap,
                        const int32_t* __restrict__ stage_dep_start, const unsigned char* __restrict__ stage_dep_t,
                        const float* __restrict__ stage_dep_load,
                        const int32_t* __restrict__ rowptr_phi, const int32_t* __restrict__ rowptr_psi,
                        const int32_t* __restrict__ dep_rowptr2,
                        int32_t* __restrict__ ptr_phi, unsigned char* __restrict__ t_phi, float* __restrict__ load_phi,
                        int32_t* __restrict__ ptr_psi, unsigned char* __restrict__ t_psi, float* __restrict__ load_psi)
{
    const int lane = threadIdx.x & 31;
    const int32_t row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= 2 * N) return;
    const int32_t e = row >= N ? 1 : 0;
    const int32_t i = row - e * N;
    const int32_t* rp = e ? rowptr_psi : rowptr_phi;
    const int32_t* drp = dep_rowptr2 + (size_t)e * (N + 1);
    int32_t* optr = e ? ptr_psi : ptr_phi;
    unsigned char* ot = e ? t_psi : t_phi;
    float* ol = e ? load_psi : load_phi;
    const int32_t beg = rp[i], len = rp[i + 1] - beg;
    const int32_t dbeg = drp[i], dlen = drp[i + 1] - dbeg;
    for (int32_t x = lane; x < len; x += 32) optr[beg + x] = dbeg + stage_dep_start[(size_t)row * stage_stride + x];
    for (int32_t x = lane; x < dlen; x += 32) {
        ot[dbeg + x] = stage_dep_t[(size_t)row * cap + x];
        ol[dbeg + x] = stage_dep_load[(size_t)row * cap + x];
    }
    if (i == N - 1 && lane == 0) optr[rp[N]] = drp[N];
}

// Re-modulation (Alg. 1 step 2 with new "learnable mask parameters (f_i)"): every entry's value is rebuilt from its
// kept deposits as sum (f_t * load) * (1/n), the products and the sum taken in the sampler's operations and order.
struct grf_remod_params { float f[2][GRF_MAX_WALK_LEN + 1]; float inv_n; };
__global__ void index_as_float_kernel(int32_t n, float* __restrict__ out)
{
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = (float)i;
}

__global__ void float_to_index_kernel(int32_t n, const float* __restrict__ in, int32_t* __restrict__ out)
{
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = (int32_t)in[i];
}

// out[x] = src[perm[x]]: Psi^T's values from Psi's
__global__ void gather_values_kernel(int32_t n, const int32_t* __restrict__ perm, const float* __restrict__ src,
                                     float* __restrict__ out)
{
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = src[perm[i]];
}

__global__ void __launch_bounds__(256)
remodulate_kernel(const __grid_constant__ grf_remod_params P, int32_t e, int64_t nnz, const int32_t* __restrict__ dep_ptr,
                  const unsigned char* __restrict__ dep_t, const float* __restrict__ dep_load, float* __restrict__ val)
{
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= nnz) return;
    const int32_t beg = dep_ptr[p], end = dep_ptr[p + 1];
    float s = 0.0f;
    for (int32_t q = beg; q < end; ++q) {
        const float term = __fmul_rn(__fmul_rn(P.f[e][dep_t[q]], dep_load[q]), P.inv_n);
        s = q == beg ? term : __fadd_rn(s, term);
    }
    val[p] = s;
}

// Copies each merged row from the fixed-stride staging area to its place in the CSR arrays.
__global__ void __launch_bounds__(256)
compact_rows_kernel(int32_t N, int32_t stage_stride, const int32_t* __restrict__ stage_col,
                    const float* __restrict__ stage_val,
                    const int32_t* __restrict__ rowptr_phi, const int32_t* __restrict__ rowptr_psi,
                    int32_t* __restrict__ col_phi, float* __restrict__ val_phi,
                    int32_t* __restrict__ col_psi, float* __restrict__ val_psi)
{
    const int lane = threadIdx.x & 31;
    const int32_t row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= 2 * N) return;
    const int32_t e = row >= N ? 1 : 0;
    const int32_t i = row - e * N;
    const int32_t* rp = e ? rowptr_psi : rowptr_phi;
    int32_t* oc = e ? col_psi : col_phi;
    float* ov = e ? val_psi : val_phi;
    const int32_t beg = rp[i], len = rp[i + 1] - beg;
    const size_t src = (size_t)row * stage_stride;
    for (int32_t x = lane; x < len; x += 32) {
        oc[beg + x] = stage_col[src + x];
        ov[beg + x] = stage_val[src + x];
    }
}

__global__ void __launch_bounds__(256)
debug_walks_kernel(const __grid_constant__ grf_walk_params P,
                   const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col, const float* __restrict__ w,
                   int32_t* __restrict__ traj, float* __restrict__ load)
{
    const int64_t total = 2ll * P.N * P.n_walks;
    const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= total) return;
    const int32_t k = (int32_t)(id % P.n_walks);
    const int64_t row = id / P.n_walks;
    const int32_t e = row >= P.N ? 1 : 0;
    const int32_t i = (int32_t)(row - (int64_t)e * P.N);
    const int32_t Lp1 = P.max_len + 1;
    int32_t* tr = traj + id * Lp1;
    float* ld = load + id * Lp1;
    Walker wk;
    wk.v = i; wk.load = 1.0f; wk.alive = true;
    wk.words[0] = wk.words[1] = wk.words[2] = wk.words[3] = 0;
    int32_t t = 0;
    for (;; ++t) {
        tr[t] = wk.v; ld[t] = wk.load;
        if (t == P.max_len) break;
        wk.advance(P, rowptr, col, w, e, i, k, t);
        if (!wk.alive) break;
    }
    for (++t; t < Lp1; ++t) { tr[t] = -1; ld[t] = 0.0f; }
}

// Consistency of a device-resident CSR graph: row pointers start at 0 and never decrease, column indices lie in
// [0, N).  A thread reads col only inside its own row's extent after checking that the extent lies inside
// [0, rowptr[N]], the length the caller vouches for.  Any violation sets *bad.
__global__ void __launch_bounds__(256)
check_graph_kernel(int32_t N, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col, int* __restrict__ bad)
{
    const int32_t E = rowptr[N];
    if (blockIdx.x == 0 && threadIdx.x == 0 && (rowptr[0] != 0 || E < 0)) *bad = 1;
    for (int32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < N; i += gridDim.x * blockDim.x) {
        const int32_t beg = rowptr[i], end = rowptr[i + 1];
        if (beg < 0 || end < beg || end > E) { *bad = 1; continue; }
        for (int32_t p = beg; p < end; ++p) {
            const int32_t c = col[p];
            if (c < 0 || c >= N) *bad = 1;
        }
    }
}

size_t walk_smem_per_warp(const grf_walk_params& P)
{
    const size_t key_slots = (1 << P.seq_bits) < 32 ? 32 : (size_t)(1 << P.seq_bits);
    return (key_slots + (size_t)P.cap) * 4;
}

}  // namespace

int grf_walk_params_init(grf_walk_params* p, int32_t N, uint64_t seed, int32_t n_walks, float p_halt,
                         int32_t max_len, const float* f_phi, const float* f_psi)
{
    if (N <= 0 || n_walks < 1 || max_len < 0 || max_len > GRF_MAX_WALK_LEN || !f_phi) return GRF_ERR_INVALID;
    if (!(p_halt >= 0.0f) || !(p_halt < 1.0f)) return GRF_ERR_INVALID;
    const int64_t cap = (int64_t)n_walks * (max_len + 1);
    if (cap > 16384) return GRF_ERR_TOO_LARGE;
    int bits = 1;
    while ((1ll << bits) < cap) ++bits;
    if (((int64_t)N << bits) > (1ll << 32)) return GRF_ERR_TOO_LARGE;
    p->N = N; p->n_walks = n_walks; p->max_len = max_len;
    p->key0 = (uint32_t)seed; p->key1 = (uint32_t)(seed >> 32);
    double thr = (double)p_halt * 4294967296.0;   // halt iff word < floor(p_halt * 2^32)
    if (thr > 4294967295.0) thr = 4294967295.0;
    p->halt_threshold = (uint32_t)thr;            // conversion truncates: floor for values >= 0
    p->inv_keep = 1.0f / (1.0f - p_halt);
    p->inv_n = 1.0f / (float)n_walks;
    p->cap = (int32_t)cap;
    p->seq_bits = bits;
    if (!f_psi) f_psi = f_phi;
    for (int t = 0; t <= GRF_MAX_WALK_LEN; ++t) {
        p->f[0][t] = t <= max_len ? f_phi[t] : 0.0f;
        p->f[1][t] = t <= max_len ? f_psi[t] : 0.0f;
    }
    return GRF_OK;
}

static int sample_into(grf_ctx* ctx, grf_features* feat, const grf_walk_params& P,
                       const int32_t* rowptr, const int32_t* col, const float* w)
{
    const int32_t N = P.N;
    const int32_t stride = P.cap < N ? P.cap : N;   // a row cannot hold more distinct columns than N
    const size_t rows2 = 2 * (size_t)N;
    GRF_TRY(grf_buf_reserve(&ctx->stage_col, rows2 * stride * sizeof(int32_t)));
    GRF_TRY(grf_buf_reserve(&ctx->stage_val, rows2 * stride * sizeof(float)));
    GRF_TRY(grf_buf_reserve(&ctx->counts, rows2 * sizeof(int32_t)));
    GRF_TRY(grf_buf_reserve(&ctx->rowptr2, 2 * ((size_t)N + 1) * sizeof(int32_t)));
    GRF_TRY(grf_csr_reserve(&feat->phi, N, N, 0));
    GRF_TRY(grf_csr_reserve(&feat->psi, N, N, 0));

    const bool keep = ctx->keep_walks;
    feat->kept.valid = false;
    feat->kept.perm_valid = false;
    if (keep) {
        GRF_TRY(grf_buf_reserve(&ctx->stage_dep_start, rows2 * stride * sizeof(int32_t)));
        GRF_TRY(grf_buf_reserve(&ctx->stage_dep_t, rows2 * (size_t)P.cap));
        GRF_TRY(grf_buf_reserve(&ctx->stage_dep_load, rows2 * (size_t)P.cap * sizeof(float)));
        GRF_TRY(grf_buf_reserve(&ctx->dep_counts, rows2 * sizeof(int32_t)));
        GRF_TRY(grf_buf_reserve(&ctx->dep_rowptr2, 2 * ((size_t)N + 1) * sizeof(int32_t)));
    }

    const size_t per_warp = walk_smem_per_warp(P);
    int warps = (int)((200u * 1024u) / per_warp);
    if (warps > 8) warps = 8;
    if (warps < 1) warps = 1;
    const size_t smem = per_warp * warps;
    static_assert(sizeof(grf_walk_params) <= 4096, "kernel parameter block too large");
    GRF_CUDA_TRY(cudaFuncSetAttribute(walk_merge_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    GRF_CUDA_TRY(cudaFuncSetAttribute(walk_merge_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    {
        grf_launch_scope scope(ctx, 0);
        if (keep)
            walk_merge_kernel<true><<<grf_ceil_div(rows2, warps), warps * 32, smem, ctx->stream>>>(
                P, rowptr, col, w, stride, (int32_t*)ctx->stage_col.ptr, (float*)ctx->stage_val.ptr,
                (int32_t*)ctx->counts.ptr, (int32_t*)ctx->stage_dep_start.ptr, (unsigned char*)ctx->stage_dep_t.ptr,
                (float*)ctx->stage_dep_load.ptr, (int32_t*)ctx->dep_counts.ptr);
        else
            walk_merge_kernel<false><<<grf_ceil_div(rows2, warps), warps * 32, smem, ctx->stream>>>(
                P, rowptr, col, w, stride, (int32_t*)ctx->stage_col.ptr, (float*)ctx->stage_val.ptr,
                (int32_t*)ctx->counts.ptr, nullptr, nullptr, nullptr, nullptr);
    }
    GRF_CUDA_TRY(cudaGetLastError());

    // counts -> row pointers of Phi (segment 0) and Psi (segment 1)
    int32_t* scan_out = (int32_t*)ctx->rowptr2.ptr;
    GRF_TRY(grf_exclusive_scan(ctx, (const int32_t*)ctx->counts.ptr, scan_out, N, 2));
    int32_t* dep_scan = (int32_t*)ctx->dep_rowptr2.ptr;
    if (keep) {
        GRF_TRY(grf_exclusive_scan(ctx, (const int32_t*)ctx->dep_counts.ptr, dep_scan, N, 2));
        GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 2, dep_scan + N, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
        GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 3, dep_scan + 2 * N + 1, sizeof(int32_t), cudaMemcpyDeviceToHost,
                                     ctx->stream));
    }
    GRF_CUDA_TRY(cudaMemcpyAsync(feat->phi.rowptr.ptr, scan_out, ((size_t)N + 1) * sizeof(int32_t),
                                 cudaMemcpyDeviceToDevice, ctx->stream));
    GRF_CUDA_TRY(cudaMemcpyAsync(feat->psi.rowptr.ptr, scan_out + N + 1, ((size_t)N + 1) * sizeof(int32_t),
                                 cudaMemcpyDeviceToDevice, ctx->stream));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 0, scan_out + N, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 1, scan_out + 2 * N + 1, sizeof(int32_t), cudaMemcpyDeviceToHost,
                                 ctx->stream));
    GRF_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    const int64_t nnz_phi = ctx->pinned[0], nnz_psi = ctx->pinned[1];

    // column/value arrays, grown with head-room so that resampling rarely reallocates
    const int64_t cap_phi = nnz_phi + nnz_phi / 8 + 64, cap_psi = nnz_psi + nnz_psi / 8 + 64;
    if (feat->phi.col.bytes < (size_t)nnz_phi * 4) GRF_TRY(grf_csr_reserve(&feat->phi, N, N, cap_phi));
    if (feat->psi.col.bytes < (size_t)nnz_psi * 4) GRF_TRY(grf_csr_reserve(&feat->psi, N, N, cap_psi));
    if (feat->psit.col.bytes < (size_t)nnz_psi * 4 || feat->psit.rowptr.bytes < ((size_t)N + 1) * 4)
        GRF_TRY(grf_csr_reserve(&feat->psit, N, N, cap_psi));
    feat->phi.nnz = nnz_phi; feat->psi.nnz = nnz_psi; feat->psit.nnz = nnz_psi;
    feat->psit.rows = N; feat->psit.cols = N;

    {
        grf_launch_scope scope(ctx, 2);
        compact_rows_kernel<<<grf_ceil_div(rows2, 8), 256, 0, ctx->stream>>>(
            N, stride, (const int32_t*)ctx->stage_col.ptr, (const float*)ctx->stage_val.ptr,
            (const int32_t*)feat->phi.rowptr.ptr, (const int32_t*)feat->psi.rowptr.ptr,
            (int32_t*)feat->phi.col.ptr, (float*)feat->phi.val.ptr,
            (int32_t*)feat->psi.col.ptr, (float*)feat->psi.val.ptr);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    if (keep) {
        grf_kept_walks& K = feat->kept;
        const int64_t nnz_e[2] = {nnz_phi, nnz_psi};
        for (int e = 0; e < 2; ++e) {
            K.deposits[e] = ctx->pinned[2 + e];
            const size_t dcap = (size_t)K.deposits[e] + (size_t)K.deposits[e] / 8 + 64;
            if (K.dep_ptr[e].bytes < ((size_t)nnz_e[e] + 1) * 4)
                GRF_TRY(grf_buf_reserve(&K.dep_ptr[e], ((size_t)nnz_e[e] + (size_t)nnz_e[e] / 8 + 65) * 4));
            if (K.dep_t[e].bytes < (size_t)K.deposits[e]) GRF_TRY(grf_buf_reserve(&K.dep_t[e], dcap));
            if (K.dep_load[e].bytes < (size_t)K.deposits[e] * 4) GRF_TRY(grf_buf_reserve(&K.dep_load[e], dcap * 4));
        }
        {
            grf_launch_scope scope(ctx, 2);
            compact_deposits_kernel<<<grf_ceil_div(rows2, 8), 256, 0, ctx->stream>>>(
                N, stride, P.cap, (const int32_t*)ctx->stage_dep_start.ptr, (const unsigned char*)ctx->stage_dep_t.ptr,
                (const float*)ctx->stage_dep_load.ptr, (const int32_t*)feat->phi.rowptr.ptr,
                (const int32_t*)feat->psi.rowptr.ptr, dep_scan,
                (int32_t*)K.dep_ptr[0].ptr, (unsigned char*)K.dep_t[0].ptr, (float*)K.dep_load[0].ptr,
                (int32_t*)K.dep_ptr[1].ptr, (unsigned char*)K.dep_t[1].ptr, (float*)K.dep_load[1].ptr);
        }
        GRF_CUDA_TRY(cudaGetLastError());
        K.n_walks = P.n_walks; K.max_len = P.max_len; K.valid = true;
        K.perm_valid = false;
    }

    GRF_TRY(grf_transpose_launch(ctx, N, N, nnz_psi, (const int32_t*)feat->psi.rowptr.ptr,
                                 (const int32_t*)feat->psi.col.ptr, (const float*)feat->psi.val.ptr,
                                 (int32_t*)feat->psit.rowptr.ptr, (int32_t*)feat->psit.col.ptr,
                                 (float*)feat->psit.val.ptr));
    feat->plan_stale = true;       // the block plan of Phi is built by the first attention call that needs it
    feat->plan_ready = false;
    grf_mask_invalidate(feat);
    return GRF_OK;
}

extern "C" int grf_sample(grf_ctx* ctx, int32_t N, const int32_t* rowptr, const int32_t* col, const float* w,
                          uint64_t seed, int32_t n_walks, float p_halt, int32_t max_len,
                          const float* f_phi, const float* f_psi, grf_features** inout)
{
    if (!ctx || !rowptr || !col || !w || !inout) return GRF_ERR_INVALID;
    grf_walk_params P;
    GRF_TRY(grf_walk_params_init(&P, N, seed, n_walks, p_halt, max_len, f_phi, f_psi));
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    if (ctx->check_graphs) {
        // debugging aid: one pass over the graph and one wait for the device before any walk is taken
        GRF_CUDA_TRY(cudaMemsetAsync(ctx->error_word + 1, 0, sizeof(int), ctx->stream));
        check_graph_kernel<<<grf_ceil_div(N, 256) > 1184 ? 1184 : grf_ceil_div(N, 256), 256, 0, ctx->stream>>>(
            N, rowptr, col, ctx->error_word + 1);
        GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 9, ctx->error_word + 1, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
        GRF_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
        if (ctx->pinned[9] != 0) return GRF_ERR_BADGRAPH;
    }
    grf_features* feat = *inout;
    if (!feat) {
        feat = new (std::nothrow) grf_features();
        if (!feat) return GRF_ERR_NOMEM;
        feat->device = ctx->device;
    }
    const int rc = sample_into(ctx, feat, P, rowptr, col, w);
    if (rc != GRF_OK) {
        if (!*inout) grf_features_free(feat);
        return rc;
    }
    *inout = feat;
    return GRF_OK;
}

extern "C" int grf_debug_walks(grf_ctx* ctx, int32_t N, const int32_t* rowptr, const int32_t* col, const float* w,
                               uint64_t seed, int32_t n_walks, float p_halt, int32_t max_len,
                               int32_t* traj, float* load)
{
    if (!ctx || !rowptr || !col || !w || !traj || !load) return GRF_ERR_INVALID;
    grf_walk_params P;
    float ones[GRF_MAX_WALK_LEN + 1];
    for (float& x : ones) x = 1.0f;
    GRF_TRY(grf_walk_params_init(&P, N, seed, n_walks, p_halt, max_len, ones, ones));
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    const int64_t total = 2ll * N * n_walks;
    {
        grf_launch_scope scope(ctx, 0);
        debug_walks_kernel<<<grf_ceil_div(total, 256), 256, 0, ctx->stream>>>(P, rowptr, col, w, traj, load);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    return GRF_OK;
}

extern "C" int grf_ctx_keep_walks(grf_ctx* ctx, int enable)
{
    if (!ctx) return GRF_ERR_INVALID;
    ctx->keep_walks = enable != 0;
    return GRF_OK;
}

extern "C" int grf_remodulate(grf_ctx* ctx, grf_features* feat, int32_t max_len, const float* f_phi, const float* f_psi)
{
    if (!ctx || !feat || !f_phi) return GRF_ERR_INVALID;
    grf_kept_walks& K = feat->kept;
    if (!K.valid || max_len != K.max_len) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    if (!f_psi) f_psi = f_phi;
    grf_remod_params P;
    for (int t = 0; t <= GRF_MAX_WALK_LEN; ++t) {
        P.f[0][t] = t <= max_len ? f_phi[t] : 0.0f;
        P.f[1][t] = t <= max_len ? f_psi[t] : 0.0f;
    }
    P.inv_n = 1.0f / (float)K.n_walks;
    grf_csr_dev* mats[2] = {&feat->phi, &feat->psi};
    for (int e = 0; e < 2; ++e) {
        if (mats[e]->nnz == 0) continue;
        grf_launch_scope scope(ctx, 2);
        remodulate_kernel<<<grf_ceil_div(mats[e]->nnz, 256), 256, 0, ctx->stream>>>(
            P, e, mats[e]->nnz, (const int32_t*)K.dep_ptr[e].ptr, (const unsigned char*)K.dep_t[e].ptr,
            (const float*)K.dep_load[e].ptr, (float*)mats[e]->val.ptr);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    // Psi^T carries copies of Psi's values in another order, which does not change with the coefficients: the first
    // re-modulation regroups the entries' own indices (exact in fp32 below 2^24 entries) and keeps the result; from then
    // on the new values are fetched through it
    const int64_t nnz_psi = feat->psi.nnz;
    if (nnz_psi > 0 && nnz_psi < (1ll << 24)) {
        const int blocks = grf_ceil_div(nnz_psi, 256);
        if (!K.perm_valid) {
            if (K.psit_perm.bytes < (size_t)nnz_psi * 4) GRF_TRY(grf_buf_reserve(&K.psit_perm, ((size_t)nnz_psi + (size_t)nnz_psi / 8 + 64) * 4));
            {
                grf_launch_scope scope(ctx, 2);
                index_as_float_kernel<<<blocks, 256, 0, ctx->stream>>>((int32_t)nnz_psi, (float*)K.psit_perm.ptr);
            }
            GRF_TRY(grf_transpose_launch(ctx, feat->psi.rows, feat->psi.cols, nnz_psi, (const int32_t*)feat->psi.rowptr.ptr,
                                         (const int32_t*)feat->psi.col.ptr, (const float*)K.psit_perm.ptr,
                                         (int32_t*)feat->psit.rowptr.ptr, (int32_t*)feat->psit.col.ptr,
                                         (float*)feat->psit.val.ptr));
            {
                grf_launch_scope scope(ctx, 2);
                float_to_index_kernel<<<blocks, 256, 0, ctx->stream>>>((int32_t)nnz_psi, (const float*)feat->psit.val.ptr,
                                                                       (int32_t*)K.psit_perm.ptr);
            }
            K.perm_valid = true;
        }
        grf_launch_scope scope(ctx, 2);
        gather_values_kernel<<<blocks, 256, 0, ctx->stream>>>((int32_t)nnz_psi, (const int32_t*)K.psit_perm.ptr,
                                                              (const float*)feat->psi.val.ptr, (float*)feat->psit.val.ptr);
    } else {
        GRF_TRY(grf_transpose_launch(ctx, feat->psi.rows, feat->psi.cols, feat->psi.nnz, (const int32_t*)feat->psi.rowptr.ptr,
                                     (const int32_t*)feat->psi.col.ptr, (const float*)feat->psi.val.ptr,
                                     (int32_t*)feat->psit.rowptr.ptr, (int32_t*)feat->psit.col.ptr,
                                     (float*)feat->psit.val.ptr));
    }
    GRF_CUDA_TRY(cudaGetLastError());
    // the structure is the same: the block plan's node lists and the mask's key lists stay; the gather kernel's
    // coefficient table and the mask's values hold the old values
    feat->plan_coef_ready = false;
    grf_mask_values_stale(feat);
    return GRF_OK;
}
