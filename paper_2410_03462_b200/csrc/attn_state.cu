// Per-node states of Alg. 1 step 5 (Eq. 12):  S_l = sum_j Psi_jl phi(k_j) v_j^T  (m x d),
// z_l = sum_j Psi_jl phi(k_j)  (m), for every problem g and node l — the rows of Phi_K^T V and
// Phi_K^T 1 of Corollary 3.4.  A segmented reduction over the column-grouped Psi^T with a fixed
// summation order (ascending j), fp32 accumulation, no atomics.
//
// This file holds the plain-ALU kernel (any supported m, d; fp32 or bf16 storage).
#include "grf_internal.cuh"

namespace {

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

// one 16-byte chunk of the tile: CH consecutive feature rows a of one column b
__device__ __forceinline__ void store_chunk(float* dst, const float (&v)[4])
{
    *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store_chunk(__nv_bfloat16* dst, const float (&v)[8])
{
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * q], v[2 * q + 1]);
        w[q] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
}

template <typename T, int M, int D>
struct StateTiling {
    static constexpr int CH = grf_tile_chunk<T>();               // feature rows per 16-byte chunk
    static constexpr int TXB = D < 32 ? D : 32;                   // threads across the columns b
    static constexpr int TB = D / TXB;                            // columns per thread (b, b+TXB, ...)
    static constexpr int KC = M / CH;                             // chunks along a
    static constexpr int THREADS = KC * TXB;
    static constexpr int JC = 8;                                  // source rows staged per step
};

// One CTA per (node l, problem g).  Thread (kc, bx) keeps the CH x TB block
// {a in chunk kc} x {b = bx + TXB*t} of the tile in registers and writes it as TB 16-byte chunks.
template <typename T, int M, int D>
__global__ void __launch_bounds__(StateTiling<T, M, D>::THREADS)
build_states_kernel(int32_t R, int32_t N, const int32_t* __restrict__ t_rowptr, const int32_t* __restrict__ t_col,
                    const float* __restrict__ t_val, const T* __restrict__ phiK, const T* __restrict__ V,
                    unsigned char* __restrict__ records)
{
    using Tl = StateTiling<T, M, D>;
    constexpr int CH = Tl::CH, TXB = Tl::TXB, TB = Tl::TB, JC = Tl::JC, THREADS = Tl::THREADS;
    __shared__ __align__(16) float ks[JC][M];
    __shared__ __align__(16) float vs[JC][D];

    const int32_t l = blockIdx.x, g = blockIdx.y;
    const int tid = threadIdx.x, bx = tid % TXB, kc = tid / TXB;
    const T* Kg = phiK + (size_t)g * N * M;
    const T* Vg = V + (size_t)g * N * D;

    float acc[TB][CH];
    float zacc[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        zacc[c] = 0.0f;
#pragma unroll
        for (int t = 0; t < TB; ++t) acc[t][c] = 0.0f;
    }

    const int32_t beg = t_rowptr[l], end = t_rowptr[l + 1];
    for (int32_t p0 = beg; p0 < end; p0 += JC) {
        const int32_t nj = min(JC, end - p0);
        for (int idx = tid; idx < JC * M; idx += THREADS) {
            const int jj = idx / M, a = idx % M;
            float x = 0.0f;
            if (jj < nj) x = t_val[p0 + jj] * to_f32(Kg[(size_t)t_col[p0 + jj] * M + a]);
            ks[jj][a] = x;
        }
        for (int idx = tid; idx < JC * D; idx += THREADS) {
            const int jj = idx / D, b = idx % D;
            vs[jj][b] = jj < nj ? to_f32(Vg[(size_t)t_col[p0 + jj] * D + b]) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int jj = 0; jj < JC; ++jj) {
            float kr[CH];
#pragma unroll
            for (int c = 0; c < CH; ++c) kr[c] = ks[jj][kc * CH + c];
#pragma unroll
            for (int t = 0; t < TB; ++t) {
                const float vb = vs[jj][bx + t * TXB];
#pragma unroll
                for (int c = 0; c < CH; ++c) acc[t][c] = fmaf(kr[c], vb, acc[t][c]);
            }
#pragma unroll
            for (int c = 0; c < CH; ++c) zacc[c] += kr[c];
        }
        __syncthreads();
    }

    unsigned char* rec = records + ((size_t)g * R + l) * grf_record_bytes<T>(M, D);
    T* Sl = reinterpret_cast<T*>(rec);
#pragma unroll
    for (int t = 0; t < TB; ++t) store_chunk(Sl + grf_tile_index<T>(kc * CH, bx + t * TXB, D), acc[t]);
    if (bx == 0) {
        float* zl = reinterpret_cast<float*>(rec + (size_t)M * D * sizeof(T));
#pragma unroll
        for (int c = 0; c < CH; ++c) zl[kc * CH + c] = zacc[c];
        if constexpr (sizeof(T) == 2) {
            __nv_bfloat16* zb = reinterpret_cast<__nv_bfloat16*>(rec + (size_t)M * D * sizeof(T) + (size_t)M * sizeof(float));
#pragma unroll
            for (int c = 0; c < CH; ++c) zb[kc * CH + c] = __float2bfloat16_rn(zacc[c]);
        }
    }
}

template <typename T, int M>
int launch_m(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, int32_t d,
             const void* phiK, const void* V, void* records)
{
    const dim3 grid(psit.rows, G);
#define GRF_STATE_CASE(DD)                                                                                  \
    case DD:                                                                                                \
        build_states_kernel<T, M, DD><<<grid, StateTiling<T, M, DD>::THREADS, 0, ctx->stream>>>(            \
            psit.rows, N, (const int32_t*)psit.rowptr.ptr, (const int32_t*)psit.col.ptr,                    \
            (const float*)psit.val.ptr, (const T*)phiK, (const T*)V, (unsigned char*)records);                            \
        break;
    {
        grf_launch_scope scope(ctx, 4);
        switch (d) {
            GRF_STATE_CASE(8) GRF_STATE_CASE(16) GRF_STATE_CASE(32) GRF_STATE_CASE(64) GRF_STATE_CASE(128)
            default: return GRF_ERR_INVALID;
        }
    }
#undef GRF_STATE_CASE
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

template <typename T>
int launch_t(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, int32_t m, int32_t d,
             const void* phiK, const void* V, void* records)
{
    switch (m) {
        case 8: return launch_m<T, 8>(ctx, psit, G, N, d, phiK, V, records);
        case 16: return launch_m<T, 16>(ctx, psit, G, N, d, phiK, V, records);
        case 32: return launch_m<T, 32>(ctx, psit, G, N, d, phiK, V, records);
        case 64: return launch_m<T, 64>(ctx, psit, G, N, d, phiK, V, records);
        case 128: return launch_m<T, 128>(ctx, psit, G, N, d, phiK, V, records);
        default: return GRF_ERR_INVALID;
    }
}

}  // namespace

int grf_build_states(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, int32_t m, int32_t d, int dtype,
                     const void* phiK, const void* V, void* records)
{
    if (G > 65535) return GRF_ERR_TOO_LARGE;
    if (dtype == GRF_DTYPE_F32) return launch_t<float>(ctx, psit, G, N, m, d, phiK, V, records);
    if (dtype == GRF_DTYPE_BF16) return launch_t<__nv_bfloat16>(ctx, psit, G, N, m, d, phiK, V, records);
    return GRF_ERR_INVALID;
}
