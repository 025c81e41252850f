// Masked attention with asymmetric graph random features (App. "Asymmetric graph random features", Alg. 2):
// with f^(2) = delta_0 the key-side features are the identity, the mask estimate is Phi itself and
//     out_i = sum_l Phi_il A_il v_l / sum_l Phi_il A_il,   A_il = phi(q_i) . phi(k_l)   (linear)
//                                                           A_il = exp(q_i . k_l)         (softmax)
// over the nodes l that the walkers out of node i visited: m + d multiply-adds per non-zero of Phi, no
// per-node states at all.
//
// One warp per query and two problems (they share the row's indices and mask values).  Non-zeros are taken
// 32 at a time: lane t computes the whole dot product of the batch's t-th key row with the query (the query
// sits in shared memory and is read as a broadcast), then
// the lanes spread over the d output columns and the batch's value rows are added one after the other, each
// read as one coalesced row.  The exponentials are taken relative to a running maximum of the scores, which
// cancels in the quotient; sums are carried in fp32 in a fixed order, so results are run-to-run identical.
#include "grf_internal.cuh"

namespace {

template <typename T> struct Row;
template <> struct Row<float> {
    static constexpr int CH = 4;
    __device__ static __forceinline__ void load(const float* p, float (&v)[4])
    {
        const float4 x = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    }
    __device__ static __forceinline__ float get(const float* p) { return __ldg(p); }
    __device__ static __forceinline__ void put(float* p, float x) { *p = x; }
};
template <> struct Row<__nv_bfloat16> {
    static constexpr int CH = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8])
    {
        const uint4 x = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            v[2 * q] = __uint_as_float(w[q] << 16);
            v[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
        }
    }
    __device__ static __forceinline__ float get(const __nv_bfloat16* p)
    {
        return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
    }
    __device__ static __forceinline__ void put(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};

constexpr int ASYM_WARPS = 8;
constexpr int ASYM_GH = 2;      // problems per warp: they share the row's indices and mask values

template <typename T, int M, int D, bool SOFTMAX>
__global__ void __launch_bounds__(ASYM_WARPS * 32)
asym_attention_kernel(int32_t G, int32_t N, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                      const float* __restrict__ val, const T* __restrict__ Q, const T* __restrict__ K,
                      const T* __restrict__ V, T* __restrict__ out, float* __restrict__ den_out)
{
    constexpr int CH = Row<T>::CH;
    constexpr int EPL = D >= 32 ? D / 32 : 1;        // output columns per lane
    constexpr int GH = ASYM_GH;
    __shared__ float qs[ASYM_WARPS][GH][M];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t i = blockIdx.x * ASYM_WARPS + warp;
    const int32_t g0 = blockIdx.y * GH;
    if (i >= N) return;
#pragma unroll
    for (int h = 0; h < GH; ++h) {
        const int32_t g = min(g0 + h, G - 1);        // a problem beyond the batch repeats the last one and is not written
        const T* qrow = Q + ((size_t)g * N + i) * M;
        for (int a = lane; a < M; a += 32) qs[warp][h][a] = Row<T>::get(qrow + a);
    }
    __syncwarp();
    const bool col_lane = lane * EPL < D;            // lanes that own output columns

    float acc[GH][EPL];
    float den[GH], run_max[GH];                      // this lane's share of the denominators; softmax: running maxima
#pragma unroll
    for (int h = 0; h < GH; ++h) {
        den[h] = 0.0f; run_max[h] = -INFINITY;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[h][e] = 0.0f;
    }

    const int32_t beg = rowptr[i], end = rowptr[i + 1];
    for (int32_t p0 = beg; p0 < end; p0 += 32) {
        const int32_t n = min(32, end - p0);
        const bool valid = lane < n;
        const int32_t l = valid ? __ldg(col + p0 + lane) : 0;
        const float phi = valid ? __ldg(val + p0 + lane) : 0.0f;
        float w[GH];
#pragma unroll
        for (int h = 0; h < GH; ++h) {
            const int32_t g = min(g0 + h, G - 1);
            // score of this lane's key: the whole dot product in one lane
            float s = 0.0f;
            if (valid) {
                const T* krow = K + ((size_t)g * N + l) * M;
#pragma unroll
                for (int c = 0; c < M / CH; ++c) {
                    float v[CH];
                    Row<T>::load(krow + c * CH, v);
#pragma unroll
                    for (int e = 0; e < CH; ++e) s = fmaf(v[e], qs[warp][h][c * CH + e], s);
                }
            }
            if (SOFTMAX) {
                float bmax = valid ? s : -INFINITY;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, off));
                const float new_max = fmaxf(run_max[h], bmax);
                const float rescale = __expf(run_max[h] - new_max);     // 0 on the first batch (run_max = -inf)
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[h][e] *= rescale;
                den[h] *= rescale;
                run_max[h] = new_max;
                w[h] = valid ? phi * __expf(s - new_max) : 0.0f;
            } else {
                w[h] = phi * s;
            }
            den[h] += w[h];
        }
        // the batch's value rows, one after the other, lanes across the output columns
        for (int32_t t = 0; t < n; ++t) {
            const int32_t lt = __shfl_sync(0xffffffffu, l, t);
#pragma unroll
            for (int h = 0; h < GH; ++h) {
                const float wt = __shfl_sync(0xffffffffu, w[h], t);
                const int32_t g = min(g0 + h, G - 1);
                if (col_lane) {
                    const T* vrow = V + ((size_t)g * N + lt) * D + lane * EPL;
                    if constexpr (sizeof(T) == 2 && EPL == 2) {
                        const uint32_t x = __ldg(reinterpret_cast<const uint32_t*>(vrow));
                        acc[h][0] = fmaf(wt, __uint_as_float(x << 16), acc[h][0]);
                        acc[h][1] = fmaf(wt, __uint_as_float(x & 0xffff0000u), acc[h][1]);
                    } else if constexpr (sizeof(T) == 2 && EPL == 4) {
                        const uint2 x = __ldg(reinterpret_cast<const uint2*>(vrow));
                        acc[h][0] = fmaf(wt, __uint_as_float(x.x << 16), acc[h][0]);
                        acc[h][1] = fmaf(wt, __uint_as_float(x.x & 0xffff0000u), acc[h][1]);
                        acc[h][2] = fmaf(wt, __uint_as_float(x.y << 16), acc[h][2]);
                        acc[h][3] = fmaf(wt, __uint_as_float(x.y & 0xffff0000u), acc[h][3]);
                    } else {
#pragma unroll
                        for (int e = 0; e < EPL; ++e) acc[h][e] = fmaf(wt, Row<T>::get(vrow + e), acc[h][e]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int h = 0; h < GH; ++h) {
        float dn = den[h];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) dn += __shfl_xor_sync(0xffffffffu, dn, off);
        if (g0 + h >= G) break;
        const float inv = dn != 0.0f ? 1.0f / dn : 0.0f;
        if (col_lane) {
            T* orow = out + ((size_t)(g0 + h) * N + i) * D + lane * EPL;
#pragma unroll
            for (int e = 0; e < EPL; ++e) Row<T>::put(orow + e, acc[h][e] * inv);
        }
        // with the softmax kernel the reported denominator is relative to exp(max score of the row)
        if (lane == 0 && den_out) den_out[(size_t)(g0 + h) * N + i] = dn;
    }
}

template <typename T, int M, int D>
int launch_md(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int kernel, const void* Q, const void* K,
              const void* V, void* out, float* den_out)
{
    const dim3 grid(grf_ceil_div(N, ASYM_WARPS), grf_ceil_div(G, ASYM_GH));
    grf_launch_scope scope(ctx, 5);
    if (kernel == GRF_KERNEL_SOFTMAX)
        asym_attention_kernel<T, M, D, true><<<grid, ASYM_WARPS * 32, 0, ctx->stream>>>(
            G, N, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr, (const float*)phi.val.ptr, (const T*)Q,
            (const T*)K, (const T*)V, (T*)out, den_out);
    else
        asym_attention_kernel<T, M, D, false><<<grid, ASYM_WARPS * 32, 0, ctx->stream>>>(
            G, N, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr, (const float*)phi.val.ptr, (const T*)Q,
            (const T*)K, (const T*)V, (T*)out, den_out);
    return GRF_OK;
}

template <typename T, int M>
int launch_m(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t d, int kernel, const void* Q,
             const void* K, const void* V, void* out, float* den_out)
{
    switch (d) {
        case 8: return launch_md<T, M, 8>(ctx, phi, G, N, kernel, Q, K, V, out, den_out);
        case 16: return launch_md<T, M, 16>(ctx, phi, G, N, kernel, Q, K, V, out, den_out);
        case 32: return launch_md<T, M, 32>(ctx, phi, G, N, kernel, Q, K, V, out, den_out);
        case 64: return launch_md<T, M, 64>(ctx, phi, G, N, kernel, Q, K, V, out, den_out);
        case 128: return launch_md<T, M, 128>(ctx, phi, G, N, kernel, Q, K, V, out, den_out);
    }
    return GRF_ERR_INVALID;
}

template <typename T>
int launch_t(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t m, int32_t d, int kernel,
             const void* Q, const void* K, const void* V, void* out, float* den_out)
{
    switch (m) {
        case 8: return launch_m<T, 8>(ctx, phi, G, N, d, kernel, Q, K, V, out, den_out);
        case 16: return launch_m<T, 16>(ctx, phi, G, N, d, kernel, Q, K, V, out, den_out);
        case 32: return launch_m<T, 32>(ctx, phi, G, N, d, kernel, Q, K, V, out, den_out);
        case 64: return launch_m<T, 64>(ctx, phi, G, N, d, kernel, Q, K, V, out, den_out);
        case 128: return launch_m<T, 128>(ctx, phi, G, N, d, kernel, Q, K, V, out, den_out);
    }
    return GRF_ERR_INVALID;
}

}  // namespace

extern "C" int grf_masked_attn_asym(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                                    int dtype, int kernel, const void* Q, const void* K, const void* V, void* out,
                                    float* den_out)
{
    if (!ctx || !feat || !Q || !K || !V || !out) return GRF_ERR_INVALID;
    if (G <= 0 || G > 65535 || N <= 0) return GRF_ERR_INVALID;
    if (kernel != GRF_KERNEL_LINEAR && kernel != GRF_KERNEL_SOFTMAX) return GRF_ERR_INVALID;
    if (dtype != GRF_DTYPE_F32 && dtype != GRF_DTYPE_BF16) return GRF_ERR_INVALID;
    if (feat->phi.rows != N || feat->phi.cols != N) return GRF_ERR_INVALID;       // the mask estimate is Phi: N x N
    if ((((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)out) & 15) != 0) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    const int rc = dtype == GRF_DTYPE_F32
                       ? launch_t<float>(ctx, feat->phi, G, N, m, d, kernel, Q, K, V, out, den_out)
                       : launch_t<__nv_bfloat16>(ctx, feat->phi, G, N, m, d, kernel, Q, K, V, out, den_out);
    if (rc != GRF_OK) return rc;
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}
