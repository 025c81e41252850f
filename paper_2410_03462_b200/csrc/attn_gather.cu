// Gather-and-contract with normalisation (Alg. 1 step 5, Eq. 12):
//   num_i = sum_l Phi_il phi(q_i)^T S_l,  den_i = sum_l Phi_il phi(q_i)^T z_l,  out_i = num_i / den_i.
// One warp per (problem g, query i).  Every S_l tile is read with 16-byte loads, a group of lanes
// per tile row; sums are carried in fp32 in a fixed order.
#include "grf_internal.cuh"

namespace {

template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const float* p, float (&v)[4])
    {
        const float4 x = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    }
    __device__ static __forceinline__ void store(float* p, const float (&v)[4])
    {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
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
    __device__ static __forceinline__ void store(__nv_bfloat16* p, const float (&v)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * q], v[2 * q + 1]);
            w[q] = *reinterpret_cast<uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

constexpr int GATHER_WARPS = 4;

template <typename T, int D> struct GatherShape {
    static constexpr int VEC = (Vec16<T>::N < D) ? Vec16<T>::N : D;   // elements per lane per tile row
    static constexpr int LPR = D / VEC;                               // lanes that share one tile row
    static constexpr int RPI = 32 / LPR;                              // tile rows per warp-wide load
};

template <typename T, int M, int D>
__global__ void __launch_bounds__(GATHER_WARPS * 32)
gather_contract_kernel(int32_t N, int32_t R, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                       const float* __restrict__ val, const T* __restrict__ phiQ, const T* __restrict__ S,
                       const float* __restrict__ z, T* __restrict__ out, float* __restrict__ den_out)
{
    constexpr int VEC = Vec16<T>::N;
    static_assert(D % VEC == 0, "head dimension must fill whole 16-byte vectors");
    constexpr int LPR = D / VEC;
    constexpr int RPI = 32 / LPR;
    static_assert(LPR >= 1 && LPR <= 32, "unsupported head dimension");
    __shared__ float qs[GATHER_WARPS][M];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t i = blockIdx.x * GATHER_WARPS + warp;
    const int32_t g = blockIdx.y;
    if (i >= N) return;
    const T* qrow = phiQ + ((size_t)g * N + i) * M;
    for (int a = lane; a < M; a += 32) qs[warp][a] = to_f32(qrow[a]);
    __syncwarp();

    const int sub = lane / LPR;         // which of the RPI rows this lane reads
    const int cg = lane % LPR;          // which 16-byte column group
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.0f;
    float den = 0.0f;

    const T* Sg = S + (size_t)g * R * M * D;
    const float* zg = z + (size_t)g * R * M;
    for (int32_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
        const int32_t l = __ldg(col + p);
        const float phi = __ldg(val + p);
        const T* tile = Sg + (size_t)l * M * D;
        const float* zl = zg + (size_t)l * M;
#pragma unroll
        for (int a0 = 0; a0 < M; a0 += RPI) {
            const int a = a0 + sub;
            if (RPI <= M || a < M) {
                const float c = phi * qs[warp][a];
                float s[VEC];
                Vec16<T>::load(tile + (size_t)a * D + cg * VEC, s);
#pragma unroll
                for (int v = 0; v < VEC; ++v) acc[v] = fmaf(c, s[v], acc[v]);
                if (cg == 0) den = fmaf(c, __ldg(zl + a), den);
            }
        }
    }
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] += __shfl_xor_sync(0xffffffffu, acc[v], off);
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) den += __shfl_xor_sync(0xffffffffu, den, off);

    if (lane < LPR) {
        const float inv = den != 0.0f ? 1.0f / den : 0.0f;
        float o[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) o[v] = acc[v] * inv;
        Vec16<T>::store(out + ((size_t)g * N + i) * D + cg * VEC, o);
    }
    if (lane == 0 && den_out) den_out[(size_t)g * N + i] = den;
}

template <typename T, int M>
int launch_m(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t d,
             const void* phiQ, const void* S, const float* z, void* out, float* den_out)
{
    const dim3 grid(grf_ceil_div(N, GATHER_WARPS), G);
#define GRF_GATHER_CASE(DD)                                                                                  \
    case DD:                                                                                                 \
        gather_contract_kernel<T, M, DD><<<grid, GATHER_WARPS * 32, 0, ctx->stream>>>(                       \
            N, phi.cols, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr,                        \
            (const float*)phi.val.ptr, (const T*)phiQ, (const T*)S, z, (T*)out, den_out);                   \
        break;
    {
    grf_launch_scope scope(ctx, 5);
    switch (d) {
        GRF_GATHER_CASE(8) GRF_GATHER_CASE(16) GRF_GATHER_CASE(32) GRF_GATHER_CASE(64) GRF_GATHER_CASE(128)
        default: return GRF_ERR_INVALID;
    }
    }
#undef GRF_GATHER_CASE
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

template <typename T>
int launch_t(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t m, int32_t d,
             const void* phiQ, const void* S, const float* z, void* out, float* den_out)
{
    switch (m) {
        case 8: return launch_m<T, 8>(ctx, phi, G, N, d, phiQ, S, z, out, den_out);
        case 16: return launch_m<T, 16>(ctx, phi, G, N, d, phiQ, S, z, out, den_out);
        case 32: return launch_m<T, 32>(ctx, phi, G, N, d, phiQ, S, z, out, den_out);
        case 64: return launch_m<T, 64>(ctx, phi, G, N, d, phiQ, S, z, out, den_out);
        case 128: return launch_m<T, 128>(ctx, phi, G, N, d, phiQ, S, z, out, den_out);
        default: return GRF_ERR_INVALID;
    }
}

}  // namespace

int grf_gather_contract(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t m, int32_t d, int dtype,
                        const void* phiQ, const void* S, const float* z, void* out, float* den_out)
{
    if (G > 65535) return GRF_ERR_TOO_LARGE;
    if (dtype == GRF_DTYPE_F32) return launch_t<float>(ctx, phi, G, N, m, d, phiQ, S, z, out, den_out);
    if (dtype == GRF_DTYPE_BF16) return launch_t<__nv_bfloat16>(ctx, phi, G, N, m, d, phiQ, S, z, out, den_out);
    return GRF_ERR_INVALID;
}
