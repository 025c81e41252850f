// Gather-and-contract with normalisation (Alg. 1 step 5, Eq. 12):
//   num_i = sum_l Phi_il phi(q_i)^T S_l,  den_i = sum_l Phi_il phi(q_i)^T z_l,  out_i = num_i / den_i.
//
// Plain-ALU kernel (any supported m, d; fp32 or bf16 storage): one warp per (problem g, query i).  A tile
// is read as consecutive 16-byte chunks (512 contiguous bytes per warp-wide load); sums are carried in
// fp32 in a fixed order.
#include "grf_internal.cuh"

namespace {

template <typename T> struct Chunk;
template <> struct Chunk<float> {
    __device__ static __forceinline__ void load(const float* p, float (&v)[4])
    {
        const float4 x = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    }
    __device__ static __forceinline__ void store1(float* p, float x) { *p = x; }
};
template <> struct Chunk<__nv_bfloat16> {
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
    __device__ static __forceinline__ void store1(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

constexpr int GATHER_WARPS = 4;

template <typename T, int M, int D>
__global__ void __launch_bounds__(GATHER_WARPS * 32)
gather_contract_kernel(int32_t N, int32_t R, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                       const float* __restrict__ val, const T* __restrict__ phiQ,
                       const unsigned char* __restrict__ records, T* __restrict__ out, float* __restrict__ den_out)
{
    constexpr int CH = grf_tile_chunk<T>();
    constexpr int NCHUNK = (M / CH) * D;            // 16-byte chunks per tile, chunk x = (a / CH) * D + b
    constexpr int NACC = D >= 32 ? D / 32 : 1;      // output columns per lane
    __shared__ float qs[GATHER_WARPS][M];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t i = blockIdx.x * GATHER_WARPS + warp;
    const int32_t g = blockIdx.y;
    if (i >= N) return;
    const T* qrow = phiQ + ((size_t)g * N + i) * M;
    for (int a = lane; a < M; a += 32) qs[warp][a] = to_f32(qrow[a]);
    __syncwarp();

    float acc[NACC];
#pragma unroll
    for (int j = 0; j < NACC; ++j) acc[j] = 0.0f;
    float den = 0.0f;

    constexpr size_t REC = grf_record_bytes<T>(M, D);
    const unsigned char* recs = records + (size_t)g * R * REC;
    for (int32_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
        const int32_t l = __ldg(col + p);
        const float phi = __ldg(val + p);
        const T* tile = reinterpret_cast<const T*>(recs + (size_t)l * REC);
        const float* zl = reinterpret_cast<const float*>(recs + (size_t)l * REC + (size_t)M * D * sizeof(T));
#pragma unroll
        for (int x0 = 0; x0 < NCHUNK; x0 += 32) {
            const int x = x0 + lane;
            if (NCHUNK % 32 == 0 || x < NCHUNK) {
                const int kc = D >= 32 ? x0 / D : x / D;
                float s[CH];
                Chunk<T>::load(tile + (size_t)x * CH, s);
                float dot = 0.0f;
#pragma unroll
                for (int c = 0; c < CH; ++c) dot = fmaf(qs[warp][kc * CH + c], s[c], dot);
                acc[D >= 32 ? (x0 % D) / 32 : 0] = fmaf(phi, dot, acc[D >= 32 ? (x0 % D) / 32 : 0]);
            }
        }
        for (int a = lane; a < M; a += 32) den = fmaf(phi * qs[warp][a], __ldg(zl + a), den);
    }
    if (D < 32) {
        // lanes with the same column b = lane % D hold partial sums over different row chunks
#pragma unroll
        for (int off = D; off < 32; off <<= 1) acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], off);
    }
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) den += __shfl_xor_sync(0xffffffffu, den, off);

    const float inv = den != 0.0f ? 1.0f / den : 0.0f;
    T* orow = out + ((size_t)g * N + i) * D;
    if (D >= 32) {
#pragma unroll
        for (int j = 0; j < NACC; ++j) Chunk<T>::store1(orow + j * 32 + lane, acc[j] * inv);
    } else if (lane < D) {
        Chunk<T>::store1(orow + lane, acc[0] * inv);
    }
    if (lane == 0 && den_out) den_out[(size_t)g * N + i] = den;
}

template <typename T, int M>
int launch_m(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t d,
             const void* phiQ, const void* records, void* out, float* den_out)
{
    const dim3 grid(grf_ceil_div(N, GATHER_WARPS), G);
#define GRF_GATHER_CASE(DD)                                                                                  \
    case DD:                                                                                                 \
        gather_contract_kernel<T, M, DD><<<grid, GATHER_WARPS * 32, 0, ctx->stream>>>(                       \
            N, phi.cols, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr,                        \
            (const float*)phi.val.ptr, (const T*)phiQ, (const unsigned char*)records, (T*)out, den_out);                   \
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
             const void* phiQ, const void* records, void* out, float* den_out)
{
    switch (m) {
        case 8: return launch_m<T, 8>(ctx, phi, G, N, d, phiQ, records, out, den_out);
        case 16: return launch_m<T, 16>(ctx, phi, G, N, d, phiQ, records, out, den_out);
        case 32: return launch_m<T, 32>(ctx, phi, G, N, d, phiQ, records, out, den_out);
        case 64: return launch_m<T, 64>(ctx, phi, G, N, d, phiQ, records, out, den_out);
        case 128: return launch_m<T, 128>(ctx, phi, G, N, d, phiQ, records, out, den_out);
        default: return GRF_ERR_INVALID;
    }
}

}  // namespace

int grf_gather_contract_alu(grf_ctx* ctx, const grf_csr_dev& phi, int32_t G, int32_t N, int32_t m, int32_t d,
                            int dtype, const void* phiQ, const void* records, void* out, float* den_out)
{
    if (G > 65535) return GRF_ERR_TOO_LARGE;
    if (dtype == GRF_DTYPE_F32) return launch_t<float>(ctx, phi, G, N, m, d, phiQ, records, out, den_out);
    if (dtype == GRF_DTYPE_BF16) return launch_t<__nv_bfloat16>(ctx, phi, G, N, m, d, phiQ, records, out, den_out);
    return GRF_ERR_INVALID;
}
