// Gather-and-contract on the 5th-generation tensor cores (Alg. 1 step 5, Eq. 12), bf16 storage.
//
// A CTA owns a block of 128 consecutive queries of one problem g.  The block's rows of Phi touch a
// union U of nodes l (the "block plan", a sorted list built once per feature object).  For every l in U
//     D[128 x d] += A_l[128 x m] * S_l[m x d],      A_l[i, a] = Phi_il * phi(q_i)_a   (0 where Phi_il = 0)
// is one or more tcgen05.mma instructions (M = 128, N = d, K = 16 each) accumulating in tensor memory:
// the sum over l of Eq. 12 becomes the K dimension of one long matrix product, evaluated in a fixed order.
//   - S_l arrives by one contiguous bulk async copy (the workspace stores tiles in operand layout),
//   - A_l is produced by the 128 "row" threads, one query each, walking their own CSR row of Phi in step
//     with the union list,
//   - one thread issues the MMAs; completion is tracked with mbarriers, every wait is bounded.
// Nodes that no query of the block touches are never loaded; a tile is loaded once per block, not once
// per query, which is where the method's "constant multiplicative cost" is paid down.
#include "grf_internal.cuh"

namespace {

constexpr int BQ = GRF_PLAN_BLOCK;  // queries per CTA = MMA M
constexpr int TC_THREADS = 192;     // warps 0-3: row threads / epilogue, warp 4: tile loader, warp 5: MMA issuer
constexpr unsigned long long WAIT_NS = 2000000000ull;   // a wait that lasts longer than this gives up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when another thread of the CTA has given up or when this wait lasted too long
// (then it raises the CTA's abort flag itself).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((it & 255u) == 0u && global_ns() - t0 > WAIT_NS) { *abort_flag = 1; return false; }
    }
}

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Shared-memory operand descriptor: unswizzled, 8-row core matrices of 128 contiguous bytes;
// lbo = byte distance between the two 16-byte K chunks of one instruction, sbo = between 8-row groups.
__device__ __forceinline__ uint64_t operand_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(sbo_bytes >> 4) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int M, int D> struct TcShape {
    static constexpr int KC = M / 8;                          // 16-byte K chunks of one A row
    static constexpr int A_BYTES = KC * BQ * 16;              // [chunk][row][16 B]
    static constexpr int B_BYTES = M * D * 2;                 // one state tile
    static constexpr int STAGE = A_BYTES + B_BYTES;
    static constexpr int STAGES = (160 * 1024 / STAGE) >= 4 ? 4 : ((160 * 1024 / STAGE) >= 3 ? 3 : 2);
    static constexpr int TMEM_COLS = D < 32 ? 32 : D;
    static constexpr size_t SMEM = (size_t)STAGES * STAGE + 1024; // + alignment slack
};

template <int M, int D>
__global__ void __launch_bounds__(TC_THREADS)
gather_contract_tc_kernel(int32_t N, int32_t R, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                          const float* __restrict__ val, const int32_t* __restrict__ plan_off,
                          const int32_t* __restrict__ plan_cnt, const int32_t* __restrict__ plan_col,
                          const __nv_bfloat16* __restrict__ phiQ, const __nv_bfloat16* __restrict__ S,
                          const float* __restrict__ z, __nv_bfloat16* __restrict__ out, float* __restrict__ den_out,
                          int* __restrict__ error_word)
{
    using Sh = TcShape<M, D>;
    constexpr int NS = Sh::STAGES;
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) unsigned long long bars[3 * NS + 1];   // a_full, b_full, empty per stage; acc_done
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t blk = blockIdx.x, g = blockIdx.y;
    const uint32_t stage_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_u32(bars);
    auto a_full = [&](int s) { return bar_base + 8u * (uint32_t)s; };
    auto b_full = [&](int s) { return bar_base + 8u * (uint32_t)(NS + s); };
    auto empty = [&](int s) { return bar_base + 8u * (uint32_t)(2 * NS + s); };
    const uint32_t acc_done = bar_base + 8u * (uint32_t)(3 * NS);

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(a_full(s), BQ); mbar_init(b_full(s), 1); mbar_init(empty(s), 1); }
        mbar_init(acc_done, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = tmem_slot;

    const int32_t cnt = plan_cnt[blk];
    const int32_t* ulist = plan_col + plan_off[blk];
    const __nv_bfloat16* Sg = S + (size_t)g * R * M * D;

    if (warp < 4) {
        // ------------------------------------------------------------ row threads: build A, then epilogue
        const int32_t row = blk * BQ + tid;
        const bool live = row < N;
        uint32_t q2[M / 2];
        if (live) {
            const uint4* qp = reinterpret_cast<const uint4*>(phiQ + ((size_t)g * N + row) * M);
#pragma unroll
            for (int c = 0; c < M / 8; ++c) {
                const uint4 x = __ldg(qp + c);
                q2[4 * c] = x.x; q2[4 * c + 1] = x.y; q2[4 * c + 2] = x.z; q2[4 * c + 3] = x.w;
            }
        } else {
#pragma unroll
            for (int c = 0; c < M / 2; ++c) q2[c] = 0u;
        }
        int32_t p = live ? rowptr[row] : 0;
        const int32_t pend = live ? rowptr[row + 1] : 0;
        int32_t next_col = p < pend ? __ldg(col + p) : -1;
        float next_val = p < pend ? __ldg(val + p) : 0.0f;
        const float* zg = z + (size_t)g * R * M;
        float den = 0.0f;
        bool ok = true;
        for (int32_t u = 0; u < cnt; ++u) {
            const int s = u % NS;
            const uint32_t ph = (uint32_t)(u / NS) & 1u;
            if (!mbar_wait(empty(s), ph ^ 1u, &abort_flag)) { ok = false; break; }
            const int32_t l = __ldg(ulist + u);
            float coef = 0.0f;
            if (next_col == l) {
                coef = next_val;
                ++p;
                next_col = p < pend ? __ldg(col + p) : -1;
                next_val = p < pend ? __ldg(val + p) : 0.0f;
            }
            const uint32_t a_stage = stage_base + (uint32_t)s * Sh::STAGE;
            if (coef != 0.0f) {
                const float4* zl = reinterpret_cast<const float4*>(zg + (size_t)l * M);
                float dot = 0.0f;
#pragma unroll
                for (int c = 0; c < M / 4; ++c) {
                    const float4 zz = __ldg(zl + c);
                    dot = fmaf(__uint_as_float(q2[2 * c] << 16), zz.x, dot);
                    dot = fmaf(__uint_as_float(q2[2 * c] & 0xffff0000u), zz.y, dot);
                    dot = fmaf(__uint_as_float(q2[2 * c + 1] << 16), zz.z, dot);
                    dot = fmaf(__uint_as_float(q2[2 * c + 1] & 0xffff0000u), zz.w, dot);
                }
                den = fmaf(coef, dot, den);
#pragma unroll
                for (int c = 0; c < M / 8; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = coef * __uint_as_float(q2[4 * c + e] << 16);
                        const float hi = coef * __uint_as_float(q2[4 * c + e] & 0xffff0000u);
                        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
                        w[e] = *reinterpret_cast<uint32_t*>(&h);
                    }
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                 ::"r"(a_stage + (uint32_t)c * (BQ * 16) + (uint32_t)tid * 16),
                                   "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
                }
            } else {
#pragma unroll
                for (int c = 0; c < M / 8; ++c)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};"
                                 ::"r"(a_stage + (uint32_t)c * (BQ * 16) + (uint32_t)tid * 16), "r"(0u) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(a_full(s));
        }
        // epilogue: this thread's row of the accumulator is TMEM lane `tid`
        if (ok && cnt > 0) ok = mbar_wait(acc_done, 0u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);   // the tensor-memory loads below are warp-wide
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const float inv = (den != 0.0f) ? 1.0f / den : 0.0f;
        __nv_bfloat16* orow = out + ((size_t)g * N + row) * D;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t r[16];
            if (ok && cnt > 0) {
                tmem_ld16(tmem_acc + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) r[e] = 0u;
            }
            if (live && ok) {
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[2 * e]) * inv, __uint_as_float(r[2 * e + 1]) * inv);
                    w[e] = *reinterpret_cast<uint32_t*>(&h);
                }
                uint4* dst = reinterpret_cast<uint4*>(orow + c0);
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            }
        }
        if (live && ok && den_out) den_out[(size_t)g * N + row] = den;
    } else if (warp == 4) {
        // ------------------------------------------------------------ tile loader
        int32_t issued = 0;
        for (int32_t u = 0; u < cnt; ++u) {
            const int s = u % NS;
            const uint32_t ph = (uint32_t)(u / NS) & 1u;
            if (!mbar_wait(empty(s), ph ^ 1u, &abort_flag)) break;
            if (lane == 0) {
                const int32_t l = __ldg(ulist + u);
                mbar_arrive_expect_tx(b_full(s), Sh::B_BYTES);
                bulk_copy_g2s(stage_base + (uint32_t)s * Sh::STAGE + Sh::A_BYTES, Sg + (size_t)l * M * D, Sh::B_BYTES,
                              b_full(s));
            }
            ++issued;
            __syncwarp();
        }
        if (abort_flag) {
            // gave up somewhere: let the copies that are still in flight land before the CTA exits
            const int32_t first = issued > NS ? issued - NS : 0;
            for (int32_t u = first; u < issued; ++u) {
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(b_full(u % NS), (uint32_t)(u / NS) & 1u) && global_ns() - t0 < WAIT_NS) {}
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = instr_desc_bf16(D);
        bool ok = true;
        for (int32_t u = 0; u < cnt; ++u) {
            const int s = u % NS;
            const uint32_t ph = (uint32_t)(u / NS) & 1u;
            if (!mbar_wait(a_full(s), ph, &abort_flag) || !mbar_wait(b_full(s), ph, &abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (lane == 0) {
                const uint32_t a_stage = stage_base + (uint32_t)s * Sh::STAGE;
                const uint32_t b_stage = a_stage + Sh::A_BYTES;
#pragma unroll
                for (int k = 0; k < M / 16; ++k) {
                    const uint64_t ad = operand_desc(a_stage + (uint32_t)k * 2u * (BQ * 16), BQ * 16, 128);
                    const uint64_t bd = operand_desc(b_stage + (uint32_t)k * 2u * (D * 16), D * 16, 128);
                    mma_bf16_ss(tmem_acc, ad, bd, idesc, (u > 0 || k > 0) ? 1u : 0u);
                }
                mma_commit(empty(s));
            }
            __syncwarp();
        }
        if (lane == 0 && cnt > 0) mma_commit(acc_done);
        __syncwarp();
        if (!ok && cnt > 0) {
            // aborted: wait (bounded) until the MMAs already issued have drained before the CTA exits
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(acc_done, 0u) && global_ns() - t0 < WAIT_NS) {}
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 5) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
    }
    if (tid == 0 && abort_flag) atomicExch(error_word, 1);
}

// ---------------------------------------------------------------------------------------------------
// Block plan: for every block of BQ consecutive rows of Phi, the sorted list of distinct columns.

__global__ void __launch_bounds__(256)
block_plan_kernel(int32_t N, int32_t R, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                  int32_t* __restrict__ plan_off, int32_t* __restrict__ plan_cnt, int32_t* __restrict__ plan_col,
                  int32_t* __restrict__ plan_total)
{
    extern __shared__ uint32_t bitmap[];        // one bit per column
    __shared__ int32_t warp_sums[8];
    __shared__ int32_t base_off;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t blk = blockIdx.x;
    const int32_t words = (R + 31) >> 5;
    for (int32_t x = tid; x < words; x += 256) bitmap[x] = 0u;
    __syncthreads();
    const int32_t r0 = blk * BQ, r1 = min(N, r0 + BQ);
    for (int32_t p = rowptr[r0] + tid; p < rowptr[r1]; p += 256) {
        const int32_t c = col[p];
        atomicOr(&bitmap[c >> 5], 1u << (c & 31));
    }
    __syncthreads();
    // each thread owns a contiguous range of words so that the output stays sorted
    const int32_t per = (words + 255) / 256;
    const int32_t w0 = min(words, tid * per), w1 = min(words, w0 + per);
    int32_t mine = 0;
    for (int32_t x = w0; x < w1; ++x) mine += __popc(bitmap[x]);
    int32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    int32_t before = inc - mine;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    if (tid == 255) {
        const int32_t total = before + mine;
        base_off = atomicAdd(plan_total, total);
        plan_off[blk] = base_off;
        plan_cnt[blk] = total;
    }
    __syncthreads();
    int32_t o = base_off + before;
    for (int32_t x = w0; x < w1; ++x) {
        uint32_t bits = bitmap[x];
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            plan_col[o++] = (x << 5) + b;
        }
    }
}

}  // namespace

int grf_build_block_plan(grf_ctx* ctx, grf_features* feat)
{
    grf_csr_dev& phi = feat->phi;
    feat->plan_ready = false;
    const int32_t N = phi.rows, R = phi.cols;
    const size_t bitmap_bytes = (size_t)((R + 31) / 32) * 4;
    if (bitmap_bytes > 200 * 1024 || phi.nnz <= 0) return GRF_OK;   // no plan: the ALU kernel serves this object
    const int32_t nblocks = grf_ceil_div(N, BQ);
    GRF_TRY(grf_buf_reserve(&feat->plan_off, sizeof(int32_t) * (size_t)nblocks));
    GRF_TRY(grf_buf_reserve(&feat->plan_cnt, sizeof(int32_t) * (size_t)nblocks));
    GRF_TRY(grf_buf_reserve(&feat->plan_col, phi.col.bytes));       // at most nnz entries in total
    GRF_TRY(grf_buf_reserve(&feat->plan_total, sizeof(int32_t)));
    GRF_CUDA_TRY(cudaMemsetAsync(feat->plan_total.ptr, 0, sizeof(int32_t), ctx->stream));
    GRF_CUDA_TRY(cudaFuncSetAttribute(block_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bitmap_bytes));
    {
        grf_launch_scope scope(ctx, 3);
        block_plan_kernel<<<nblocks, 256, bitmap_bytes, ctx->stream>>>(
            N, R, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr, (int32_t*)feat->plan_off.ptr,
            (int32_t*)feat->plan_cnt.ptr, (int32_t*)feat->plan_col.ptr, (int32_t*)feat->plan_total.ptr);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    feat->plan_blocks = nblocks;
    feat->plan_ready = true;
    return GRF_OK;
}

template <int M, int D>
static int launch_tc(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N,
                     const void* phiQ, const void* S, const float* z, void* out, float* den_out)
{
    using Sh = TcShape<M, D>;
    const grf_csr_dev& phi = feat->phi;
    GRF_CUDA_TRY(cudaFuncSetAttribute(gather_contract_tc_kernel<M, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)Sh::SMEM));
    const dim3 grid(feat->plan_blocks, G);
    {
        grf_launch_scope scope(ctx, 5);
        gather_contract_tc_kernel<M, D><<<grid, TC_THREADS, Sh::SMEM, ctx->stream>>>(
            N, phi.cols, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr, (const float*)phi.val.ptr,
            (const int32_t*)feat->plan_off.ptr, (const int32_t*)feat->plan_cnt.ptr, (const int32_t*)feat->plan_col.ptr,
            (const __nv_bfloat16*)phiQ, (const __nv_bfloat16*)S, z, (__nv_bfloat16*)out, den_out, ctx->error_word);
    }
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

// Returns GRF_OK after launching, or 1 when this shape/object has no tensor-core path (caller falls back).
int grf_gather_contract_tc(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                           const void* phiQ, const void* S, const float* z, void* out, float* den_out)
{
    if (!feat->plan_ready || G > 65535) return 1;
#define GRF_TC_CASE(MM, DD) \
    if (m == MM && d == DD) return launch_tc<MM, DD>(ctx, feat, G, N, phiQ, S, z, out, den_out);
    GRF_TC_CASE(16, 16) GRF_TC_CASE(16, 32) GRF_TC_CASE(16, 64) GRF_TC_CASE(16, 128)
    GRF_TC_CASE(32, 16) GRF_TC_CASE(32, 32) GRF_TC_CASE(32, 64) GRF_TC_CASE(32, 128)
    GRF_TC_CASE(64, 16) GRF_TC_CASE(64, 32) GRF_TC_CASE(64, 64) GRF_TC_CASE(64, 128)
    GRF_TC_CASE(128, 16) GRF_TC_CASE(128, 32) GRF_TC_CASE(128, 64) GRF_TC_CASE(128, 128)
#undef GRF_TC_CASE
    return 1;
}
