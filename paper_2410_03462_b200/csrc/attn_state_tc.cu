// Per-node states on the 5th-generation tensor cores (Alg. 1 step 5, Eq. 12), bf16 storage, d <= 64:
//     S_l^T [d x m] = sum_j v_j (Psi_jl phi(k_j))^T,     z_l [m] = sum_j 1 * (Psi_jl phi(k_j))
// For one node l the sum over its c_l keys j is the K dimension of a small matrix product with
//     A [128 x c_l] : rows 0..d-1 = the gathered value rows v_j (column j), row d = all ones, other rows zero,
//     B [c_l x m]   : the gathered key features phi(k_j) scaled by Psi_jl,
// so rows 0..d-1 of the accumulator are S_l^T and row d is z_l: the denominators' ingredient comes out of
// the same instructions.  M = 128 costs the tensor pipe no more time than M = 64 at these widths.
//
// A CTA walks a range of nodes of one problem.  Keys are processed in items of up to 64 (four K = 16 steps):
//   producers (4 warps)  gather v_j and Psi_jl * phi(k_j) into shared memory in the unswizzled MN-major
//                        operand layout (16-byte pieces of a row go to 8x16-byte core matrices),
//   one warp             issues the tcgen05.mma instructions, accumulating a node in tensor memory,
//   epilogue (4 warps)   read the accumulator (two buffers, so the next node overlaps), round to bf16 and
//                        write the node's record: the tile in the gather kernel's operand layout, then z_l.
// The summation order over j is fixed by the instruction order (ascending j), so results are reproducible.
// All mbarrier waits are bounded; a wait that gives up raises the context's error word.
#include "grf_internal.cuh"

namespace {

constexpr long long WAIT_CYCLES = 4000000000ll;
constexpr int ITEM_KEYS = 64;        // keys per item = 4 K-steps of 16
constexpr int NODES_PER_CTA = 64;
constexpr int ST_THREADS = 288;      // warps 0-3 epilogue, warp 4 MMA issuer, warps 5-8 producers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_CYCLES) { *abort_flag = 1; return false; }
        }
    }
}

// Unswizzled MN-major operand: 8 (K) x 16-byte core matrices; lbo = bytes between K blocks of 8,
// sbo = bytes between blocks of 8 along M/N.
__device__ __forceinline__ uint64_t operand_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(sbo_bytes >> 4) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    return d;
}
// bf16 x bf16 -> fp32, both operands MN-major, M = 128, N = n
__host__ __device__ constexpr uint32_t instr_desc_mn(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
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

template <int M, int D> struct StShape {
    static constexpr int A_LBO = 16 * 128;                    // 16 blocks of 8 rows (M = 128), 128 bytes each
    static constexpr int A_KSTEP = 2 * A_LBO;                 // one K = 16 step of A
    static constexpr int A_BYTES = (ITEM_KEYS / 16) * A_KSTEP;
    static constexpr int B_LBO = (M / 8) * 128;
    static constexpr int B_KSTEP = 2 * B_LBO;
    static constexpr int B_BYTES = (ITEM_KEYS / 16) * B_KSTEP;
    static constexpr int STAGE = A_BYTES + B_BYTES;
    static constexpr int NS = (100 * 1024 / STAGE) >= 4 ? 4 : ((100 * 1024 / STAGE) >= 3 ? 3 : 2);
    static constexpr int ACC_COLS = M < 32 ? 32 : M;          // columns of one accumulator buffer
    static constexpr int TMEM_COLS = 2 * ACC_COLS < 32 ? 32 : 2 * ACC_COLS;
    static constexpr size_t SMEM = (size_t)NS * STAGE + 1024;
};

template <int M, int D>
__global__ void __launch_bounds__(ST_THREADS)
build_states_tc_kernel(int32_t R, int32_t N, const int32_t* __restrict__ t_rowptr, const int32_t* __restrict__ t_col,
                       const float* __restrict__ t_val, const __nv_bfloat16* __restrict__ phiK,
                       const __nv_bfloat16* __restrict__ V, unsigned char* __restrict__ records,
                       int* __restrict__ error_word)
{
    using Sh = StShape<M, D>;
    constexpr int NS = Sh::NS;
    static_assert(D <= 64 && D % 8 == 0 && M % 16 == 0 && M <= 128, "shape not covered by this kernel");
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) unsigned long long bars[2 * NS + 4];   // full, empty per stage; acc_full[2], acc_free[2]
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t g = blockIdx.y;
    const int32_t l0 = blockIdx.x * NODES_PER_CTA, l1 = min(R, l0 + NODES_PER_CTA);
    const uint32_t stage_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* stage_generic = smem_dyn + (stage_base - smem_u32(smem_dyn));
    const uint32_t bar_base = smem_u32(bars);
    auto full = [&](int s) { return bar_base + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar_base + 8u * (uint32_t)(NS + s); };
    auto acc_full = [&](int b) { return bar_base + 8u * (uint32_t)(2 * NS + b); };
    auto acc_free = [&](int b) { return bar_base + 8u * (uint32_t)(2 * NS + 2 + b); };

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full(s), 4); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_free(b), 4); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // constant part of every A buffer: zeros, and ones in row D (the row that sums Psi_jl phi(k_j) into z_l)
    for (int x = tid; x < NS * Sh::A_BYTES / 16; x += ST_THREADS) {
        const int s = x / (Sh::A_BYTES / 16), y = x % (Sh::A_BYTES / 16);
        *reinterpret_cast<uint4*>(stage_generic + (size_t)s * Sh::STAGE + (size_t)y * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();
    for (int x = tid; x < NS * ITEM_KEYS; x += ST_THREADS) {
        const int s = x / ITEM_KEYS, jj = x % ITEM_KEYS;
        // key jj of the item: K step jj / 16, K block (jj % 16) / 8, row jj % 8 of the core matrix; M block D / 8
        unsigned char* p = stage_generic + (size_t)s * Sh::STAGE + (size_t)(jj / 16) * Sh::A_KSTEP +
                           (size_t)((jj % 16) / 8) * Sh::A_LBO + (size_t)(D / 8) * 128 + (size_t)(jj % 8) * 16;
        *reinterpret_cast<unsigned short*>(p) = 0x3F80u;   // bf16 1.0 at row D (element 0 of the block)
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    const __nv_bfloat16* Kg = phiK + (size_t)g * N * M;
    const __nv_bfloat16* Vg = V + (size_t)g * N * D;

    if (warp >= 5) {
        // ------------------------------------------------------------ producers
        // Software pipeline over items: while item q is written to shared memory, the rows of item q+1 and
        // the (key, Psi) pairs of item q+2 are already on their way from L2.
        const int ptid = tid - 160;            // 0..127: key row jj = ptid / 2, half h = ptid % 2 of its pieces
        const int jj = ptid >> 1, h = ptid & 1;
        const uint32_t a_row = (uint32_t)(jj / 16) * Sh::A_KSTEP + (uint32_t)((jj % 16) / 8) * Sh::A_LBO + (uint32_t)(jj % 8) * 16;
        const uint32_t b_row = (uint32_t)(jj / 16) * Sh::B_KSTEP + (uint32_t)((jj % 16) / 8) * Sh::B_LBO + (uint32_t)(jj % 8) * 16;
        constexpr int NV = (D / 8 + 1) / 2, NK = (M / 8 + 1) / 2;

        struct Walk {          // position in the CTA's item sequence
            int32_t l, it, beg, c;
            __device__ __forceinline__ void load(const int32_t* rp, int32_t lend) {
                if (l < lend) { beg = __ldg(rp + l); c = __ldg(rp + l + 1) - beg; } else { beg = 0; c = 0; }
            }
            __device__ __forceinline__ void advance(const int32_t* rp, int32_t lend) {
                const int32_t nitems = c > 0 ? (c + ITEM_KEYS - 1) / ITEM_KEYS : 1;
                if (++it >= nitems) { ++l; it = 0; load(rp, lend); }
            }
            __device__ __forceinline__ int32_t keys() const { return min(ITEM_KEYS, c - it * ITEM_KEYS); }
        };
        struct Idx { int32_t j; float psi; bool real; };
        auto fetch_idx = [&](const Walk& w) {
            Idx x; x.j = 0; x.psi = 0.0f;
            x.real = w.l < l1 && jj < w.keys();
            if (x.real) { x.j = __ldg(t_col + w.beg + w.it * ITEM_KEYS + jj); x.psi = __ldg(t_val + w.beg + w.it * ITEM_KEYS + jj); }
            return x;
        };
        struct Rows { uint4 v[NV], k[NK]; };
        auto fetch_rows = [&](const Idx& x) {
            Rows r;
#pragma unroll
            for (int y = 0; y < NV; ++y) r.v[y] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int y = 0; y < NK; ++y) r.k[y] = make_uint4(0u, 0u, 0u, 0u);
            if (x.real) {
#pragma unroll
                for (int y = 0; y < NV; ++y)
                    if (h + 2 * y < D / 8) r.v[y] = __ldg(reinterpret_cast<const uint4*>(Vg + (size_t)x.j * D) + h + 2 * y);
#pragma unroll
                for (int y = 0; y < NK; ++y)
                    if (h + 2 * y < M / 8) r.k[y] = __ldg(reinterpret_cast<const uint4*>(Kg + (size_t)x.j * M) + h + 2 * y);
            }
            return r;
        };

        Walk w0; w0.l = l0; w0.it = 0; w0.load(t_rowptr, l1);
        Walk w2 = w0;
        Idx idx_cur = fetch_idx(w2);
        w2.advance(t_rowptr, l1);
        Idx idx_nxt = fetch_idx(w2);
        w2.advance(t_rowptr, l1);
        Rows rows_cur = fetch_rows(idx_cur);
        int32_t q = 0;
        bool ok = true;
        while (w0.l < l1) {
            const Rows rows_nxt = fetch_rows(idx_nxt);        // item q+1
            const Idx idx_nxt2 = fetch_idx(w2);               // item q+2
            w2.advance(t_rowptr, l1);
            const int s = q % NS;
            const int32_t n = w0.keys();
            const int32_t rows = n > 0 ? ((n + 15) & ~15) : 16;         // rows the MMAs will read
            if (!mbar_wait(empty(s), ((uint32_t)(q / NS) & 1u) ^ 1u, &abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (jj < rows) {
                unsigned char* a_dst = stage_generic + (size_t)s * Sh::STAGE + a_row;
                unsigned char* b_dst = stage_generic + (size_t)s * Sh::STAGE + Sh::A_BYTES + b_row;
#pragma unroll
                for (int y = 0; y < NV; ++y)
                    if (h + 2 * y < D / 8) *reinterpret_cast<uint4*>(a_dst + (size_t)(h + 2 * y) * 128) = rows_cur.v[y];
#pragma unroll
                for (int y = 0; y < NK; ++y)
                    if (h + 2 * y < M / 8) {
                        const uint32_t w[4] = {rows_cur.k[y].x, rows_cur.k[y].y, rows_cur.k[y].z, rows_cur.k[y].w};
                        uint32_t r[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float lo = idx_cur.psi * __uint_as_float(w[e] << 16);
                            const float hi = idx_cur.psi * __uint_as_float(w[e] & 0xffff0000u);
                            __nv_bfloat162 t2 = __floats2bfloat162_rn(lo, hi);
                            r[e] = *reinterpret_cast<uint32_t*>(&t2);
                        }
                        *reinterpret_cast<uint4*>(b_dst + (size_t)(h + 2 * y) * 128) = make_uint4(r[0], r[1], r[2], r[3]);
                    }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(full(s));
            ++q;
            w0.advance(t_rowptr, l1);
            idx_cur = idx_nxt; idx_nxt = idx_nxt2; rows_cur = rows_nxt;
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = instr_desc_mn(M);
        int32_t q = 0, nn = 0;
        bool ok = true;
        for (int32_t l = l0; l < l1 && ok; ++l, ++nn) {
            const int32_t c = t_rowptr[l + 1] - t_rowptr[l];
            const int32_t nitems = c > 0 ? (c + ITEM_KEYS - 1) / ITEM_KEYS : 1;
            const int buf = nn & 1;
            // the accumulator buffer must have been read out by the epilogue of the node two back
            if (!mbar_wait(acc_free(buf), ((uint32_t)(nn >> 1) & 1u) ^ 1u, &abort_flag)) { ok = false; break; }
            const uint32_t acc = tmem_base + (uint32_t)(buf * Sh::ACC_COLS);
            for (int32_t it = 0; it < nitems; ++it, ++q) {
                const int s = q % NS;
                const int32_t n = min(ITEM_KEYS, c - it * ITEM_KEYS);
                const int32_t ksteps = n > 0 ? (n + 15) / 16 : 1;
                if (!mbar_wait(full(s), (uint32_t)(q / NS) & 1u, &abort_flag)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (lane == 0) {
                    const uint32_t a_op = stage_base + (uint32_t)s * Sh::STAGE;
                    const uint32_t b_op = a_op + Sh::A_BYTES;
                    for (int32_t ks = 0; ks < ksteps; ++ks) {
                        const uint64_t ad = operand_desc(a_op + (uint32_t)ks * Sh::A_KSTEP, Sh::A_LBO, 128);
                        const uint64_t bd = operand_desc(b_op + (uint32_t)ks * Sh::B_KSTEP, Sh::B_LBO, 128);
                        mma_bf16_ss(acc, ad, bd, idesc, (it > 0 || ks > 0) ? 1u : 0u);
                    }
                    mma_commit(empty(s));
                    if (it == nitems - 1) mma_commit(acc_full(buf));
                }
                __syncwarp();
            }
        }
        if (!ok) {
            // aborted: let the MMAs already issued drain (bounded) before tensor memory is released
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000ll) {}
        }
    } else {
        // ------------------------------------------------------------ epilogue: accumulator -> record
        constexpr size_t REC = grf_record_bytes<__nv_bfloat16>(M, D);
        const int row = warp * 32 + lane;                   // accumulator row = TMEM lane
        const bool warp_has_rows = warp * 32 <= D;          // S rows 0..D-1 and the z row D
        int32_t nn = 0;
        bool ok = true;
        for (int32_t l = l0; l < l1; ++l, ++nn) {
            const int buf = nn & 1;
            if (ok && !mbar_wait(acc_full(buf), (uint32_t)(nn >> 1) & 1u, &abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (warp_has_rows) {
                unsigned char* rec = records + ((size_t)g * R + l) * REC;
                __nv_bfloat16* tile = reinterpret_cast<__nv_bfloat16*>(rec);
                float* zl = reinterpret_cast<float*>(rec + (size_t)M * D * 2);
                const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * Sh::ACC_COLS);
#pragma unroll
                for (int c0 = 0; c0 < M; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)c0, r);
                    if (row < D) {
                        // columns c0..c0+15 of row b = feature rows a of column b: two 16-byte chunks of the tile
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(r[8 * half + 2 * e]),
                                                                          __uint_as_float(r[8 * half + 2 * e + 1]));
                                w[e] = *reinterpret_cast<uint32_t*>(&t2);
                            }
                            *reinterpret_cast<uint4*>(tile + grf_tile_index<__nv_bfloat16>(c0 + 8 * half, row, D)) =
                                make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    } else if (row == D) {
#pragma unroll
                        for (int e = 0; e < 16; e += 4)
                            *reinterpret_cast<float4*>(zl + c0 + e) = make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]),
                                                                                  __uint_as_float(r[e + 2]), __uint_as_float(r[e + 3]));
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_free(buf));
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
    }
    if (tid == 0 && abort_flag) atomicExch(error_word, 1);
}

template <int M, int D>
int launch_state_tc(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, const void* phiK, const void* V,
                    void* records)
{
    using Sh = StShape<M, D>;
    GRF_CUDA_TRY(cudaFuncSetAttribute(build_states_tc_kernel<M, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Sh::SMEM));
    const dim3 grid(grf_ceil_div(psit.rows, NODES_PER_CTA), G);
    {
        grf_launch_scope scope(ctx, 4);
        build_states_tc_kernel<M, D><<<grid, ST_THREADS, Sh::SMEM, ctx->stream>>>(
            psit.rows, N, (const int32_t*)psit.rowptr.ptr, (const int32_t*)psit.col.ptr, (const float*)psit.val.ptr,
            (const __nv_bfloat16*)phiK, (const __nv_bfloat16*)V, (unsigned char*)records, ctx->error_word);
    }
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

}  // namespace

// Returns GRF_OK after launching, or 1 when this shape has no tensor-core path (the caller falls back).
int grf_build_states_tc(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, int32_t m, int32_t d,
                        const void* phiK, const void* V, void* records)
{
    if (G > 65535) return 1;
#define GRF_ST_CASE(MM, DD) \
    if (m == MM && d == DD) return launch_state_tc<MM, DD>(ctx, psit, G, N, phiK, V, records);
    GRF_ST_CASE(16, 16) GRF_ST_CASE(16, 32) GRF_ST_CASE(16, 64)
    GRF_ST_CASE(32, 16) GRF_ST_CASE(32, 32) GRF_ST_CASE(32, 64)
    GRF_ST_CASE(64, 16) GRF_ST_CASE(64, 32) GRF_ST_CASE(64, 64)
    GRF_ST_CASE(128, 16) GRF_ST_CASE(128, 32) GRF_ST_CASE(128, 64)
#undef GRF_ST_CASE
    return 1;
}
