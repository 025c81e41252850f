// Per-node states on the 5th-generation tensor cores (Alg. 1 step 5, Eq. 12), bf16 storage, d <= 64:
//     S_l^T [d x m] = sum_j v_j (Psi_jl phi(k_j))^T,     z_l [m] = sum_j 1 * (Psi_jl phi(k_j))
// For one node l the sum over its c_l keys j is the K dimension of a small matrix product with
//     A [128 x c_l] : rows 0..d-1 = the gathered value rows v_j (column j), row d = all ones, other rows zero,
//     B [c_l x m]   : the gathered key features phi(k_j) scaled by Psi_jl,
// so rows 0..d-1 of the accumulator are S_l^T and row d is z_l: the denominators' ingredient comes out of
// the same instructions.  M = 128 costs the tensor pipe no more time than M = 64 at these widths.
//
// A CTA walks a range of nodes of one problem.  Keys are processed in items of up to 64 (four K = 16 steps):
//   producers (4 warps)  each warp owns one shared-memory stage and every fourth item: it gathers v_j and
//                        phi(k_j) into the stage in the tensor cores' MN-major operand layout and scales the
//                        phi(k_j) rows by Psi_jl in place.  Two kernels differ in how the rows travel:
//                        asynchronous 16-byte copies into the unswizzled layout (any d <= 64), or, for d = 64,
//                        the tensor-map copy engine gathering whole rows into the swizzled layout,
//   one warp             issues the tcgen05.mma instructions, accumulating a node in tensor memory,
//   epilogue (4 warps)   read the accumulator (two buffers, so the next node overlaps), round to bf16 and
//                        write the node's record: the tile in the gather kernel's operand layout, then z_l.
// The summation order over j is fixed by the instruction order (ascending j), so results are reproducible.
// All mbarrier waits are bounded; a wait that gives up raises the context's error word.
#include "tc_common.cuh"

namespace {

constexpr int ITEM_KEYS = 64;        // keys per item = 4 K-steps of 16
constexpr int NODES_PER_CTA = 64;
constexpr int ST_THREADS = 288;      // warps 0-3 epilogue, warp 4 MMA issuer, warps 5-8 producers

using namespace grf_tc;

template <int M, int D> struct StShape {
    // Blocks of 8 along M/N sit 144, 160 or 192 bytes apart, not 128: the eight lanes of a quarter warp copy
    // 16-byte pieces of 1, 2 or 4 neighbouring keys (rows 8, 4 or 2 pieces long), and with these strides their
    // destinations fall into eight different bank groups.
    static constexpr int pad_stride(int pieces) { return pieces >= 8 ? 144 : (pieces == 4 ? 160 : 192); }
    static constexpr int A_SBO = pad_stride(D / 8);
    static constexpr int B_SBO = pad_stride(M / 8);
    static constexpr int A_LBO = 16 * A_SBO;                  // 16 blocks of 8 rows (M = 128)
    static constexpr int A_KSTEP = 2 * A_LBO;                 // one K = 16 step of A
    static constexpr int A_BYTES = (ITEM_KEYS / 16) * A_KSTEP;
    static constexpr int B_LBO = (M / 8) * B_SBO;
    static constexpr int B_KSTEP = 2 * B_LBO;
    static constexpr int B_BYTES = (ITEM_KEYS / 16) * B_KSTEP;
    static constexpr int STAGE = A_BYTES + B_BYTES;
    static constexpr int NS = (100 * 1024 / STAGE) >= 4 ? 4 : ((100 * 1024 / STAGE) >= 3 ? 3 : 2);
    static constexpr int ACC_COLS = M < 32 ? 32 : M;          // columns of one accumulator buffer
    static constexpr int TMEM_COLS = 2 * ACC_COLS < 32 ? 32 : 2 * ACC_COLS;
    static constexpr size_t SMEM = (size_t)NS * STAGE + 1024;
};

constexpr long long DRAIN_CYCLES = 20000000ll;   // after an abort: how long a warp waits for its own work in flight

// MMA issuer of both kernels: walks the CTA's nodes in order, item by item; `descs(s, ks, ad, bd)` gives the two
// operand descriptors of K step ks of stage s.  Barriers are addressed as base + 8 * index.
template <int M, int NS, int ACC_COLS, class Descs>
__device__ __forceinline__ void state_mma_issuer(int32_t nnodes, const int32_t* node_beg, uint32_t full0, uint32_t empty0,
                                                 uint32_t acc_full0, uint32_t acc_free0, uint32_t drain_bar,
                                                 uint32_t tmem_base, volatile int* abort_flag, Descs descs)
{
    constexpr uint32_t idesc = instr_desc(M, true, true);
    int32_t q = 0;
    bool ok = true;
    for (int32_t nn = 0; nn < nnodes && ok; ++nn) {
        const int32_t c = node_beg[nn + 1] - node_beg[nn];
        const int32_t nitems = c > 0 ? (c + ITEM_KEYS - 1) / ITEM_KEYS : 1;
        const int buf = nn & 1;
        // the accumulator buffer must have been read out by the epilogue of the node two back
        if (!__all_sync(0xffffffffu, mbar_wait(acc_free0 + 8u * buf, ((uint32_t)(nn >> 1) & 1u) ^ 1u, abort_flag))) { ok = false; break; }
        const uint32_t acc = tmem_base + (uint32_t)(buf * ACC_COLS);
        for (int32_t it = 0; it < nitems; ++it, ++q) {
            const int s = q % NS;
            const int32_t n = min(ITEM_KEYS, c - it * ITEM_KEYS);
            const int32_t ksteps = n > 0 ? (n + 15) / 16 : 1;
            if (!__all_sync(0xffffffffu, mbar_wait(full0 + 8u * s, (uint32_t)(q / NS) & 1u, abort_flag))) { ok = false; break; }
            fence_after_sync();
            for (int32_t ks = 0; ks < ksteps; ++ks) {
                uint64_t ad, bd;
                descs(s, ks, ad, bd);
                mma_bf16_ss(acc, ad, bd, idesc, (it > 0 || ks > 0) ? 1u : 0u);
            }
            mma_commit(empty0 + 8u * s);
            if (it == nitems - 1) mma_commit(acc_full0 + 8u * buf);
        }
    }
    if (!ok) {
        // aborted: the products already issued must have drained before tensor memory is released
        mma_commit(drain_bar);
        mbar_drain(drain_bar, 0u, DRAIN_CYCLES);
    }
}

// Epilogue of both kernels (warps 0-3): accumulator rows -> the node's record (tile in the gather kernel's operand
// layout, z_l in fp32 and once more in bf16).
template <int M, int D, int ACC_COLS>
__device__ __forceinline__ void state_epilogue(int warp, int lane, int32_t g, int32_t R, int32_t l0, int32_t l1,
                                               uint32_t acc_full0, uint32_t acc_free0, uint32_t tmem_base,
                                               volatile int* abort_flag, unsigned char* __restrict__ records)
{
    constexpr size_t REC = grf_record_bytes<__nv_bfloat16>(M, D);
    const int row = warp * 32 + lane;                   // accumulator row = TMEM lane
    const bool warp_has_rows = warp * 32 <= D;          // S rows 0..D-1 and the z row D
    int32_t nn = 0;
    bool ok = true;
    for (int32_t l = l0; l < l1; ++l, ++nn) {
        const int buf = nn & 1;
        if (ok && !mbar_wait(acc_full0 + 8u * buf, (uint32_t)(nn >> 1) & 1u, abort_flag)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        fence_after_sync();
        if (warp_has_rows) {
            unsigned char* rec = records + ((size_t)g * R + l) * REC;
            __nv_bfloat16* tile = reinterpret_cast<__nv_bfloat16*>(rec);
            float* zl = reinterpret_cast<float*>(rec + (size_t)M * D * 2);
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * ACC_COLS);
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
                    // and once more in bf16, for the denominators kernel
                    uint32_t zw[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                        zw[e] = *reinterpret_cast<uint32_t*>(&t2);
                    }
                    uint4* zb = reinterpret_cast<uint4*>(rec + (size_t)M * D * 2 + (size_t)M * 4 + (size_t)c0 * 2);
                    zb[0] = make_uint4(zw[0], zw[1], zw[2], zw[3]);
                    zb[1] = make_uint4(zw[4], zw[5], zw[6], zw[7]);
                }
            }
        }
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_free0 + 8u * buf);
    }
}

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
    __shared__ __align__(8) unsigned long long bars[2 * NS + 5];   // full, empty per stage; acc_full[2], acc_free[2]; drain
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int32_t node_beg[NODES_PER_CTA + 1];   // row pointers of the CTA's nodes

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
    const uint32_t drain_bar = bar_base + 8u * (uint32_t)(2 * NS + 4);   // used only after an abort

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_free(b), 4); }
        mbar_init(drain_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid <= NODES_PER_CTA) node_beg[tid] = t_rowptr[min(l0 + tid, R)];
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
                           (size_t)((jj % 16) / 8) * Sh::A_LBO + (size_t)(D / 8) * Sh::A_SBO + (size_t)(jj % 8) * 16;
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
        // Producer warp w owns stage w and the items q = w, w + NW, ...: the warps work on different items, so the
        // waits of one item (stage free, copies landed, proxy fence) overlap the copies of the others.
        // A warp copy instruction (16 bytes per lane, asynchronous, straight into the operand layout) covers
        // whole rows: consecutive lanes take consecutive pieces of one key's row.  The lane that copied a piece
        // of phi(k_j) scales it by Psi_jl afterwards.  Keys and Psi values of the warp's next item are read
        // while the current one is in flight.
        constexpr int NW = NS;                              // one producer warp per stage (NS <= 4)
        static_assert(NS <= 4, "more stages than producer warps");
        const int pw = warp - 5;
        constexpr int CV = D / 8, CK = M / 8;             // 16-byte pieces per value row / per key-feature row
        constexpr int KPV = 32 / CV, KPK = CK >= 32 ? 1 : 32 / CK;   // keys per copy instruction
        constexpr int NIV = ITEM_KEYS / KPV, NIK = ITEM_KEYS / KPK;  // copy instructions per item
        static_assert(CV <= 8 && CK <= 16, "rows longer than a warp's copy");
        auto key_offset = [](int key, int kstep_bytes, int lbo) {
            return (uint32_t)(key / 16) * (uint32_t)kstep_bytes + (uint32_t)((key % 16) / 8) * (uint32_t)lbo +
                   (uint32_t)(key % 8) * 16u;
        };
        // destination of this lane's piece in instruction 0; instruction y adds key_offset(KP * y) (the
        // offsets add up because KP divides 16)
        const uint32_t a_lane = key_offset(lane / CV, Sh::A_KSTEP, Sh::A_LBO) + (uint32_t)(lane % CV) * Sh::A_SBO;
        const uint32_t b_lane = key_offset(lane / CK, Sh::B_KSTEP, Sh::B_LBO) + (uint32_t)(lane % CK) * Sh::B_SBO + Sh::A_BYTES;
        const int32_t nn = l1 - l0;
        if (pw < NW) {
            const int s = pw;
            const uint32_t st = stage_base + (uint32_t)s * Sh::STAGE;
            unsigned char* st_generic = stage_generic + (size_t)s * Sh::STAGE;
            // walker over the CTA's items
            int32_t wn = 0, wit = 0, wbeg = node_beg[0], wc = node_beg[1] - node_beg[0];
            auto advance = [&]() {
                const int32_t nitems = wc > 0 ? (wc + ITEM_KEYS - 1) / ITEM_KEYS : 1;
                if (++wit >= nitems) { ++wn; wit = 0; wbeg = node_beg[min(wn, nn)]; wc = node_beg[min(wn + 1, nn)] - wbeg; }
            };
            int32_t j0, j1, nkeys; float p0, p1;
            auto read_idx = [&](int32_t& nk, int32_t& ja, int32_t& jb, float& pa, float& pb) {
                ja = -1; jb = -1; pa = 0.0f; pb = 0.0f; nk = 0;
                if (wn < nn) {
                    nk = min(ITEM_KEYS, wc - wit * ITEM_KEYS);
                    const int32_t pos = wbeg + wit * ITEM_KEYS + lane;
                    if (lane < nk) { ja = __ldg(t_col + pos); pa = __ldg(t_val + pos); }
                    if (lane + 32 < nk) { jb = __ldg(t_col + pos + 32); pb = __ldg(t_val + pos + 32); }
                }
            };
            for (int k = 0; k < pw; ++k) advance();
            read_idx(nkeys, j0, j1, p0, p1);
            bool ok = true;
            for (uint32_t use = 0; wn < nn; ++use) {
                const int32_t rows = nkeys > 0 ? ((nkeys + 15) & ~15) : 16;     // rows the MMAs will read
                if (!mbar_wait(empty(s), (use & 1u) ^ 1u, &abort_flag)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
#pragma unroll
                for (int y = 0; y < NIV; ++y) {
                    if (KPV * y < rows) {
                        const int32_t j = __shfl_sync(0xffffffffu, y < NIV / 2 ? j0 : j1, (KPV * y + lane / CV) & 31);
                        const __nv_bfloat16* src = Vg + (size_t)max(j, 0) * D + (lane % CV) * 8;
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;"
                                     ::"r"(st + a_lane + key_offset(KPV * y, Sh::A_KSTEP, Sh::A_LBO)), "l"(src),
                                       "r"(j >= 0 ? 16u : 0u) : "memory");       // no such key: zero-filled
                    }
                }
#pragma unroll
                for (int y = 0; y < NIK; ++y) {
                    if (KPK * y < rows) {
                        const int32_t j = __shfl_sync(0xffffffffu, y < NIK / 2 ? j0 : j1, (KPK * y + lane / CK) & 31);
                        const __nv_bfloat16* src = Kg + (size_t)max(j, 0) * M + (lane % CK) * 8;
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;"
                                     ::"r"(st + b_lane + key_offset(KPK * y, Sh::B_KSTEP, Sh::B_LBO)), "l"(src),
                                       "r"(j >= 0 ? 16u : 0u) : "memory");
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                // the warp's next item: keys and Psi values on their way while this one lands
                for (int k = 0; k < NW; ++k) advance();
                int32_t nkeys_n, jn0, jn1; float pn0, pn1;
                read_idx(nkeys_n, jn0, jn1, pn0, pn1);
                asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
                for (int y = 0; y < NIK; ++y) {
                    if (KPK * y < rows) {
                        const float psi = __shfl_sync(0xffffffffu, y < NIK / 2 ? p0 : p1, (KPK * y + lane / CK) & 31);
                        const __nv_bfloat162 p2 = __float2bfloat162_rn(psi);
                        unsigned char* pc = st_generic + b_lane + key_offset(KPK * y, Sh::B_KSTEP, Sh::B_LBO);
                        uint4 w = *reinterpret_cast<uint4*>(pc);
                        __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&w);
#pragma unroll
                        for (int x = 0; x < 4; ++x) e[x] = __hmul2(e[x], p2);
                        *reinterpret_cast<uint4*>(pc) = w;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(full(s));
                nkeys = nkeys_n; j0 = jn0; j1 = jn1; p0 = pn0; p1 = pn1;
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------ MMA issuer
        state_mma_issuer<M, NS, Sh::ACC_COLS>(l1 - l0, node_beg, full(0), empty(0), acc_full(0), acc_free(0), drain_bar,
                                              tmem_base, &abort_flag,
                                              [&](int s, int32_t ks, uint64_t& ad, uint64_t& bd) {
            const uint32_t a_op = stage_base + (uint32_t)s * Sh::STAGE;
            ad = operand_desc(a_op + (uint32_t)ks * Sh::A_KSTEP, Sh::A_LBO, Sh::A_SBO);
            bd = operand_desc(a_op + Sh::A_BYTES + (uint32_t)ks * Sh::B_KSTEP, Sh::B_LBO, Sh::B_SBO);
        });
    } else {
        // ------------------------------------------------------------ epilogue: accumulator -> record
        state_epilogue<M, D, Sh::ACC_COLS>(warp, lane, g, R, l0, l1, acc_full(0), acc_free(0), tmem_base, &abort_flag, records);
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


// ---------------------------------------------------------------------------------------------------------
// d = 64: the same product with the rows gathered by the tensor-map copy engine (TMA, tile::gather4: four
// rows of a 2-D tensor per instruction, row indices given in registers), so the gather does not pass through
// the load/store units.  A gathered v_j row is 128 bytes: 64 rows stacked at a 128-byte pitch, written with
// the 128-byte swizzle, ARE the MN-major swizzled operand (8 keys x 128 bytes per swizzle atom).  The second
// atom along M (rows 64..127: the ones row that yields z_l, then zeros) is one constant 2 KB region shared by
// all stages and K steps, reached through the descriptor's leading-dimension offset.  The copy engine sustains about one
// four-row gather per 15 cycles per SM whatever the rows' length, so the shorter phi(k_j) rows do not go
// through it as well: they travel as asynchronous 16-byte copies through the load/store units (which would
// otherwise idle) into the padded unswizzled layout of the kernel above, and are scaled in place by Psi_jl.
template <int M> struct TmaShape {
    static constexpr int D = 64;
    static constexpr int A_BYTES = ITEM_KEYS * 128;             // gathered value rows of an item
    static constexpr int B_SBO = StShape<M, 64>::B_SBO;
    static constexpr int B_LBO = (M / 8) * B_SBO;
    static constexpr int B_KSTEP = 2 * B_LBO;
    static constexpr int B_BYTES = (ITEM_KEYS / 16) * B_KSTEP;
    static constexpr int STAGE = A_BYTES + B_BYTES;
    static constexpr int NS = 4;                                // one stage per producer warp
    static constexpr int ACC_COLS = M < 32 ? 32 : M;
    static constexpr int TMEM_COLS = 2 * ACC_COLS < 32 ? 32 : 2 * ACC_COLS;
    static constexpr int CONST_BYTES = 2048;                    // the constant second atom of A: one K step (16 keys)
    static constexpr size_t SMEM = (size_t)NS * STAGE + CONST_BYTES + 1024;
    static_assert(STAGE % 1024 == 0, "stages must keep the swizzle phase");
};

template <int M>
__global__ void __launch_bounds__(ST_THREADS)
build_states_tma_kernel(int32_t R, int32_t N, const int32_t* __restrict__ t_rowptr, const int32_t* __restrict__ t_col,
                        const float* __restrict__ t_val, const __nv_bfloat16* __restrict__ phiK,
                        const __grid_constant__ CUtensorMap map_v, unsigned char* __restrict__ records,
                        int* __restrict__ error_word)
{
    using Sh = TmaShape<M>;
    constexpr int NS = Sh::NS, D = Sh::D;
    extern __shared__ unsigned char smem_dyn[];
    __shared__ __align__(8) unsigned long long bars[3 * NS + 5];   // landed, full, empty per stage; acc_full[2], acc_free[2]; drain
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int32_t node_beg[NODES_PER_CTA + 1];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t g = blockIdx.y;
    const int32_t l0 = blockIdx.x * NODES_PER_CTA, l1 = min(R, l0 + NODES_PER_CTA);
    const uint32_t stage_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* stage_generic = smem_dyn + (stage_base - smem_u32(smem_dyn));
    const uint32_t const_base = stage_base + (uint32_t)NS * Sh::STAGE;     // the constant second atom of A
    const uint32_t bar_base = smem_u32(bars);
    auto landed = [&](int s) { return bar_base + 8u * (uint32_t)s; };
    auto full = [&](int s) { return bar_base + 8u * (uint32_t)(NS + s); };
    auto empty = [&](int s) { return bar_base + 8u * (uint32_t)(2 * NS + s); };
    auto acc_full = [&](int b) { return bar_base + 8u * (uint32_t)(3 * NS + b); };
    auto acc_free = [&](int b) { return bar_base + 8u * (uint32_t)(3 * NS + 2 + b); };
    const uint32_t drain_bar = bar_base + 8u * (uint32_t)(3 * NS + 4);   // used only after an abort

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(landed(s), 1); mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_free(b), 4); }
        mbar_init(drain_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid <= NODES_PER_CTA) node_beg[tid] = t_rowptr[min(l0 + tid, R)];
    // stages start as zeros (pad rows are multiplied before they are ever written); the constant atom is zero
    // except for bf16 1.0 in element 0 of logical piece 0 of every key row, which the swizzle puts at piece r % 8
    for (int x = tid; x < (NS * Sh::STAGE + Sh::CONST_BYTES) / 16; x += ST_THREADS)
        *reinterpret_cast<uint4*>(stage_generic + (size_t)x * 16) = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    for (int r = tid; r < 16; r += ST_THREADS)
        *reinterpret_cast<unsigned short*>(stage_generic + (size_t)NS * Sh::STAGE + (size_t)r * 128 + (size_t)(r % 8) * 16) = 0x3F80u;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    if (warp >= 5) {
        // ------------------------------------------------------------ producers: warp w owns stage w, items w, w+4, ...
        const int s = warp - 5;
        const int32_t nn = l1 - l0;
        const uint32_t st = stage_base + (uint32_t)s * Sh::STAGE;
        unsigned char* st_generic = stage_generic + (size_t)s * Sh::STAGE;
        constexpr int CK = M / 8;                         // 16-byte pieces of a phi(k_j) row
        constexpr int KPK = 32 / CK, NIK = ITEM_KEYS / KPK;   // keys per copy instruction, instructions per item
        const int y4 = lane & 15;                         // lanes 0-15 gather the value rows of keys 4*y4 .. 4*y4+3
        const int32_t row0 = g * N;
        auto key_offset = [](int key) {
            return (uint32_t)(key / 16) * (uint32_t)Sh::B_KSTEP + (uint32_t)((key % 16) / 8) * (uint32_t)Sh::B_LBO +
                   (uint32_t)(key % 8) * 16u;
        };
        // this lane's piece of phi(k_j) in copy instruction 0; instruction y adds key_offset(KPK * y)
        const uint32_t b_lane = Sh::A_BYTES + key_offset(lane / CK) + (uint32_t)(lane % CK) * Sh::B_SBO;
        const __nv_bfloat16* Kg = phiK + (size_t)g * N * M + (lane % CK) * 8;
        int32_t wn = 0, wit = 0, wbeg = node_beg[0], wc = node_beg[1] - node_beg[0];
        auto advance = [&]() {
            const int32_t nitems = wc > 0 ? (wc + ITEM_KEYS - 1) / ITEM_KEYS : 1;
            if (++wit >= nitems) { ++wn; wit = 0; wbeg = node_beg[min(wn, nn)]; wc = node_beg[min(wn + 1, nn)] - wbeg; }
        };
        struct Idx { int32_t nkeys, jlo, jhi; float p0, p1; };    // lane x holds key x (jlo) and key x + 32 (jhi)
        auto read_idx = [&]() {
            Idx x; x.nkeys = 0; x.p0 = 0.0f; x.p1 = 0.0f; x.jlo = -1; x.jhi = -1;
            if (wn < nn) {
                x.nkeys = min(ITEM_KEYS, wc - wit * ITEM_KEYS);
                const int32_t pos = wbeg + wit * ITEM_KEYS;
                if (lane < x.nkeys) { x.jlo = __ldg(t_col + pos + lane); x.p0 = __ldg(t_val + pos + lane); }
                if (lane + 32 < x.nkeys) { x.jhi = __ldg(t_col + pos + lane + 32); x.p1 = __ldg(t_val + pos + lane + 32); }
            }
            return x;
        };
        for (int k = 0; k < s; ++k) advance();
        Idx cur = read_idx();
        bool ok = true;
        for (uint32_t use = 0; wn < nn; ++use) {
            const int32_t rows = cur.nkeys > 0 ? ((cur.nkeys + 15) & ~15) : 16;     // rows the MMAs will read
            if (!mbar_wait(empty(s), (use & 1u) ^ 1u, &abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane == 0)
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                             ::"r"(landed(s)), "r"((uint32_t)rows * 128u) : "memory");
            __syncwarp();
            // lane y (< 16) gathers the value rows of keys 4y .. 4y+3; the keys come from the lanes that hold them;
            // beyond the item's keys its last key is repeated (the row meets a zero row of phi(k))
            int32_t r4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int32_t key = min(4 * y4 + e, max(cur.nkeys - 1, 0));
                const int32_t a = __shfl_sync(0xffffffffu, cur.jlo, key & 31), b = __shfl_sync(0xffffffffu, cur.jhi, key & 31);
                r4[e] = row0 + max(key < 32 ? a : b, 0);
            }
            if (lane < 16 && 4 * y4 < rows)
                tma_gather4(st + (uint32_t)y4 * 512u, &map_v, r4[0], r4[1], r4[2], r4[3], landed(s));
#pragma unroll
            for (int y = 0; y < NIK; ++y) {
                const int32_t j = __shfl_sync(0xffffffffu, y < NIK / 2 ? cur.jlo : cur.jhi, (KPK * y + lane / CK) & 31);
                if (KPK * y < rows)
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;"
                                 ::"r"(st + b_lane + key_offset(KPK * y)), "l"(Kg + (size_t)max(j, 0) * M),
                                   "r"(j >= 0 ? 16u : 0u) : "memory");       // no such key: zero-filled
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            // the warp's next item: keys and Psi values on their way while this one lands
            for (int k = 0; k < NS; ++k) advance();
            const Idx nxt = read_idx();
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            // Psi_jl * phi(k_j), in place: every lane scales the pieces it copied
            constexpr int BATCH = NIK < 8 ? NIK : 8;
#pragma unroll
            for (int y0 = 0; y0 < NIK; y0 += BATCH) {
                uint4 w[BATCH];
#pragma unroll
                for (int u = 0; u < BATCH; ++u)
                    w[u] = *reinterpret_cast<const uint4*>(st_generic + b_lane + key_offset(KPK * (y0 + u)));
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    const float psi = __shfl_sync(0xffffffffu, y0 + u < NIK / 2 ? cur.p0 : cur.p1, (KPK * (y0 + u) + lane / CK) & 31);
                    const __nv_bfloat162 p2 = __float2bfloat162_rn(psi);
                    __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&w[u]);
#pragma unroll
                    for (int x = 0; x < 4; ++x) e[x] = __hmul2(e[x], p2);
                }
#pragma unroll
                for (int u = 0; u < BATCH; ++u)
                    if (KPK * (y0 + u) < rows) *reinterpret_cast<uint4*>(st_generic + b_lane + key_offset(KPK * (y0 + u))) = w[u];
            }
            if (!mbar_wait(landed(s), use & 1u, &abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                // gave up with this item's gathers possibly still in flight: let them land (bounded) before the
                // CTA's shared memory is released
                mbar_drain(landed(s), use & 1u, DRAIN_CYCLES);
                break;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(full(s));
            cur = nxt;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else if (warp == 4) {
        // ------------------------------------------------------------ MMA issuer
        state_mma_issuer<M, NS, Sh::ACC_COLS>(l1 - l0, node_beg, full(0), empty(0), acc_full(0), acc_free(0), drain_bar,
                                              tmem_base, &abort_flag,
                                              [&](int s, int32_t ks, uint64_t& ad, uint64_t& bd) {
            // A: two atoms along M (gathered rows, then the constant atom), 8-key groups 1024 bytes apart
            // (every K step points its second atom at the same constant 2 KB)
            const uint32_t a_op = stage_base + (uint32_t)s * Sh::STAGE + (uint32_t)ks * 2048u;
            ad = swizzled_desc(a_op, const_base - a_op, 1024u, 2);
            bd = operand_desc(stage_base + (uint32_t)s * Sh::STAGE + Sh::A_BYTES + (uint32_t)ks * Sh::B_KSTEP, Sh::B_LBO, Sh::B_SBO);
        });
    } else {
        // ------------------------------------------------------------ epilogue: accumulator -> record
        state_epilogue<M, D, Sh::ACC_COLS>(warp, lane, g, R, l0, l1, acc_full(0), acc_free(0), tmem_base, &abort_flag, records);
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
    }
    if (tid == 0 && abort_flag) atomicExch(error_word, 1);
}

// 1 when the tensor maps cannot be made (the caller then takes the kernel above)
template <int M>
int launch_state_tma(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, const void* phiK, const void* V,
                     void* records)
{
    using Sh = TmaShape<M>;
    if ((int64_t)G * N > 0x7fffffffll) return 1;
    CUtensorMap map_v;
    if ((reinterpret_cast<uintptr_t>(phiK) & 15u) != 0 || !grf_make_row_gather_map(&map_v, V, (uint64_t)G * N, 64)) return 1;
    GRF_CUDA_TRY(cudaFuncSetAttribute(build_states_tma_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Sh::SMEM));
    const dim3 grid(grf_ceil_div(psit.rows, NODES_PER_CTA), G);
    {
        grf_launch_scope scope(ctx, 4);
        build_states_tma_kernel<M><<<grid, ST_THREADS, Sh::SMEM, ctx->stream>>>(
            psit.rows, N, (const int32_t*)psit.rowptr.ptr, (const int32_t*)psit.col.ptr, (const float*)psit.val.ptr,
            (const __nv_bfloat16*)phiK, map_v, (unsigned char*)records, ctx->error_word);
    }
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

}  // namespace

// Returns GRF_OK after launching, or 1 when this shape has no tensor-core path (the caller falls back).
int grf_build_states_tc(grf_ctx* ctx, const grf_csr_dev& psit, int32_t G, int32_t N, int32_t m, int32_t d,
                        const void* phiK, const void* V, void* records)
{
    if (G > 65535) return 1;
    if (d == 64 && (m == 16 || m == 32 || m == 64)) {
        const int rc = m == 16 ? launch_state_tma<16>(ctx, psit, G, N, phiK, V, records)
                     : m == 32 ? launch_state_tma<32>(ctx, psit, G, N, phiK, V, records)
                               : launch_state_tma<64>(ctx, psit, G, N, phiK, V, records);
        if (rc != 1) return rc;
    }
#define GRF_ST_CASE(MM, DD) \
    if (m == MM && d == DD) return launch_state_tc<MM, DD>(ctx, psit, G, N, phiK, V, records);
    GRF_ST_CASE(16, 16) GRF_ST_CASE(16, 32) GRF_ST_CASE(16, 64)
    GRF_ST_CASE(32, 16) GRF_ST_CASE(32, 32) GRF_ST_CASE(32, 64)
    GRF_ST_CASE(64, 16) GRF_ST_CASE(64, 32) GRF_ST_CASE(64, 64)
    GRF_ST_CASE(128, 16) GRF_ST_CASE(128, 32) GRF_ST_CASE(128, 64)
#undef GRF_ST_CASE
    return 1;
}
