// Gather-and-contract on the 5th-generation tensor cores (Alg. 1 step 5, Eq. 12), bf16 storage.
//
// A CTA owns a block of 128 consecutive queries of one problem g.  The block's rows of Phi touch a
// union U of nodes l (the "block plan", a sorted list built once per feature object).  For every l in U
//     D[128 x d] += A_l[128 x m] * S_l[m x d],      A_l[i, a] = Phi_il * phi(q_i)_a   (0 where Phi_il = 0)
// is m/16 tcgen05.mma instructions (M = 128, N = d, K = 16) accumulating in tensor memory: the sum over l
// of Eq. 12 becomes the K dimension of one long matrix product, evaluated in a fixed order.
//   - the state tile of node l (S_l in operand layout, the head of its record) arrives by one contiguous bulk
//     async copy into a ring of shared-memory slots, four tiles per landing barrier; the loader reads the node
//     indices one group ahead of the copies;
//   - A_l lives in tensor memory: each of the 128 "row" threads owns one query (= one TMEM lane), reads its
//     coefficients Phi_il from the plan's dense table and stores its scaled phi(q) (zeros for most rows) with
//     tcgen05.st, so the MMA reads only S_l from shared memory; three groups of A operands are in flight;
//   - one warp issues the MMAs: its loop is warp-uniform and an elected lane issues (the same instruction
//     issued from a single-lane branch costs about three times as much); one tcgen05.commit per group frees
//     both the A slots and the record slots of that group; the epilogue divides by the denominators (a
//     separate kernel, below) and writes the block's outputs;
//   - every mbarrier wait is bounded: a wait that outlasts its limit raises an error word and the CTA drains
//     its copies and MMAs, frees its tensor memory and exits.
// Nodes that no query of the block touches are never loaded; a tile is loaded once per block, not once
// per query, which is where the method's "constant multiplicative cost" is paid down.
#include "tc_common.cuh"

namespace {

constexpr int BQ = GRF_PLAN_BLOCK;  // queries per CTA = MMA M
using namespace grf_tc;

constexpr int pow2_at_least(int x) { return x <= 32 ? 32 : (x <= 64 ? 64 : (x <= 128 ? 128 : (x <= 256 ? 256 : 512))); }

template <int M, int D> struct TcShape {
    static constexpr int A_COLS = M / 2;                      // TMEM columns of one union entry's A operand
    static constexpr int GU = M <= 32 ? 4 : (M == 64 ? 2 : 1); // union entries per group (one commit per group)
    static constexpr int NA = 3;                              // A stages: groups written ahead of the one being multiplied
    static constexpr int TMEM_COLS = pow2_at_least(D + NA * GU * A_COLS);       // accumulator + A ring
    static constexpr int TILE_BYTES = M * D * 2;
    static constexpr int REC_BYTES = TILE_BYTES + M * 4 + M * 2;   // state tile, z (fp32), z (bf16)
    static constexpr int CHUNK_BYTES = GU * TILE_BYTES;        // only the tiles are copied to shared memory
    static constexpr int SMEM_BUDGET = TMEM_COLS <= 256 ? 104 * 1024 : 200 * 1024;   // two CTAs per SM, or one
    static constexpr int NBC_WANT = SMEM_BUDGET / CHUNK_BYTES;
    static constexpr int NBC = NBC_WANT > 8 ? 8 : (NBC_WANT < 2 ? 2 : NBC_WANT);     // record chunks in flight
    static constexpr size_t SMEM = (size_t)NBC * CHUNK_BYTES + 1024;                  // + alignment slack
};

// warps 0-3: row threads (A operand, epilogue); warp 4: record loader; warp 5: MMA issuer
constexpr int TC_THREADS = 192;

template <int M, int D>
__global__ void __launch_bounds__(TC_THREADS)
gather_contract_tc_kernel(int32_t G, int32_t nblocks, int32_t N, int32_t R, const int32_t* __restrict__ plan_off,
                          const int32_t* __restrict__ plan_cnt, const int32_t* __restrict__ plan_col,
                          const uint2* __restrict__ plan_coef,
                          const __nv_bfloat16* __restrict__ phiQ, const unsigned char* __restrict__ records,
                          __nv_bfloat16* __restrict__ out, const float* __restrict__ den_in, int* __restrict__ error_word)
{
    using Sh = TcShape<M, D>;
    constexpr int NA = Sh::NA, NBC = Sh::NBC, GU = Sh::GU, NREC = NBC * GU;
    extern __shared__ unsigned char smem_dyn[];
    // a_full per A stage; rec_full and done per record chunk (= per group of GU union entries); acc_done per issuer
    __shared__ __align__(8) unsigned long long bars[NA + NBC + NBC + 1];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Launch order.  The blocks' union sizes differ by up to a factor of three and the CTAs that start last
    // decide when the kernel ends, so the last quarter of the problems is taken block by block in order of
    // decreasing union size (all of these problems for a block together); the first three quarters keep the
    // order of the rows, in which neighbouring blocks run together and share their tiles in L2.
    int32_t blk, g;
    {
        const int32_t tail_g = G / 4, head_g = G - tail_g;
        const uint32_t idx = blockIdx.x;
        if (idx < (uint32_t)head_g * (uint32_t)nblocks) {
            g = (int32_t)(idx / (uint32_t)nblocks);
            blk = (int32_t)(idx % (uint32_t)nblocks);
        } else {
            const uint32_t j = idx - (uint32_t)head_g * (uint32_t)nblocks;
            g = head_g + (int32_t)(j % (uint32_t)tail_g);
            blk = plan_cnt[nblocks + (int32_t)(j / (uint32_t)tail_g)];
        }
    }
    const uint32_t b_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const unsigned char* b_generic = smem_dyn + (b_base - smem_u32(smem_dyn));
    const uint32_t bar_base = smem_u32(bars);
    auto a_full = [&](int s) { return bar_base + 8u * (uint32_t)s; };
    auto rec_full = [&](int s) { return bar_base + 8u * (uint32_t)(NA + s); };
    auto done = [&](int s) { return bar_base + 8u * (uint32_t)(NA + NBC + s); };
    const uint32_t acc_done = bar_base + 8u * (uint32_t)(NA + NBC + NBC);

    if (tid == 0) {
        for (int s = 0; s < NA; ++s) mbar_init(a_full(s), 4);
        for (int s = 0; s < NBC; ++s) mbar_init(rec_full(s), 1);
        for (int s = 0; s < NBC; ++s) mbar_init(done(s), 1);
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
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tmem_a = tmem_base + (uint32_t)D;   // A ring behind the accumulator

    const int32_t cnt = plan_cnt[blk];
    const int32_t ngroups = (cnt + GU - 1) / GU;
    const int32_t* ulist = plan_col + plan_off[blk];
    const unsigned char* recs = records + (size_t)g * R * Sh::REC_BYTES;

    if (warp < 4) {
        // ------------------------------------------------------------ row threads: A operand, denominators, epilogue
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
        // this row's coefficients Phi_il for the block's union entries, four entries (bf16) per 8-byte word,
        // read two words ahead of their use
        const uint2* tab = plan_coef + (size_t)(plan_off[blk] >> 2) * BQ + tid;
        const int32_t nquads = cnt >> 2;
        uint2 cur = make_uint2(0u, 0u);
        uint2 nxt1 = nquads > 0 ? __ldg(tab) : make_uint2(0u, 0u);
        uint2 nxt2 = nquads > 1 ? __ldg(tab + BQ) : make_uint2(0u, 0u);
        const float den = live ? den_in[(size_t)g * N + row] : 0.0f;
        bool ok = true;
        const uint32_t lane_field = (uint32_t)(warp * 32) << 16;
        for (int32_t gi = 0; gi < ngroups; ++gi) {
            const int32_t u0 = gi * GU;
            if ((u0 & 3) == 0) {
                const int32_t q = u0 >> 2;
                cur = nxt1; nxt1 = nxt2;
                nxt2 = q + 2 < nquads ? __ldg(tab + (size_t)(q + 2) * BQ) : make_uint2(0u, 0u);
            }
            const unsigned long long quad = ((unsigned long long)cur.y << 32) | cur.x;
            const int st = gi % NA;
            // the A slots of this stage are free once the group that used them NA groups ago has been multiplied
            if (gi >= NA && !mbar_wait(done((gi - NA) % NBC), (uint32_t)((gi - NA) / NBC) & 1u, &abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int j = 0; j < GU; ++j) {
                // A_l[row, :] = Phi_il * phi(q_row): zeros for most rows; products are taken in packed bf16
                const uint32_t cbits = (uint32_t)(quad >> (16 * ((u0 + j) & 3))) & 0xffffu;
                // (no branch on a zero coefficient: the product is then a signed zero, which adds nothing)
                const uint32_t cpair = cbits | (cbits << 16);
                const __nv_bfloat162 c2 = *reinterpret_cast<const __nv_bfloat162*>(&cpair);
                uint32_t w[M / 2];
#pragma unroll
                for (int e = 0; e < M / 2; ++e) {
                    const __nv_bfloat162 h = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&q2[e]), c2);
                    w[e] = *reinterpret_cast<const uint32_t*>(&h);
                }
                const uint32_t a_slot = tmem_a + lane_field + (uint32_t)((st * GU + j) * Sh::A_COLS);
                if constexpr (M >= 32) {
#pragma unroll
                    for (int c = 0; c < M / 32; ++c) {
                        uint32_t w16[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) w16[e] = w[16 * c + e];
                        tmem_st16(a_slot + (uint32_t)c * 16u, w16);
                    }
                } else {
                    uint32_t w8[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) w8[e] = w[e];
                    tmem_st8(a_slot, w8);
                }
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(a_full(st));
        }
        // epilogue: this thread's row of the accumulator is TMEM lane `tid`
        if (ok && ngroups > 0) ok = mbar_wait(acc_done, 0u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);   // the tensor-memory loads below are warp-wide
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const float inv = (den != 0.0f) ? 1.0f / den : 0.0f;
        __nv_bfloat16* orow = out + ((size_t)g * N + row) * D;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 16) {
            uint32_t r[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) r[e] = 0u;
            if (ok && ngroups > 0) tmem_ld16(tmem_base + lane_field + (uint32_t)c0, r);
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
    } else if (warp == 4) {
        // ------------------------------------------------------------ record loader (runs NBC chunks ahead)
        // (the whole warp runs the loop in step; one elected lane issues).  The node indices of a group are
        // read one group ahead of their use, all at once, so that no copy waits for an index load.  The ring is
        // deep enough to cover the latency of HBM: separate L2 prefetches only cost issue slots.
        int32_t issued = 0;
        int32_t l_cur[GU], l_nxt[GU];
        auto read_indices = [&](int32_t gq, int32_t (&l)[GU]) {
#pragma unroll
            for (int j = 0; j < GU; ++j) l[j] = gq * GU + j < cnt ? __ldg(ulist + gq * GU + j) : 0;
        };
        read_indices(0, l_cur);
        for (int32_t gi = 0; gi < ngroups; ++gi) {
            read_indices(gi + 1, l_nxt);
            if (gi >= NBC && !__all_sync(0xffffffffu, mbar_wait(done(gi % NBC), (uint32_t)((gi - NBC) / NBC) & 1u, &abort_flag))) break;
            const int32_t uend = min(cnt, (gi + 1) * GU);
            // one barrier per chunk: it completes when all of the chunk's records have landed
            expect_tx_elected(rec_full(gi % NBC), (uint32_t)(uend - gi * GU) * Sh::TILE_BYTES);
#pragma unroll
            for (int j = 0; j < GU; ++j) {
                const int32_t u = gi * GU + j;
                if (u < uend)
                    bulk_load_elected(b_base + (uint32_t)(u % NREC) * Sh::TILE_BYTES, recs + (size_t)l_cur[j] * Sh::REC_BYTES,
                                        Sh::TILE_BYTES, rec_full(gi % NBC));
            }
            issued = uend;
#pragma unroll
            for (int j = 0; j < GU; ++j) l_cur[j] = l_nxt[j];
        }
        if (abort_flag) {
            // gave up somewhere: let the copies that are still in flight land before the CTA exits
            const int32_t glast = (issued + GU - 1) / GU;
            for (int32_t gq = glast > NBC ? glast - NBC : 0; gq < glast; ++gq) {
                const long long t0 = clock64();
                while (!mbar_try_wait(rec_full(gq % NBC), (uint32_t)(gq / NBC) & 1u) && clock64() - t0 < WAIT_CYCLES) {}
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issuer: all groups, in list order
        // The whole warp runs the loop in step (every exit is voted on), so that the issuing helpers meet a
        // converged warp.
        constexpr uint32_t idesc = instr_desc(D, false, false);
        const uint32_t acc = tmem_base;
        bool ok = true;
        bool first = true;
        for (int32_t gi = 0; gi < ngroups && ok; ++gi) {
            const int st = gi % NA;
            if (!__all_sync(0xffffffffu, mbar_wait(a_full(st), (uint32_t)(gi / NA) & 1u, &abort_flag))) { ok = false; break; }
            if (!__all_sync(0xffffffffu, mbar_wait(rec_full(gi % NBC), (uint32_t)(gi / NBC) & 1u, &abort_flag))) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int32_t uend = min(cnt, (gi + 1) * GU);
            for (int32_t u = gi * GU; u < uend; ++u) {
                const int sr = u % NREC;
                const uint32_t a_op = tmem_a + (uint32_t)((st * GU + (u - gi * GU)) * Sh::A_COLS);
                const uint32_t b_op = b_base + (uint32_t)sr * Sh::TILE_BYTES;
#pragma unroll
                for (int k = 0; k < M / 16; ++k) {
                    const uint64_t bd = operand_desc(b_op + (uint32_t)k * 2u * (D * 16), D * 16, 128);
                    mma_bf16_ts(acc, a_op + (uint32_t)k * 8u, bd, idesc, (first && k == 0) ? 0u : 1u);
                }
                first = false;
            }
            if (ok) mma_commit(done(gi % NBC));
        }
        if (ngroups > 0) mma_commit(acc_done);
        if (!ok && ngroups > 0) {
            // aborted: wait (bounded) until the MMAs already issued have drained before the CTA exits
            const long long t0 = clock64();
            while (!mbar_try_wait(acc_done, 0u) && clock64() - t0 < WAIT_CYCLES) {}
        }
        __syncwarp();
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 5) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Sh::TMEM_COLS) : "memory");
    }
    if (tid == 0 && abort_flag) atomicExch(error_word, 1);
}

// ---------------------------------------------------------------------------------------------------
// Denominators of Eq. 12 for the tensor-core path: den_i = phi(q_i) . (sum_l Phi_il z_l), one warp per
// (problem, query); m/4 lanes take one node's z_l (its bf16 copy in the record, four components = 8 bytes per lane),
// so a warp handles 128/m nodes side by side; the sums run on packed pairs of fp32.

constexpr int DEN_GH = 4;   // problems per warp of the denominators kernel: they share the row's indices and coefficients

__device__ __forceinline__ uint64_t den_pack2(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ uint64_t den_fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

template <int M, int D>
__global__ void __launch_bounds__(256)
row_denominators_kernel(int32_t G, int32_t N, int32_t R, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                        const float* __restrict__ val, const __nv_bfloat16* __restrict__ phiQ,
                        const unsigned char* __restrict__ records, float* __restrict__ den)
{
    constexpr int LPL = M / 4;                              // lanes per node: each takes four components (bf16 x 4)
    constexpr int LPW = 32 / LPL;                           // nodes handled side by side in a warp
    constexpr size_t REC = (size_t)M * D * 2 + (size_t)M * 4 + (size_t)M * 2;
    static_assert(LPL >= 1 && LPL <= 32 && REC % 8 == 0, "layout");
    const int lane = threadIdx.x & 31;
    const int sub = lane / LPL, pl = lane % LPL;
    const int32_t i = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int32_t g0 = blockIdx.y * DEN_GH;
    if (i >= N) return;
    const size_t gstride = (size_t)R * REC;                 // from one problem's records to the next one's
    const unsigned char* zbase = records + (size_t)g0 * gstride + (size_t)M * D * 2 + (size_t)M * 4 + (size_t)pl * 8;   // the bf16 copy of z
    uint64_t z01[DEN_GH], z23[DEN_GH];                      // components 0,1 and 2,3 of this lane's four
#pragma unroll
    for (int h = 0; h < DEN_GH; ++h) { z01[h] = 0ull; z23[h] = 0ull; }
    const int32_t beg = rowptr[i], end = rowptr[i + 1];
    for (int32_t p0 = beg; p0 < end; p0 += 32) {
        const int32_t n = min(32, end - p0);
        const int32_t c_mine = lane < n ? __ldg(col + p0 + lane) : 0;
        const float v_mine = lane < n ? __ldg(val + p0 + lane) : 0.0f;
        for (int32_t j = 0; j < n; j += LPW) {
            const int32_t jj = j + sub;
            const int32_t l = __shfl_sync(0xffffffffu, c_mine, jj & 31);
            const float phi = __shfl_sync(0xffffffffu, v_mine, jj & 31);
            if (jj < n) {
                const unsigned char* zl = zbase + (size_t)l * REC;
                uint2 w[DEN_GH];
#pragma unroll
                for (int h = 0; h < DEN_GH; ++h)
                    w[h] = g0 + h < G ? __ldg(reinterpret_cast<const uint2*>(zl + (size_t)h * gstride)) : make_uint2(0u, 0u);
                const uint64_t phi2 = den_pack2(__float_as_uint(phi), __float_as_uint(phi));
#pragma unroll
                for (int h = 0; h < DEN_GH; ++h) {
                    z01[h] = den_fma2(phi2, den_pack2(w[h].x << 16, w[h].x & 0xffff0000u), z01[h]);
                    z23[h] = den_fma2(phi2, den_pack2(w[h].y << 16, w[h].y & 0xffff0000u), z23[h]);
                }
            }
        }
    }
#pragma unroll
    for (int h = 0; h < DEN_GH; ++h) {
        if (g0 + h >= G) break;
        const uint2 q = __ldg(reinterpret_cast<const uint2*>(phiQ + ((size_t)(g0 + h) * N + i) * M) + pl);
        float a0, a1, a2, a3;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(z01[h]));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(a2), "=f"(a3) : "l"(z23[h]));
        float d = __uint_as_float(q.x << 16) * a0;
        d = fmaf(__uint_as_float(q.x & 0xffff0000u), a1, d);
        d = fmaf(__uint_as_float(q.y << 16), a2, d);
        d = fmaf(__uint_as_float(q.y & 0xffff0000u), a3, d);
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
        if (lane == 0) den[(size_t)(g0 + h) * N + i] = d;
    }
}

// ---------------------------------------------------------------------------------------------------
// Self-test of the bounded waits: a barrier that nothing ever arrives at is waited for with the kernels' own wait
// routine and a short limit; the wait must give up, raise the CTA's flag and the context's error word.
__global__ void __launch_bounds__(32) wait_timeout_probe_kernel(long long limit_cycles, int* __restrict__ error_word)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_cycles);
    if (!__all_sync(0xffffffffu, ok) && threadIdx.x == 0 && abort_flag) atomicExch(error_word, 1);
}

// ---------------------------------------------------------------------------------------------------
// Block plan: for every block of BQ consecutive rows of Phi, the sorted list of distinct columns.

constexpr int PLAN_THREADS = 1024;   // one CTA per block: the passes over the block's non-zeros use all of them,
                                     // the ordered parts (one contiguous range of bitmap words per thread) the first 256

__global__ void __launch_bounds__(PLAN_THREADS)
block_plan_kernel(int32_t N, int32_t R, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                  int32_t* __restrict__ plan_off, int32_t* __restrict__ plan_cnt, int32_t* __restrict__ plan_col,
                  int32_t* __restrict__ plan_total)
{
    extern __shared__ uint32_t bitmap[];        // one bit per column
    __shared__ int32_t warp_sums[8];
    __shared__ int32_t base_off, block_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t blk = blockIdx.x;
    const int32_t words = (R + 31) >> 5;
    for (int32_t x = tid; x < words; x += PLAN_THREADS) bitmap[x] = 0u;
    __syncthreads();
    const int32_t r0 = blk * BQ, r1 = min(N, r0 + BQ);
    for (int32_t p = rowptr[r0] + tid; p < rowptr[r1]; p += PLAN_THREADS) {
        const int32_t c = col[p];
        atomicOr(&bitmap[c >> 5], 1u << (c & 31));
    }
    __syncthreads();
    // each of the first 256 threads owns a contiguous range of words so that the output stays sorted
    const int32_t per = (words + 255) / 256;
    const int32_t w0 = min(words, min(tid, 256) * per), w1 = tid < 256 ? min(words, w0 + per) : w0;
    int32_t mine = 0;
    for (int32_t x = w0; x < w1; ++x) mine += __popc(bitmap[x]);
    int32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31 && warp < 8) warp_sums[warp] = inc;
    __syncthreads();
    int32_t before = inc - mine;
    for (int w = 0; w < min(warp, 8); ++w) before += warp_sums[w];
    if (tid == 255) {
        // lists are padded to a multiple of four entries (the last column repeated, with zero coefficients)
        const int32_t total = before + mine, padded = (total + 3) & ~3;
        base_off = atomicAdd(plan_total, padded);
        block_total = total;
        plan_off[blk] = base_off;
        plan_cnt[blk] = padded;
    }
    __syncthreads();
    if (tid >= 256) return;
    int32_t o = base_off + before;
    for (int32_t x = w0; x < w1; ++x) {
        uint32_t bits = bitmap[x];
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            plan_col[o++] = (x << 5) + b;
        }
    }
    if (before + mine == block_total && block_total > 0) {
        // the thread that holds the end of the list: w1 may be below `words` only for trailing empty ranges
        bool last = true;
        for (int32_t x = w1; x < words && last; ++x) last = bitmap[x] == 0u;
        if (last && mine > 0) {
            const int32_t last_col = plan_col[base_off + block_total - 1];
            for (int32_t e = block_total; e < ((block_total + 3) & ~3); ++e) plan_col[base_off + e] = last_col;
        }
    }
}

// Second pass of the plan: the block's coefficients as a dense table, four union entries (bf16) per 8-byte
// word, [quad][row][4], so that a row thread of the gather kernel reads its coefficients with one coalesced
// load per four union entries.
__global__ void __launch_bounds__(PLAN_THREADS)
block_coef_kernel(int32_t N, int32_t R, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                  const float* __restrict__ val, const int32_t* __restrict__ plan_off,
                  const int32_t* __restrict__ plan_cnt, __nv_bfloat16* __restrict__ plan_coef)
{
    extern __shared__ uint32_t smem_plan[];     // bitmap, then the number of set bits before each word
    __shared__ int32_t warp_sums[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t blk = blockIdx.x;
    const int32_t words = (R + 31) >> 5;
    uint32_t* bitmap = smem_plan;
    int32_t* before_word = reinterpret_cast<int32_t*>(smem_plan + words);
    for (int32_t x = tid; x < words; x += PLAN_THREADS) bitmap[x] = 0u;
    __syncthreads();
    const int32_t r0 = blk * BQ, r1 = min(N, r0 + BQ);
    for (int32_t p = rowptr[r0] + tid; p < rowptr[r1]; p += PLAN_THREADS) {
        const int32_t c = col[p];
        atomicOr(&bitmap[c >> 5], 1u << (c & 31));
    }
    // zero this block's part of the table meanwhile
    const int32_t off = plan_off[blk], cnt = plan_cnt[blk];
    uint4* tab4 = reinterpret_cast<uint4*>(plan_coef + (size_t)off * BQ);
    for (int32_t x = tid; x < cnt * (BQ * 2 / 16); x += PLAN_THREADS) tab4[x] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    const int32_t per = (words + 255) / 256;
    const int32_t w0 = min(words, min(tid, 256) * per), w1 = tid < 256 ? min(words, w0 + per) : w0;
    int32_t mine = 0;
    for (int32_t x = w0; x < w1; ++x) mine += __popc(bitmap[x]);
    int32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31 && warp < 8) warp_sums[warp] = inc;
    __syncthreads();
    int32_t run = inc - mine;
    for (int w = 0; w < min(warp, 8); ++w) run += warp_sums[w];
    for (int32_t x = w0; x < w1; ++x) { before_word[x] = run; run += __popc(bitmap[x]); }
    __syncthreads();
    __nv_bfloat16* tab = plan_coef + (size_t)off * BQ;
    for (int32_t r = r0 + warp; r < r1; r += PLAN_THREADS / 32)
        for (int32_t p = rowptr[r] + lane; p < rowptr[r + 1]; p += 32) {
            const int32_t c = col[p];
            const int32_t u = before_word[c >> 5] + __popc(bitmap[c >> 5] & ((1u << (c & 31)) - 1u));
            tab[((size_t)(u >> 2) * BQ + (r - r0)) * 4 + (u & 3)] = __float2bfloat16_rn(val[p]);
        }
}

// order[r] = the block with the r-th largest union (ties: lower index first), stored behind the counts
__global__ void __launch_bounds__(256) block_order_kernel(int32_t nblocks, int32_t* __restrict__ plan_cnt)
{
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nblocks) return;
    const int32_t c = plan_cnt[i];
    int32_t rank = 0;
    for (int32_t j = 0; j < nblocks; ++j) {
        const int32_t cj = plan_cnt[j];
        rank += (cj > c || (cj == c && j < i)) ? 1 : 0;
    }
    plan_cnt[nblocks + rank] = i;
}

}  // namespace

// The coefficient table of the tensor-core gather (Phi's values per union entry and row), for a plan that is ready.
static int build_plan_coefficients(grf_ctx* ctx, grf_features* feat)
{
    grf_csr_dev& phi = feat->phi;
    const int32_t N = phi.rows, R = phi.cols;
    const size_t words = (size_t)(R + 31) / 32;
    const size_t table_bytes = (size_t)feat->plan_entries * BQ * sizeof(__nv_bfloat16);
    if (feat->plan_coef.bytes < table_bytes) GRF_TRY(grf_buf_reserve(&feat->plan_coef, table_bytes + table_bytes / 8));
    GRF_CUDA_TRY(cudaFuncSetAttribute(block_coef_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(words * 8)));
    {
        grf_launch_scope scope(ctx, 7);
        block_coef_kernel<<<feat->plan_blocks, PLAN_THREADS, words * 8, ctx->stream>>>(
            N, R, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr, (const float*)phi.val.ptr,
            (const int32_t*)feat->plan_off.ptr, (const int32_t*)feat->plan_cnt.ptr, (__nv_bfloat16*)feat->plan_coef.ptr);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    feat->plan_coef_ready = true;
    return GRF_OK;
}

int grf_build_block_plan(grf_ctx* ctx, grf_features* feat, bool with_coef)
{
    grf_csr_dev& phi = feat->phi;
    feat->plan_ready = false;
    feat->plan_coef_ready = false;
    const int32_t N = phi.rows, R = phi.cols;
    const size_t words = (size_t)(R + 31) / 32;
    if (words * 8 > 200 * 1024 || phi.nnz <= 0) return GRF_OK;   // no plan: the ALU kernel serves this object
    const int32_t nblocks = grf_ceil_div(N, BQ);
    GRF_TRY(grf_buf_reserve(&feat->plan_off, sizeof(int32_t) * (size_t)nblocks));
    GRF_TRY(grf_buf_reserve(&feat->plan_cnt, sizeof(int32_t) * 2 * (size_t)nblocks));   // counts, then blocks by decreasing count
    GRF_TRY(grf_buf_reserve(&feat->plan_col, phi.col.bytes + sizeof(int32_t) * 3 * (size_t)nblocks));
    GRF_TRY(grf_buf_reserve(&feat->plan_total, sizeof(int32_t)));
    GRF_CUDA_TRY(cudaMemsetAsync(feat->plan_total.ptr, 0, sizeof(int32_t), ctx->stream));
    GRF_CUDA_TRY(cudaFuncSetAttribute(block_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(words * 4)));
    {
        grf_launch_scope scope(ctx, 7);
        block_plan_kernel<<<nblocks, PLAN_THREADS, words * 4, ctx->stream>>>(
            N, R, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr, (int32_t*)feat->plan_off.ptr,
            (int32_t*)feat->plan_cnt.ptr, (int32_t*)feat->plan_col.ptr, (int32_t*)feat->plan_total.ptr);
    }
    {
        grf_launch_scope scope(ctx, 7);
        block_order_kernel<<<grf_ceil_div(nblocks, 256), 256, 0, ctx->stream>>>(nblocks, (int32_t*)feat->plan_cnt.ptr);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    // the table's size is known only now
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 4, feat->plan_total.ptr, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    GRF_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    const size_t entries = (size_t)ctx->pinned[4];
    const size_t table_bytes = entries * BQ * sizeof(__nv_bfloat16);
    if (table_bytes > ((size_t)2 << 30)) return GRF_OK;           // too little sharing between neighbouring rows
    feat->plan_blocks = nblocks;
    feat->plan_entries = (int64_t)entries;
    feat->plan_ready = true;
    return with_coef ? build_plan_coefficients(ctx, feat) : GRF_OK;
}

extern "C" int grf_debug_wait_timeout(grf_ctx* ctx, int64_t limit_cycles)
{
    if (!ctx || limit_cycles < 1 || limit_cycles > 2000000000ll) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    wait_timeout_probe_kernel<<<1, 32, 0, ctx->stream>>>((long long)limit_cycles, ctx->error_word);
    ctx->launches += 1;
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

extern "C" int grf_plan_stats(grf_ctx* ctx, const grf_features* feat, int32_t* blocks, int64_t* entries)
{
    if (!ctx || !feat) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    GRF_TRY(grf_ensure_block_plan(ctx, feat));
    if (!feat->plan_ready) return GRF_ERR_TOO_LARGE;
    if (blocks) *blocks = feat->plan_blocks;
    if (entries) *entries = feat->plan_entries;
    return GRF_OK;
}

template <int M, int D>
static int launch_tc(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N,
                     const void* phiQ, const void* records, void* out, float* den_out)
{
    using Sh = TcShape<M, D>;
    const grf_csr_dev& phi = feat->phi;
    GRF_CUDA_TRY(cudaFuncSetAttribute(gather_contract_tc_kernel<M, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)Sh::SMEM));
    float* den = den_out;
    if (!den) {
        GRF_TRY(grf_buf_reserve(&ctx->den_scratch, sizeof(float) * (size_t)G * N));
        den = (float*)ctx->den_scratch.ptr;
    }
    // (Running the denominators on a side stream beside the gather kernel was measured: both draw on the same
    // L2 bandwidth, the pair ends 0.1 ms earlier at most, and the rows then need a second pass to be divided.)
    {
        grf_launch_scope scope(ctx, 6);
        row_denominators_kernel<M, D><<<dim3(grf_ceil_div(N, 8), grf_ceil_div(G, DEN_GH)), 256, 0, ctx->stream>>>(
            G, N, phi.cols, (const int32_t*)phi.rowptr.ptr, (const int32_t*)phi.col.ptr, (const float*)phi.val.ptr,
            (const __nv_bfloat16*)phiQ, (const unsigned char*)records, den);
    }
    const dim3 grid((unsigned)feat->plan_blocks * (unsigned)G);
    {
        grf_launch_scope scope(ctx, 5);
        gather_contract_tc_kernel<M, D><<<grid, TC_THREADS, Sh::SMEM, ctx->stream>>>(
            G, feat->plan_blocks, N, phi.cols, (const int32_t*)feat->plan_off.ptr, (const int32_t*)feat->plan_cnt.ptr,
            (const int32_t*)feat->plan_col.ptr, (const uint2*)feat->plan_coef.ptr, (const __nv_bfloat16*)phiQ,
            (const unsigned char*)records, (__nv_bfloat16*)out, den, ctx->error_word);
    }
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

// The plan is a cache inside the feature object, built on first use (the asymmetric route never needs it); the
// route over the materialised mask uses its node lists but not the coefficient table, which is then left out until
// the gather kernel asks for it.
int grf_ensure_block_plan(grf_ctx* ctx, const grf_features* feat, bool with_coef)
{
    grf_features* f = const_cast<grf_features*>(feat);
    if (feat->plan_stale) {
        GRF_TRY(grf_build_block_plan(ctx, f, with_coef));
        f->plan_stale = false;
        return GRF_OK;
    }
    if (with_coef && feat->plan_ready && !feat->plan_coef_ready) return build_plan_coefficients(ctx, f);
    return GRF_OK;
}

// Returns GRF_OK after launching, or 1 when this shape/object has no tensor-core path (caller falls back).
int grf_gather_contract_tc(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                           const void* phiQ, const void* records, void* out, float* den_out)
{
    if (G > 65535) return 1;
    GRF_TRY(grf_ensure_block_plan(ctx, feat));
    if (!feat->plan_ready) return 1;
#define GRF_TC_CASE(MM, DD) \
    if (m == MM && d == DD) return launch_tc<MM, DD>(ctx, feat, G, N, phiQ, records, out, den_out);
    GRF_TC_CASE(16, 16) GRF_TC_CASE(16, 32) GRF_TC_CASE(16, 64) GRF_TC_CASE(16, 128)
    GRF_TC_CASE(32, 16) GRF_TC_CASE(32, 32) GRF_TC_CASE(32, 64) GRF_TC_CASE(32, 128)
    GRF_TC_CASE(64, 16) GRF_TC_CASE(64, 32) GRF_TC_CASE(64, 64) GRF_TC_CASE(64, 128)
    GRF_TC_CASE(128, 16) GRF_TC_CASE(128, 32) GRF_TC_CASE(128, 64) GRF_TC_CASE(128, 128)
#undef GRF_TC_CASE
    return 1;
}
