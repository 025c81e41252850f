// Masked attention with the mask estimate materialised (Eqs. 1-2 with Mhat = Phi Psi^T, Sec. 3.3), bf16 storage.
//
// Instead of going through the per-node states of Eq. 12, the sparse product Mhat = Phi Psi^T is formed once per
// feature object and the attention is evaluated from its definition,
//     out_i = sum_j Mhat_ij (phi(q_i) . phi(k_j)) v_j / sum_j Mhat_ij (phi(q_i) . phi(k_j)),
// over the non-zeros of Mhat only.  On graphs whose node numbering keeps neighbours together, the rows of a block
// of 128 consecutive queries reach a few thousand keys between them and about a quarter of that block of Mhat is
// non-zero: dense enough for the tensor cores.  Per block the mask is stored densely (bf16) over the block's key
// list, and one CTA per (block, problem) runs a two-product pipeline over tiles of 64 keys:
//     S = phi(Q_blk) phi(K_tile)^T   (tcgen05, accumulator in tensor memory)
//     P = S * Mhat_tile              (row threads: tensor memory -> registers -> tensor memory, bf16)
//     O += P V_tile                  (tcgen05, P read from tensor memory)
// and the row sums of P (taken in fp32, before its rounding) give the denominators.  Key and value rows are gathered
// by key index with 16-byte asynchronous copies: value rows into the 128-byte-swizzled MN-major operand layout,
// key-feature rows into the unswizzled K-major layout.
//
// Building the mask (once per feature object): the key list of a block is the union of the rows of Psi^T over the
// block's node list (the block plan of Phi); the values are accumulated row by row, one warp per row, in ascending
// order of the node l, each lane owning distinct keys, so the sums are reproducible without atomics.
#include "tc_common.cuh"

namespace {

using namespace grf_tc;

constexpr int BQ = GRF_PLAN_BLOCK;      // queries per block
constexpr int KT = GRF_MASK_TILE;       // keys per tile

// ---------------------------------------------------------------------------------------------------
// Key sets: one CTA per block of rows marks, in a bitmap, the keys of Psi^T's rows over the block's node list.
// A warp takes 32 nodes at a time (lane x holds node x's extent in Psi^T) and fetches the keys of four nodes
// together, so that several loads are in flight.  The bitmap and the count (padded to whole tiles) are kept.

constexpr int MASK_BITMAP_THREADS = 1024;     // one CTA per block: many warps, each with a few batches of 32 nodes

__global__ void __launch_bounds__(MASK_BITMAP_THREADS)
mask_bitmap_kernel(int32_t Nk, const int32_t* __restrict__ plan_off, const int32_t* __restrict__ plan_cnt,
                   const int32_t* __restrict__ plan_col, const int32_t* __restrict__ t_rowptr,
                   const int32_t* __restrict__ t_col, uint32_t* __restrict__ bits, int32_t* __restrict__ mk_cnt)
{
    extern __shared__ uint32_t bitmap[];        // one bit per key
    __shared__ int32_t warp_sums[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t blk = blockIdx.x;
    const int32_t words = (Nk + 31) >> 5;
    for (int32_t x = tid; x < words; x += MASK_BITMAP_THREADS) bitmap[x] = 0u;
    __syncthreads();
    const int32_t* ulist = plan_col + plan_off[blk];
    const int32_t ucnt = plan_cnt[blk];
    for (int32_t u0 = warp * 32; u0 < ucnt; u0 += MASK_BITMAP_THREADS) {
        const int32_t n = min(32, ucnt - u0);
        const int32_t my_l = lane < n ? __ldg(ulist + u0 + lane) : 0;
        const int32_t my_beg = lane < n ? __ldg(t_rowptr + my_l) : 0;
        const int32_t my_end = lane < n ? __ldg(t_rowptr + my_l + 1) : 0;
        for (int32_t e0 = 0; e0 < n; e0 += 4) {
            int32_t jj[4][4];
            int32_t ebeg[4], eend[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                ebeg[e] = e0 + e < n ? __shfl_sync(0xffffffffu, my_beg, (e0 + e) & 31) : 0;
                eend[e] = e0 + e < n ? __shfl_sync(0xffffffffu, my_end, (e0 + e) & 31) : 0;
#pragma unroll
                for (int sl = 0; sl < 4; ++sl) {
                    const int32_t q = ebeg[e] + sl * 32 + lane;
                    jj[e][sl] = q < eend[e] ? __ldg(t_col + q) : -1;
                }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
#pragma unroll
                for (int sl = 0; sl < 4; ++sl)
                    if (jj[e][sl] >= 0) atomicOr(&bitmap[jj[e][sl] >> 5], 1u << (jj[e][sl] & 31));
                for (int32_t q = ebeg[e] + 128 + lane; q < eend[e]; q += 32) {
                    const int32_t j = __ldg(t_col + q);
                    atomicOr(&bitmap[j >> 5], 1u << (j & 31));
                }
            }
        }
    }
    __syncthreads();
    // the bitmap, and behind it the number of set bits before each of its words (the first 256 threads)
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
    if (tid >= 256) return;
    int32_t run = inc - mine;
    for (int w = 0; w < warp; ++w) run += warp_sums[w];
    uint32_t* dst = bits + (size_t)blk * 2 * words;
    for (int32_t x = w0; x < w1; ++x) {
        const uint32_t b = bitmap[x];
        dst[x] = b;
        dst[words + x] = (uint32_t)run;
        run += __popc(b);
    }
    if (tid == 255) mk_cnt[blk] = (run + KT - 1) / KT * KT;
}

// Key lists: the set bits of a block's bitmap in ascending order, padded to whole tiles with the last key
// (whose mask values in the padding are zeros).
__global__ void __launch_bounds__(256)
mask_list_kernel(int32_t Nk, const uint32_t* __restrict__ bits, const int32_t* __restrict__ mk_off,
                 const int32_t* __restrict__ mk_cnt, int32_t* __restrict__ mk_key)
{
    __shared__ int32_t warp_sums[8];
    __shared__ int32_t block_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t blk = blockIdx.x;
    const int32_t words = (Nk + 31) >> 5;
    const uint32_t* bitmap = bits + (size_t)blk * 2 * words;
    // each thread owns a contiguous range of words so that the list comes out sorted
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
    if (tid == 255) block_total = before + mine;
    const int32_t base_off = mk_off[blk];
    int32_t o = base_off + before;
    for (int32_t x = w0; x < w1; ++x) {
        uint32_t b = bitmap[x];
        while (b) {
            const int k = __ffs(b) - 1;
            b &= b - 1;
            mk_key[o++] = (x << 5) + k;
        }
    }
    __syncthreads();
    const int32_t padded = mk_cnt[blk];
    if (block_total > 0)
        for (int32_t e = block_total + tid; e < padded; e += 256) mk_key[base_off + e] = mk_key[base_off + block_total - 1];
}

// order[r] = the block with the r-th largest key list (ties: lower index first), stored behind the counts
__global__ void __launch_bounds__(256) mask_order_kernel(int32_t nblocks, int32_t* __restrict__ mk_cnt)
{
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nblocks) return;
    const int32_t c = mk_cnt[i];
    int32_t rank = 0;
    for (int32_t j = 0; j < nblocks; ++j) {
        const int32_t cj = mk_cnt[j];
        rank += (cj > c || (cj == c && j < i)) ? 1 : 0;
    }
    mk_cnt[nblocks + rank] = i;
}

// ---------------------------------------------------------------------------------------------------
// Mask values: Mhat_ij = sum_l Phi_il Psi_jl for the rows i of one block and the keys j of its list.
// A CTA takes MASK_ROWS rows of one block (the blocks with the longest key lists first), one warp per row at a
// time.  The warp keeps the row's accumulators (fp32, one per key of a segment of the list) in shared memory; for
// every non-zero Phi_il, taken in ascending l, its lanes add Phi_il * Psi_jl at the position of key j, found from
// the bitmap of the block's keys and the number of set bits before each bitmap word.  Keys of one l are distinct,
// so no two lanes meet at one position, and the warp is synchronised between two l: the order of every sum is
// fixed.  The keys of four nodes are fetched together and the next four are on their way while these are added.
// Lists longer than a segment take further passes.

constexpr int MASK_SEG = 4096;          // accumulators per warp
constexpr int MASK_WARPS = 4;
constexpr int MASK_ROWS = 8;            // rows of a block per CTA

struct MaskGroup {                      // the keys of four nodes l, up to 128 each: lane x holds keys x, x+32, x+64, x+96
    int32_t j[4][4];
    float v[4][4];
    int32_t beg[4], end[4];
};

__global__ void __launch_bounds__(MASK_WARPS * 32)
mask_values_kernel(int32_t N, int32_t Nk, const int32_t* __restrict__ phi_rowptr, const int32_t* __restrict__ phi_col,
                   const float* __restrict__ phi_val, const int32_t* __restrict__ t_rowptr,
                   const int32_t* __restrict__ t_col, const float* __restrict__ t_val,
                   const int32_t* __restrict__ mk_off, const int32_t* __restrict__ mk_cnt,
                   const uint32_t* __restrict__ bits, __nv_bfloat16* __restrict__ mk_val)
{
    extern __shared__ uint32_t smem_mask[];     // bitmap, set bits before each word, accumulators
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int GROUPS = BQ / MASK_ROWS;
    const int32_t nblocks = (N + BQ - 1) / BQ;
    const int32_t blk = mk_cnt[nblocks + blockIdx.x / GROUPS];     // blocks by decreasing key count
    const int32_t rg = blockIdx.x % GROUPS;
    const int32_t words = (Nk + 31) >> 5;
    const int32_t words_al = (words + 1) & ~1;
    uint32_t* bitmap = smem_mask;
    int32_t* before_word = reinterpret_cast<int32_t*>(smem_mask + words_al);
    // (the accumulators are read as float4: they start at a multiple of 16 bytes)
    float* acc = reinterpret_cast<float*>(smem_mask + 2 * (size_t)words_al) + (size_t)warp * MASK_SEG;
    const int32_t off = mk_off[blk], cnt = mk_cnt[blk];
    // the block's bitmap and prefix counts as the key-set kernel left them
    const uint32_t* src = bits + (size_t)blk * 2 * words;
    for (int32_t x = tid; x < words; x += MASK_WARPS * 32) {
        bitmap[x] = src[x];
        before_word[x] = (int32_t)src[words + x];
    }
    for (int32_t x = lane; x < MASK_SEG; x += 32) acc[x] = 0.0f;
    __syncthreads();
    const int32_t r0 = blk * BQ;
    for (int32_t seg0 = 0; seg0 < cnt; seg0 += MASK_SEG) {
        const int32_t seglen = min(MASK_SEG, cnt - seg0);       // a multiple of the tile, hence of 8
        auto position = [&](int32_t j) {
            const int32_t ps = before_word[j >> 5] + __popc(bitmap[j >> 5] & ((1u << (j & 31)) - 1u)) - seg0;
            return (ps >= 0 && ps < seglen) ? ps : -1;
        };
        for (int32_t rr = rg * MASK_ROWS + warp; rr < (rg + 1) * MASK_ROWS; rr += MASK_WARPS) {
            const int32_t r = r0 + rr;
            if (r < N) {
                const int32_t pbeg = phi_rowptr[r], pend = phi_rowptr[r + 1];
                for (int32_t p0 = pbeg; p0 < pend; p0 += 32) {
                    // 32 non-zeros of the row at a time: lane x holds node l_x, Phi_il and the extent of row l_x of Psi^T
                    const int32_t n = min(32, pend - p0);
                    const int32_t my_l = lane < n ? __ldg(phi_col + p0 + lane) : 0;
                    const float my_phi = lane < n ? __ldg(phi_val + p0 + lane) : 0.0f;
                    const int32_t my_beg = lane < n ? __ldg(t_rowptr + my_l) : 0;
                    const int32_t my_end = lane < n ? __ldg(t_rowptr + my_l + 1) : 0;
                    auto fetch = [&](int32_t e0, MaskGroup& gq) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            gq.beg[e] = e0 + e < n ? __shfl_sync(0xffffffffu, my_beg, (e0 + e) & 31) : 0;
                            gq.end[e] = e0 + e < n ? __shfl_sync(0xffffffffu, my_end, (e0 + e) & 31) : 0;
#pragma unroll
                            for (int sl = 0; sl < 4; ++sl) {
                                const int32_t q = gq.beg[e] + sl * 32 + lane;
                                const bool valid = q < gq.end[e];
                                gq.j[e][sl] = valid ? __ldg(t_col + q) : -1;
                                gq.v[e][sl] = valid ? __ldg(t_val + q) : 0.0f;
                            }
                        }
                    };
                    auto add = [&](int32_t e0, MaskGroup& gq) {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
#pragma unroll
                            for (int sl = 0; sl < 4; ++sl) gq.j[e][sl] = gq.j[e][sl] >= 0 ? position(gq.j[e][sl]) : -1;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float phi = __shfl_sync(0xffffffffu, my_phi, (e0 + e) & 31);
                            float a[4];
                            // one node's keys are distinct: a lane's four additions go side by side
#pragma unroll
                            for (int sl = 0; sl < 4; ++sl) a[sl] = gq.j[e][sl] >= 0 ? acc[gq.j[e][sl]] : 0.0f;
#pragma unroll
                            for (int sl = 0; sl < 4; ++sl)
                                if (gq.j[e][sl] >= 0) acc[gq.j[e][sl]] = fmaf(phi, gq.v[e][sl], a[sl]);
                            for (int32_t q = gq.beg[e] + 128 + lane; q < gq.end[e]; q += 32) {   // nodes with more than 128 keys
                                const int32_t ps = position(__ldg(t_col + q));
                                if (ps >= 0) acc[ps] = fmaf(phi, __ldg(t_val + q), acc[ps]);
                            }
                            __syncwarp();
                        }
                    };
                    MaskGroup ga, gb;
                    fetch(0, ga);
                    for (int32_t e0 = 0; e0 < n; e0 += 8) {
                        if (e0 + 4 < n) fetch(e0 + 4, gb);
                        add(e0, ga);
                        if (e0 + 4 < n) {
                            if (e0 + 8 < n) fetch(e0 + 8, ga);
                            add(e0 + 4, gb);
                        }
                    }
                }
            }
            // the row's values of this segment, eight keys (16 bytes) per lane at a time; the accumulators are
            // cleared for the next row as they are read
            for (int32_t c8 = lane; c8 < seglen / 8; c8 += 32) {
                float4* a4 = reinterpret_cast<float4*>(acc + c8 * 8);
                const float4 x0 = a4[0], x1 = a4[1];
                a4[0] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                a4[1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(x0.x, x0.y), h1 = __floats2bfloat162_rn(x0.z, x0.w);
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(x1.x, x1.y), h3 = __floats2bfloat162_rn(x1.z, x1.w);
                uint4* dst = reinterpret_cast<uint4*>(mk_val + ((size_t)((off + seg0) / 8 + c8) * BQ + rr) * 8);
                *dst = make_uint4(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1),
                                  *reinterpret_cast<const uint32_t*>(&h2), *reinterpret_cast<const uint32_t*>(&h3));
            }
            __syncwarp();
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// The same sums with the positions looked up once per (block, node) instead of once per (row, node): a node of a
// block's list is used by nine of the block's rows on average, and the look-up (two shared-memory reads and a
// population count per key) was most of the work of every addition.
//   mask_node_offsets_kernel  per block: where each node's positions start (running sum of the lengths of the
//                             nodes' rows of Psi^T over the block's list) and the block's total;
//   mask_positions_kernel     per block: the position in the block's key list of every key of every node of the
//                             list (16 bits each), and for every non-zero Phi_il of the block's rows where the
//                             positions of node l start;
//   mask_values_pos_kernel    the row-by-row accumulation, reading positions instead of keys.

__global__ void __launch_bounds__(256)
mask_node_offsets_kernel(const int32_t* __restrict__ plan_off, const int32_t* __restrict__ plan_cnt,
                         const int32_t* __restrict__ plan_col, const int32_t* __restrict__ t_rowptr,
                         int32_t* __restrict__ node_off, int32_t* __restrict__ blk_total,
                         const int32_t* __restrict__ mk_cnt, int32_t* __restrict__ longest_list)
{
    __shared__ int32_t warp_sums[8];
    __shared__ int32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t blk = blockIdx.x;
    const int32_t uoff = plan_off[blk], ucnt = plan_cnt[blk];
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int32_t base = 0; base < ucnt; base += 256) {
        const int32_t u = base + tid;
        int32_t len = 0;
        if (u < ucnt) {
            const int32_t l = plan_col[uoff + u];
            len = t_rowptr[l + 1] - t_rowptr[l];
        }
        int32_t inc = len;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        if (lane == 31) warp_sums[warp] = inc;
        __syncthreads();
        int32_t before = carry_s + inc - len;
        for (int w = 0; w < warp; ++w) before += warp_sums[w];
        if (u < ucnt) node_off[uoff + u] = before;
        __syncthreads();
        if (tid == 255) carry_s = before + len;
        __syncthreads();
    }
    if (tid == 0) {
        blk_total[blk] = carry_s;
        atomicMax(longest_list, mk_cnt[blk]);        // positions are kept in 16 bits: the host checks this
    }
}

constexpr int MASK_POS_PARTS = 4;

__global__ void __launch_bounds__(256)
mask_positions_kernel(int32_t N, int32_t Nk, int32_t R, const int32_t* __restrict__ phi_rowptr,
                      const int32_t* __restrict__ phi_col, const int32_t* __restrict__ plan_off,
                      const int32_t* __restrict__ plan_cnt, const int32_t* __restrict__ plan_col,
                      const int32_t* __restrict__ t_rowptr, const int32_t* __restrict__ t_col,
                      const uint32_t* __restrict__ bits, const int32_t* __restrict__ node_off,
                      const int32_t* __restrict__ blk_pos, unsigned short* __restrict__ pos16, int32_t* __restrict__ phi_pos)
{
    extern __shared__ uint32_t smem_pos[];      // key bitmap, its prefix counts, node bitmap, its prefix counts
    __shared__ int32_t warp_sums[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // MASK_POS_PARTS CTAs share a block: each takes every MASK_POS_PARTS-th batch of nodes and slice of non-zeros
    const int32_t blk = blockIdx.x / MASK_POS_PARTS, part = blockIdx.x % MASK_POS_PARTS;
    const int32_t wk = (Nk + 31) >> 5, wr = (R + 31) >> 5;
    uint32_t* kbits = smem_pos;
    int32_t* kbefore = reinterpret_cast<int32_t*>(smem_pos + wk);
    uint32_t* nbits = smem_pos + 2 * wk;
    int32_t* nbefore = reinterpret_cast<int32_t*>(smem_pos + 2 * wk + wr);
    const uint32_t* src = bits + (size_t)blk * 2 * wk;
    for (int32_t x = tid; x < wk; x += 256) { kbits[x] = src[x]; kbefore[x] = (int32_t)src[wk + x]; }
    for (int32_t x = tid; x < wr; x += 256) nbits[x] = 0u;
    __syncthreads();
    const int32_t uoff = plan_off[blk], ucnt = plan_cnt[blk];
    const int32_t* ulist = plan_col + uoff;
    for (int32_t u = tid; u < ucnt; u += 256) {
        const int32_t l = ulist[u];
        atomicOr(&nbits[l >> 5], 1u << (l & 31));
    }
    __syncthreads();
    {
        const int32_t per = (wr + 255) / 256;
        const int32_t w0 = min(wr, tid * per), w1 = min(wr, w0 + per);
        int32_t mine = 0;
        for (int32_t x = w0; x < w1; ++x) mine += __popc(nbits[x]);
        int32_t inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t y = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += y;
        }
        if (lane == 31) warp_sums[warp] = inc;
        __syncthreads();
        int32_t run = inc - mine;
        for (int w = 0; w < warp; ++w) run += warp_sums[w];
        for (int32_t x = w0; x < w1; ++x) { nbefore[x] = run; run += __popc(nbits[x]); }
    }
    __syncthreads();
    const int32_t base = blk_pos[blk];
    // positions of the keys of every node of the list; a warp takes 32 nodes at a time (lane x holds node x's extent
    // in Psi^T and the start of its positions) and fetches the keys of four nodes together
    for (int32_t u0 = (part * 8 + warp) * 32; u0 < ucnt; u0 += MASK_POS_PARTS * 8 * 32) {
        const int32_t n = min(32, ucnt - u0);
        const int32_t my_l = lane < n ? __ldg(ulist + u0 + lane) : 0;
        const int32_t my_beg = lane < n ? __ldg(t_rowptr + my_l) : 0;
        const int32_t my_end = lane < n ? __ldg(t_rowptr + my_l + 1) : 0;
        const int32_t my_dst = lane < n ? base + node_off[uoff + u0 + lane] : 0;
        for (int32_t e0 = 0; e0 < n; e0 += 4) {
            int32_t jj[4][4];
            int32_t ebeg[4], eend[4], edst[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                ebeg[e] = e0 + e < n ? __shfl_sync(0xffffffffu, my_beg, (e0 + e) & 31) : 0;
                eend[e] = e0 + e < n ? __shfl_sync(0xffffffffu, my_end, (e0 + e) & 31) : 0;
                edst[e] = __shfl_sync(0xffffffffu, my_dst, (e0 + e) & 31);
#pragma unroll
                for (int sl = 0; sl < 4; ++sl) {
                    const int32_t q = ebeg[e] + sl * 32 + lane;
                    jj[e][sl] = q < eend[e] ? __ldg(t_col + q) : -1;
                }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
#pragma unroll
                for (int sl = 0; sl < 4; ++sl) {
                    const int32_t j = jj[e][sl];
                    if (j >= 0)
                        pos16[(size_t)edst[e] + sl * 32 + lane] =
                            (unsigned short)(kbefore[j >> 5] + __popc(kbits[j >> 5] & ((1u << (j & 31)) - 1u)));
                }
                for (int32_t q = ebeg[e] + 128 + lane; q < eend[e]; q += 32) {        // nodes with more than 128 keys
                    const int32_t j = __ldg(t_col + q);
                    pos16[(size_t)edst[e] + (q - ebeg[e])] =
                        (unsigned short)(kbefore[j >> 5] + __popc(kbits[j >> 5] & ((1u << (j & 31)) - 1u)));
                }
            }
        }
    }
    // where the positions of its node start, for every non-zero of the block's rows of Phi (the list holds a node
    // once, apart from the padding at its end, which repeats the last node: the first occurrence counts)
    const int32_t r0 = blk * BQ, r1 = min(N, r0 + BQ);
    for (int32_t p = phi_rowptr[r0] + part * 256 + tid; p < phi_rowptr[r1]; p += MASK_POS_PARTS * 256) {
        const int32_t l = __ldg(phi_col + p);
        const int32_t u = nbefore[l >> 5] + __popc(nbits[l >> 5] & ((1u << (l & 31)) - 1u));
        phi_pos[p] = base + node_off[uoff + u];
    }
}

struct MaskPosGroup {                   // the keys of four nodes l, up to 128 each: lane x holds keys x, x+32, x+64, x+96
    int32_t ps[4][4];
    float v[4][4];
    int32_t len[4], beg[4], pbeg[4];
};

__global__ void __launch_bounds__(MASK_WARPS * 32)
mask_values_pos_kernel(int32_t N, const int32_t* __restrict__ phi_rowptr, const int32_t* __restrict__ phi_col,
                       const float* __restrict__ phi_val, const int32_t* __restrict__ phi_pos,
                       const int32_t* __restrict__ t_rowptr, const float* __restrict__ t_val,
                       const unsigned short* __restrict__ pos16, const int32_t* __restrict__ mk_off,
                       const int32_t* __restrict__ mk_cnt, __nv_bfloat16* __restrict__ mk_val)
{
    extern __shared__ float smem_acc[];         // the warps' accumulators
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int GROUPS = BQ / MASK_ROWS;
    const int32_t nblocks = (N + BQ - 1) / BQ;
    const int32_t blk = mk_cnt[nblocks + blockIdx.x / GROUPS];     // blocks by decreasing key count
    const int32_t rg = blockIdx.x % GROUPS;
    float* acc = smem_acc + (size_t)warp * MASK_SEG;
    const int32_t off = mk_off[blk], cnt = mk_cnt[blk];
    for (int32_t x = lane; x < MASK_SEG; x += 32) acc[x] = 0.0f;
    __syncwarp();
    const int32_t r0 = blk * BQ;
    for (int32_t seg0 = 0; seg0 < cnt; seg0 += MASK_SEG) {
        const int32_t seglen = min(MASK_SEG, cnt - seg0);       // a multiple of the tile, hence of 8
        for (int32_t rr = rg * MASK_ROWS + warp; rr < (rg + 1) * MASK_ROWS; rr += MASK_WARPS) {
            const int32_t r = r0 + rr;
            if (r < N) {
                const int32_t pbeg = phi_rowptr[r], pend = phi_rowptr[r + 1];
                for (int32_t p0 = pbeg; p0 < pend; p0 += 32) {
                    // 32 non-zeros of the row at a time: lane x holds Phi_il, the start and length of row l_x of Psi^T
                    // and the start of node l_x's positions
                    const int32_t n = min(32, pend - p0);
                    const int32_t my_l = lane < n ? __ldg(phi_col + p0 + lane) : 0;
                    const float my_phi = lane < n ? __ldg(phi_val + p0 + lane) : 0.0f;
                    const int32_t my_pbeg = lane < n ? __ldg(phi_pos + p0 + lane) : 0;
                    const int32_t my_beg = lane < n ? __ldg(t_rowptr + my_l) : 0;
                    const int32_t my_len = lane < n ? __ldg(t_rowptr + my_l + 1) - my_beg : 0;
                    auto fetch = [&](int32_t e0, MaskPosGroup& gq) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            gq.beg[e] = __shfl_sync(0xffffffffu, my_beg, (e0 + e) & 31);
                            gq.pbeg[e] = __shfl_sync(0xffffffffu, my_pbeg, (e0 + e) & 31);
                            gq.len[e] = e0 + e < n ? __shfl_sync(0xffffffffu, my_len, (e0 + e) & 31) : 0;
#pragma unroll
                            for (int sl = 0; sl < 4; ++sl) {
                                const int32_t x = sl * 32 + lane;
                                const bool valid = x < gq.len[e];
                                gq.ps[e][sl] = valid ? (int32_t)__ldg(pos16 + (size_t)gq.pbeg[e] + x) : -1;
                                gq.v[e][sl] = valid ? __ldg(t_val + gq.beg[e] + x) : 0.0f;
                            }
                        }
                    };
                    auto add = [&](int32_t e0, MaskPosGroup& gq) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float phi = __shfl_sync(0xffffffffu, my_phi, (e0 + e) & 31);
                            float a[4];
                            int32_t ps[4];
                            // one node's keys are distinct: a lane's four additions go side by side
#pragma unroll
                            for (int sl = 0; sl < 4; ++sl) {
                                const int32_t x = gq.ps[e][sl] - seg0;
                                ps[sl] = (gq.ps[e][sl] >= 0 && x >= 0 && x < seglen) ? x : -1;
                                a[sl] = ps[sl] >= 0 ? acc[ps[sl]] : 0.0f;
                            }
#pragma unroll
                            for (int sl = 0; sl < 4; ++sl)
                                if (ps[sl] >= 0) acc[ps[sl]] = fmaf(phi, gq.v[e][sl], a[sl]);
                            for (int32_t x = 128 + lane; x < gq.len[e]; x += 32) {      // nodes with more than 128 keys
                                const int32_t y = (int32_t)__ldg(pos16 + (size_t)gq.pbeg[e] + x) - seg0;
                                if (y >= 0 && y < seglen) acc[y] = fmaf(phi, __ldg(t_val + gq.beg[e] + x), acc[y]);
                            }
                            __syncwarp();
                        }
                    };
                    MaskPosGroup ga, gb;
                    fetch(0, ga);
                    for (int32_t e0 = 0; e0 < n; e0 += 8) {
                        if (e0 + 4 < n) fetch(e0 + 4, gb);
                        add(e0, ga);
                        if (e0 + 4 < n) {
                            if (e0 + 8 < n) fetch(e0 + 8, ga);
                            add(e0 + 4, gb);
                        }
                    }
                }
            }
            // the row's values of this segment, eight keys (16 bytes) per lane at a time; the accumulators are
            // cleared for the next row as they are read
            for (int32_t c8 = lane; c8 < seglen / 8; c8 += 32) {
                float4* a4 = reinterpret_cast<float4*>(acc + c8 * 8);
                const float4 x0 = a4[0], x1 = a4[1];
                a4[0] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                a4[1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(x0.x, x0.y), h1 = __floats2bfloat162_rn(x0.z, x0.w);
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(x1.x, x1.y), h3 = __floats2bfloat162_rn(x1.z, x1.w);
                uint4* dst = reinterpret_cast<uint4*>(mk_val + ((size_t)((off + seg0) / 8 + c8) * BQ + rr) * 8);
                *dst = make_uint4(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1),
                                  *reinterpret_cast<const uint32_t*>(&h2), *reinterpret_cast<const uint32_t*>(&h3));
            }
            __syncwarp();
        }
    }
}

// Dense rows of the mask for checking and export: out[x][j] = Mhat[rows[x]][j] (zeros elsewhere), one CTA per row.
__global__ void __launch_bounds__(256)
mask_rows_kernel(int32_t Nk, const int32_t* __restrict__ rows, const int32_t* __restrict__ mk_off,
                 const int32_t* __restrict__ mk_cnt, const int32_t* __restrict__ mk_key,
                 const __nv_bfloat16* __restrict__ mk_val, float* __restrict__ out)
{
    const int32_t r = rows[blockIdx.x];
    float* o = out + (size_t)blockIdx.x * Nk;
    for (int32_t j = threadIdx.x; j < Nk; j += 256) o[j] = 0.0f;
    __syncthreads();
    const int32_t blk = r / BQ, rr = r % BQ;
    const int32_t off = mk_off[blk], cnt = mk_cnt[blk];
    // padding entries repeat the last key with the value 0: skip an entry whose predecessor has the same key
    for (int32_t e = threadIdx.x; e < cnt; e += 256) {
        const int32_t j = mk_key[off + e];
        if (e > 0 && mk_key[off + e - 1] == j) continue;
        o[j] = __bfloat162float(mk_val[((size_t)((off + e) / 8) * BQ + rr) * 8 + ((off + e) & 7)]);
    }
}

// ---------------------------------------------------------------------------------------------------
// The attention kernel.  One CTA = 128 queries of one head; the block's keys come in tiles of 64.
//   warps 0-3, 4-7  two groups of row threads (one query = one tensor-memory lane each): a group multiplies the
//                   scores of every other tile by the mask, in place (fp32 scores -> bf16 pairs), and sums its rows
//   warp 8          issues S_t = Q K_t^T into one of three score buffers
//   warp 9          issues O += P_t V_t once the rows of tile t are masked, and frees the tile's stage and buffer
//   warps 10-13     producers: a quarter of every tile's key-feature and value rows each, by 16-byte async copies
// An instruction of the tensor pipe costs its issuing thread about fifty cycles, whatever its size, so the two
// products have a thread each; three score buffers let the first product run two tiles ahead of the masking.
// (A round trip to tensor memory is about 230 cycles and the hand-overs add several hundred per tile: what bounds
// the kernel is the length of that chain, not a pipe.)

template <int M> struct MhShape {
    static constexpr int D = 64;
    // key/value stages in flight: two CTAs' rings then leave the SM the larger part of its L1, which serves the mask
    // values and the rows that neighbouring keys share (eight stages were 8 % slower at the point cloud, 25 % at the grid)
    static constexpr int NS = M <= 32 ? 5 : 3;
    static constexpr int NB = 3;                          // score buffers
    static constexpr int V_BYTES = KT * 128;              // 64 value rows of 128 bytes, 128-byte swizzle
    static constexpr int K_BYTES = KT * M * 2;            // [M/8][KT keys][8] bf16: K-major, unswizzled
    static constexpr int STAGE = V_BYTES + K_BYTES;
    static constexpr int Q_BYTES = BQ * M * 2;            // [M/8][128 rows][8] bf16
    static constexpr int S_COLS = KT;                     // one score buffer; P (bf16 pairs) reuses its first half
    static constexpr int O_COL = NB * S_COLS;
    static constexpr int TMEM_COLS = 256;                 // 3 score buffers + the output accumulator
    static constexpr size_t SMEM = (size_t)NS * STAGE + Q_BYTES + 1024;
    static_assert(STAGE % 1024 == 0, "stages must keep the swizzle phase");
    static_assert(O_COL + D <= TMEM_COLS, "tensor memory");
};

constexpr int MH_THREADS = 448;

// two fp32 values in one 64-bit register: the packed multiply and add take one issue slot for both
__device__ __forceinline__ uint64_t pack_f32x2(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
constexpr int MH_ISSUER_S = 8, MH_ISSUER_O = 9, MH_PRODUCER0 = 10;

template <int M>
__global__ void __launch_bounds__(MH_THREADS, 2)
mhat_attention_kernel(int32_t G, int32_t nblocks, int32_t N, const int32_t* __restrict__ mk_off,
                      const int32_t* __restrict__ mk_cnt, const int32_t* __restrict__ mk_key,
                      const uint4* __restrict__ mk_val, const __nv_bfloat16* __restrict__ phiQ,
                      const __nv_bfloat16* __restrict__ phiK, const __nv_bfloat16* __restrict__ Vg,
                      __nv_bfloat16* __restrict__ out, float* __restrict__ den_out, int* __restrict__ error_word)
{
    using Sh = MhShape<M>;
    constexpr int NS = Sh::NS, NB = Sh::NB, D = Sh::D;
    extern __shared__ unsigned char smem_dyn[];
    // kv_full, kv_empty per stage; s_full, p_full per score buffer; acc_done; den_ready; one drain barrier per issuer
    __shared__ __align__(8) unsigned long long bars[2 * NS + 2 * NB + 4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float den_odd[BQ];                  // row sums of the odd tiles, handed to the first group

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t g = (int32_t)(blockIdx.x % (uint32_t)G);
    const int32_t blk = mk_cnt[nblocks + (int32_t)(blockIdx.x / (uint32_t)G)];   // blocks by decreasing key count
    const uint32_t stage_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* stage_generic = smem_dyn + (stage_base - smem_u32(smem_dyn));
    const uint32_t q_base = stage_base + (uint32_t)NS * Sh::STAGE;
    const uint32_t bar_base = smem_u32(bars);
    auto kv_full = [&](int s) { return bar_base + 8u * (uint32_t)s; };
    auto kv_empty = [&](int s) { return bar_base + 8u * (uint32_t)(NS + s); };
    auto s_full = [&](int b) { return bar_base + 8u * (uint32_t)(2 * NS + b); };
    auto p_full = [&](int b) { return bar_base + 8u * (uint32_t)(2 * NS + NB + b); };
    const uint32_t acc_done = bar_base + 8u * (uint32_t)(2 * NS + 2 * NB);
    const uint32_t den_ready = acc_done + 8u;
    const uint32_t drain_s = acc_done + 16u, drain_o = acc_done + 24u;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(kv_full(s), 128); mbar_init(kv_empty(s), 1); }
        for (int b = 0; b < NB; ++b) { mbar_init(s_full(b), 1); mbar_init(p_full(b), 4); }
        mbar_init(acc_done, 1);
        mbar_init(den_ready, 4);
        mbar_init(drain_s, 1);
        mbar_init(drain_o, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MH_ISSUER_S) tmem_alloc(&tmem_slot, (uint32_t)Sh::TMEM_COLS);
    // the block's queries in the K-major operand layout: 16-byte chunk c of row r at (c * 128 + r) * 16
    if (tid < BQ) {
        const int32_t row = blk * BQ + tid;
        const uint4* qp = reinterpret_cast<const uint4*>(phiQ + ((size_t)g * N + min(row, N - 1)) * M);
#pragma unroll
        for (int c = 0; c < M / 8; ++c) {
            const uint4 x = row < N ? __ldg(qp + c) : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(stage_generic + (size_t)NS * Sh::STAGE + ((size_t)c * BQ + tid) * 16) = x;
        }
    }
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem_base = tmem_slot;

    const int32_t off = mk_off[blk];
    const int32_t T = mk_cnt[blk] / KT;                   // key tiles of this block

    if (warp < 8) {
        // ------------------------------------------------------------ row threads: P = S * Mhat, row sums, epilogue
        const int grp = warp >> 2;                               // 0: even tiles, 1: odd tiles
        const int rr = (warp & 3) * 32 + lane;                   // row of the block = tensor-memory lane
        const int32_t row = blk * BQ + rr;
        const uint32_t lane_field = (uint32_t)((warp & 3) * 32) << 16;
        const uint4* mrow = mk_val + (size_t)(off / 8) * BQ + rr;       // chunk x of this row: mrow[x * BQ]
        uint64_t den2[2] = {0ull, 0ull};                         // row sums, four partial sums in two packed pairs
        uint4 mk[KT / 8];
        if (grp < T) {
#pragma unroll
            for (int c = 0; c < KT / 8; ++c) mk[c] = __ldg(mrow + (size_t)(grp * (KT / 8) + c) * BQ);
        }
        bool ok = true;
        int buf = grp;                                           // t % NB and the parity of t / NB, kept in step
        uint32_t par = 0u;
        for (int32_t t = grp; t < T; t += 2) {
            if (!mbar_wait(s_full(buf), par, &abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            fence_after_sync();
            const uint32_t s_addr = tmem_base + lane_field + (uint32_t)(buf * Sh::S_COLS);
#pragma unroll
            for (int c16 = 0; c16 < KT / 16; ++c16) {
                uint32_t sv[16];
                tmem_ld16(s_addr + (uint32_t)(c16 * 16), sv);
                uint32_t pw[8];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint4 mm = mk[2 * c16 + h];
                    const uint32_t mw[4] = {mm.x, mm.y, mm.z, mm.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        // two masked scores at a time; the denominator adds them in fp32, before the rounding to bf16
                        const uint64_t p2 = mul_f32x2(pack_f32x2(sv[8 * h + 2 * e], sv[8 * h + 2 * e + 1]),
                                                      pack_f32x2(mw[e] << 16, mw[e] & 0xffff0000u));
                        den2[e & 1] = add_f32x2(den2[e & 1], p2);
                        float p0, p1;
                        unpack_f32x2(p2, p0, p1);
                        const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
                        pw[4 * h + e] = *reinterpret_cast<const uint32_t*>(&pb);
                    }
                }
                tmem_st8(s_addr + (uint32_t)(c16 * 8), pw);
            }
            // this group's next tile: its mask values travel while the products run
            if (t + 2 < T) {
#pragma unroll
                for (int c = 0; c < KT / 8; ++c) mk[c] = __ldg(mrow + (size_t)((t + 2) * (KT / 8) + c) * BQ);
            }
            tmem_st_wait();
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full(buf));
            buf += 2;
            if (buf >= NB) { buf -= NB; par ^= 1u; }
        }
        float den;
        {
            float d0, d1, d2, d3;
            unpack_f32x2(den2[0], d0, d1);
            unpack_f32x2(den2[1], d2, d3);
            den = (d0 + d1) + (d2 + d3);
        }
        if (grp == 1) {
            // hand the odd tiles' row sums to the first group, which writes the block's outputs
            den_odd[rr] = den;
            __syncwarp();
            if (lane == 0) mbar_arrive(den_ready);
        } else {
            if (ok && !mbar_wait(den_ready, 0u, &abort_flag)) ok = false;
            den += den_odd[rr];
            if (ok && T > 0) ok = mbar_wait(acc_done, 0u, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            fence_after_sync();
            const bool live = row < N;
            const float inv = (den != 0.0f) ? 1.0f / den : 0.0f;
            if (live && ok && den_out) den_out[(size_t)g * N + row] = den;
            __nv_bfloat16* orow = out + ((size_t)g * N + row) * D;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 16) {
                uint32_t r[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) r[e] = 0u;
                if (ok && T > 0) tmem_ld16(tmem_base + lane_field + (uint32_t)(Sh::O_COL + c0), r);
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
        }
    } else if (warp >= MH_PRODUCER0) {
        // ------------------------------------------------------------ producers: warp w takes keys 16w .. 16w+15 of every tile
        // Lanes x and x + 16 hold key x of the warp's sixteen.  Rows travel as 16-byte pieces.  Value rows (128
        // bytes): eight consecutive lanes copy one row, piece c of tile row r going to r * 128 + ((c ^ (r & 7)) * 16),
        // the 128-byte swizzle the second product's operand descriptor names.  Key-feature rows: piece c of key y
        // goes to (c * 64 + y) * 16; lanes 0-15 copy the even pieces, lanes 16-31 the odd ones.  A warp's copies of
        // one tile arrive on the stage's barrier by themselves as they land (the barrier counts all 128 producer
        // threads), so a producer never waits for its own copies; the issuing threads run the proxy fence between
        // their wait on that barrier and the product that reads the stage.  Key indices are read three tiles ahead.
        const int pw = warp - MH_PRODUCER0;
        const __nv_bfloat16* Kg = phiK + (size_t)g * N * M;
        const __nv_bfloat16* Vh = Vg + (size_t)g * N * D;
        const int ky = pw * 16 + (lane & 15);                   // this lane's key within the tile
        const int vc = lane & 7;                                // its piece of a value row
        bool ok = true;
        const int32_t* kp = mk_key + off + ky;
        int32_t k1 = T > 0 ? __ldg(kp) : 0, k2 = T > 1 ? __ldg(kp + KT) : 0, k3 = T > 2 ? __ldg(kp + 2 * KT) : 0;
        for (int32_t t = 0; t < T; ++t) {
            const int s = t % NS;
            const int32_t k = k1;
            k1 = k2; k2 = k3;
            if (t + 3 < T) k3 = __ldg(kp + (size_t)(t + 3) * KT);
            if (t >= NS && !mbar_wait(kv_empty(s), (uint32_t)(t / NS - 1) & 1u, &abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t v_st = stage_base + (uint32_t)s * Sh::STAGE, k_st = v_st + Sh::V_BYTES;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int y = (lane >> 3) + 4 * i;              // key of the warp's sixteen
                const int32_t kv = __shfl_sync(0xffffffffu, k, y);
                const int r = pw * 16 + y;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                             ::"r"(v_st + (uint32_t)(r * 128 + ((vc ^ (r & 7)) << 4))), "l"(Vh + (size_t)kv * D + vc * 8) : "memory");
            }
#pragma unroll
            for (int c2 = 0; c2 < M / 16; ++c2) {
                const int c = 2 * c2 + (lane >> 4);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                             ::"r"(k_st + (uint32_t)(c * KT + ky) * 16u), "l"(Kg + (size_t)k * M + c * 8) : "memory");
            }
            // every thread's arrival on the stage's barrier happens when its own copies above have landed
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(kv_full(s)) : "memory");
        }
        asm volatile("cp.async.wait_all;" ::: "memory");         // also after giving up: no copy outlives the CTA
    } else if (warp == MH_ISSUER_S) {
        // ------------------------------------------------------------ S_t = Q K_t^T (the whole warp runs the loop in step)
        constexpr uint32_t idesc_s = instr_desc(KT, false, false);     // both operands K-major
        bool ok = true;
        int buf = 0;
        for (int32_t t = 0; t < T; ++t) {
            const int s = t % NS;
            if (!__all_sync(0xffffffffu, mbar_wait(kv_full(s), (uint32_t)(t / NS) & 1u, &abort_flag))) { ok = false; break; }
            // the score buffer is free once the second product of the tile three back, which read its P, is complete
            if (t >= NB && !__all_sync(0xffffffffu, mbar_wait(kv_empty((t - NB) % NS), (uint32_t)((t - NB) / NS) & 1u, &abort_flag))) { ok = false; break; }
            fence_async_smem();                                        // the copies wrote through the generic proxy
            fence_after_sync();
            const uint32_t k_st = stage_base + (uint32_t)s * Sh::STAGE + Sh::V_BYTES;
#pragma unroll
            for (int k = 0; k < M / 16; ++k) {
                const uint64_t ad = operand_desc(q_base + (uint32_t)k * 2u * (BQ * 16), BQ * 16, 128);
                const uint64_t bd = operand_desc(k_st + (uint32_t)k * 2u * (KT * 16), KT * 16, 128);
                mma_bf16_ss(tmem_base + (uint32_t)(buf * Sh::S_COLS), ad, bd, idesc_s, k > 0 ? 1u : 0u);
            }
            mma_commit(s_full(buf));
            if (++buf == NB) buf = 0;
        }
        if (!ok) {
            mma_commit(drain_s);
            mbar_drain(drain_s, 0u, 20000000ll);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ O += P_t V_t (the whole warp runs the loop in step)
        constexpr uint32_t idesc_o = instr_desc(D, false, true);       // V is MN-major (rows of d values)
        bool ok = true;
        int buf = 0;
        uint32_t par = 0u;
        for (int32_t t = 0; t < T; ++t) {
            const int s = t % NS;
            if (!__all_sync(0xffffffffu, mbar_wait(p_full(buf), par, &abort_flag))) { ok = false; break; }
            // (complete since the first product of this tile ran; waited on here for this thread's own view of the stage)
            if (!__all_sync(0xffffffffu, mbar_wait(kv_full(s), (uint32_t)(t / NS) & 1u, &abort_flag))) { ok = false; break; }
            fence_async_smem();
            fence_after_sync();
            const uint32_t p_op = tmem_base + (uint32_t)(buf * Sh::S_COLS);
            const uint32_t v_st = stage_base + (uint32_t)s * Sh::STAGE;
#pragma unroll
            for (int ks = 0; ks < KT / 16; ++ks) {
                const uint64_t bd = swizzled_desc(v_st + (uint32_t)ks * 2048u, 1024u, 1024u, 2);
                mma_bf16_ts(tmem_base + (uint32_t)Sh::O_COL, p_op + (uint32_t)ks * 8u, bd, idesc_o, (t > 0 || ks > 0) ? 1u : 0u);
            }
            mma_commit(kv_empty(s));                                   // frees the stage and the score buffer
            if (++buf == NB) { buf = 0; par ^= 1u; }
        }
        if (ok && T > 0) mma_commit(acc_done);
        if (!ok) {
            mma_commit(drain_o);
            mbar_drain(drain_o, 0u, 20000000ll);
        }
        __syncwarp();
    }

    fence_before_sync();
    __syncthreads();
    if (warp == MH_ISSUER_S) tmem_dealloc(tmem_base, (uint32_t)Sh::TMEM_COLS);
    if (tid == 0 && abort_flag) atomicExch(error_word, 1);
}

}  // namespace

void grf_mask_invalidate(grf_features* feat) { feat->mask.ready = false; feat->mask.structure_ready = false; }
// Phi's and Psi's values changed, their structure did not (re-modulation): key lists and positions stay
void grf_mask_values_stale(grf_features* feat) { feat->mask.ready = false; }

namespace {
// The values of the mask from the present values of Phi and Psi^T, over key lists (and positions) that are in place.
int launch_mask_values(grf_ctx* ctx, grf_features* feat, bool by_position)
{
    grf_mask_dev& K = feat->mask;
    const int32_t N = feat->phi.rows, Nk = feat->psi.rows, nblocks = feat->plan_blocks;
    const size_t words = ((size_t)Nk + 31) / 32;
    if (by_position) {
        const size_t smem_acc = (size_t)MASK_WARPS * MASK_SEG * sizeof(float);
        GRF_CUDA_TRY(cudaFuncSetAttribute(mask_values_pos_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_acc));
        grf_launch_scope scope(ctx, 8);
        mask_values_pos_kernel<<<nblocks * (BQ / MASK_ROWS), MASK_WARPS * 32, smem_acc, ctx->stream>>>(
            N, (const int32_t*)feat->phi.rowptr.ptr, (const int32_t*)feat->phi.col.ptr, (const float*)feat->phi.val.ptr,
            (const int32_t*)K.phi_pos.ptr, (const int32_t*)feat->psit.rowptr.ptr, (const float*)feat->psit.val.ptr,
            (const unsigned short*)K.pos16.ptr, (const int32_t*)K.off.ptr, (const int32_t*)K.cnt.ptr,
            (__nv_bfloat16*)K.val.ptr);
    } else {
        const size_t smem_values = ((words + 1) & ~(size_t)1) * 8 + (size_t)MASK_WARPS * MASK_SEG * sizeof(float);
        GRF_CUDA_TRY(cudaFuncSetAttribute(mask_values_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_values));
        grf_launch_scope scope(ctx, 8);
        mask_values_kernel<<<nblocks * (BQ / MASK_ROWS), MASK_WARPS * 32, smem_values, ctx->stream>>>(
            N, Nk, (const int32_t*)feat->phi.rowptr.ptr, (const int32_t*)feat->phi.col.ptr, (const float*)feat->phi.val.ptr,
            (const int32_t*)feat->psit.rowptr.ptr, (const int32_t*)feat->psit.col.ptr, (const float*)feat->psit.val.ptr,
            (const int32_t*)K.off.ptr, (const int32_t*)K.cnt.ptr, (const uint32_t*)K.bits.ptr, (__nv_bfloat16*)K.val.ptr);
    }
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}
}  // namespace

void grf_mask_release(grf_features* feat)
{
    grf_mask_dev& K = feat->mask;
    grf_buf_release(&K.off); grf_buf_release(&K.cnt); grf_buf_release(&K.key); grf_buf_release(&K.bits); grf_buf_release(&K.val); grf_buf_release(&K.node_off);
    grf_buf_release(&K.blk_pos); grf_buf_release(&K.pos16); grf_buf_release(&K.phi_pos);
    K.ready = false;
    K.structure_ready = false;
}

extern "C" int grf_features_materialise(grf_ctx* ctx, grf_features* feat)
{
    if (!ctx || !feat) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    grf_mask_dev& K = feat->mask;
    K.ready = false;
    if (K.structure_ready && feat->plan_ready && !feat->plan_stale) {
        // same walks, new coefficients: the key lists and positions still hold
        GRF_TRY(launch_mask_values(ctx, feat, K.by_position));
        K.ready = true;
        return GRF_OK;
    }
    K.structure_ready = false;
    const int32_t N = feat->phi.rows, Nk = feat->psi.rows;
    const size_t words = ((size_t)Nk + 31) / 32;
    // the values kernel keeps the key bitmap, its prefix counts and the accumulators in shared memory
    const size_t smem_values = ((words + 1) & ~(size_t)1) * 8 + (size_t)MASK_WARPS * MASK_SEG * sizeof(float);
    if (smem_values > 200 * 1024) return GRF_ERR_TOO_LARGE;
    GRF_TRY(grf_ensure_block_plan(ctx, feat, false));         // the node lists only
    if (!feat->plan_ready) return GRF_ERR_TOO_LARGE;          // rows of a block share too little
    const int32_t nblocks = feat->plan_blocks;
    GRF_TRY(grf_buf_reserve(&K.cnt, sizeof(int32_t) * 2 * (size_t)nblocks));
    GRF_TRY(grf_buf_reserve(&K.off, sizeof(int32_t) * ((size_t)nblocks + 1)));
    GRF_TRY(grf_buf_reserve(&K.bits, sizeof(uint32_t) * 2 * (size_t)nblocks * words));
    GRF_CUDA_TRY(cudaFuncSetAttribute(mask_bitmap_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(words * 4)));
    {
        grf_launch_scope scope(ctx, 8);
        mask_bitmap_kernel<<<nblocks, MASK_BITMAP_THREADS, words * 4, ctx->stream>>>(
            Nk, (const int32_t*)feat->plan_off.ptr, (const int32_t*)feat->plan_cnt.ptr, (const int32_t*)feat->plan_col.ptr,
            (const int32_t*)feat->psit.rowptr.ptr, (const int32_t*)feat->psit.col.ptr, (uint32_t*)K.bits.ptr,
            (int32_t*)K.cnt.ptr);
    }
    GRF_CUDA_TRY(cudaGetLastError());
    GRF_TRY(grf_exclusive_scan(ctx, (const int32_t*)K.cnt.ptr, (int32_t*)K.off.ptr, nblocks, 1));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 5, (const int32_t*)K.off.ptr + nblocks, sizeof(int32_t),
                                 cudaMemcpyDeviceToHost, ctx->stream));
    // where every node's key positions will start (per block, then over the blocks), and the longest key list
    const int32_t R = feat->psit.rows;
    // (buffers whose size follows the sample grow with head-room: resampling changes the sizes a little every time,
    // and a reallocation stalls the device)
    auto reserve_with_headroom = [](grf_buf* b, size_t bytes) {
        return b->bytes >= bytes ? GRF_OK : grf_buf_reserve(b, bytes + bytes / 8 + 256);
    };
    GRF_TRY(reserve_with_headroom(&K.node_off, sizeof(int32_t) * (size_t)(feat->plan_entries > 0 ? feat->plan_entries : 1)));
    GRF_TRY(grf_buf_reserve(&K.blk_pos, sizeof(int32_t) * (2 * (size_t)nblocks + 2)));
    int32_t* blk_pos = (int32_t*)K.blk_pos.ptr;                 // offsets [nblocks + 1], totals [nblocks], longest list
    GRF_CUDA_TRY(cudaMemsetAsync(blk_pos + 2 * nblocks + 1, 0, sizeof(int32_t), ctx->stream));
    {
        grf_launch_scope scope(ctx, 8);
        mask_node_offsets_kernel<<<nblocks, 256, 0, ctx->stream>>>(
            (const int32_t*)feat->plan_off.ptr, (const int32_t*)feat->plan_cnt.ptr, (const int32_t*)feat->plan_col.ptr,
            (const int32_t*)feat->psit.rowptr.ptr, (int32_t*)K.node_off.ptr, blk_pos + nblocks + 1,
            (const int32_t*)K.cnt.ptr, blk_pos + 2 * nblocks + 1);
    }
    GRF_TRY(grf_exclusive_scan(ctx, blk_pos + nblocks + 1, blk_pos, nblocks, 1));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 6, blk_pos + nblocks, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    GRF_CUDA_TRY(cudaMemcpyAsync(ctx->pinned + 7, blk_pos + 2 * nblocks + 1, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    GRF_CUDA_TRY(cudaStreamSynchronize(ctx->stream));          // the sizes of the key lists are known only now
    const int64_t entries = ctx->pinned[5];
    if (entries < 0) return GRF_ERR_TOO_LARGE;
    // positions are looked up once per (block, node) when they fit 16 bits, their number fits an int32 (a negative
    // total means it did not) and both bitmaps fit shared memory; otherwise once per (row, node)
    const int64_t total_pos = ctx->pinned[6];
    const size_t smem_pos = (words + ((size_t)R + 31) / 32) * 8;
    const bool by_position = total_pos >= 0 && ctx->pinned[7] <= 65535 && smem_pos <= 96 * 1024;
    const size_t val_bytes = (size_t)entries * BQ * sizeof(__nv_bfloat16);
    if (val_bytes > ((size_t)8 << 30)) return GRF_ERR_TOO_LARGE;   // no locality: the S/z route serves this object
    if (K.key.bytes < (size_t)entries * 4) GRF_TRY(grf_buf_reserve(&K.key, ((size_t)entries + (size_t)entries / 8 + 64) * 4));
    if (K.val.bytes < val_bytes) GRF_TRY(grf_buf_reserve(&K.val, val_bytes + val_bytes / 8 + 256));
    {
        grf_launch_scope scope(ctx, 8);
        mask_list_kernel<<<nblocks, 256, 0, ctx->stream>>>(Nk, (const uint32_t*)K.bits.ptr, (const int32_t*)K.off.ptr,
                                                           (const int32_t*)K.cnt.ptr, (int32_t*)K.key.ptr);
    }
    {
        grf_launch_scope scope(ctx, 8);
        mask_order_kernel<<<grf_ceil_div(nblocks, 256), 256, 0, ctx->stream>>>(nblocks, (int32_t*)K.cnt.ptr);
    }
    if (by_position) {
        GRF_TRY(reserve_with_headroom(&K.pos16, sizeof(unsigned short) * (size_t)(total_pos + 1)));
        GRF_TRY(reserve_with_headroom(&K.phi_pos, sizeof(int32_t) * (size_t)(feat->phi.nnz + 1)));
        GRF_CUDA_TRY(cudaFuncSetAttribute(mask_positions_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_pos));
        {
            grf_launch_scope scope(ctx, 8);
            mask_positions_kernel<<<nblocks * MASK_POS_PARTS, 256, smem_pos, ctx->stream>>>(
                N, Nk, R, (const int32_t*)feat->phi.rowptr.ptr, (const int32_t*)feat->phi.col.ptr,
                (const int32_t*)feat->plan_off.ptr, (const int32_t*)feat->plan_cnt.ptr, (const int32_t*)feat->plan_col.ptr,
                (const int32_t*)feat->psit.rowptr.ptr, (const int32_t*)feat->psit.col.ptr, (const uint32_t*)K.bits.ptr,
                (const int32_t*)K.node_off.ptr, blk_pos, (unsigned short*)K.pos16.ptr, (int32_t*)K.phi_pos.ptr);
        }
    }
    GRF_TRY(launch_mask_values(ctx, feat, by_position));
    GRF_CUDA_TRY(cudaGetLastError());
    K.blocks = nblocks;
    K.entries = entries;
    K.by_position = by_position;
    K.structure_ready = true;
    K.ready = true;
    return GRF_OK;
}

extern "C" int grf_mask_stats(const grf_features* feat, int32_t* blocks, int64_t* key_entries, int64_t* bytes)
{
    if (!feat || !feat->mask.ready) return GRF_ERR_INVALID;
    if (blocks) *blocks = feat->mask.blocks;
    if (key_entries) *key_entries = feat->mask.entries;
    if (bytes) *bytes = feat->mask.entries * (int64_t)(BQ * sizeof(__nv_bfloat16) + sizeof(int32_t));
    return GRF_OK;
}

extern "C" int grf_mask_rows(grf_ctx* ctx, const grf_features* feat, int32_t n, const int32_t* rows, float* out)
{
    if (!ctx || !feat || n <= 0 || !rows || !out) return GRF_ERR_INVALID;
    if (!feat->mask.ready) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    const grf_mask_dev& K = feat->mask;
    {
        grf_launch_scope scope(ctx, 8);
        mask_rows_kernel<<<n, 256, 0, ctx->stream>>>(feat->psi.rows, rows, (const int32_t*)K.off.ptr, (const int32_t*)K.cnt.ptr,
                                                     (const int32_t*)K.key.ptr, (const __nv_bfloat16*)K.val.ptr, out);
    }
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

template <int M>
static int launch_mhat(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, const void* phiQ, const void* phiK,
                       const void* V, void* out, float* den_out)
{
    using Sh = MhShape<M>;
    const grf_mask_dev& K = feat->mask;
    // at most two CTAs per SM: each holds half of the SM's tensor memory
    const size_t smem = Sh::SMEM > 78 * 1024 ? Sh::SMEM : 78 * 1024;
    GRF_CUDA_TRY(cudaFuncSetAttribute(mhat_attention_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    {
        grf_launch_scope scope(ctx, 9);
        mhat_attention_kernel<M><<<(unsigned)K.blocks * (unsigned)G, MH_THREADS, smem, ctx->stream>>>(
            G, K.blocks, N, (const int32_t*)K.off.ptr, (const int32_t*)K.cnt.ptr, (const int32_t*)K.key.ptr,
            (const uint4*)K.val.ptr, (const __nv_bfloat16*)phiQ, (const __nv_bfloat16*)phiK, (const __nv_bfloat16*)V,
            (__nv_bfloat16*)out, den_out, ctx->error_word);
    }
    return cudaGetLastError() == cudaSuccess ? GRF_OK : GRF_ERR_CUDA;
}

extern "C" int grf_masked_attn_mhat(grf_ctx* ctx, const grf_features* feat, int32_t G, int32_t N, int32_t m, int32_t d,
                                    int dtype, const void* phiQ, const void* phiK, const void* V, void* out, float* den_out)
{
    if (!ctx || !feat || !phiQ || !phiK || !V || !out || G <= 0 || N <= 0) return GRF_ERR_INVALID;
    if (dtype != GRF_DTYPE_BF16 || d != 64 || (m != 16 && m != 32 && m != 64)) return GRF_ERR_INVALID;
    if (!feat->mask.ready || feat->phi.rows != N || feat->psi.rows != N) return GRF_ERR_INVALID;
    if ((int64_t)G * N > 0x7fffffffll || (int64_t)G * feat->mask.blocks > 0x7fffffffll) return GRF_ERR_TOO_LARGE;
    if (((uintptr_t)phiQ | (uintptr_t)phiK | (uintptr_t)V | (uintptr_t)out) & 15u) return GRF_ERR_INVALID;
    GRF_CUDA_TRY(cudaSetDevice(ctx->device));
    if (m == 16) return launch_mhat<16>(ctx, feat, G, N, phiQ, phiK, V, out, den_out);
    if (m == 32) return launch_mhat<32>(ctx, feat, G, N, phiQ, phiK, V, out, den_out);
    return launch_mhat<64>(ctx, feat, G, N, phiQ, phiK, V, out, den_out);
}
