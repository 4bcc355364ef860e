// Gram matrices S = X^T X of the refresh (the orthonormalisations of Section 3.5 and the small SVD) on the
// integer tensor cores, exact.
//
// X (rows x k, FP32) has a condition number of 10^4 and more, so S must be known to about 1e-10 relative to
// |x_i| |x_j| before a Cholesky factorisation can use it; FP32 accumulation is far from that, and the FP64
// tensor path that does it directly runs at 1/70 of the 8-bit integer rate.  Integer arithmetic gives the same
// result without rounding at all:
//   1. every column j is scaled by a power of two to |y| <= 1/2 (exponent e_j from the column's largest entry);
//   2. y is cut into six signed 7-bit digits, y = sum_s d_s 2^(-7(s+1)), d_s in [-64, 64] (each digit the
//      rounded remainder of the previous one, all steps exact in FP32); what is dropped is below 2^-43;
//   3. for every pair of digit planes (s, t) with s + t <= 5 the products D_s^T D_t are integer matrix products,
//      |d_s d_t| <= 2^12, summed over at most 2^15 rows and the at most six pairs of one level s + t: below 2^31,
//      so the INT32 accumulators of tcgen05.mma.kind::i8 hold them exactly;
//   4. S_ij = 2^(e_i + e_j) sum_level 2^(-7(level + 2)) A_level(i, j), formed in FP64 in the epilogue.
// The digit planes are stored transposed (k x rows, the row index of X contiguous), which is the K-major operand
// layout the MMAs want; one tile of the product loads the six planes of its rows and columns once per 64 rows of
// X and forms all 21 pair products from them.  An MMA reads its whole A operand from shared memory again, so 21
// narrow MMAs (N = 64) would keep the tensor pipe waiting for shared memory more than half of the time.  The
// products of one A plane s with the B planes t = 0 .. 5 - s go to consecutive levels s + t, i.e. to consecutive
// accumulators: stacked along N they are ONE wide MMA.  In a CTA pair the first half of an MMA's N rows comes from
// the leader's shared memory and the second half from its peer's, at the same offsets, so the leader keeps the B
// planes {0, 1, 4} and the peer {2, 3, 5} (each for all 64 columns of the tile): eight MMAs per 32 rows of X do
// the work of 21 (see the table at the MMA loop); the columns past the sixth level take products nobody reads.
//
// Kernels: gram_slabmax_kernel + gram_colexp_kernel (column exponents), gram_digits_kernel (digit planes), gram_i8_kernel (CTA pairs,
// persistent over a tile table: producer / MMA / epilogue warps as in the BF16 GEMM), then the existing
// gram_reduce_kernel adds the row chunks in fixed order and mirrors the upper triangle.
#include "tsr_internal.h"
#include "tsr_umma.cuh"

namespace tsr {

constexpr int GI_DIGITS = 6;
constexpr int GI_BN = 64;                    // tile: 256 (pair) x 64 outputs
constexpr int GI_BK = 64;                    // rows of X per stage (64-byte operand rows, 64-byte swizzle)
constexpr int GI_STAGES = 3;
constexpr int GI_A_BYTES = UM_BM * GI_BK;            // one digit plane of this CTA's 128 rows: 8 KB
constexpr int GI_B_BYTES = GI_BN * GI_BK;            // one digit plane of the tile's 64 columns: 4 KB
constexpr int GI_B_SLOTS = 3;                        // B planes a CTA keeps: {0, 1, 4} (leader) or {2, 3, 5} (peer)
constexpr int GI_STAGE_BYTES = GI_DIGITS * GI_A_BYTES + GI_B_SLOTS * GI_B_BYTES;   // 60 KB
constexpr int GI_BAR_OFFSET = GI_STAGES * GI_STAGE_BYTES;
constexpr int GI_NBARS = 2 * GI_STAGES + 2;
constexpr int GI_SMEM = GI_BAR_OFFSET + GI_NBARS * 8 + 64 + 1024;
constexpr int GI_THREADS = 384;
constexpr uint32_t GI_TMEM_COLS = 512;       // six levels of 64 INT32 columns (384) + 128 columns of products past the sixth level

// ---------------------------------------------------------------------------------------------------------
// Column exponents: e_j = smallest integer with max_i |x_ij| <= 2^(e_j - 1); 0 for an all-zero column.
// Two steps without atomics: gram_slabmax_kernel writes the column maxima of every slab of RG_ROWS rows (into the
// Gram partial-sum buffer, which is free until the products are stored), gram_colexp_kernel reduces them.
// A non-finite entry flags the block.
// ---------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gram_slabmax_kernel(const RefreshDev *__restrict__ rd, const RowItem *__restrict__ items, int side, int src_sel)
{
    const RowItem it = items[blockIdx.y];
    const RefreshDev &d = rd[it.block];
    const int k = d.k, rows = side ? d.n : d.m;
    const int c0 = blockIdx.x * 32;
    if (c0 >= k) return;
    const float *__restrict__ X = d.buf[src_sel];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int col = c0 + tx;
    float mx = 0.f;
    bool bad = false;
    if (col < k) {
        float v[RG_ROWS / 8];
#pragma unroll
        for (int u = 0; u < RG_ROWS / 8; ++u) {
            const int row = it.row0 + ty + 8 * u;
            v[u] = (row < rows) ? fabsf(X[(int64_t)row * k + col]) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < RG_ROWS / 8; ++u) {
            if (!(v[u] <= 3.0e38f)) bad = true;     // NaN or Inf
            mx = fmaxf(mx, v[u]);
        }
    }
    __shared__ float s_mx[8][33];
    __shared__ int s_bad;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    s_mx[ty][tx] = mx;
    if (bad) s_bad = 1;
    __syncthreads();
    if (ty == 0 && col < k) {
        float m = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) m = fmaxf(m, s_mx[w][tx]);
        ((float *)d.gpart)[(int64_t)(it.row0 / RG_ROWS) * k + col] = m;
    }
    if (threadIdx.x == 0 && s_bad) atomicMax(d.status, (int)TSR_ERR_NONFINITE);
}

__global__ void __launch_bounds__(256)
gram_colexp_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int side)
{
    const RefreshDev &d = rd[list[blockIdx.y]];
    const int k = d.k, rows = side ? d.n : d.m;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int col = blockIdx.x * 32 + tx;
    if (blockIdx.x * 32 >= k) return;
    const int nslab = (rows + RG_ROWS - 1) / RG_ROWS;
    const float *__restrict__ sm = (const float *)d.gpart;
    float m = 0.f;
    if (col < k)
        for (int sl = ty; sl < nslab; sl += 8) m = fmaxf(m, sm[(int64_t)sl * k + col]);
    __shared__ float s_mx[8][33];
    s_mx[ty][tx] = m;
    __syncthreads();
    if (ty == 0 && col < k) {
#pragma unroll
        for (int w = 1; w < 8; ++w) m = fmaxf(m, s_mx[w][tx]);
        int e = 0;
        if (m > 0.f && m <= 3.0e38f) {
            (void)frexpf(m, &e);            // m = f 2^e with f in [1/2, 1)  =>  m < 2^e
            e += 1;                         // m 2^-e < 1/2
        }
        d.col_exp[col] = e;
    }
}

// ---------------------------------------------------------------------------------------------------------
// Digit planes.  planes[s][col][row] (INT8, row pitch ldp) for a slab of 128 rows x 32 columns per CTA:
// the tile is read row-wise, transposed through shared memory, and every thread writes 16 consecutive rows of
// one column as one 16-byte word per plane.
// ---------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gram_digits_kernel(const RefreshDev *__restrict__ rd, const RowItem *__restrict__ items, int side, int src_sel)
{
    const RowItem it = items[blockIdx.y];
    const RefreshDev &d = rd[it.block];
    const int k = d.k, rows = side ? d.n : d.m;
    const int c0 = blockIdx.x * 32;
    if (c0 >= k) return;
    const float *__restrict__ X = d.buf[src_sel];
    __shared__ float tile[RG_ROWS][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < RG_ROWS; i += 8) {
        const int row = it.row0 + i, col = c0 + tx;
        tile[i][tx] = (row < rows && col < k) ? X[(int64_t)row * k + col] : 0.f;
    }
    __syncthreads();
    const int c = threadIdx.x >> 3, g = threadIdx.x & 7;      // column of the tile, group of 16 rows
    const int col = c0 + c;
    if (col >= k) return;
    const int row_first = it.row0 + 16 * g;
    if (row_first >= d.ldp) return;                            // past the padded row count: nothing to write
    const float scale = ldexpf(1.0f, 7 - d.col_exp[col]);      // y 2^7 = x 2^(7 - e)
    uint32_t w[GI_DIGITS][4];
#pragma unroll
    for (int s = 0; s < GI_DIGITS; ++s)
#pragma unroll
        for (int u = 0; u < 4; ++u) w[s][u] = 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float r = tile[16 * g + i][c] * scale;                 // |r| <= 64 (rows past the end are zero)
        if (!(fabsf(r) <= 64.f)) r = 0.f;                      // a non-finite entry (the block is flagged already)
#pragma unroll
        for (int s = 0; s < GI_DIGITS; ++s) {
            // round to nearest even by adding 1.5 * 2^23: the sum's low mantissa bits are the integer in two's
            // complement (|r| <= 64), and taking the constant off again gives it back as a float -- the same value
            // as rintf(r), without the conversion unit
            const float t = __fadd_rn(r, 12582912.f);
            const float dgt = __fadd_rn(t, -12582912.f);       // in [-64, 64]
            w[s][i >> 2] |= (__float_as_uint(t) & 0xffu) << (8 * (i & 3));
            r = (r - dgt) * 128.f;                             // exact: the remainder, |.| <= 1/2, scaled by 2^7
        }
    }
#pragma unroll
    for (int s = 0; s < GI_DIGITS; ++s) {
        int8_t *dst = d.planes + ((int64_t)s * k + col) * d.ldp + row_first;
        *(uint4 *)dst = make_uint4(w[s][0], w[s][1], w[s][2], w[s][3]);
    }
}

// ---------------------------------------------------------------------------------------------------------
// The integer products.  Shared-memory matrix descriptor of a K-major operand tile written by TMA with 64-byte
// rows and the 64-byte swizzle: 8-row groups are 512 bytes apart.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t umma_desc_sw64(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(512 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)4 << 61;
    return d;
}
// Instruction descriptor: signed 8-bit operands, both K-major, INT32 accumulator, M = 256 (CTA pair), N columns.
__host__ __device__ constexpr uint32_t gi_idesc(int n) { return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24); }

__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// probs[b].tmA / tmB: the digit planes of block b as a (6 k) x rows INT8 matrix (plane s starts at row s k), boxes of
// 64 bytes x 128 rows and 64 bytes x 32 rows (two of them per B plane).  A tile: rows m0 .. m0 + 255 and columns n0 .. n0 + 63 of S, the
// rows [64 kb0, 64 kb1) of X; it writes its part of the chunk's partial sum (FP64, row pitch k).
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GI_THREADS, 1)
gram_i8_kernel(const UmmaProblem *__restrict__ probs, const UmmaTile *__restrict__ tiles, int num_tiles, long long budget_in,
               int32_t *__restrict__ status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + GI_BAR_OFFSET);
    uint64_t *bar_full = bars, *bar_empty = bars + GI_STAGES;
    uint64_t *bar_acc_full = bars + 2 * GI_STAGES, *bar_acc_empty = bar_acc_full + 1;
    uint32_t *tmem_slot = (uint32_t *)(bars + GI_NBARS);
    __shared__ int s_timeout;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long budget = budget_in > 0 ? budget_in : UM_WAIT_CLOCKS;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, stride = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        s_timeout = 0;
        for (int s = 0; s < GI_STAGES; ++s) { mbar_init(smem_u32(bar_full + s), 1); mbar_init(smem_u32(bar_empty + s), 1); }
        mbar_init(smem_u32(bar_acc_full), 1);
        mbar_init(smem_u32(bar_acc_empty), 2 * 8);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1)
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(GI_TMEM_COLS)
                     : "memory");
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // the pair's permit to allocate is given up only once both CTAs hold their tensor memory
    if (warp == 1) asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;                   // stage and phase of the operand ring this thread fills next
            uint32_t ph = 0;
            bool ok = true;
            for (int t = pair; t < num_tiles && ok; t += stride) {
                const UmmaTile tile = tiles[t];
                const UmmaProblem *P = probs + tile.prob;
                const int k = P->M;
                for (int kb = tile.kb0; kb < tile.kb1; ++kb, s = (s + 1 == GI_STAGES ? 0 : s + 1), ph ^= (s == 0 ? 1u : 0u)) {
                    if (!mbar_wait(smem_u32(bar_empty + s), ph ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                    const uint32_t full = leader_addr(smem_u32(bar_full + s));
                    if (rank == 0) mbar_expect_tx(smem_u32(bar_full + s), 2u * (uint32_t)GI_STAGE_BYTES);
                    uint8_t *st = smem + s * GI_STAGE_BYTES;
#pragma unroll
                    for (int dg = 0; dg < GI_DIGITS; ++dg)
                        tma_load_2d_pair(smem_u32(st + dg * GI_A_BYTES), &P->tmA, full, kb * GI_BK,
                                         dg * k + tile.m0 + (int)rank * UM_BM);
#pragma unroll
                    for (int sl = 0; sl < GI_B_SLOTS; ++sl) {
                        const int dg = sl == 2 ? 4 + (int)rank : 2 * (int)rank + sl;     // leader {0, 1, 4}, peer {2, 3, 5}
                        uint8_t *dst = st + GI_DIGITS * GI_A_BYTES + sl * GI_B_BYTES;
                        tma_load_2d_pair(smem_u32(dst), &P->tmB, full, kb * GI_BK, dg * k + tile.n0);
                        tma_load_2d_pair(smem_u32(dst + GI_B_BYTES / 2), &P->tmB, full, kb * GI_BK, dg * k + tile.n0 + GI_BN / 2);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            uint32_t tc = 0;
            int s = 0;                   // stage and phase of the operand ring this thread consumes next
            uint32_t ph = 0;
            bool ok = true;
            for (int t = pair; t < num_tiles && ok; t += stride, ++tc) {
                const UmmaTile tile = tiles[t];
                if (!mbar_wait(smem_u32(bar_acc_empty), (tc & 1u) ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                tc_fence_after();
                for (int kb = tile.kb0; kb < tile.kb1; ++kb, s = (s + 1 == GI_STAGES ? 0 : s + 1), ph ^= (s == 0 ? 1u : 0u)) {
                    if (!mbar_wait(smem_u32(bar_full + s), ph, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_base = smem_u32(smem + s * GI_STAGE_BYTES);
                    const uint32_t b_base = a_base + GI_DIGITS * GI_A_BYTES;
                    const bool first_kb = (kb == tile.kb0);
                    // A plane s against the stacked B planes, accumulator columns from 64 s on (level s + t at 64 (s + t)):
                    //   N = 256 over slots 0, 1: leader's planes 0, 1 -> levels s, s + 1; peer's planes 2, 3 -> levels s + 2, s + 3
                    //   N = 128 over slot 2:     leader's plane 4 -> level s + 4; peer's plane 5 -> level s + 5
                    //   N = 128 over slot 0:     leader's plane 0 -> level s;     peer's plane 2 -> level s + 1 (used for s = 5 only)
                    // Levels past 5 fall into columns 384 .. 511, which are never read.  The two MMAs of s = 0 cover all six
                    // levels and start them afresh on the tile's first rows.
#pragma unroll
                    for (int k2 = 0; k2 < GI_BK / 32; ++k2) {
                        const uint32_t fresh = (first_kb && k2 == 0) ? 0u : 1u;
#pragma unroll
                        for (int da = 0; da < GI_DIGITS; ++da) {
                            const uint64_t adesc = umma_desc_sw64(a_base + da * GI_A_BYTES + k2 * 32);
                            const uint32_t d_tmem = tmem_base + (uint32_t)(da * GI_BN);
                            if (da < 5)
                                tc_mma_i8_pair(d_tmem, adesc, umma_desc_sw64(b_base + k2 * 32), gi_idesc(256), da == 0 ? fresh : 1u);
                            else
                                tc_mma_i8_pair(d_tmem, adesc, umma_desc_sw64(b_base + k2 * 32), gi_idesc(128), 1u);
                            if (da < 2)
                                tc_mma_i8_pair(d_tmem + 4 * GI_BN, adesc, umma_desc_sw64(b_base + 2 * GI_B_BYTES + k2 * 32), gi_idesc(128),
                                               da == 0 ? fresh : 1u);
                        }
                    }
                    tc_commit_pair(smem_u32(bar_empty + s));
                }
                tc_commit_pair(smem_u32(bar_acc_full));
            }
        }
    } else if (warp >= 4) {
        const int q = warp & 3, half = (warp - 4) >> 2;
        uint32_t tc = 0;
        bool ok = true;
        for (int t = pair; t < num_tiles && ok; t += stride, ++tc) {
            const UmmaTile tile = tiles[t];
            const UmmaProblem *__restrict__ P = probs + tile.prob;
            const int k = P->M;
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(bar_acc_full), tc & 1u, budget))) { note_timeout(&s_timeout, t); ok = false; break; }
            tc_fence_after();
            double acc[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) acc[j] = 0.0;
#pragma unroll
            for (int lv = 0; lv < GI_DIGITS; ++lv) {
                uint32_t v[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(lv * GI_BN + half * 32), v);
                const double wgt = ldexp(1.0, -7 * (lv + 2));
#pragma unroll
                for (int j = 0; j < 32; ++j) acc[j] = fma((double)(int)v[j], wgt, acc[j]);
            }
            tc_fence_before();
            if (lane == 0) mbar_arrive_leader(smem_u32(bar_acc_empty));
            const int row = tile.m0 + (int)rank * UM_BM + q * 32 + lane;
            const int col0 = tile.n0 + half * 32;
            if (row < k && col0 < k && col0 + 31 >= (row & ~7)) {     // the reduction reads 8 x 8 sub-tiles on or above the diagonal
                const int32_t *__restrict__ ce = P->col_exp;
                const int er = ce[row];
                double *out = (double *)P->out + (int64_t)tile.split * P->split_stride + (int64_t)row * k + col0;
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < k) out[j] = ldexp(acc[j], er + ce[col0 + j]);
            }
        }
    }
    if (s_timeout) __nanosleep(2000000);
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(GI_TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && s_timeout && status)
        for (int t = s_timeout - 1; t < num_tiles; t += stride) atomicMax(status + probs[tiles[t].prob].block, (int)TSR_ERR_TIMEOUT);
}

cudaError_t gram_i8_configure()
{
    return cudaFuncSetAttribute(gram_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GI_SMEM);
}

cudaError_t gram_i8_prepare(const RefreshDev *rd, const RowItem *items128, int nitems128, const int32_t *list, int nlist,
                            int side, int src_sel, int kmax, cudaStream_t stream)
{
    if (nitems128 <= 0 || nlist <= 0) return cudaSuccess;
    const int t = (kmax + 31) / 32;
    gram_slabmax_kernel<<<dim3(t, nitems128), 256, 0, stream>>>(rd, items128, side, src_sel);
    gram_colexp_kernel<<<dim3(t, nlist), 256, 0, stream>>>(rd, list, side);
    gram_digits_kernel<<<dim3(t, nitems128), 256, 0, stream>>>(rd, items128, side, src_sel);
    return cudaGetLastError();
}

cudaError_t gram_i8_launch(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms, long long wait_clocks,
                           int32_t *status, cudaStream_t stream)
{
    if (num_tiles <= 0) return cudaSuccess;
    const int pairs = num_tiles < num_sms / 2 ? num_tiles : num_sms / 2;
    gram_i8_kernel<<<2 * pairs, GI_THREADS, GI_SMEM, stream>>>(probs, tiles, num_tiles, wait_clocks, status);
    return cudaGetLastError();
}

}  // namespace tsr
