// Grouped, persistent BF16 GEMM on the 5th-generation tensor cores (tcgen05) for sm_100a.
//
//   D[M x N] = A[M x K] * B[N x K]^T     A, B BF16 with K contiguous, FP32 accumulation
//
// The grid is one CTA per SM, grouped into clusters of two (a CTA pair).  Every pair walks a
// device-resident tile table (tiles of all matrix blocks of a model share one launch; static
// round-robin over pairs).  A tile is 256 x BN outputs over a range of 64-wide K blocks: CTA c of
// the pair owns output rows 128 c .. 128 c + 127 and holds that half of the accumulator in its
// own tensor memory.  Roles inside each CTA:
//   warp 0    one lane issues the TMA loads (128-byte swizzled 64-wide K slices) of this CTA's
//             128 rows of A and of HALF of the tile's B rows into a ring of shared-memory stages;
//             the bytes of both CTAs complete on the LEADER's "full" mbarrier (its address is
//             mapped into the peer with mapa), so each SM ingests only half of B per K block.
//             No load uses cluster multicast;
//   warp 1    allocates tensor memory (two accumulators of BN columns).  In the leader CTA one
//             lane issues tcgen05.mma.cta_group::2 (256 x N x 16 per instruction, N = the tile's
//             width rounded up to 16; it reads A and B halves from both CTAs' shared memory) and
//             commits, multicast to both CTAs, to the stage's "empty" mbarrier and, per tile, to
//             the accumulator's "full" mbarrier.  The MMAs of tile i+1 overlap the epilogue of
//             tile i;
//   warps 4-11 read the accumulator with tcgen05.ld (lane = output row, 32 columns at a time;
//             warp e owns TMEM lanes 32 (e % 4).. and the column half (e - 4) / 4 of the tile) and
//             release it by arriving on the leader's "accumulator empty" mbarrier.
//             Epilogues: plain FP32 / BF16 stores (each lane writes whole 32-byte sectors of its
//             own row), the transposed BF16 store, and the fused core update of Section 3.4,
//             which goes through a warp-private shared-memory transpose so that its moment
//             read-modify-write touches full 128-byte row segments, with the moment tiles
//             prefetched to L2 while the tile's MMAs run.
// A cluster barrier at entry orders barrier initialisation before remote arrivals, and one at
// exit keeps either CTA from leaving while its peer still reads its shared or tensor memory.
// Ragged edges rely on TMA zero fill for loads and on predicated stores.
// Every mbarrier wait is bounded by a clock budget; on expiry the CTA records
// TSR_ERR_TIMEOUT, stops storing and still releases its tensor memory before it exits.
#include "tsr_device.cuh"
#include "tsr_internal.h"
#include "tsr_umma.cuh"

namespace tsr {

constexpr int UG_THREADS = 384;   // warps 0-1: TMA / MMA, warps 2-3 idle, warps 4-11: epilogue
constexpr int UG_EPI_WARPS = 8;

// PLANES = 1, 2: BF16 operands, B in one or two planes (hi + lo) accumulated into the same D.
// PLANES = 3: FP32 data as three TF32 products.  A and B each come as a plane of values truncated
// to TF32 and a plane of remainders (both FP32 containers, K blocks of 32 elements); D accumulates
// A_hi B_hi + A_hi B_lo + A_lo B_hi, which carries about 21 mantissa bits of each operand.
template <int BN, int PLANES>
struct UmmaSmem {
    static constexpr int A_PLANES = PLANES == 3 ? 2 : 1;
    static constexpr int B_PLANES = PLANES == 3 ? 2 : PLANES;
    static constexpr int BK_ELEMS = PLANES == 3 ? 32 : UM_BK;        // elements per 128-byte K block
    static constexpr int A_BYTES = UM_BM * 128;                       // one plane of this CTA's A rows
    static constexpr int B_BYTES = (BN / 2) * 128;                    // each CTA of the pair stages half of the B rows
    static constexpr int STAGE_BYTES = A_PLANES * A_BYTES + B_PLANES * B_BYTES;
    static constexpr int STAGES = (192 * 1024) / STAGE_BYTES > 6 ? 6 : (192 * 1024) / STAGE_BYTES;
    static constexpr int PATCH_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int PATCH_BYTES = 32 * 33 * 4;                  // per epilogue warp
    static constexpr int BAR_OFFSET = PATCH_OFFSET + UG_EPI_WARPS * PATCH_BYTES;
    static constexpr int NBARS = 2 * STAGES + 4;
    static constexpr int TOTAL = BAR_OFFSET + NBARS * 8 + 64 + 1024;  // + slack for 1024-byte alignment
};

template <int BN, int EPI, int PLANES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(UG_THREADS, 1)
umma_gemm_kernel(const UmmaProblem *__restrict__ probs, const UmmaTile *__restrict__ tiles, int num_tiles,
                 StepScalars sc, int32_t *__restrict__ status)
{
    using SM = UmmaSmem<BN, PLANES>;
    constexpr int STAGES = SM::STAGES;
    constexpr uint32_t TMEM_COLS = 2 * BN;   // 256 or 512

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + SM::BAR_OFFSET);
    uint64_t *bar_full = bars, *bar_empty = bars + STAGES;
    uint64_t *bar_acc_full = bars + 2 * STAGES, *bar_acc_empty = bar_acc_full + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + SM::NBARS);
    __shared__ int s_timeout;   // 0, or 1 + the first tile (table index) this CTA gave up on

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long budget = wait_budget(sc);
    const uint32_t rank = cluster_ctarank();          // 0 = leader of the CTA pair
    const int pair = blockIdx.x >> 1;
    const int stride = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        s_timeout = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(bar_full + s), 1); mbar_init(smem_u32(bar_empty + s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(bar_acc_full + b), 1); mbar_init(smem_u32(bar_acc_empty + b), 2 * UG_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs allocates the pair's tensor memory
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();      // the peer's barriers are initialised before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = pair; t < num_tiles && ok; t += stride) {
                const UmmaTile tile = tiles[t];
                const UmmaProblem *P = probs + tile.prob;
                if (P->starve) {   // diagnostic: nothing is loaded for this tile, so every consumer's bounded wait runs out
                    note_timeout(&s_timeout, t);
                    break;
                }
                int n_eff = P->N - tile.n0;
                n_eff = tile.nw > 0 ? tile.nw : (n_eff >= BN ? BN : ((n_eff + 15) & ~15));
                const int b_row = tile.n0 + (int)rank * (n_eff / 2);   // this CTA's half of the B rows
                for (int kb = tile.kb0; kb < tile.kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(smem_u32(bar_empty + s), ph ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                    // both CTAs' copies report their bytes to the leader's "full" barrier
                    const uint32_t full = leader_addr(smem_u32(bar_full + s));
                    if (rank == 0) mbar_expect_tx(smem_u32(bar_full + s), 2u * (uint32_t)SM::STAGE_BYTES);
                    uint8_t *st = smem + s * SM::STAGE_BYTES;
#pragma unroll
                    for (int pl = 0; pl < SM::A_PLANES; ++pl)
                        tma_load_2d_pair(smem_u32(st + pl * SM::A_BYTES), &P->tmA, full, kb * SM::BK_ELEMS,
                                         tile.m0 + (int)rank * UM_BM + pl * P->a_plane_rows);
#pragma unroll
                    for (int pl = 0; pl < SM::B_PLANES; ++pl)
                        tma_load_2d_pair(smem_u32(st + SM::A_PLANES * SM::A_BYTES + pl * SM::B_BYTES), &P->tmB, full,
                                         kb * SM::BK_ELEMS, b_row + pl * P->plane_rows);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {   // the leader issues the pair's MMAs (256 x N x 16 each)
            uint32_t it = 0, tc = 0;
            bool ok = true;
            for (int t = pair; t < num_tiles && ok; t += stride, ++tc) {
                const UmmaTile tile = tiles[t];
                int n_eff = probs[tile.prob].N - tile.n0;
                n_eff = tile.nw > 0 ? tile.nw : (n_eff >= BN ? BN : ((n_eff + 15) & ~15));
                const uint32_t idesc = PLANES == 3 ? umma_idesc_pair_tf32(n_eff) : umma_idesc_pair(n_eff);
                const uint32_t buf = tc & 1u;
                if (!mbar_wait(smem_u32(bar_acc_empty + buf), ((tc >> 1) & 1u) ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = tile.kb0; kb < tile.kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(smem_u32(bar_full + s), ph, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_base = smem_u32(smem + s * SM::STAGE_BYTES);
                    if (PLANES == 3) {
                        // (A plane, B plane) = (hi, hi), (hi, lo), (lo, hi); 32 bytes of K per instruction
#pragma unroll
                        for (int pr = 0; pr < 3; ++pr) {
                            const uint32_t a_pl = a_base + (pr == 2 ? SM::A_BYTES : 0);
                            const uint32_t b_pl = a_base + 2 * SM::A_BYTES + (pr == 1 ? SM::B_BYTES : 0);
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4)
                                tc_mma_tf32_pair(d_tmem, umma_desc_sw128(a_pl + k4 * 32), umma_desc_sw128(b_pl + k4 * 32),
                                                 idesc, ((kb - tile.kb0) | pr | k4) ? 1u : 0u);
                        }
                    } else {
#pragma unroll
                        for (int pl = 0; pl < SM::B_PLANES; ++pl) {
                            const uint32_t b_base = a_base + SM::A_BYTES + pl * SM::B_BYTES;
#pragma unroll
                            for (int k4 = 0; k4 < UM_BK / 16; ++k4)
                                tc_mma_bf16_pair(d_tmem, umma_desc_sw128(a_base + k4 * 32), umma_desc_sw128(b_base + k4 * 32),
                                                 idesc, ((kb - tile.kb0) | pl | k4) ? 1u : 0u);
                        }
                    }
                    tc_commit_pair(smem_u32(bar_empty + s));       // frees the stage in both CTAs
                }
                tc_commit_pair(smem_u32(bar_acc_full + buf));      // accumulator ready, in both CTAs
            }
        }
    } else if (warp >= 4) {
        // eight epilogue warps: warp e reads TMEM lanes 32 (e % 4) .. + 31 (the quarter a warp may
        // access is fixed by its index modulo 4) and the column half e / 4 of the tile
        const int q = warp & 3;
        const int half = (warp - 4) >> 2;
        float *patch = (float *)(smem + SM::PATCH_OFFSET + (warp - 4) * SM::PATCH_BYTES);   // [32][33]
        uint32_t nbox = 0;       // EPI_STORE_BF16 through TMA: boxes written so far
        uint32_t tc = 0;
        bool ok = true;
        for (int t = pair; t < num_tiles && ok; t += stride, ++tc) {
            const UmmaTile tile = tiles[t];
            const UmmaProblem *__restrict__ P = probs + tile.prob;
            const uint32_t buf = tc & 1u;
            const int N = P->N, M = P->M;
            const int Nt = tile.nw > 0 ? min(N, tile.n0 + tile.nw) : N;   // first column past this tile
            const int row0 = tile.m0 + (int)rank * UM_BM + q * 32;   // this CTA holds rows 128 rank .. of the tile
            // a split-K problem inside a core-update launch only stores its slab
            const bool store_f32 = (EPI == EPI_STORE_F32) || (EPI == EPI_CORE_UPDATE && P->epilogue == EPI_STORE_F32);
            if (EPI == EPI_CORE_UPDATE && !store_f32) {
                // pull this warp's slice of the moments towards L2 while the MMAs of the tile run
                const int prow = row0 + lane;
                if (prow < M) {
                    const int w = min(BN / 2, N - tile.n0 - half * (BN / 2));
                    const char *a1 = (const char *)(P->mom1 + (int64_t)prow * N + tile.n0 + half * (BN / 2));
                    const char *a2 = (const char *)(P->mom2 + (int64_t)prow * N + tile.n0 + half * (BN / 2));
                    for (int o = 0; o < w * 4; o += 128) {
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(a1 + o));
                        if (sc.rule != TSR_RULE_SGD) asm volatile("prefetch.global.L2 [%0];" ::"l"(a2 + o));
                    }
                }
            }
            if (!mbar_wait(smem_u32(bar_acc_full + buf), (tc >> 1) & 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
            tc_fence_after();
            const int nrows = min(32, M - row0);        // may be <= 0
            const int c_begin = half * (BN / 2), c_end = c_begin + BN / 2;
            if (tile.n0 + c_begin >= Nt) {   // this warp's column half lies outside the tile
                tc_fence_before();
                if (lane == 0) mbar_arrive_leader(smem_u32(bar_acc_empty + buf));
                continue;
            }
#pragma unroll 1
            for (int c0 = c_begin; c0 < c_end; c0 += 32) {
                const int col0 = tile.n0 + c0;
                if (col0 >= Nt) break;
                uint32_t v[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN + (uint32_t)c0, v);
                if (c0 + 32 >= c_end || col0 + 32 >= Nt) {   // this warp's last chunk of the tile: release the accumulator
                    tc_fence_before();
                    if (lane == 0) mbar_arrive_leader(smem_u32(bar_acc_empty + buf));
                }
                if (nrows <= 0) continue;
                const int ncols = min(32, Nt - col0);
                if (EPI == EPI_STORE_BF16_T) {
                    // out[col][row]: for a fixed column the 32 lanes hold 32 consecutive rows
                    bf16 *out = (bf16 *)P->out + (int64_t)col0 * P->ld_out + row0 + lane;
                    if (lane < nrows) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (j < ncols) out[(int64_t)j * P->ld_out] = __float2bfloat16_rn(__uint_as_float(v[j]));
                    }
                    continue;
                }
                // Fast paths (full 32 x 32 chunk): transpose through the warp's patch so that lane = column;
                // every global access is then one full row segment (128 bytes of FP32, 64 of BF16).
                const bool full_chunk = (ncols == 32) && (nrows == 32);
                if (store_f32 && ncols == 32 && (P->ld_out & 3) == 0 && (col0 & 3) == 0 &&
                    (((uintptr_t)P->out) & 15) == 0 && (P->split_stride & 3) == 0) {
                    // lane = row: each lane writes 128 contiguous bytes of its own row
                    if (lane < nrows) {
                        float *out = (float *)P->out + (int64_t)tile.split * P->split_stride + (int64_t)(row0 + lane) * P->ld_out + col0;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *(float4 *)(out + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                               __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                    }
                    continue;
                }
                if (EPI == EPI_STORE_BF16 && P->out_tma) {
                    // The chunk goes to a 32 x 32 BF16 box in shared memory (64-byte rows, 64-byte swizzle;
                    // two boxes per warp inside the patch area) and leaves as one TMA store, which writes
                    // whole lines and clips at the matrix edge.  Direct stores from the lane = row layout
                    // cost one 16-byte write request per lane and instruction and were the bound of P = U D.
                    uint8_t *box = smem + SM::PATCH_OFFSET + (((warp - 4) * 2 + (int)(nbox & 1u)) << 11);
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 pk;
                        __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1]));
                        __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
                        __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
                        pk.x = *(uint32_t *)&h0; pk.y = *(uint32_t *)&h1; pk.z = *(uint32_t *)&h2; pk.w = *(uint32_t *)&h3;
                        *(uint4 *)(box + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) = pk;
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&P->tmW, smem_u32(box), col0, row0);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                    ++nbox;
                    continue;
                }
                if (EPI == EPI_STORE_BF16 && ncols == 32 && (P->ld_out & 7) == 0 && (col0 & 7) == 0 &&
                    (((uintptr_t)P->out) & 15) == 0) {
                    if (lane < nrows) {
                        bf16 *out = (bf16 *)P->out + (int64_t)(row0 + lane) * P->ld_out + col0;
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            uint4 pk;
                            __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                            __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                            __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                            pk.x = *(uint32_t *)&h0; pk.y = *(uint32_t *)&h1; pk.z = *(uint32_t *)&h2; pk.w = *(uint32_t *)&h3;
                            *(uint4 *)(out + j) = pk;
                        }
                    }
                    continue;
                }
                if (full_chunk && EPI == EPI_CORE_UPDATE && !store_f32) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) patch[lane * 33 + j] = __uint_as_float(v[j]);
                    __syncwarp();
                    {
                        const int64_t e0 = (int64_t)row0 * N + col0 + lane;   // C, M, Vm are dense r x r (N = r)
                        float *cp = (float *)P->out + e0;
                        float *m1p = P->mom1 + e0;
                        float *m2p = P->mom2 + e0;
                        bf16 *dp = P->d_bf16 ? P->d_bf16 + (int64_t)row0 * P->ldd + col0 + lane : nullptr;
                        const int64_t ldd = P->ldd;
                        const bool sgd = (sc.rule == TSR_RULE_SGD);
#pragma unroll
                        for (int i0 = 0; i0 < 32; i0 += 16) {
                            float m1[16], m2[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i) m1[i] = m1p[(int64_t)(i0 + i) * N];
#pragma unroll
                            for (int i = 0; i < 16; ++i) m2[i] = sgd ? 0.f : m2p[(int64_t)(i0 + i) * N];
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const float c = patch[(i0 + i) * 33 + lane];
                                const float dd = core_update_elem(c, m1[i], m2[i], sc);
                                cp[(int64_t)(i0 + i) * N] = c;
                                m1p[(int64_t)(i0 + i) * N] = m1[i];
                                if (!sgd) m2p[(int64_t)(i0 + i) * N] = m2[i];
                                if (dp) dp[(int64_t)(i0 + i) * ldd] = __float2bfloat16_rn(dd);
                                patch[(i0 + i) * 33 + lane] = dd;
                            }
                        }
                        __syncwarp();
                        // D^T: back to lane = row
                        bf16 *dtp = P->dt_bf16 + (int64_t)col0 * ldd + row0 + lane;
#pragma unroll
                        for (int j = 0; j < 32; ++j) dtp[(int64_t)j * ldd] = __float2bfloat16_rn(patch[lane * 33 + j]);
                    }
                    __syncwarp();
                    continue;
                }
                // Ragged or unaligned chunk: transpose through the patch so that lane = column and
                // the loop index = row; accesses stay row-contiguous.
#pragma unroll
                for (int j = 0; j < 32; ++j) patch[lane * 33 + j] = __uint_as_float(v[j]);
                __syncwarp();
                const int col = col0 + lane;
                const bool col_ok = lane < ncols;
                if (store_f32) {
                    float *out = (float *)P->out + (int64_t)tile.split * P->split_stride + (int64_t)row0 * P->ld_out + col;
                    if (col_ok)
                        for (int i = 0; i < nrows; ++i) out[(int64_t)i * P->ld_out] = patch[i * 33 + lane];
                } else if (EPI == EPI_STORE_BF16) {
                    bf16 *out = (bf16 *)P->out + (int64_t)row0 * P->ld_out + col;
                    if (col_ok)
                        for (int i = 0; i < nrows; ++i) out[(int64_t)i * P->ld_out] = __float2bfloat16_rn(patch[i * 33 + lane]);
                } else if (EPI == EPI_CORE_UPDATE && !store_f32) {
                    // C, M, Vm are dense r x r (N = r)
                    if (col_ok) {
                        for (int i = 0; i < nrows; ++i) {
                            const int64_t e = (int64_t)(row0 + i) * N + col;
                            const float c = patch[i * 33 + lane];
                            float m1 = P->mom1[e];
                            float m2 = (sc.rule == TSR_RULE_SGD) ? 0.f : P->mom2[e];
                            const float dd = core_update_elem(c, m1, m2, sc);
                            ((float *)P->out)[e] = c;
                            P->mom1[e] = m1;
                            if (sc.rule != TSR_RULE_SGD) P->mom2[e] = m2;
                            if (P->d_bf16) P->d_bf16[(int64_t)(row0 + i) * P->ldd + col] = __float2bfloat16_rn(dd);
                            patch[i * 33 + lane] = dd;
                        }
                    }
                    __syncwarp();
                    // D^T: back to lane = row
                    if (lane < nrows) {
                        bf16 *dt = P->dt_bf16 + (int64_t)col0 * P->ldd + row0 + lane;
                        for (int j = 0; j < ncols; ++j) dt[(int64_t)j * P->ldd] = __float2bfloat16_rn(patch[lane * 33 + j]);
                    }
                }
                __syncwarp();
            }
        }
        // TMA stores read their boxes asynchronously: they must have done so before the CTA goes away
        if (EPI == EPI_STORE_BF16 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    if (s_timeout) __nanosleep(2000000);   // let copies in flight land before the CTA goes away
    tc_fence_before();
    __syncthreads();
    cluster_sync();      // neither CTA may leave while the peer still uses its shared or tensor memory
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    // every block that owns a tile this CTA did not finish is flagged
    if (threadIdx.x == 0 && s_timeout && status)
        for (int t = s_timeout - 1; t < num_tiles; t += stride) atomicMax(status + probs[tiles[t].prob].block, (int)TSR_ERR_TIMEOUT);
}

template <int BN, int EPI, int PLANES>
static cudaError_t launch_one(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms,
                              const StepScalars &sc, int32_t *status, cudaStream_t stream)
{
    using SM = UmmaSmem<BN, PLANES>;
    const int pairs = num_tiles < num_sms / 2 ? num_tiles : num_sms / 2;
    umma_gemm_kernel<BN, EPI, PLANES><<<2 * pairs, UG_THREADS, SM::TOTAL, stream>>>(probs, tiles, num_tiles, sc, status);
    return cudaGetLastError();
}

template <int BN, int EPI, int PLANES>
static cudaError_t configure_one()
{
    using SM = UmmaSmem<BN, PLANES>;
    return cudaFuncSetAttribute(umma_gemm_kernel<BN, EPI, PLANES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                SM::TOTAL);
}

cudaError_t umma_configure()
{
    cudaError_t e;
    if ((e = configure_one<128, EPI_STORE_F32, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<256, EPI_STORE_F32, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_STORE_F32, 2>()) != cudaSuccess) return e;
    if ((e = configure_one<256, EPI_STORE_F32, 2>()) != cudaSuccess) return e;
    if ((e = configure_one<256, EPI_STORE_F32, 3>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_STORE_BF16, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<256, EPI_STORE_BF16, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_STORE_BF16_T, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<256, EPI_STORE_BF16_T, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_CORE_UPDATE, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<256, EPI_CORE_UPDATE, 1>()) != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t umma_gemm_launch(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms, int bn,
                             int epilogue, int planes, const StepScalars &sc, int32_t *status, cudaStream_t stream)
{
    if (num_tiles <= 0) return cudaSuccess;
#define TSR_UG(BN_, EPI_, PL_) return launch_one<BN_, EPI_, PL_>(probs, tiles, num_tiles, num_sms, sc, status, stream)
    if (planes == 2) {
        if (bn == 128 && epilogue == EPI_STORE_F32) TSR_UG(128, EPI_STORE_F32, 2);
        if (bn == 256 && epilogue == EPI_STORE_F32) TSR_UG(256, EPI_STORE_F32, 2);
        return cudaErrorInvalidValue;
    }
    if (planes == 3) {
        if (bn == 256 && epilogue == EPI_STORE_F32) TSR_UG(256, EPI_STORE_F32, 3);
        return cudaErrorInvalidValue;
    }
    if (bn == 128) {
        switch (epilogue) {
        case EPI_STORE_F32: TSR_UG(128, EPI_STORE_F32, 1);
        case EPI_STORE_BF16: TSR_UG(128, EPI_STORE_BF16, 1);
        case EPI_STORE_BF16_T: TSR_UG(128, EPI_STORE_BF16_T, 1);
        case EPI_CORE_UPDATE: TSR_UG(128, EPI_CORE_UPDATE, 1);
        default: return cudaErrorInvalidValue;
        }
    }
    if (bn == 256) {
        switch (epilogue) {
        case EPI_STORE_F32: TSR_UG(256, EPI_STORE_F32, 1);
        case EPI_STORE_BF16: TSR_UG(256, EPI_STORE_BF16, 1);
        case EPI_STORE_BF16_T: TSR_UG(256, EPI_STORE_BF16_T, 1);
        case EPI_CORE_UPDATE: TSR_UG(256, EPI_CORE_UPDATE, 1);
        default: return cudaErrorInvalidValue;
        }
    }
#undef TSR_UG
    return cudaErrorInvalidValue;
}

}  // namespace tsr
