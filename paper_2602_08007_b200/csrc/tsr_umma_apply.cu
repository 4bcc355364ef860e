// Persistent back-projection + weight update (Section 3.4) on tcgen05 tensor cores:
//
//   W[m x n] <- decay * W - step_scale * (P V^T),   P = U D (m x r, BF16),  V (n x r, BF16)
//
// The lifted update never reaches memory: each 128 x BN tile of P V^T (BN = 128, or 256 for r >= 512)
// is accumulated in tensor memory and consumed by the epilogue, which streams the matching W tile
// through shared memory with TMA (read-modify-write of 8 bytes per weight is what bounds this kernel).
//
// One CTA per SM loops over the tiles of all blocks (static round-robin over a device-resident
// tile table).  Roles:
//   warp 0      TMA producer for the P / V operand stages (128-byte swizzle, ring of stages)
//   warp 1      tensor-memory allocation; one lane issues the MMAs into one of two BN-column
//               accumulators, so the MMAs of tile i+1 overlap the epilogue of tile i
//   warps 4-7   epilogue; warp q owns accumulator rows 32q..32q+31 and a private ring of
//               32 x 32 FP32 W boxes (4 KB, 128-byte swizzle): it prefetches its W boxes
//               several boxes (more than a tile) ahead, combines them with the accumulator
//               (tcgen05.ld, lane = row), writes the result back into the same box and issues
//               the TMA store.  TMA zero-fills loads and clips stores at ragged edges, so no
//               predicate is needed.
// All waits are bounded (see mbar_wait); on expiry the CTA flags TSR_ERR_TIMEOUT and drains.
#include "tsr_internal.h"
#include "tsr_umma.cuh"
#include "tsr_pdl.cuh"

namespace tsr {

constexpr int AP_THREADS = 256;
constexpr int AP_LAG = 2;                    // a box is refilled AP_LAG stores after its own store
constexpr int AP_BOX_BYTES = 4096;

// Tile width 128: four operand stages and six W boxes per epilogue warp.  Tile width 256 (the P tile
// is then used for twice as many outputs, which lowers the operand bytes an SM has to pull in per
// byte of W): three stages of 16 KB (P) + 32 KB (V), five W boxes per warp, both accumulators fill
// the 512 columns of tensor memory.
template <int BN>
struct ApplyCfg {
    static constexpr int STAGES = BN == 256 ? 3 : 4;
    static constexpr int STAGE_BYTES = 16384 + BN * 128;
    static constexpr int NBOX = BN == 256 ? 5 : 6;
    static constexpr int CHUNKS = BN / 32;
    static constexpr int WBOX_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int BAR_OFFSET = WBOX_OFFSET + 4 * NBOX * AP_BOX_BYTES;
    static constexpr int NBARS = 2 * STAGES + 4 + 4 * NBOX;
    static constexpr int SMEM = BAR_OFFSET + NBARS * 8 + 64 + 1024;
    static constexpr uint32_t TMEM_COLS = 2 * BN;
};

struct ChunkCursor {   // walks the (tile, 32-column chunk) sequence of this CTA
    int tile_idx;      // index into the tile table; >= num_tiles: exhausted
    int c;             // chunk inside the tile
    int m0, n0, prob, N, M;
};

__device__ __forceinline__ void cursor_load(ChunkCursor &cur, const UmmaTile *tiles, const UmmaProblem *probs,
                                            int num_tiles)
{
    if (cur.tile_idx < num_tiles) {
        const UmmaTile t = tiles[cur.tile_idx];
        cur.m0 = t.m0; cur.n0 = t.n0; cur.prob = t.prob;
        cur.N = probs[t.prob].N;
        cur.M = probs[t.prob].M;
    }
}
template <int CHUNKS>
__device__ __forceinline__ void cursor_next(ChunkCursor &cur, const UmmaTile *tiles, const UmmaProblem *probs,
                                            int num_tiles, int stride)
{
    cur.c++;
    if (cur.c >= CHUNKS || cur.n0 + cur.c * 32 >= cur.N) {
        cur.c = 0;
        cur.tile_idx += stride;
        cursor_load(cur, tiles, probs, num_tiles);
    }
}

template <int BN, int WB>
__global__ void __launch_bounds__(AP_THREADS, 1)
umma_apply_kernel(const UmmaProblem *__restrict__ probs, const UmmaTile *__restrict__ tiles, int num_tiles,
                  StepScalars sc, int32_t *__restrict__ status)
{
    using CF = ApplyCfg<BN>;
    constexpr int AP_STAGES = CF::STAGES, AP_STAGE_BYTES = CF::STAGE_BYTES, AP_NBOX = CF::NBOX;
    constexpr int AP_WBOX_OFFSET = CF::WBOX_OFFSET, AP_BAR_OFFSET = CF::BAR_OFFSET, AP_NBARS = CF::NBARS;
    constexpr int AP_BN = BN;
    constexpr uint32_t W_BOX_BYTES = 32 * 32 * WB;   // FP32 weights: 4 KB boxes, 128-byte swizzle; BF16: 2 KB, 64-byte swizzle
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + AP_BAR_OFFSET);
    uint64_t *bar_full = bars;                       // [AP_STAGES]
    uint64_t *bar_empty = bars + AP_STAGES;          // [AP_STAGES]
    uint64_t *bar_acc_full = bars + 2 * AP_STAGES;   // [2]
    uint64_t *bar_acc_empty = bar_acc_full + 2;      // [2]
    uint64_t *bar_w = bar_acc_empty + 2;             // [4][AP_NBOX]
    uint32_t *tmem_slot = (uint32_t *)(bars + AP_NBARS);
    __shared__ int s_timeout;   // 0, or 1 + the first tile (table index) this CTA gave up on

    pdl_trigger();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stride = gridDim.x;
    const long long budget = wait_budget(sc);

    if (threadIdx.x == 0) {
        s_timeout = 0;
        for (int s = 0; s < AP_STAGES; ++s) { mbar_init(smem_u32(bar_full + s), 1); mbar_init(smem_u32(bar_empty + s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(bar_acc_full + b), 1); mbar_init(smem_u32(bar_acc_empty + b), 4); }
        for (int i = 0; i < 4 * AP_NBOX; ++i) mbar_init(smem_u32(bar_w + i), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(CF::TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();      // set-up done; P = U D of the kernel before this one is read from here on

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;                   // stage and phase of the operand ring this thread fills next
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += stride) {
                const UmmaTile tile = tiles[t];
                const UmmaProblem *P = probs + tile.prob;
                const int nkb = (P->K + UM_BK - 1) / UM_BK;
                const CUtensorMap *tmA = &P->tmA, *tmB = &P->tmB;
                const int m0 = tile.m0, n0 = tile.n0;
                // (nothing in this loop reads global memory: it is on the critical path of the operand pipeline)
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(smem_u32(bar_empty + s), ph ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                    const uint32_t full = smem_u32(bar_full + s);
                    mbar_expect_tx(full, (uint32_t)AP_STAGE_BYTES);
                    const uint32_t st = smem_u32(smem + s * AP_STAGE_BYTES);
                    tma_load_2d(st, tmA, full, kb * UM_BK, m0);
                    tma_load_2d(st + 16384, tmB, full, kb * UM_BK, n0);
                    if (BN == 256) tma_load_2d(st + 32768, tmB, full, kb * UM_BK, n0 + 128);
                    if (++s == AP_STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(AP_BN);
            uint32_t tc = 0;
            int cs = 0;                  // stage and phase of the operand ring this thread consumes next
            uint32_t cph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += stride, ++tc) {
                const UmmaTile tile = tiles[t];
                const int nkb = (probs[tile.prob].K + UM_BK - 1) / UM_BK;
                const uint32_t buf = tc & 1u;
                if (!mbar_wait(smem_u32(bar_acc_empty + buf), ((tc >> 1) & 1u) ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * AP_BN;
                for (int kb = 0; kb < nkb; ++kb) {
                    const int s = cs;
                    if (!mbar_wait(smem_u32(bar_full + s), cph, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                    if (++cs == AP_STAGES) { cs = 0; cph ^= 1u; }
                    tc_fence_after();
                    const uint32_t a_base = smem_u32(smem + s * AP_STAGE_BYTES);
                    const uint32_t b_base = a_base + 16384;
#pragma unroll
                    for (int k4 = 0; k4 < UM_BK / 16; ++k4)
                        tc_mma_bf16(d_tmem, umma_desc_sw128(a_base + k4 * 32), umma_desc_sw128(b_base + k4 * 32), idesc,
                                    (kb | k4) ? 1u : 0u);
                    tc_commit(smem_u32(bar_empty + s));
                }
                tc_commit(smem_u32(bar_acc_full + buf));
            }
        }
    } else if (warp >= 4) {
        const int q = warp & 3;
        uint8_t *boxes = smem + AP_WBOX_OFFSET + q * AP_NBOX * AP_BOX_BYTES;
        uint64_t *wbar = bar_w + q * AP_NBOX;
        ChunkCursor pre, cur;
        pre.tile_idx = blockIdx.x; pre.c = 0; pre.m0 = pre.n0 = pre.prob = 0; pre.N = 0; pre.M = 0;
        cursor_load(pre, tiles, probs, num_tiles);
        cur = pre;
        uint32_t issued = 0, cons = 0, tc = 0;
        bool ok = true;
        // initial prefetch: AP_NBOX - AP_LAG boxes
        for (int i = 0; i < AP_NBOX - AP_LAG && pre.tile_idx < num_tiles; ++i) {
            if (lane == 0) {
                const uint32_t slot = issued % AP_NBOX;
                mbar_expect_tx(smem_u32(wbar + slot), W_BOX_BYTES);
                tma_load_2d(smem_u32(boxes + slot * AP_BOX_BYTES), &probs[pre.prob].tmW, smem_u32(wbar + slot),
                            pre.n0 + pre.c * 32, pre.m0 + q * 32);
            }
            ++issued;
            cursor_next<CF::CHUNKS>(pre, tiles, probs, num_tiles, stride);
        }
        while (cur.tile_idx < num_tiles && ok) {
            const uint32_t buf = tc & 1u;
            if (cur.c == 0) {
                if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(bar_acc_full + buf), (tc >> 1) & 1u, budget))) { note_timeout(&s_timeout, cur.tile_idx); ok = false; break; }
                tc_fence_after();
            }
            const uint32_t slot = cons % AP_NBOX;
            uint32_t v[32];
            tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * AP_BN + (uint32_t)(cur.c * 32), v);
            const bool last_chunk = (cur.c == CF::CHUNKS - 1) || (cur.n0 + (cur.c + 1) * 32 >= cur.N);
            if (last_chunk) {   // accumulator fully read by this warp: hand it back to the MMA warp
                tc_fence_before();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar_acc_empty + buf)) : "memory");
            }
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(wbar + slot), (cons / AP_NBOX) & 1u, budget))) { note_timeout(&s_timeout, cur.tile_idx); ok = false; break; }
            if (WB == 4) {
                uint8_t *box = boxes + slot * AP_BOX_BYTES + lane * 128;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float4 *p = (float4 *)(box + ((j ^ (lane & 7)) << 4));
                    float4 x = *p;
                    x.x = __fmaf_rn(-sc.step_scale, __uint_as_float(v[4 * j + 0]), __fmul_rn(sc.decay, x.x));
                    x.y = __fmaf_rn(-sc.step_scale, __uint_as_float(v[4 * j + 1]), __fmul_rn(sc.decay, x.y));
                    x.z = __fmaf_rn(-sc.step_scale, __uint_as_float(v[4 * j + 2]), __fmul_rn(sc.decay, x.z));
                    x.w = __fmaf_rn(-sc.step_scale, __uint_as_float(v[4 * j + 3]), __fmul_rn(sc.decay, x.w));
                    *p = x;
                }
            } else {
                // BF16 weights: a row of the box is 64 bytes (four 16-byte chunks, 64-byte swizzle); the update
                // is formed in FP32 and rounded to nearest even
                uint8_t *box = boxes + slot * AP_BOX_BYTES + lane * 64;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 *p = (uint4 *)(box + ((j ^ ((lane >> 1) & 3)) << 4));
                    uint4 x = *p;
                    uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float w0 = __uint_as_float(w[u] << 16), w1 = __uint_as_float(w[u] & 0xffff0000u);
                        const float y0 = __fmaf_rn(-sc.step_scale, __uint_as_float(v[8 * j + 2 * u]), __fmul_rn(sc.decay, w0));
                        const float y1 = __fmaf_rn(-sc.step_scale, __uint_as_float(v[8 * j + 2 * u + 1]), __fmul_rn(sc.decay, w1));
                        const __nv_bfloat162 h = __floats2bfloat162_rn(y0, y1);
                        w[u] = *(const uint32_t *)&h;
                    }
                    *p = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if (cur.m0 + q * 32 < cur.M)   // rows past the end were zero-filled on load; nothing to store
                    tma_store_2d(&probs[cur.prob].tmW, smem_u32(boxes + slot * AP_BOX_BYTES), cur.n0 + cur.c * 32, cur.m0 + q * 32);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            ++cons;
            // refill the box whose store was issued AP_LAG stores ago
            if (pre.tile_idx < num_tiles) {
                if (lane == 0) {
                    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(AP_LAG - 1) : "memory");
                    const uint32_t pslot = issued % AP_NBOX;
                    mbar_expect_tx(smem_u32(wbar + pslot), W_BOX_BYTES);
                    tma_load_2d(smem_u32(boxes + pslot * AP_BOX_BYTES), &probs[pre.prob].tmW, smem_u32(wbar + pslot),
                                pre.n0 + pre.c * 32, pre.m0 + q * 32);
                }
                ++issued;
                cursor_next<CF::CHUNKS>(pre, tiles, probs, num_tiles, stride);
            }
            if (last_chunk) ++tc;
            cursor_next<CF::CHUNKS>(cur, tiles, probs, num_tiles, stride);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    if (s_timeout) __nanosleep(2000000);   // let copies in flight land before the CTA goes away
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(CF::TMEM_COLS) : "memory");
    }
    // every block that owns a tile this CTA did not finish is flagged
    if (threadIdx.x == 0 && s_timeout && status)
        for (int t = s_timeout - 1; t < num_tiles; t += stride) atomicMax(status + probs[tiles[t].prob].block, (int)TSR_ERR_TIMEOUT);
}

cudaError_t umma_apply_configure()
{
    cudaError_t e;
#define TSR_AP_CFG(BN_, WB_)                                                                                           \
    if ((e = cudaFuncSetAttribute(umma_apply_kernel<BN_, WB_>, cudaFuncAttributeMaxDynamicSharedMemorySize,            \
                                  ApplyCfg<BN_>::SMEM)) != cudaSuccess)                                                \
        return e
    TSR_AP_CFG(128, 4); TSR_AP_CFG(256, 4); TSR_AP_CFG(128, 2); TSR_AP_CFG(256, 2);
#undef TSR_AP_CFG
    return cudaSuccess;
}

cudaError_t umma_apply_launch(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms, int bn,
                              int w_bytes, const StepScalars &sc, int32_t *status, cudaStream_t stream)
{
    if (num_tiles <= 0) return cudaSuccess;
    const int grid = num_tiles < num_sms ? num_tiles : num_sms;
    if (bn == 256 && w_bytes == 4)
        return launch_dependent(umma_apply_kernel<256, 4>, dim3(grid), dim3(AP_THREADS), (size_t)ApplyCfg<256>::SMEM, stream, 1, probs, tiles, num_tiles, sc, status);
    else if (bn == 256)
        return launch_dependent(umma_apply_kernel<256, 2>, dim3(grid), dim3(AP_THREADS), (size_t)ApplyCfg<256>::SMEM, stream, 1, probs, tiles, num_tiles, sc, status);
    else if (w_bytes == 4)
        return launch_dependent(umma_apply_kernel<128, 4>, dim3(grid), dim3(AP_THREADS), (size_t)ApplyCfg<128>::SMEM, stream, 1, probs, tiles, num_tiles, sc, status);
    else
        return launch_dependent(umma_apply_kernel<128, 2>, dim3(grid), dim3(AP_THREADS), (size_t)ApplyCfg<128>::SMEM, stream, 1, probs, tiles, num_tiles, sc, status);
}

}  // namespace tsr
