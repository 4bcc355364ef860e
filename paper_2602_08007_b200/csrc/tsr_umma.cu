// Grouped BF16 GEMM on the 5th-generation tensor cores (tcgen05) for sm_100a.
//
//   D[M x N] = A[M x K] * B[N x K]^T     A, B BF16 with K contiguous, FP32 accumulation
//
// One CTA computes one 128 x BN output tile listed in a device-resident tile table (tiles of
// all matrix blocks of a model share one launch).  Roles inside the CTA:
//   warp 0    one lane issues the TMA loads (128-byte swizzled 64-wide K slices) into a ring of
//             shared-memory stages and signals "full" mbarriers with the byte count;
//   warp 1    allocates tensor memory; one lane issues tcgen05.mma (128 x BN x 16 per
//             instruction) from shared-memory descriptors into the TMEM accumulator and
//             commits to the "empty" mbarrier of the stage, finally to the "accumulator ready"
//             mbarrier;
//   warps 2-5 read the accumulator with tcgen05.ld (lane = output row) and run the epilogue:
//             plain / transposed stores, the fused core update of Section 3.4, or the fused
//             weight update W <- decay * W - step_scale * acc (the lifted update never reaches
//             memory).
// Ragged edges rely on TMA zero fill for loads and on predicated stores.
// Every mbarrier wait is bounded by a clock budget; on expiry the CTA records
// TSR_ERR_TIMEOUT in the block's status word, skips its stores and still releases its tensor
// memory before it exits.
#include "tsr_device.cuh"
#include "tsr_internal.h"
#include "tsr_umma.cuh"

namespace tsr {

template <int EPI>
struct UmmaCfg {
    static constexpr int STAGES = (EPI == EPI_APPLY || EPI == EPI_STORE_BF16) ? 2 : 4;
};

template <int BN, int PLANES, int STAGES>
struct UmmaSmem {
    static constexpr int A_BYTES = UM_BM * UM_BK * 2;
    static constexpr int B_BYTES = BN * UM_BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + PLANES * B_BYTES;
    static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;  // barriers + slack for 1024-byte alignment
};

template <int BN, int EPI, int PLANES>
__global__ void __launch_bounds__(UM_THREADS)
umma_gemm_kernel(const UmmaProblem *__restrict__ probs, const UmmaTile *__restrict__ tiles, StepScalars sc,
                 int32_t *__restrict__ status)
{
    constexpr int STAGES = UmmaCfg<EPI>::STAGES;
    using SM = UmmaSmem<BN, PLANES, STAGES>;
    constexpr uint32_t TMEM_COLS = (BN <= 32) ? 32 : (BN <= 64 ? 64 : (BN <= 128 ? 128 : 256));

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + SM::BAR_OFFSET);
    // bars[0..STAGES) full, [STAGES..2*STAGES) empty, [2*STAGES] accumulator ready
    uint32_t *tmem_slot = (uint32_t *)(bars + 2 * STAGES + 1);
    __shared__ int s_timeout;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const UmmaTile tile = tiles[blockIdx.x];
    const UmmaProblem *__restrict__ P = probs + tile.prob;
    const int nkb = tile.kb1 - tile.kb0;

    if (threadIdx.x == 0) {
        s_timeout = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(bars + s), 1);
            mbar_init(smem_u32(bars + STAGES + s), 1);
        }
        mbar_init(smem_u32(bars + 2 * STAGES), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < nkb; ++i) {
                const int s = i % STAGES;
                const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
                if (!mbar_wait(smem_u32(bars + STAGES + s), ph ^ 1u)) { s_timeout = 1; break; }
                const uint32_t full = smem_u32(bars + s);
                mbar_expect_tx(full, (uint32_t)SM::STAGE_BYTES);
                uint8_t *st = smem + s * SM::STAGE_BYTES;
                const int kx = (tile.kb0 + i) * UM_BK;
                tma_load_2d(smem_u32(st), &P->tmA, full, kx, tile.m0);
#pragma unroll
                for (int pl = 0; pl < PLANES; ++pl)
                    tma_load_2d(smem_u32(st + SM::A_BYTES + pl * SM::B_BYTES), &P->tmB, full, kx,
                                tile.n0 + pl * P->plane_rows);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(BN);
            bool ok = true;
            for (int i = 0; i < nkb && ok; ++i) {
                const int s = i % STAGES;
                const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
                if (!mbar_wait(smem_u32(bars + s), ph)) { s_timeout = 1; ok = false; break; }
                tc_fence_after();
                const uint32_t a_base = smem_u32(smem + s * SM::STAGE_BYTES);
#pragma unroll
                for (int pl = 0; pl < PLANES; ++pl) {
                    const uint32_t b_base = a_base + SM::A_BYTES + pl * SM::B_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < UM_BK / 16; ++k4) {
                        const uint64_t adesc = umma_desc_sw128(a_base + k4 * 32);
                        const uint64_t bdesc = umma_desc_sw128(b_base + k4 * 32);
                        tc_mma_bf16(tmem_base, adesc, bdesc, idesc, (i | pl | k4) ? 1u : 0u);
                    }
                }
                tc_commit(smem_u32(bars + STAGES + s));
            }
            tc_commit(smem_u32(bars + 2 * STAGES));
        }
    } else {
        // epilogue: warps 2..5 own TMEM lane quarters (warp % 4)
        const int quarter = warp & 3;
        bool ok = mbar_wait(smem_u32(bars + 2 * STAGES), 0);
        if (!ok) s_timeout = 1;
        ok = ok && (s_timeout == 0);
        tc_fence_after();
        const int row = tile.m0 + quarter * 32 + lane;
        const bool row_ok = ok && row < P->M;
        const int N = P->N;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
            if (tile.n0 + c0 >= N) break;
            uint32_t v[32];
            tc_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, v);
            if (!row_ok) continue;
            const int col0 = tile.n0 + c0;
            const bool full_chunk = (col0 + 32 <= N);
            if (EPI == EPI_STORE_F32) {
                float *out = (float *)P->out + (int64_t)tile.split * P->split_stride + (int64_t)row * P->ld_out + col0;
                if (full_chunk && (P->ld_out & 3) == 0 && (col0 & 3) == 0) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *(float4 *)(out + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                           __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                } else {
                    for (int j = 0; j < 32 && col0 + j < N; ++j) out[j] = __uint_as_float(v[j]);
                }
            } else if (EPI == EPI_STORE_BF16) {
                bf16 *out = (bf16 *)P->out + (int64_t)row * P->ld_out + col0;
                if (full_chunk && (P->ld_out & 7) == 0) {
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
                } else {
                    for (int j = 0; j < 32 && col0 + j < N; ++j) out[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
                }
            } else if (EPI == EPI_STORE_BF16_T) {
                bf16 *out = (bf16 *)P->out + (int64_t)col0 * P->ld_out + row;
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < N) out[(int64_t)j * P->ld_out] = __float2bfloat16_rn(__uint_as_float(v[j]));
            } else if (EPI == EPI_CORE_UPDATE) {
                const int64_t base = (int64_t)row * N + col0;  // C, M, Vm are dense r x r (N = r)
                float *Cc = (float *)P->out + base;
                float *m1p = P->mom1 + base;
                float *m2p = P->mom2 + base;
                bf16 *dp = P->d_bf16 + (int64_t)row * P->ldd + col0;
                bf16 *dtp = P->dt_bf16 + (int64_t)col0 * P->ldd + row;
                for (int j = 0; j < 32 && col0 + j < N; ++j) {
                    const float c = __uint_as_float(v[j]);
                    float m1 = m1p[j];
                    float m2 = (sc.rule == TSR_RULE_SGD) ? 0.f : m2p[j];
                    const float dd = core_update_elem(c, m1, m2, sc);
                    Cc[j] = c;
                    m1p[j] = m1;
                    if (sc.rule != TSR_RULE_SGD) m2p[j] = m2;
                    const bf16 db = __float2bfloat16_rn(dd);
                    dp[j] = db;
                    dtp[(int64_t)j * P->ldd] = db;
                }
            } else if (EPI == EPI_APPLY) {
                float *w = (float *)P->out + (int64_t)row * P->ld_out + col0;
                if (full_chunk && (P->ld_out & 3) == 0 && (col0 & 3) == 0) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float4 x = *(float4 *)(w + j);
                        x.x = __fmaf_rn(-sc.step_scale, __uint_as_float(v[j]), __fmul_rn(sc.decay, x.x));
                        x.y = __fmaf_rn(-sc.step_scale, __uint_as_float(v[j + 1]), __fmul_rn(sc.decay, x.y));
                        x.z = __fmaf_rn(-sc.step_scale, __uint_as_float(v[j + 2]), __fmul_rn(sc.decay, x.z));
                        x.w = __fmaf_rn(-sc.step_scale, __uint_as_float(v[j + 3]), __fmul_rn(sc.decay, x.w));
                        *(float4 *)(w + j) = x;
                    }
                } else {
                    for (int j = 0; j < 32 && col0 + j < N; ++j)
                        w[j] = __fmaf_rn(-sc.step_scale, __uint_as_float(v[j]), __fmul_rn(sc.decay, w[j]));
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && s_timeout && status) atomicMax(status + P->block, (int)TSR_ERR_TIMEOUT);
}

template <int BN, int EPI, int PLANES>
static cudaError_t launch_one(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, const StepScalars &sc,
                              int32_t *status, cudaStream_t stream)
{
    using SM = UmmaSmem<BN, PLANES, UmmaCfg<EPI>::STAGES>;
    umma_gemm_kernel<BN, EPI, PLANES><<<num_tiles, UM_THREADS, SM::TOTAL, stream>>>(probs, tiles, sc, status);
    return cudaGetLastError();
}

template <int BN, int EPI, int PLANES>
static cudaError_t configure_one()
{
    using SM = UmmaSmem<BN, PLANES, UmmaCfg<EPI>::STAGES>;
    return cudaFuncSetAttribute(umma_gemm_kernel<BN, EPI, PLANES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                SM::TOTAL);
}

cudaError_t umma_configure()
{
    cudaError_t e;
    if ((e = configure_one<128, EPI_STORE_F32, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_STORE_F32, 2>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_STORE_BF16, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_STORE_BF16_T, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_CORE_UPDATE, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<128, EPI_APPLY, 1>()) != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t umma_gemm_launch(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int bn, int epilogue,
                             int planes, const StepScalars &sc, int32_t *status, cudaStream_t stream)
{
    if (num_tiles <= 0) return cudaSuccess;
    if (bn != 128) return cudaErrorInvalidValue;
    switch (epilogue) {
    case EPI_STORE_F32:
        return planes == 2 ? launch_one<128, EPI_STORE_F32, 2>(probs, tiles, num_tiles, sc, status, stream)
                           : launch_one<128, EPI_STORE_F32, 1>(probs, tiles, num_tiles, sc, status, stream);
    case EPI_STORE_BF16: return launch_one<128, EPI_STORE_BF16, 1>(probs, tiles, num_tiles, sc, status, stream);
    case EPI_STORE_BF16_T: return launch_one<128, EPI_STORE_BF16_T, 1>(probs, tiles, num_tiles, sc, status, stream);
    case EPI_CORE_UPDATE: return launch_one<128, EPI_CORE_UPDATE, 1>(probs, tiles, num_tiles, sc, status, stream);
    case EPI_APPLY: return launch_one<128, EPI_APPLY, 1>(probs, tiles, num_tiles, sc, status, stream);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace tsr
