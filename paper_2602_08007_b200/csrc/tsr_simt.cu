// CUDA-core kernels of libtsr: the all-FP32 path (FP32 gradients, or buffers that miss the
// 16-byte alignment the tensor-core path needs), the stand-alone core update (Section 3.4),
// operand conversion for the tensor-core path, and the Gaussian generator for Omega.
#include "tsr_internal.h"
#include "tsr_device.cuh"
#include "tsr_pdl.cuh"
#include <cooperative_groups.h>
#include <type_traits>

namespace tsr {

// ---------------------------------------------------------------------------------------
// Generic strided FP32 GEMM, 64 x 64 output tile, 16-deep K slices, 4 x 4 outputs per thread.
// Products with few output tiles and a long contraction (T = G V of a single matrix: 16 tiles,
// K = 1376) are split along K over the CTAs of a thread-block cluster (gridDim.z = cluster size
// <= 8): every CTA sums its slab of K, parks its 64 x 64 partial tile in its own shared memory,
// and the cluster's first CTA adds the others' tiles through distributed shared memory in rank
// order -- a fixed order, so the result does not depend on timing -- and runs the epilogue.
// ---------------------------------------------------------------------------------------
template <typename TA>
__device__ __forceinline__ float load_as_float(const TA *p);
template <>
__device__ __forceinline__ float load_as_float<float>(const float *p) { return *p; }
template <>
__device__ __forceinline__ float load_as_float<bf16>(const bf16 *p) { return __bfloat162float(*p); }

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16;
constexpr int SG_LD = SG_BM * SG_BK / 256;   // elements of each operand slice a thread moves
constexpr int SG_NST = 3;                      // shared-memory stages of the FP32 operand slices

template <typename TA, typename TB, int EPI>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(int M, int N, int K, const TA *__restrict__ A, int64_t sa_i, int64_t sa_k,
                 const TB *__restrict__ B, int64_t sb_k, int64_t sb_j, float *__restrict__ D, int64_t ldd,
                 float decay, float step_scale)
{
    // K slices of both operands, SG_NST stages of [k][row] and [k][column]; after the main loop the same storage holds
    // this CTA's partial tile for the cluster's reduction
    __shared__ __align__(16) float smem_ab[SG_NST * 2 * SG_BK * (SG_BM + 4)];
    float (*As)[SG_BK][SG_BM + 4] = (float (*)[SG_BK][SG_BM + 4])smem_ab;
    float (*Bs)[SG_BK][SG_BN + 4] = (float (*)[SG_BK][SG_BN + 4])(smem_ab + SG_NST * SG_BK * (SG_BM + 4));
    float *red = smem_ab;                    // [a][b][thread]: read and written without bank conflicts
    pdl_trigger();
    pdl_wait();                              // nothing to set up: the operands are the predecessor's results
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
    // this CTA's slab of the contraction: whole K slices, the same count for every rank
    const int nslab = (int)gridDim.z, slab = (int)blockIdx.z;
    const int slices = (K + SG_BK - 1) / SG_BK;
    const int per = (slices + nslab - 1) / nslab;
    const int k_begin = min(K, slab * per * SG_BK), k_end = min(K, (slab + 1) * per * SG_BK);

    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    // Loader index maps: put the unit-stride index on consecutive threads.
    const bool a_k_fast = (sa_k == 1);
    const bool b_j_fast = (sb_j == 1);
    auto a_index = [&](int e, int &ai, int &ak) { if (a_k_fast) { ak = e % SG_BK; ai = e / SG_BK; } else { ai = e % SG_BM; ak = e / SG_BM; } };
    auto b_index = [&](int e, int &bj, int &bk) { if (b_j_fast) { bj = e % SG_BN; bk = e / SG_BN; } else { bk = e % SG_BK; bj = e / SG_BK; } };
    auto compute = [&](int stage) {
#pragma unroll
        for (int kk = 0; kk < SG_BK; ++kk) {
            const float4 a4 = *(const float4 *)&As[stage][kk][ty * 4];
            const float4 b4 = *(const float4 *)&Bs[stage][kk][tx * 4];
            const float av[4] = {a4.x, a4.y, a4.z, a4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
        }
    };

    constexpr bool ASYNC = std::is_same<TA, float>::value && std::is_same<TB, float>::value;
    if (ASYNC) {
        // FP32 operands go from global to shared memory with 4-byte asynchronous copies (any stride, any alignment;
        // elements past an edge are zero-filled), SG_NST - 1 slices ahead of the arithmetic: with a handful of slices
        // per CTA the kernel is a chain of global-memory latencies, and this takes two of every three off it.
        const float *Af = (const float *)A, *Bf = (const float *)B;
        auto issue = [&](int stage, int k0) {
#pragma unroll
            for (int l = 0; l < SG_LD; ++l) {
                const int e = tid + l * 256;
                int ai, ak, bj, bk;
                a_index(e, ai, ak);
                b_index(e, bj, bk);
                const int gi = m0 + ai, gk = k0 + ak, gj = n0 + bj, gk2 = k0 + bk;
                const bool va = gi < M && gk < k_end, vb = gj < N && gk2 < k_end;
                const float *pa = va ? Af + (int64_t)gi * sa_i + (int64_t)gk * sa_k : Af;
                const float *pb = vb ? Bf + (int64_t)gk2 * sb_k + (int64_t)gj * sb_j : Bf;
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(&As[stage][ak][ai])),
                             "l"(pa), "r"(va ? 4 : 0) : "memory");
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(&Bs[stage][bk][bj])),
                             "l"(pb), "r"(vb ? 4 : 0) : "memory");
            }
        };
        const int nsteps = (k_end - k_begin + SG_BK - 1) / SG_BK;
        for (int st = 0; st < SG_NST - 1; ++st) {
            if (st < nsteps) issue(st, k_begin + st * SG_BK);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        for (int st = 0; st < nsteps; ++st) {
            asm volatile("cp.async.wait_group %0;" ::"n"(SG_NST - 2) : "memory");
            __syncthreads();                 // slice st has landed for every thread, and slice st - 1 has been used by all
            const int nx = st + SG_NST - 1;
            if (nx < nsteps) issue(nx % SG_NST, k_begin + nx * SG_BK);
            asm volatile("cp.async.commit_group;" ::: "memory");
            compute(st % SG_NST);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
    } else {
        // global -> registers -> shared, with the next K slice in flight while the current one is used
        float ra[SG_LD], rb[SG_LD];
        auto fetch = [&](int k0) {
#pragma unroll
            for (int l = 0; l < SG_LD; ++l) {
                const int e = tid + l * 256;  // 0 .. 64 * SG_BK - 1
                int ai, ak, bj, bk;
                a_index(e, ai, ak);
                b_index(e, bj, bk);
                const int gi = m0 + ai, gk = k0 + ak;
                ra[l] = (gi < M && gk < k_end) ? load_as_float<TA>(A + (int64_t)gi * sa_i + (int64_t)gk * sa_k) : 0.f;
                const int gj = n0 + bj, gk2 = k0 + bk;
                rb[l] = (gj < N && gk2 < k_end) ? load_as_float<TB>(B + (int64_t)gk2 * sb_k + (int64_t)gj * sb_j) : 0.f;
            }
        };
        if (k_begin < k_end) fetch(k_begin);
        for (int k0 = k_begin; k0 < k_end; k0 += SG_BK) {
#pragma unroll
            for (int l = 0; l < SG_LD; ++l) {
                const int e = tid + l * 256;
                int ai, ak, bj, bk;
                a_index(e, ai, ak);
                b_index(e, bj, bk);
                As[0][ak][ai] = ra[l];
                Bs[0][bk][bj] = rb[l];
            }
            __syncthreads();
            if (k0 + SG_BK < k_end) fetch(k0 + SG_BK);
            compute(0);
            __syncthreads();
        }
    }
    if (nslab > 1) {
        namespace cg = cooperative_groups;
        cg::cluster_group cluster = cg::this_cluster();
        if (slab != 0) {
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) red[(a * 4 + b) * 256 + tid] = acc[a][b];
        }
        cluster.sync();                                   // every partial tile is in place
        if (slab == 0) {
            for (int sl = 1; sl < nslab; ++sl) {          // rank order: the sum does not depend on timing
                const float *peer = cluster.map_shared_rank(red, sl);
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) acc[a][b] += peer[(a * 4 + b) * 256 + tid];
            }
        }
        cluster.sync();                                   // nobody leaves while its tile may still be read
        if (slab != 0) return;
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int gi = m0 + ty * 4 + a;
        if (gi >= M) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int gj = n0 + tx * 4 + b;
            if (gj >= N) continue;
            if (EPI == SIMT_APPLY_BF16) {   // D holds BF16 weights: update in FP32, round to nearest even
                bf16 *dw = (bf16 *)D + (int64_t)gi * ldd + gj;
                *dw = __float2bfloat16_rn(__fmaf_rn(-step_scale, acc[a][b], __fmul_rn(decay, __bfloat162float(*dw))));
                continue;
            }
            float *d = D + (int64_t)gi * ldd + gj;
            if (EPI == SIMT_APPLY) {
                *d = __fmaf_rn(-step_scale, acc[a][b], __fmul_rn(decay, *d));
            } else {
                *d = acc[a][b];
            }
        }
    }
}

// FP32 A (any strides) times a BF16 or FP32 B, plain store: the one-sided projection C = U^T G.
// K slabs for a product with `tiles` output tiles: doubled while the grid stays within about one wave of CTAs
// (148 SMs, several CTAs each) and every slab keeps at least four K slices; a power of two up to the portable
// cluster size of 8.
static int simt_slabs(int tiles, int K)
{
    int s = 1;
    while (s < 8 && tiles * s * 2 <= 296 && K / (s * 2) >= 4 * SG_BK) s *= 2;
    return s;
}

template <typename Kern, typename... Args>
static cudaError_t simt_launch(Kern kern, dim3 grid, int slabs, cudaStream_t stream, Args... args)
{
    return launch_dependent(kern, dim3(grid.x, grid.y, (unsigned)slabs), dim3(256), 0, stream, slabs, args...);
}

cudaError_t simt_gemm_bt(int M, int N, int K, const float *A, int64_t sa_i, int64_t sa_k, const void *B, int b_dtype,
                         int64_t sb_k, int64_t sb_j, float *D, int64_t ldd, cudaStream_t stream)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    dim3 grid((N + SG_BN - 1) / SG_BN, (M + SG_BM - 1) / SG_BM);
    const int slabs = simt_slabs((int)(grid.x * grid.y), K);
    if (b_dtype == TSR_BF16)
        return simt_launch(simt_gemm_kernel<float, bf16, SIMT_STORE>, grid, slabs, stream, M, N, K, A, sa_i, sa_k, (const bf16 *)B,
                           sb_k, sb_j, D, ldd, 0.f, 0.f);
    return simt_launch(simt_gemm_kernel<float, float, SIMT_STORE>, grid, slabs, stream, M, N, K, A, sa_i, sa_k, (const float *)B,
                       sb_k, sb_j, D, ldd, 0.f, 0.f);
}

cudaError_t simt_gemm(int M, int N, int K, const void *A, int a_dtype, int64_t sa_i, int64_t sa_k, const float *B,
                      int64_t sb_k, int64_t sb_j, float *D, int64_t ldd, int epilogue, float decay, float step_scale,
                      cudaStream_t stream)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    dim3 grid((N + SG_BN - 1) / SG_BN, (M + SG_BM - 1) / SG_BM);
    const int slabs = simt_slabs((int)(grid.x * grid.y), K);
#define TSR_SG(TA_, EPI_)                                                                                              \
    return simt_launch(simt_gemm_kernel<TA_, float, EPI_>, grid, slabs, stream, M, N, K, (const TA_ *)A, sa_i, sa_k, B, sb_k, \
                       sb_j, D, ldd, decay, step_scale)
    if (a_dtype == TSR_BF16) {
        if (epilogue == SIMT_APPLY) TSR_SG(bf16, SIMT_APPLY);
        else if (epilogue == SIMT_APPLY_BF16) TSR_SG(bf16, SIMT_APPLY_BF16);
        else TSR_SG(bf16, SIMT_STORE);
    } else {
        if (epilogue == SIMT_APPLY) TSR_SG(float, SIMT_APPLY);
        else if (epilogue == SIMT_APPLY_BF16) TSR_SG(float, SIMT_APPLY_BF16);
        else TSR_SG(float, SIMT_STORE);
    }
#undef TSR_SG
}

// ---------------------------------------------------------------------------------------
// Core-space update (Section 3.4; Algorithm 2 for the SGD rule).  The same arithmetic, with
// the same explicit rounding steps, is used by the tensor-core projection epilogue so that
// the fused and the unfused orders agree bit for bit.
// ---------------------------------------------------------------------------------------
// mode 0: full update; mode 1: only sum the split-K slabs into Cout.
// One CTA per 32 x 128 strip of the core (four 32 x 32 tiles): every global access is a full
// 128-byte (FP32) or 64-byte (BF16) row segment, the loads of a tile are issued before its
// arithmetic, and the transposed BF16 copy of D goes through shared memory.
constexpr int CU_TILES = 4;

__global__ void __launch_bounds__(256)
core_update_kernel(const CoreUpdateArgs *__restrict__ args, const int32_t *__restrict__ list, StepScalars sc, int mode,
                   int ntile)
{
    // ntile (1 .. CU_TILES) tiles of 32 x 32 per CTA: small launches take one, so that more CTAs share the work
    pdl_trigger();
    pdl_wait();
    const CoreUpdateArgs a = args[list[blockIdx.z]];
    const int r = a.r, nc = a.nc;   // rows, columns of the core (square except for a one-sided block)
    const int r0 = blockIdx.y * 32;
    if (r0 >= r || blockIdx.x * 32 * ntile >= nc) return;
    __shared__ float tile[CU_TILES][32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const bool sgd = (sc.rule == TSR_RULE_SGD);
#pragma unroll
    for (int tt = 0; tt < CU_TILES; ++tt) {
        if (tt >= ntile) break;
        const int c0 = (blockIdx.x * ntile + tt) * 32;
        const int col = c0 + tx;
        float c[4], m1[4], m2[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int row = r0 + ty + 8 * u;
            const bool in = (row < r && col < nc);
            const int64_t e = (int64_t)row * nc + col;
            c[u] = in ? a.C[e] : 0.f;
            if (in && a.nsplit > 1) {
                // slabs are added in slab order; eight loads are in flight at a time
                for (int s0 = 1; s0 < a.nsplit; s0 += 8) {
                    float part[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) part[j] = (s0 + j < a.nsplit) ? a.C[e + (int64_t)(s0 + j) * a.split_stride] : 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (s0 + j < a.nsplit) c[u] = __fadd_rn(c[u], part[j]);
                }
            }
            m1[u] = (in && mode == 0) ? a.mom1[e] : 0.f;
            m2[u] = (in && mode == 0 && !sgd) ? a.mom2[e] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int row = r0 + ty + 8 * u;
            const bool in = (row < r && col < nc);
            const int64_t e = (int64_t)row * nc + col;
            float d = 0.f;
            if (in) {
                if (a.nsplit > 1) a.Cout[e] = c[u];
                if (mode == 0) {
                    d = core_update_elem(c[u], m1[u], m2[u], sc);
                    a.mom1[e] = m1[u];
                    if (!sgd) a.mom2[e] = m2[u];
                    if (a.d_f32) a.d_f32[e] = d;
                    if (a.d_bf16) a.d_bf16[(int64_t)row * a.ldd + col] = __float2bfloat16_rn(d);
                }
            }
            tile[tt][ty + 8 * u][tx] = d;
        }
    }
    if (mode != 0 || a.dt_bf16 == nullptr) return;
    __syncthreads();
#pragma unroll
    for (int tt = 0; tt < CU_TILES; ++tt) {
        if (tt >= ntile) break;
        const int c0 = (blockIdx.x * ntile + tt) * 32;
        for (int i = ty; i < 32; i += 8) {
            const int col = c0 + i, row = r0 + tx;
            if (row < r && col < nc) a.dt_bf16[(int64_t)col * a.ldd + row] = __float2bfloat16_rn(tile[tt][tx][i]);
        }
    }
}

cudaError_t core_update_launch(const CoreUpdateArgs *args_dev, const int32_t *list_dev, int nblocks, int max_r,
                               int max_cols, const StepScalars &sc, int mode, cudaStream_t stream)
{
    if (nblocks <= 0) return cudaSuccess;
    const int t = (max_r + 31) / 32, tc = (max_cols + 31) / 32;
    const int ntile = ((int64_t)t * tc * nblocks >= 4 * 148 * CU_TILES) ? CU_TILES : 1;
    return launch_dependent(core_update_kernel, dim3((tc + ntile - 1) / ntile, t, nblocks), dim3(256), 0, stream, 1, args_dev, list_dev,
                            sc, mode, ntile);
}

// ---------------------------------------------------------------------------------------
// Operand conversion
// ---------------------------------------------------------------------------------------
// The transposing kernels below work on tiles of 64 rows x 32 columns: in the transposed copy a lane
// writes two consecutive rows as one 32-bit word, so a warp stores 128 contiguous bytes.  The row
// pitches of the transposed copies are multiples of 8 elements, which keeps those words aligned.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *(const uint32_t *)&h;
}

__global__ void shadows_kernel(const float *__restrict__ X, int rows, int r, bf16 *__restrict__ Xb, int64_t ldb,
                               bf16 *__restrict__ Xbt, int64_t ldt)
{
    __shared__ float tile[64][33];
    const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 32;
    for (int i = threadIdx.y; i < 64; i += blockDim.y) {
        const int row = r0 + i, col = c0 + threadIdx.x;
        float v = 0.f;
        if (row < rows && col < r) {
            v = X[(int64_t)row * r + col];
            if (Xb) Xb[(int64_t)row * ldb + col] = __float2bfloat16_rn(v);
        }
        tile[i][threadIdx.x] = v;
    }
    __syncthreads();
    if (Xbt) {
        for (int i = threadIdx.y; i < 32; i += blockDim.y) {
            const int col = c0 + i, row = r0 + 2 * threadIdx.x;
            if (col >= r || row >= rows) continue;
            bf16 *dst = Xbt + (int64_t)col * ldt + row;
            if (row + 1 < rows) *(uint32_t *)dst = pack_bf16x2(tile[2 * threadIdx.x][i], tile[2 * threadIdx.x + 1][i]);
            else *dst = __float2bfloat16_rn(tile[2 * threadIdx.x][i]);
        }
    }
}

cudaError_t make_shadows(const float *X, int rows, int r, bf16 *Xb, int64_t ldb, bf16 *Xbt, int64_t ldt,
                         cudaStream_t stream)
{
    dim3 grid((r + 31) / 32, (rows + 63) / 64);
    shadows_kernel<<<grid, dim3(32, 8), 0, stream>>>(X, rows, r, Xb, ldb, Xbt, ldt);
    return cudaGetLastError();
}

// X (rows x k) FP32 -> X^T as BF16 planes: hi = bf16(x), lo = bf16(x - hi).
__global__ void split_transpose_kernel(const float *__restrict__ X, int rows, int k, bf16 *__restrict__ out,
                                       int64_t ldo, int plane_rows, int planes)
{
    __shared__ float tile[64][33];
    const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 32;
    for (int i = threadIdx.y; i < 64; i += blockDim.y) {
        const int row = r0 + i, col = c0 + threadIdx.x;
        tile[i][threadIdx.x] = (row < rows && col < k) ? X[(int64_t)row * k + col] : 0.f;
    }
    __syncthreads();
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        const int col = c0 + i, row = r0 + 2 * threadIdx.x;
        if (col >= k || row >= rows) continue;
        const float v0 = tile[2 * threadIdx.x][i], v1 = tile[2 * threadIdx.x + 1][i];
        const bf16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
        bf16 *dhi = out + (int64_t)col * ldo + row;
        bf16 *dlo = out + ((int64_t)plane_rows + col) * ldo + row;
        if (row + 1 < rows) {
            *(uint32_t *)dhi = (uint32_t)(*(const uint16_t *)&h0) | ((uint32_t)(*(const uint16_t *)&h1) << 16);
            if (planes > 1) *(uint32_t *)dlo = pack_bf16x2(v0 - __bfloat162float(h0), v1 - __bfloat162float(h1));
        } else {
            *dhi = h0;
            if (planes > 1) *dlo = __float2bfloat16_rn(v0 - __bfloat162float(h0));
        }
    }
}

cudaError_t split_transpose(const float *X, int rows, int k, bf16 *out, int64_t ldo, int plane_rows, int planes,
                            cudaStream_t stream)
{
    dim3 grid((k + 31) / 32, (rows + 63) / 64);
    split_transpose_kernel<<<grid, dim3(32, 8), 0, stream>>>(X, rows, k, out, ldo, plane_rows, planes);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Counter-based N(0,1) generator for Omega (Algorithm 1, "Sample shared Omega (shared RNG
// seed)"): element e of stream `stream_id` hashes (seed, stream_id, e) with two rounds of a
// 64-bit mixer, then Box-Muller on the two 32-bit halves.  Independent of the launch shape.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__global__ void gaussian_kernel(float *__restrict__ out, int64_t count, uint64_t seed, uint64_t stream_id)
{
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += (int64_t)gridDim.x * blockDim.x) {
        const uint64_t h = mix64(mix64(seed ^ (stream_id * 0xD1342543DE82EF95ull)) + (uint64_t)e);
        const uint32_t a = (uint32_t)h, b = (uint32_t)(h >> 32);
        const float u1 = ((float)(a >> 8) + 0.5f) * (1.0f / 16777216.0f);  // (0,1)
        const float u2 = ((float)(b >> 8) + 0.5f) * (1.0f / 16777216.0f);
        out[e] = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
    }
}

cudaError_t fill_gaussian(float *out, int64_t count, uint64_t seed, uint64_t stream_id, cudaStream_t stream)
{
    if (count <= 0) return cudaSuccess;
    int64_t blocks = (count + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    gaussian_kernel<<<(int)blocks, 256, 0, stream>>>(out, count, seed, stream_id);
    return cudaGetLastError();
}

cudaError_t fill_zero_f32(float *p, int64_t count, cudaStream_t stream)
{
    return cudaMemsetAsync(p, 0, (size_t)count * sizeof(float), stream);
}

}  // namespace tsr
