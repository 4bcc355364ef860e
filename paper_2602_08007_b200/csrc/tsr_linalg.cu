// Small dense linear algebra of the subspace refresh (Section 3.5), batched over blocks:
// Gram matrices in FP64, Cholesky factor and its inverse (orth = Cholesky-QR applied twice),
// tall-times-small products, and a cyclic Jacobi eigen-solver on the k x k Gram matrix of B^T
// that yields the small SVD.
//
// All kernels are bounded loops; anything that goes wrong numerically (a non-positive pivot,
// a non-finite entry, the sweep limit) is written to the block's status word.
#include "tsr_internal.h"

namespace tsr {

// ---------------------------------------------------------------------------------------
// S = X^T X, X rows x k FP32, accumulation in FP64.  Rows are cut into slabs of GRAM_ROWS;
// each slab writes its own partial (upper-triangular part only), a second kernel adds the
// partials in slab order and mirrors the result, so the sum is deterministic.
// The products run on the FP64 tensor-core path (mma.sync m8n8k4: FP32 inputs convert to FP64
// exactly, FP64 fused accumulation): a CTA owns a 64 x 64 tile of S, its eight warps 32 x 16
// regions of it as 4 x 2 sub-tiles of 8 x 8.  Sub-tiles below the diagonal or past column k are
// skipped, so the work follows the upper triangle to a granularity of 8.
// ---------------------------------------------------------------------------------------
constexpr int GR_T = 64;   // output tile edge
constexpr int GR_S = 8;    // sub-tile edge (the MMA shape)
constexpr int GR_PITCH = 72;   // floats per staged row: 72 = 8 mod 32 keeps the fragment loads conflict-free

__device__ __forceinline__ void dmma_8x8x4(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c0), "+d"(c1)
                 : "d"(a), "d"(b));
}

__global__ void __launch_bounds__(256)
gram_partial_kernel(const RefreshDev *__restrict__ rd, const RowItem *__restrict__ items, int side, int src_sel)
{
    const RowItem it = items[blockIdx.z];
    const RefreshDev &d = rd[it.block];
    const int k = d.k;
    const int ti = blockIdx.y, tj = blockIdx.x;
    if (tj < ti || ti * GR_T >= k || tj * GR_T >= k) return;
    const int rows = side ? d.n : d.m;
    const float *__restrict__ X = d.buf[src_sel];
    __shared__ __align__(16) float Xi[16][GR_PITCH];
    __shared__ __align__(16) float Xj[16][GR_PITCH];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wi = warp >> 2, wj = warp & 3;         // warp grid 2 x 4: rows 32 wi .., columns 16 wj ..
    const int g = lane >> 2, q = lane & 3;           // fragment coordinates
    const int row_begin = it.row0;
    const int row_end = min(rows, row_begin + GRAM_ROWS);
    // which of the warp's 4 x 2 sub-tiles hold anything to compute
    bool need[4][2];
    bool any = false;
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            const int si = ti * (GR_T / GR_S) + wi * 4 + a, sj = tj * (GR_T / GR_S) + wj * 2 + b;
            need[a][b] = (sj >= si) && (si * GR_S < k) && (sj * GR_S < k);
            any = any || need[a][b];
        }
    double acc[4][2][2];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
    float ri[4], rj[4];
    auto fetch = [&](int r0) {
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = threadIdx.x + l * 256;
            const int rr = e / GR_T, cc = e % GR_T;
            const int row = r0 + rr;
            const int ci = ti * GR_T + cc, cj = tj * GR_T + cc;
            ri[l] = (row < row_end && ci < k) ? X[(int64_t)row * k + ci] : 0.f;
            rj[l] = (row < row_end && cj < k) ? X[(int64_t)row * k + cj] : 0.f;
        }
    };
    fetch(row_begin);
    for (int r0 = row_begin; r0 < row_end; r0 += 16) {
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = threadIdx.x + l * 256;
            Xi[e / GR_T][e % GR_T] = ri[l];
            Xj[e / GR_T][e % GR_T] = rj[l];
        }
        __syncthreads();
        if (r0 + 16 < row_end) fetch(r0 + 16);
        if (any) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {             // four rows of X per MMA
                double af[4], bf[2];
#pragma unroll
                for (int a = 0; a < 4; ++a) af[a] = (double)Xi[kk * 4 + q][wi * 32 + a * GR_S + g];
#pragma unroll
                for (int b = 0; b < 2; ++b) bf[b] = (double)Xj[kk * 4 + q][wj * 16 + b * GR_S + g];
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 2; ++b)
                        if (need[a][b]) dmma_8x8x4(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
            }
        }
        __syncthreads();
    }
    double *P = d.gpart + (int64_t)(it.row0 / GRAM_ROWS) * k * k;
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            if (!need[a][b]) continue;
            const int i = ti * GR_T + wi * 32 + a * GR_S + g;
            const int j = tj * GR_T + wj * 16 + b * GR_S + 2 * q;
            if (i < k && j < k) P[(int64_t)i * k + j] = acc[a][b][0];
            if (i < k && j + 1 < k) P[(int64_t)i * k + j + 1] = acc[a][b][1];
        }
}

// S = sum of the chunks' partial sums, in fixed order, for one 32 x 32 tile per CTA.  Only 8 x 8 sub-tiles on or
// above the diagonal were written: a tile below the diagonal is the transpose of its mirror image, a tile on the
// diagonal takes its lower sub-tiles from its own transpose (both through shared memory).
__global__ void __launch_bounds__(256)
gram_reduce_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int side)
{
    const RefreshDev &d = rd[list[blockIdx.z]];
    const int k = d.k;
    const int ti = blockIdx.y, tj = blockIdx.x;
    if (ti * 32 >= k || tj * 32 >= k) return;
    const int chunks = gram_chunks(side ? d.n : d.m);
    const int64_t total = (int64_t)k * k;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int si = ti <= tj ? ti : tj, sj = ti <= tj ? tj : ti;     // the tile that was written
    __shared__ double t[32][33];
    const double *__restrict__ gp = d.gpart;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int i = si * 32 + ty + 8 * u, j = sj * 32 + tx;
        double s = 0.0;
        if (i < k && j < k && (j / GR_S) >= (i / GR_S))
            for (int c = 0; c < chunks; ++c) s += gp[(int64_t)c * total + (int64_t)i * k + j];
        t[ty + 8 * u][tx] = s;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int li = ty + 8 * u, lj = tx;
        const int i = ti * 32 + li, j = tj * 32 + lj;
        if (i >= k || j >= k) continue;
        double v;
        if (ti < tj) v = t[li][lj];
        else if (ti > tj) v = t[lj][li];
        else v = (lj / GR_S) >= (li / GR_S) ? t[li][lj] : t[lj][li];
        d.S[(int64_t)i * k + j] = v;
    }
}

cudaError_t gram_batched(const RefreshDev *rd, const RowItem *items, int nitems, const int32_t *list, int nlist,
                         int side, int src_sel, int kmax, cudaStream_t stream)
{
    if (nitems <= 0 || nlist <= 0) return cudaSuccess;
    const int t = (kmax + GR_T - 1) / GR_T;
    gram_partial_kernel<<<dim3(t, t, nitems), 256, 0, stream>>>(rd, items, side, src_sel);
    return gram_reduce_batched(rd, list, nlist, side, kmax, stream);
}

cudaError_t gram_reduce_batched(const RefreshDev *rd, const int32_t *list, int nlist, int side, int kmax, cudaStream_t stream)
{
    if (nlist <= 0) return cudaSuccess;
    const int t = (kmax + 31) / 32;
    gram_reduce_kernel<<<dim3(t, t, nlist), 256, 0, stream>>>(rd, list, side);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Cholesky S = R^T R with R upper triangular (one CTA per matrix, FP64, in place), followed by
// Rinv = R^{-1} written as FP32.  Both halves are blocked by 16, synchronise the CTA a few times per
// block, and run their products on the FP64 tensor path (mma m8n8k4):
//   factorisation (right-looking): a 16-row panel of S sits in shared memory; one warp factors its
//   16 x 16 diagonal block R11 and inverts it in registers (lane = column, rows exchanged by
//   shuffles); the rest of the panel is R12 = R11^{-T} S12, one 16 x 8 tile of columns per warp
//   and trip; the trailing upper triangle then gets the rank-16 update S22 -= R12^T R12 in 8 x 8
//   tiles, a row of tiles per warp, eight tiles of S in flight per lane as 16-byte accesses (the
//   update is bound by the number of cache lines a warp visits, not by arithmetic);
//   inverse (X = R^{-1}, block rows from the bottom up): with the 16 rows of R staged in shared
//   memory, a warp accumulates the 16 x 8 tile sum_l R[I][l] X[l][c] over the rows l of X that are
//   already known (FP64 copy in Xw) and multiplies it by -R11^{-1} through a private patch.
// A pivot that is not safely positive is replaced by a floor relative to the largest diagonal
// entry and the block is flagged TSR_ERR_RANK_DEFICIENT.
// ---------------------------------------------------------------------------------------
constexpr int CH_NB = 16;
constexpr int CH_THREADS = 512;

__global__ void __launch_bounds__(CH_THREADS)
chol_inverse_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int kpad)
{
    extern __shared__ __align__(16) double ch_smem[];   // P[CH_NB][kpad], then a 16 x 8 patch per warp
    const RefreshDev d = rd[list[blockIdx.x]];
    const int k = d.k;
    double *__restrict__ S = d.S;
    double *__restrict__ X = d.Xw;
    double *P = ch_smem;
    __shared__ double dinv[CH_NB][CH_NB + 1];    // inverse of the current diagonal block (upper triangular)
    __shared__ double s_floor;
    __shared__ int s_flag;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int warp = tid >> 5, lane = tid & 31, nwarps = nt >> 5;
    if (warp == 0) {
        double mx = 0.0;
        int bad = 0;
        for (int i = lane; i < k; i += 32) {
            const double v = S[(int64_t)i * k + i];
            if (!(v == v) || v > 1e300 || v < -1e300) bad = 1;
            if (v > mx) mx = v;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            bad |= __shfl_xor_sync(0xffffffffu, bad, off);
        }
        if (lane == 0) {
            s_floor = mx * 1e-13;
            if (!(s_floor > 0.0)) s_floor = 1e-300;
            s_flag = bad ? TSR_ERR_NONFINITE : 0;
        }
    }
    __syncthreads();
    // ---- factorisation
    for (int jb = 0; jb < k; jb += CH_NB) {
        const int nb = min(CH_NB, k - jb);
        const int w = k - jb;                       // panel width: columns jb..k-1
        for (int e = tid; e < nb * w; e += nt) {    // P[j][c] = S[jb + j][jb + c]
            const int j = e / w, c = e - j * w;
            P[j * kpad + c] = (c >= j) ? S[(int64_t)(jb + j) * k + jb + c] : 0.0;
        }
        __syncthreads();
        if (warp == 0) {
            // The nb x nb diagonal block and its inverse, in registers: lane c (< 16) holds column c of the
            // block; row j of the factor reaches the other lanes by shuffles (all loops unrolled, so every
            // register index is static).  Lanes 16..31 only take part in the shuffles.
            const double floor_v = s_floor;
            const int c = lane & 15;
            double col[CH_NB], rinv_d[CH_NB];
#pragma unroll
            for (int i = 0; i < CH_NB; ++i) col[i] = (i <= c && c < nb && i < nb) ? P[i * kpad + c] : 0.0;
            bool floored = false;
#pragma unroll
            for (int j = 0; j < CH_NB; ++j) {
                rinv_d[j] = 0.0;
                if (j < nb) {                                   // uniform over the warp
                    double v = __shfl_sync(0xffffffffu, col[j], j);
                    if (!(v > floor_v)) { floored = true; v = floor_v; }
                    const double rpiv = rsqrt(v);
                    const double piv = v * rpiv;
                    rinv_d[j] = rpiv;
                    col[j] = (c == j) ? piv : col[j] * rpiv;    // R[j][c] for c >= j (zero for c < j)
#pragma unroll
                    for (int i = j + 1; i < CH_NB; ++i) {
                        const double rji = __shfl_sync(0xffffffffu, col[j], i);   // R[j][i]
                        col[i] -= rji * col[j];                 // only entries with c >= i are used later
                    }
                }
            }
            if (floored && lane == 0 && s_flag == 0) s_flag = TSR_ERR_RANK_DEFICIENT;
            // column c of R11^{-1} by back substitution; R[i][l] comes from lane l
            double x[CH_NB];
#pragma unroll
            for (int i = CH_NB - 1; i >= 0; --i) {
                double acc = (i == c) ? 1.0 : 0.0;
#pragma unroll
                for (int l = i + 1; l < CH_NB; ++l) {
                    const double ril = __shfl_sync(0xffffffffu, col[i], l);
                    if (l <= c) acc -= ril * x[l];
                }
                x[i] = (i <= c && c < nb && i < nb) ? acc * rinv_d[i] : 0.0;
            }
            if (lane < CH_NB) {
#pragma unroll
                for (int i = 0; i < CH_NB; ++i) {
                    if (i <= c && c < nb) P[i * kpad + c] = col[i];
                    dinv[i][c] = x[i];
                    if (i < nb && c < nb) {
                        X[(int64_t)(jb + i) * k + jb + c] = x[i];
                        d.Rinv[(int64_t)(jb + i) * k + jb + c] = (float)x[i];
                    }
                }
            }
        }
        __syncthreads();
        {   // R12 = R11^{-T} S12 on the FP64 tensor path: (16 x 16 lower triangular) times 16 x 8 column tiles,
            // in place (a tile's columns belong to one warp, which reads them before it writes)
            const int g = lane >> 2, q = lane & 3;
            for (int c0 = nb + 8 * warp; c0 < w; c0 += 8 * nwarps) {
                double bfr[4];
#pragma unroll
                for (int st = 0; st < 4; ++st) bfr[st] = P[(4 * st + q) * kpad + min(c0 + g, w - 1)];
                double y[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
#pragma unroll
                for (int st = 0; st < 4; ++st) {
                    if (st < 2) dmma_8x8x4(y[0][0], y[0][1], dinv[4 * st + q][g], bfr[st]);   // rows 0..7 end at l = 7
                    dmma_8x8x4(y[1][0], y[1][1], dinv[4 * st + q][8 + g], bfr[st]);
                }
                __syncwarp();
#pragma unroll
                for (int jt = 0; jt < 2; ++jt)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int col = c0 + 2 * q + h;
                        if (col < w) P[(jt * 8 + g) * kpad + col] = y[jt][h];
                    }
            }
        }
        __syncthreads();
        for (int e = tid; e < nb * w; e += nt) {    // the finished rows of R
            const int j = e / w, c = e - j * w;
            if (c >= j) S[(int64_t)(jb + j) * k + jb + c] = P[j * kpad + c];
        }
        // rank-nb update of the trailing upper triangle on the FP64 tensor path: S22 -= R12^T R12 in
        // 8 x 8 tiles (mma m8n8k4, four steps over the 16 panel rows).  A warp owns the row tiles
        // warp, warp + nwarps, ... and takes eight column tiles per trip, all their loads issued
        // before the first product (the update is bound by the latency of those loads).  Tiles that
        // straddle the diagonal are updated whole: entries below the diagonal are never read.
        if (nb == CH_NB) {
            const int g = lane >> 2, q = lane & 3;
            const int nt8 = (k + 7) >> 3;
            const bool k_even = (k & 1) == 0;   // then every pair (l, l + 1) with l even is 16-byte aligned and inside the row
            for (int ti = ((jb + CH_NB) >> 3) + warp; ti < nt8; ti += nwarps) {
                const int row = ti * 8 + g;
                const bool row_ok = row < k;
                double af[4];
#pragma unroll
                for (int st = 0; st < 4; ++st) af[st] = P[(4 * st + q) * kpad + min(row, k - 1) - jb];
                double *srow = S + (int64_t)min(row, k - 1) * k;
                double cv[8][2], nv[8][2];
                auto cload = [&](int tj0, double (&v)[8][2]) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int l = (tj0 + u) * 8 + 2 * q;
                        if (k_even) {   // both entries as one 16-byte access: half as many cache-line visits
                            const double2 t = (row_ok && l < k) ? *(const double2 *)(srow + l) : make_double2(0.0, 0.0);
                            v[u][0] = t.x; v[u][1] = t.y;
                        } else {
                            v[u][0] = (row_ok && l < k) ? srow[l] : 0.0;
                            v[u][1] = (row_ok && l + 1 < k) ? srow[l + 1] : 0.0;
                        }
                    }
                };
                cload(ti, cv);
                for (int tj0 = ti; tj0 < nt8; tj0 += 8) {
                    cload(tj0 + 8, nv);              // the next trip's tiles are in flight during this trip's products
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (tj0 + u < nt8) {
                            double a0 = 0.0, a1 = 0.0, b0 = 0.0, b1 = 0.0;   // two chains of two products each
#pragma unroll
                            for (int st = 0; st < 4; ++st) {
                                const double bfr = P[(4 * st + q) * kpad + min((tj0 + u) * 8 + g, k - 1) - jb];
                                if (st & 1) dmma_8x8x4(b0, b1, af[st], bfr);
                                else dmma_8x8x4(a0, a1, af[st], bfr);
                            }
                            const int l = (tj0 + u) * 8 + 2 * q;
                            if (k_even) {
                                if (row_ok && l < k) *(double2 *)(srow + l) = make_double2(cv[u][0] - (a0 + b0), cv[u][1] - (a1 + b1));
                            } else {
                                if (row_ok && l < k) srow[l] = cv[u][0] - (a0 + b0);
                                if (row_ok && l + 1 < k) srow[l + 1] = cv[u][1] - (a1 + b1);
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) { cv[u][0] = nv[u][0]; cv[u][1] = nv[u][1]; }
                }
            }
        }
        __syncthreads();
    }
    // ---- X = R^{-1}, block rows from the bottom up (the diagonal blocks are already in place)
    const int nblk = (k + CH_NB - 1) / CH_NB;
    for (int I = nblk - 1; I >= 0; --I) {
        const int i0 = I * CH_NB, nb = min(CH_NB, k - i0);
        const int l0 = i0 + nb;                      // first row of X that is already known (a multiple of 16)
        for (int e = tid; e < nb * (k - l0); e += nt) {   // P[j][c] = R[i0 + j][c], c >= l0
            const int j = e / (k - l0), c = l0 + (e - j * (k - l0));
            P[j * kpad + c] = S[(int64_t)(i0 + j) * k + c];
        }
        if (tid < 4 * CH_NB) P[(tid >> 2) * kpad + k + (tid & 3)] = 0.0;   // a group may reach three columns past k - 1
        if (tid < CH_NB * CH_NB) {
            const int i = tid / CH_NB, c = tid % CH_NB;
            dinv[i][c] = (i < nb && c < nb && c >= i) ? X[(int64_t)(i0 + i) * k + i0 + c] : 0.0;
        }
        __syncthreads();
        {   // acc = R[I][l0 ..] X[l0 .., c] on the FP64 tensor path: a warp owns 16 x 8 tiles of columns
            // (two mma row tiles) and runs over l in steps of four; X is zero below its diagonal, so the
            // sum stops at the last column of the tile.  Eight steps of X values are in flight per lane.
            const int g = lane >> 2, q = lane & 3;
            const int nct = (k - l0 + 7) >> 3;
            double *patch = ch_smem + CH_NB * kpad + warp * 128;    // 16 x 8, private to the warp
            for (int ct = warp; ct < nct; ct += nwarps) {
                const int c0 = l0 + ct * 8;
                const int cg = min(c0 + g, k - 1);                  // columns past k - 1 are computed and dropped
                const int lend = min(c0 + 8, k);
                double lo0 = 0.0, lo1 = 0.0, hi0 = 0.0, hi1 = 0.0;
                auto bload = [&](int l) -> double {
                    const int row = l + q;
                    return (row < lend) ? X[(int64_t)row * k + cg] : 0.0;
                };
                double bq[8], nq[8];
#pragma unroll
                for (int pp = 0; pp < 8; ++pp) bq[pp] = bload(l0 + 4 * pp);
                for (int l = l0; l < lend; l += 32) {
#pragma unroll
                    for (int pp = 0; pp < 8; ++pp) nq[pp] = bload(l + 32 + 4 * pp);
#pragma unroll
                    for (int pp = 0; pp < 8; ++pp) {
                        const int ll = l + 4 * pp;
                        if (ll < lend) {
                            const double a_lo = P[g * kpad + ll + q], a_hi = P[(8 + g) * kpad + ll + q];
                            dmma_8x8x4(lo0, lo1, a_lo, bq[pp]);
                            dmma_8x8x4(hi0, hi1, a_hi, bq[pp]);
                        }
                    }
#pragma unroll
                    for (int pp = 0; pp < 8; ++pp) bq[pp] = nq[pp];
                }
                // X[I][c] = -R11^{-1} acc: the tile goes through the patch to become the B operand
                patch[g * 8 + 2 * q] = lo0; patch[g * 8 + 2 * q + 1] = lo1;
                patch[(8 + g) * 8 + 2 * q] = hi0; patch[(8 + g) * 8 + 2 * q + 1] = hi1;
                __syncwarp();
                double y[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
#pragma unroll
                for (int st = 0; st < 4; ++st) {
                    const double bfr = patch[(4 * st + q) * 8 + g];
                    dmma_8x8x4(y[0][0], y[0][1], dinv[g][4 * st + q], bfr);
                    if (st >= 2) dmma_8x8x4(y[1][0], y[1][1], dinv[8 + g][4 * st + q], bfr);   // R11^{-1} is upper triangular
                }
#pragma unroll
                for (int jt = 0; jt < 2; ++jt) {
                    const int j = jt * 8 + g;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int col = c0 + 2 * q + h;
                        if (j < nb && col < k) {
                            const double v = -y[jt][h];
                            X[(int64_t)(i0 + j) * k + col] = v;
                            d.Rinv[(int64_t)(i0 + j) * k + col] = (float)v;
                        }
                    }
                }
                __syncwarp();
            }
        }
        for (int e = tid; e < nb * i0; e += nt) {    // zeros left of the diagonal block
            const int j = e / i0, c = e - j * i0;
            X[(int64_t)(i0 + j) * k + c] = 0.0;
            d.Rinv[(int64_t)(i0 + j) * k + c] = 0.f;
        }
        __syncthreads();
    }
    if (tid == 0 && s_flag != 0) atomicMax(d.status, s_flag);
}

cudaError_t chol_inverse_batched(const RefreshDev *rd, const int32_t *list, int nlist, int kmax, cudaStream_t stream)
{
    if (nlist <= 0) return cudaSuccess;
    const int kpad = (kmax + 5) & ~1;   // even row pitch (in doubles): pairs of a row are read as one 16-byte word
    const size_t bytes = ((size_t)CH_NB * kpad + (CH_THREADS / 32) * 128) * sizeof(double);   // panel + one 16 x 8 patch per warp
    static size_t configured = 0;
    if (bytes > configured) {
        cudaError_t e = cudaFuncSetAttribute(chol_inverse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) return e;
        configured = bytes;
    }
    chol_inverse_kernel<<<nlist, CH_THREADS, bytes, stream>>>(rd, list, kpad);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// dst[rows x N] = src[rows x k] * Mat[k x N]   (FP32; 128 x 64 tiles, one slab of RG_ROWS = 128 rows
// per item, 8 x 4 outputs per thread)
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
rows_gemm_kernel(const RefreshDev *__restrict__ rd, const RowItem *__restrict__ items, int side, int src_sel,
                 int mat_sel, int dst_sel)
{
    const RowItem it = items[blockIdx.y];
    const RefreshDev &d = rd[it.block];
    const int K = d.k;
    const int N = (mat_sel == 0) ? d.k : d.r;
    const int n0 = blockIdx.x * 64;
    if (n0 >= N) return;
    const int rows = side ? d.n : d.m;
    const float *__restrict__ A = d.buf[src_sel];
    const float *__restrict__ B = (mat_sel == 0) ? d.Rinv : (mat_sel == 1 ? d.Wu : d.Wv);
    float *__restrict__ D = (dst_sel < 3) ? d.buf[dst_sel] : (dst_sel == 3 ? d.U : d.V);
    const int m0 = it.row0;

    __shared__ __align__(16) float As[16][RG_ROWS + 4];
    __shared__ __align__(16) float Bs[16][64 + 4];
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    float acc[8][4];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    // global -> registers -> shared, with the next K slice in flight while the current one is used
    float ra[8], rb[4];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int l = 0; l < 8; ++l) {
            const int e = tid + l * 256;
            const int ak = e % 16, ai = e / 16;
            const int gi = m0 + ai, gk = k0 + ak;
            ra[l] = (gi < rows && gk < K) ? A[(int64_t)gi * K + gk] : 0.f;
        }
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = tid + l * 256;
            const int bj = e % 64, bk = e / 64;
            const int gj = n0 + bj, gk2 = k0 + bk;
            rb[l] = (gj < N && gk2 < K) ? B[(int64_t)gk2 * N + gj] : 0.f;
        }
    };
    // Rinv is upper triangular: columns n0 .. n0 + 63 of the product only need rows 0 .. n0 + 63 of it
    const int Kend = (mat_sel == 0) ? min(K, n0 + 64) : K;
    fetch(0);
    for (int k0 = 0; k0 < Kend; k0 += 16) {
#pragma unroll
        for (int l = 0; l < 8; ++l) {
            const int e = tid + l * 256;
            As[e % 16][e / 16] = ra[l];
        }
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = tid + l * 256;
            Bs[e / 64][e % 64] = rb[l];
        }
        __syncthreads();
        if (k0 + 16 < Kend) fetch(k0 + 16);
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            const float4 a0 = *(const float4 *)&As[kk][ty * 8];
            const float4 a1 = *(const float4 *)&As[kk][ty * 8 + 4];
            const float4 bf = *(const float4 *)&Bs[kk][tx * 4];
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float bv[4] = {bf.x, bf.y, bf.z, bf.w};
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        const int gi = m0 + ty * 8 + a;
        if (gi >= rows) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int gj = n0 + tx * 4 + b;
            if (gj < N) D[(int64_t)gi * N + gj] = acc[a][b];
        }
    }
}

// The same product on 128 x 128 tiles (8 x 8 outputs per thread as four 4 x 4 quadrants, two shared-memory
// stages so that a K slice costs one barrier): used when the small matrix is at least 512 columns wide,
// where the wider tile nearly halves the shared-memory traffic per multiply-add.
__global__ void __launch_bounds__(256, 2)
rows_gemm128_kernel(const RefreshDev *__restrict__ rd, const RowItem *__restrict__ items, int side, int src_sel,
                    int mat_sel, int dst_sel)
{
    const RowItem it = items[blockIdx.y];
    const RefreshDev &d = rd[it.block];
    const int K = d.k;
    const int N = (mat_sel == 0) ? d.k : d.r;
    const int n0 = blockIdx.x * 128;
    if (n0 >= N) return;
    const int rows = side ? d.n : d.m;
    const float *__restrict__ A = d.buf[src_sel];
    const float *__restrict__ B = (mat_sel == 0) ? d.Rinv : (mat_sel == 1 ? d.Wu : d.Wv);
    float *__restrict__ D = (dst_sel < 3) ? d.buf[dst_sel] : (dst_sel == 3 ? d.U : d.V);
    const int m0 = it.row0;

    __shared__ __align__(16) float As[2][16][128 + 4];
    __shared__ __align__(16) float Bs[2][16][128 + 4];
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    float acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = 0.f;
    const bool a_vec = (K & 3) == 0, b_vec = (N & 3) == 0;
    float4 ra[2], rb[2];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int l = 0; l < 2; ++l) {
            const int e = tid + l * 256;
            {   // A: row e / 4 of the tile, four consecutive k
                const int ai = e >> 2, gk = k0 + 4 * (e & 3), gi = m0 + ai;
                const float *src = A + (int64_t)gi * K + gk;
                if (gi < rows && a_vec && gk + 3 < K) ra[l] = *(const float4 *)src;
                else {
                    ra[l].x = (gi < rows && gk < K) ? src[0] : 0.f;
                    ra[l].y = (gi < rows && gk + 1 < K) ? src[1] : 0.f;
                    ra[l].z = (gi < rows && gk + 2 < K) ? src[2] : 0.f;
                    ra[l].w = (gi < rows && gk + 3 < K) ? src[3] : 0.f;
                }
            }
            {   // B: k row e / 32 of the slice, four consecutive columns
                const int bk = e >> 5, gj = n0 + 4 * (e & 31), gk = k0 + bk;
                const float *src = B + (int64_t)gk * N + gj;
                if (gk < K && b_vec && gj + 3 < N) rb[l] = *(const float4 *)src;
                else {
                    rb[l].x = (gk < K && gj < N) ? src[0] : 0.f;
                    rb[l].y = (gk < K && gj + 1 < N) ? src[1] : 0.f;
                    rb[l].z = (gk < K && gj + 2 < N) ? src[2] : 0.f;
                    rb[l].w = (gk < K && gj + 3 < N) ? src[3] : 0.f;
                }
            }
        }
    };
    auto stage = [&](int buf) {
#pragma unroll
        for (int l = 0; l < 2; ++l) {
            const int e = tid + l * 256;
            const int ai = e >> 2, ak = 4 * (e & 3);
            As[buf][ak][ai] = ra[l].x; As[buf][ak + 1][ai] = ra[l].y; As[buf][ak + 2][ai] = ra[l].z; As[buf][ak + 3][ai] = ra[l].w;
            *(float4 *)&Bs[buf][e >> 5][4 * (e & 31)] = rb[l];
        }
    };
    // Rinv is upper triangular: columns n0 .. n0 + 127 of the product only need rows 0 .. n0 + 127 of it
    const int Kend = (mat_sel == 0) ? min(K, n0 + 128) : K;
    fetch(0);
    stage(0);
    __syncthreads();
    int buf = 0;
    for (int k0 = 0; k0 < Kend; k0 += 16, buf ^= 1) {
        const bool more = k0 + 16 < Kend;
        if (more) fetch(k0 + 16);
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            const float4 a0 = *(const float4 *)&As[buf][kk][ty * 4];
            const float4 a1 = *(const float4 *)&As[buf][kk][64 + ty * 4];
            const float4 b0 = *(const float4 *)&Bs[buf][kk][tx * 4];
            const float4 b1 = *(const float4 *)&Bs[buf][kk][64 + tx * 4];
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
                for (int b = 0; b < 8; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
        }
        if (more) stage(buf ^ 1);    // the other stage was last read before the previous barrier
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        const int gi = m0 + (a < 4 ? ty * 4 + a : 64 + ty * 4 + (a - 4));
        if (gi >= rows) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int gj = n0 + h * 64 + tx * 4;
            float *dst = D + (int64_t)gi * N + gj;
            if (b_vec && gj + 3 < N) {
                *(float4 *)dst = make_float4(acc[a][4 * h], acc[a][4 * h + 1], acc[a][4 * h + 2], acc[a][4 * h + 3]);
            } else {
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    if (gj + b < N) dst[b] = acc[a][4 * h + b];
                }
            }
        }
    }
}

cudaError_t rows_gemm_batched(const RefreshDev *rd, const RowItem *items, int nitems, int side, int src_sel,
                              int mat_sel, int dst_sel, int nmax, cudaStream_t stream)
{
    if (nitems <= 0) return cudaSuccess;
    if (nmax >= 512)
        rows_gemm128_kernel<<<dim3((nmax + 127) / 128, nitems), 256, 0, stream>>>(rd, items, side, src_sel, mat_sel, dst_sel);
    else
        rows_gemm_kernel<<<dim3((nmax + 63) / 64, nitems), 256, 0, stream>>>(rd, items, side, src_sel, mat_sel, dst_sel);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Operand planes for the tensor-core form of dst = buf[src] * Mat (three TF32 products).
// Every FP32 value x is written as hi = x with the low 13 mantissa bits cleared (a TF32 number) and
// lo = x - hi (exact).  Rows: Xs[row][c] = hi, Xs[mx + row][c] = lo with mx = max(m, n).
// Small matrix, transposed so that the contraction index is contiguous: Bts[j][l] = hi(Mat[l][j]),
// Bts[k + j][l] = lo(Mat[l][j]).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float tf32_hi(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

__global__ void __launch_bounds__(256)
split_rows_kernel(const RefreshDev *__restrict__ rd, const RowItem *__restrict__ items, int side, int src_sel)
{
    const RowItem it = items[blockIdx.x];
    const RefreshDev &d = rd[it.block];
    const int k = d.k;
    const int rows = side ? d.n : d.m;
    const int64_t mx = max(d.m, d.n);
    const int nrow = min(RG_ROWS, rows - it.row0);
    const float4 *__restrict__ X = (const float4 *)(d.buf[src_sel] + (int64_t)it.row0 * k);
    float4 *__restrict__ H = (float4 *)(d.Xs + (int64_t)it.row0 * k);
    float4 *__restrict__ Lo = (float4 *)(d.Xs + (mx + it.row0) * k);
    const int n4 = nrow * k / 4;                  // k is a multiple of 4 on this path
    for (int e = threadIdx.x; e < n4; e += 256) {
        const float4 x = X[e];
        float4 h, l;
        h.x = tf32_hi(x.x); h.y = tf32_hi(x.y); h.z = tf32_hi(x.z); h.w = tf32_hi(x.w);
        l.x = x.x - h.x; l.y = x.y - h.y; l.z = x.z - h.z; l.w = x.w - h.w;
        H[e] = h;
        Lo[e] = l;
    }
}

__global__ void __launch_bounds__(256)
split_mat_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int mat_sel)
{
    const RefreshDev d = rd[list[blockIdx.z]];
    const int k = d.k;
    const int N = (mat_sel == 0) ? d.k : d.r;
    const int l0 = blockIdx.y * 32, j0 = blockIdx.x * 32;   // Mat[l][j], l < k, j < N
    if (l0 >= k || j0 >= N) return;
    const float *__restrict__ M = (mat_sel == 0) ? d.Rinv : (mat_sel == 1 ? d.Wu : d.Wv);
    __shared__ float t[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int a = ty; a < 32; a += 8) {
        const int l = l0 + a, j = j0 + tx;
        t[a][tx] = (l < k && j < N) ? M[(int64_t)l * N + j] : 0.f;
    }
    __syncthreads();
    for (int a = ty; a < 32; a += 8) {
        const int j = j0 + a, l = l0 + tx;
        if (j < N && l < k) {
            const float x = t[tx][a], h = tf32_hi(x);
            d.Bts[(int64_t)j * k + l] = h;
            d.Bts[(int64_t)(k + j) * k + l] = x - h;
        }
    }
}

cudaError_t split_operands_batched(const RefreshDev *rd, const RowItem *items, int nitems, const int32_t *list, int nlist,
                                   int side, int src_sel, int mat_sel, int kmax, cudaStream_t stream)
{
    if (nitems <= 0 || nlist <= 0) return cudaSuccess;
    split_rows_kernel<<<nitems, 256, 0, stream>>>(rd, items, side, src_sel);
    const int t = (kmax + 31) / 32;
    split_mat_kernel<<<dim3(t, t, nlist), 256, 0, stream>>>(rd, list, mat_sel);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Cyclic Jacobi eigen-solver for a symmetric k x k matrix (FP64), one CTA per matrix.
// Round-robin ordering: every round rotates k/2 disjoint index pairs at once; the two-sided
// update S <- J^T S J is done on 2 x 2 blocks (pair A rows x pair B columns), the eigenvector
// accumulation W <- W J on rows of W.  Stops after a sweep without any rotation, or after
// max_sweeps (then flags TSR_ERR_NOT_CONVERGED).
// Afterwards eigenvalues are ranked in descending order and the leading r eigenvectors are
// written out: Wu = W[:, :r]; Wv = W[:, :r] / sqrt(lambda)  (B^T W / sigma = right vectors).
// ---------------------------------------------------------------------------------------
constexpr int JAC_MAX_K = 1056;

__global__ void __launch_bounds__(1024)
jacobi_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int max_sweeps)
{
    const RefreshDev d = rd[list[blockIdx.x]];
    const int k = d.k, r = d.r;
    double *__restrict__ S = d.S;
    double *__restrict__ W = d.Wj;
    __shared__ double s_c[JAC_MAX_K / 2], s_s[JAC_MAX_K / 2];
    __shared__ short s_p[JAC_MAX_K / 2], s_q[JAC_MAX_K / 2];
    __shared__ int s_rot;
    __shared__ int s_flag;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int ke = (k + 1) & ~1;  // even number of slots; slot k (if any) is a bye
    const int np = ke / 2;

    for (int64_t e = tid; e < (int64_t)k * k; e += nt) W[e] = ((e / k) == (e % k)) ? 1.0 : 0.0;
    if (tid == 0) s_flag = 0;
    __syncthreads();

    bool converged = false;
    const int sweep_limit = d.max_sweeps > 0 ? d.max_sweeps : max_sweeps;   // per-block limit, when one was set
    for (int sweep = 0; sweep < sweep_limit && !converged; ++sweep) {
        if (tid == 0) s_rot = 0;
        __syncthreads();
        for (int round = 0; round < ke - 1; ++round) {
            for (int i = tid; i < np; i += nt) {
                int a, b;
                if (i == 0) { a = ke - 1; b = round % (ke - 1); }
                else { a = (round + i) % (ke - 1); b = (round + ke - 1 - i) % (ke - 1); }
                int p = min(a, b), q = max(a, b);
                double c = 1.0, s = 0.0;
                if (q < k) {
                    const double spp = S[(int64_t)p * k + p], sqq = S[(int64_t)q * k + q], spq = S[(int64_t)p * k + q];
                    if (spq != 0.0 && fabs(spq) > 1e-15 * sqrt(fabs(spp * sqq))) {
                        const double zeta = (sqq - spp) / (2.0 * spq);
                        const double t = ((zeta >= 0.0) ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                        c = 1.0 / sqrt(1.0 + t * t);
                        s = c * t;
                        atomicAdd(&s_rot, 1);
                    }
                } else {
                    q = -1;  // bye: p has no partner this round
                }
                s_c[i] = c; s_s[i] = s; s_p[i] = (short)p; s_q[i] = (short)q;
            }
            __syncthreads();
            // S <- J^T S J on 2 x 2 blocks; every entry belongs to exactly one (A, B) block
            for (int e = tid; e < np * np; e += nt) {
                const int A = e / np, B = e % np;
                const int pA = s_p[A], qA = s_q[A], pB = s_p[B], qB = s_q[B];
                const double cA = s_c[A], sA = s_s[A], cB = s_c[B], sB = s_s[B];
                if (sA == 0.0 && sB == 0.0) continue;
                if (qA < 0 && qB < 0) continue;
                if (qA < 0) {  // single row pA, column pair B
                    const double x = S[(int64_t)pA * k + pB], y = S[(int64_t)pA * k + qB];
                    S[(int64_t)pA * k + pB] = cB * x - sB * y;
                    S[(int64_t)pA * k + qB] = sB * x + cB * y;
                    continue;
                }
                if (qB < 0) {  // row pair A, single column pB
                    const double x = S[(int64_t)pA * k + pB], y = S[(int64_t)qA * k + pB];
                    S[(int64_t)pA * k + pB] = cA * x - sA * y;
                    S[(int64_t)qA * k + pB] = sA * x + cA * y;
                    continue;
                }
                double x00 = S[(int64_t)pA * k + pB], x01 = S[(int64_t)pA * k + qB];
                double x10 = S[(int64_t)qA * k + pB], x11 = S[(int64_t)qA * k + qB];
                const double r00 = cA * x00 - sA * x10, r01 = cA * x01 - sA * x11;  // rows: J_A^T
                const double r10 = sA * x00 + cA * x10, r11 = sA * x01 + cA * x11;
                x00 = cB * r00 - sB * r01; x01 = sB * r00 + cB * r01;                // columns: J_B
                x10 = cB * r10 - sB * r11; x11 = sB * r10 + cB * r11;
                if (A == B) { x01 = 0.0; x10 = 0.0; }
                S[(int64_t)pA * k + pB] = x00; S[(int64_t)pA * k + qB] = x01;
                S[(int64_t)qA * k + pB] = x10; S[(int64_t)qA * k + qB] = x11;
            }
            // W <- W J
            for (int e = tid; e < k * np; e += nt) {
                const int i = e / np, B = e % np;
                const int qB = s_q[B];
                const double sB = s_s[B];
                if (qB < 0 || sB == 0.0) continue;
                const int pB = s_p[B];
                const double cB = s_c[B];
                const double x = W[(int64_t)i * k + pB], y = W[(int64_t)i * k + qB];
                W[(int64_t)i * k + pB] = cB * x - sB * y;
                W[(int64_t)i * k + qB] = sB * x + cB * y;
            }
            __syncthreads();
        }
        converged = (s_rot == 0);
        __syncthreads();
    }
    if (tid == 0 && !converged) s_flag = TSR_ERR_NOT_CONVERGED;
    __syncthreads();

    // rank eigenvalues (descending; ties by index) and emit the leading r columns
    for (int j = tid; j < k; j += nt) {
        const double lj = S[(int64_t)j * k + j];
        if (!(lj == lj)) s_flag = TSR_ERR_NONFINITE;
        int rank = 0;
        for (int l = 0; l < k; ++l) {
            const double ll = S[(int64_t)l * k + l];
            rank += (ll > lj || (ll == lj && l < j)) ? 1 : 0;
        }
        d.lam[rank] = lj;
        if (rank < r) {
            double inv = 0.0;
            if (lj > 1e-300) inv = 1.0 / sqrt(lj);
            else s_flag = TSR_ERR_RANK_DEFICIENT;
            for (int i = 0; i < k; ++i) {
                const double w = W[(int64_t)i * k + j];
                d.Wu[(int64_t)i * r + rank] = (float)w;
                d.Wv[(int64_t)i * r + rank] = (float)(w * inv);
            }
        }
    }
    __syncthreads();
    if (tid == 0 && s_flag != 0) atomicMax(d.status, s_flag);
}

cudaError_t jacobi_batched(const RefreshDev *rd, const int32_t *list, int nlist, int max_sweeps, cudaStream_t stream)
{
    if (nlist <= 0) return cudaSuccess;
    jacobi_kernel<<<nlist, 1024, 0, stream>>>(rd, list, max_sweeps);
    return cudaGetLastError();
}

}  // namespace tsr
