// Internal declarations shared by the translation units of libtsr (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "tsr.h"

namespace tsr {

typedef __nv_bfloat16 bf16;

inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// ---------------------------------------------------------------------------------------
// Tensor-core grouped GEMM:  D[M x N] = A[M x K] * B[N x K]^T, both operands BF16 with K
// contiguous ("K-major"), FP32 accumulation in tensor memory.  B may come as two planes
// (hi + lo) that are accumulated into the same D.  planes = 3 selects FP32 data as three TF32
// products (both operands in a truncated and a remainder plane, K blocks of 32 elements).
// ---------------------------------------------------------------------------------------
enum UmmaEpilogue : int {
    EPI_STORE_F32 = 0,     // out_f32[row * ld + col] = acc
    EPI_STORE_BF16 = 1,    // out_bf16[row * ld + col] = bf16(acc)
    EPI_STORE_BF16_T = 2,  // out_bf16[col * ld + row] = bf16(acc)          (transposed)
    EPI_CORE_UPDATE = 3,   // acc is a tile of the core C: write C, update M / Vm, write D, D^T as BF16
    EPI_APPLY = 4,         // W[row * ld + col] = decay * W - step_scale * acc
    EPI_RUNTIME = 5        // kernel instantiation whose epilogue is chosen per tile (the merged projection launch)
};

struct alignas(64) UmmaProblem {
    CUtensorMap tmA;       // box 64 (K) x 128 (M rows), 128-byte swizzle
    CUtensorMap tmB;       // box 64 (K) x BN (N rows); plane 1 lives plane_rows rows below plane 0
    CUtensorMap tmW;       // apply: FP32 W, box 32 columns x 32 rows, 128-byte swizzle; EPI_STORE_BF16 with out_tma: the
                           // BF16 output, box 32 columns x 32 rows, 64-byte swizzle
    int32_t M, N, K;
    int32_t planes;        // 1 or 2
    int32_t plane_rows;    // row offset of the second plane inside the B tensor map
    int32_t block;         // plan index of the matrix block (for status words)
    int32_t epilogue;      // UmmaEpilogue
    int32_t a_plane_rows;  // three-product mode: row offset of the remainder plane inside the A tensor map
    void *out;             // EPI_STORE_*: destination; EPI_APPLY: W; EPI_CORE_UPDATE: C (split-K: partial buffer)
    int64_t ld_out;
    int64_t split_stride;  // elements between split-K partial slabs (EPI_STORE_F32 with split tiles)
    float *mom1;           // EPI_CORE_UPDATE
    float *mom2;
    bf16 *d_bf16;          // D   [r x ldd]
    bf16 *dt_bf16;         // D^T [r x ldd]
    int64_t ldd;
    int32_t out_tma;       // EPI_STORE_BF16: tmW describes the output, chunks leave through TMA stores
    int32_t a_mn;          // A is given as [K x M] with M contiguous (the same form for the other operand: G^T X reads G itself)
    const int32_t *col_exp; // integer Gram kernel: the column exponents of the matrix whose digit planes tmA / tmB describe
    int32_t starve;        // diagnostic (tsr_set_limits): the producer issues no loads for this problem's tiles
    int32_t b_mn;          // B is given as [K x N] with N contiguous (a row-major matrix contracted over its rows): tmB has
                           // boxes of 64 columns (N) x 64 rows (K), and the MMA reads the operand MN-major
};

// 512 bytes: the three tensor maps of every entry of a problem table then start on 128-byte lines (at 576 bytes, with
// half of the maps straddling two lines, the grouped GEMMs of a step ran a tenth slower)
static_assert(sizeof(UmmaProblem) == 512, "UmmaProblem must stay a multiple of 128 bytes");

struct UmmaTile {
    int32_t prob;
    int32_t m0, n0;        // element offsets of the tile
    int32_t kb0, kb1;      // range of 64-wide K blocks [kb0, kb1)
    int32_t split;         // split-K slab index (0 when not split)
    int32_t nw;            // width of the tile in columns (a multiple of 16, at most the kernel's tile width); 0: the full width
    // merged projection launch only (zero elsewhere)
    int32_t kind;          // 0: a tile of T~ = (G V)^T (first problem table); 1: a tile of the core C = U^T T (second table)
    int32_t wait_slot;     // kind 1: counter that must reach wait_count before the tile's B operand (T~) may be loaded; -1: none
    int32_t wait_count;
    int32_t signal_slot;   // kind 0: counter every epilogue warp of the tile increments once its stores are visible; -1: none
};

struct StepScalars {       // per-step scalars shared by all blocks
    float beta1, beta2, eps;
    float omb1, omb2;       // 1 - beta, formed in FP64 from the FP32 betas the caller passed
    float inv_bc1, inv_bc2; // 1 / (1 - beta^t)
    float decay;            // 1 - lr * weight_decay
    float step_scale;       // lr * scale
    int32_t rule;           // tsr_rule
    long long wait_clocks;  // bound of every device-side wait in SM clock ticks; <= 0: the default
};

// Launchers (tsr_umma.cu).  tiles / probs are device pointers.  bn = 128 or 256 (tile width).
cudaError_t umma_gemm_launch(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms, int bn,
                             int epilogue, int planes, const StepScalars &sc, int32_t *status, cudaStream_t stream);
cudaError_t umma_configure();  // sets the dynamic shared-memory attributes once per process
// Arrivals one finished tile of kind 0 adds to its counter (every epilogue warp of both CTAs of the pair).
constexpr int UMMA_SIGNALS_PER_TILE = 16;
// The merged projection launch (Section 3.3 in one kernel): tiles of T~ = (G V)^T (problems probs_t) and, a few blocks
// behind them in the same table, the tiles of C = U^T T (problems probs_c) that read T~ back while it is still in L2.
// A core tile waits (bounded) on a counter in `counters` that the T~ tiles it depends on advance; the launch is
// cooperative, so that all CTAs are resident while any of them waits.  fuse != 0: core tiles run the fused core update.
// counters: nslots dependency counters (one per block) followed by the tile counter (nslots + 1 words); they must
// be zero at launch.  Returns cudaErrorNotSupported when the device cannot hold the whole grid at once.
cudaError_t umma_project_launch(const UmmaProblem *probs_t, const UmmaProblem *probs_c, const UmmaTile *tiles, int num_tiles,
                                int num_sms, int bn, int fuse, int32_t *counters, const StepScalars &sc, int32_t *status,
                                cudaStream_t stream, int nslots);
// Persistent apply kernel (tsr_umma_apply.cu): W <- decay W - step_scale P V^T over a tile table.
cudaError_t umma_apply_configure();
// w_bytes: 4 = FP32 weights, 2 = BF16 weights (the tile table must not mix them).
cudaError_t umma_apply_launch(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms, int bn,
                              int w_bytes, const StepScalars &sc, int32_t *status, cudaStream_t stream);

// ---------------------------------------------------------------------------------------
// CUDA-core helpers (tsr_simt.cu)
// ---------------------------------------------------------------------------------------
enum SimtEpilogue : int { SIMT_STORE = 0, SIMT_APPLY = 1, SIMT_APPLY_BF16 = 2 };   // _BF16: D holds BF16 weights

// D[M x N] (ldd) = sum_k A(i,k) B(k,j),  A(i,k) = A[i*sa_i + k*sa_k],  B(k,j) = B[k*sb_k + j*sb_j].
// a_dtype: TSR_F32 or TSR_BF16; B and D are FP32.  SIMT_APPLY: D = decay * D - step_scale * acc.
cudaError_t simt_gemm(int M, int N, int K, const void *A, int a_dtype, int64_t sa_i, int64_t sa_k, const float *B,
                      int64_t sb_k, int64_t sb_j, float *D, int64_t ldd, int epilogue, float decay, float step_scale,
                      cudaStream_t stream);
// The same product with an FP32 A and a B of either type (b_dtype), plain store.
cudaError_t simt_gemm_bt(int M, int N, int K, const float *A, int64_t sa_i, int64_t sa_k, const void *B, int b_dtype,
                         int64_t sb_k, int64_t sb_j, float *D, int64_t ldd, cudaStream_t stream);

struct CoreUpdateArgs {     // one entry per block for the stand-alone core update
    const float *C;         // r x r, or split-K partial slabs
    float *Cout;            // where the summed core goes when nsplit > 1 (else unused)
    float *mom1, *mom2;
    float *d_f32;           // may be NULL
    bf16 *d_bf16, *dt_bf16; // may be NULL
    int64_t ldd;
    int64_t split_stride;
    int32_t r, nsplit;
    int32_t nc;             // columns of C, mom1, mom2 (r; n for a one-sided block)
};
// Runs the core update for the blocks args_dev[list_dev[0..nblocks)].  mode 0: full update;
// mode 1: only sum split-K slabs into Cout.
cudaError_t core_update_launch(const CoreUpdateArgs *args_dev, const int32_t *list_dev, int nblocks, int max_r,
                               int max_cols, const StepScalars &sc, int mode, cudaStream_t stream);

// BF16 operand copies of a basis X (rows x r, FP32): Xb[rows x ldb] and Xbt[r x ldt].
cudaError_t make_shadows(const float *X, int rows, int r, bf16 *Xb, int64_t ldb, bf16 *Xbt, int64_t ldt,
                         cudaStream_t stream);
// out[cols x ldo] = in[rows x ldi]^T (BF16)
// X (rows x k FP32) -> planes hi / lo of X^T: out[plane][k x ldo]; plane stride = plane_rows * ldo elements.
cudaError_t split_transpose(const float *X, int rows, int k, bf16 *out, int64_t ldo, int plane_rows, int planes,
                            cudaStream_t stream);
cudaError_t fill_gaussian(float *out, int64_t count, uint64_t seed, uint64_t stream_id, cudaStream_t stream);
cudaError_t fill_zero_f32(float *p, int64_t count, cudaStream_t stream);

// ---------------------------------------------------------------------------------------
// Small dense linear algebra for the refresh (tsr_linalg.cu).  All launchers are batched over
// a list of blocks; the per-block pointers live in a device-resident RefreshDev table.
// ---------------------------------------------------------------------------------------
struct RefreshDev {
    int32_t m, n, k, r;
    float *buf[3];      // three scratch matrices, each max(m, n) x k FP32
    double *S;          // k x k Gram matrix / Cholesky factor
    double *Xw;         // k x k work (inverse factor)
    double *Wj;         // k x k eigenvectors
    double *gpart;      // Gram partial sums, gram_chunks(max(m, n)) * k * k
    double *lam;        // k eigenvalues, descending
    float *Rinv;        // k x k
    float *Wu, *Wv;     // k x r
    float *Xs, *Bts;    // TF32 operand planes of the tensor-core row products (may be NULL)
    float *U, *V;       // the block's bases (FP32 masters)
    int32_t *status;    // the block's status word
    // exact integer Gram matrices (tsr_gram_i8.cu): power-of-two exponent of every column, and the six INT8 digit
    // planes of the matrix, transposed: planes[s][col][row], row pitch ldp bytes
    int32_t *col_exp;
    int8_t *planes;
    int64_t ldp;
    // tridiagonal eigen-solver (tsr_eig.cu)
    double *tau, *dvec, *evec;   // k each: reflector scales, diagonal / eigenvalues, off-diagonal
    double2 *rot;                // logged plane rotations (c, s)
    int2 *sweeps;                // per QL sweep: column of the first rotation, count
    int2 *groups;                // skewed log: per group of 32 sweeps (first row, stream elements)
    int32_t *nsweeps;            // number of logged sweeps
    int32_t *rank;               // k: descending rank of each eigenvalue
    int32_t rot_cap, sweep_cap;
    int32_t max_sweeps;          // eigen-solver limit (Jacobi sweeps / QL iterations per eigenvalue); <= 0: the default
    // divide-and-conquer merge of the two halves of the tridiagonal problem (tsr_eig.cu)
    double *dc_z;                // k: the rank-one vector in the basis of the halves' eigenvectors
    int32_t *dc_nd;              // coordinates that take part in the secular problem, ascending eigenvalue
    int2 *dc_rot_idx;            // deflation rotations: coordinate pair
    double2 *dc_rot_cs;          //                      (c, s)
    double *dc_scal;             // [0] rho
    int32_t *dc_info;            // [0] K (size of the secular problem), [1] number of deflation rotations
};
struct RowItem { int32_t block; int32_t row0; };   // a slab of rows of one block

constexpr int GRAM_ROWS = 2048;   // rows per Gram work item
constexpr int RG_ROWS = 128;      // rows per rows_gemm work item
__host__ __device__ inline int gram_chunks(int64_t rows) { return (int)((rows + GRAM_ROWS - 1) / GRAM_ROWS); }

// side: 0 = matrices with m rows, 1 = matrices with n rows.
// S = X^T X with X = buf[src_sel] (FP32), FP64 accumulation, deterministic.
cudaError_t gram_batched(const RefreshDev *rd, const RowItem *items, int nitems, const int32_t *list, int nlist,
                         int side, int src_sel, int kmax, cudaStream_t stream);
// The same Gram matrix on the integer tensor cores, exact (tsr_gram_i8.cu): gram_i8_prepare writes the column
// exponents and digit planes of buf[src_sel] (items128: slabs of RG_ROWS rows), gram_i8_launch runs the products over a
// tile table (problems: digit-plane tensor maps, out = gpart), gram_reduce_batched adds the chunks into S.
cudaError_t gram_i8_configure();
cudaError_t gram_i8_prepare(const RefreshDev *rd, const RowItem *items128, int nitems128, const int32_t *list, int nlist,
                            int side, int src_sel, int kmax, cudaStream_t stream);
cudaError_t gram_i8_launch(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms, long long wait_clocks,
                           int32_t *status, cudaStream_t stream);
cudaError_t gram_reduce_batched(const RefreshDev *rd, const int32_t *list, int nlist, int side, int kmax, cudaStream_t stream);
// Cholesky S = R^T R in place and Rinv = float(R^{-1}).
cudaError_t chol_inverse_batched(const RefreshDev *rd, const int32_t *list, int nlist, int kmax, cudaStream_t stream);
// dst = buf[src_sel] * Mat;  mat_sel: 0 Rinv (k x k), 1 Wu (k x r), 2 Wv (k x r);
// dst_sel: 0..2 buf[], 3 = U, 4 = V.
cudaError_t rows_gemm_batched(const RefreshDev *rd, const RowItem *items, int nitems, int side, int src_sel,
                              int mat_sel, int dst_sel, int nmax, cudaStream_t stream);
// Operand planes for the tensor-core form of the product above: every value as a TF32 part and a
// remainder; rows of buf[src_sel] into Xs, the transposed small matrix into Bts.
cudaError_t split_operands_batched(const RefreshDev *rd, const RowItem *items, int nitems, const int32_t *list, int nlist,
                                   int side, int src_sel, int mat_sel, int kmax, cudaStream_t stream);
// Eigen-decomposition of S by cyclic Jacobi, descending sort, Wu = W[:, :r], Wv = W[:, :r] / sqrt(lambda).
// The same result through Householder tridiagonalisation + implicit QL with logged rotations
// (for k too large for the Jacobi solver).  panel_items: (block, row0) slabs of eig_panel_rows(kmax)
// rows of the k x k eigenvector matrix.  eig_rot_capacity(k): entries of the rotation log to provide.
int eig_panel_rows(int kmax);
int64_t eig_rot_capacity(int k);
cudaError_t eig_tridiag_batched(const RefreshDev *rd, const int32_t *list, int nlist, const RowItem *panel_items,
                                int npanels, int kmax, cudaStream_t stream);
cudaError_t jacobi_batched(const RefreshDev *rd, const int32_t *list, int nlist, int max_sweeps, cudaStream_t stream);

}  // namespace tsr
