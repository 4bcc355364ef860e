/*
 * tsr.h -- C ABI of libtsr: the per-step optimizer hot path of TSR-Adam
 * (two-sided low-rank Adam) on one NVIDIA B200 (sm_100a).
 *
 * For every m x n weight block W with local gradient G the method keeps two
 * orthonormal bases U (m x r) and V (n x r) and Adam moments M, Vm of the
 * r x r core (Algorithm 1 of the paper; Sections 3.3-3.5):
 *
 *     C  = U^T G V                                   core projection
 *     M  = b1 M + (1-b1) C ;  Vm = b2 Vm + (1-b2) C o C
 *     D  = (M / (1-b1^t)) / (sqrt(Vm / (1-b2^t)) + eps)
 *     W  = W - lr (scale * U D V^T + weight_decay * W)
 *
 * and, every K steps, refreshes (U, V) from the current gradient by a
 * randomized SVD with k = r + p sketch columns and q power iterations.
 *
 * General rules
 *   - Every pointer in tsr_mat_ptrs and every `workspace` pointer is a DEVICE
 *     pointer owned by the caller; the library never frees or reallocates it.
 *     Descriptor / index / hyper-parameter arguments are HOST pointers.  The
 *     only calls that take HOST data buffers are the *_host entry points.
 *   - All matrices are row-major.  G and W carry explicit leading dimensions
 *     (in elements); U is m x r, V is n x r, M / Vm / C are r x r, all dense
 *     FP32.  Buffers of different roles must not alias.
 *   - G is read-only.  W, U, V, M, Vm, C are updated in place.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream) unless stated otherwise, and calls on
 *     one context must be issued from one host thread at a time.
 *   - Every call returns a tsr_status.  Argument errors are detected on the
 *     host before anything is launched and leave all buffers untouched.
 *     Conditions detected on the device (a rank-deficient sketch, an
 *     eigen-solver that ran out of sweeps, a non-finite value) are recorded per
 *     block and read back with tsr_poll_status; no kernel traps or spins
 *     without a bound.
 *   - There is no CPU fallback: without a CUDA device every compute call
 *     returns TSR_ERR_CUDA.
 *   - Gradients in BF16 with 16-byte aligned pointers and row pitches take the
 *     tensor-core path (tcgen05 MMAs fed by TMA, FP32 accumulation; U, V, the
 *     intermediate products and D are rounded to BF16 as MMA operands).
 *     FP32 gradients, or buffers that miss the alignment rule, take an
 *     all-FP32 CUDA-core path.
 */
#ifndef TSR_H_
#define TSR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define TSR_API
#else
#define TSR_API __attribute__((visibility("default")))
#endif

typedef struct tsr_ctx tsr_ctx; /* opaque plan: shapes, bound pointers, device tables */

typedef enum {
    TSR_OK = 0,
    TSR_ERR_INVALID_ARG = 1,    /* null pointer, bad index, bad enum                      */
    TSR_ERR_SHAPE = 2,          /* non-positive size, ld < cols, r + p > min(m, n) or > 1056 */
    TSR_ERR_ALIGNMENT = 3,      /* a pointer that must be 16-byte aligned is not          */
    TSR_ERR_WORKSPACE = 4,      /* workspace missing or too small                         */
    TSR_ERR_CUDA = 5,           /* a CUDA runtime / driver call failed, or no device      */
    TSR_ERR_UNSUPPORTED = 6,    /* dtype or option not implemented                        */
    TSR_ERR_NOT_CONVERGED = 7,  /* device: eigen-solver hit its sweep limit               */
    TSR_ERR_RANK_DEFICIENT = 8, /* device: a sketch lost rank; bases are still orthonormal only approximately */
    TSR_ERR_NONFINITE = 9,      /* device: NaN / Inf met in a refresh                     */
    TSR_ERR_TIMEOUT = 10,       /* device: a bounded wait ran out                         */
    TSR_ERR_NOT_BOUND = 11      /* compute call before tsr_bind                           */
} tsr_status;

typedef enum { TSR_F32 = 0, TSR_BF16 = 1 } tsr_dtype;

/* Update rule in core space: Algorithm 1 (Adam) or Algorithm 2 (momentum SGD, D = M,
 * no second moment, no weight decay, no bias correction; beta1 is its momentum). */
typedef enum { TSR_RULE_ADAM = 0, TSR_RULE_SGD = 1 } tsr_rule;

/* Per-block options.  TSR_BLOCK_REEXPRESS_MOMENT: at every refresh (not at tsr_init_subspace,
 * whose moments are zero) replace the first moment by M' = Unew^T (Uold M Vold^T) Vnew, i.e. keep
 * the lifted moment, projected onto the refreshed subspaces -- the "refresh alignment" the
 * paper's convergence analysis assumes.  Algorithm 1 as printed leaves M untouched (flag clear).
 * The second moment is never re-expressed.  Costs (m + n) r + 3 r^2 floats of extra scratch.
 * TSR_BLOCK_ONE_SIDED: the one-sided arm of the paper's comparison (Table 1 and the ablation of
 * Section 5: synchronized object C = U^T G of size r x n): the step of this block is
 * C = U^T G, moments and D in that r x n space, W <- (1 - lr wd) W - lr scale U D.  M, Vm and C of
 * the block are then r x n (row-major, dense); V is still bound and still written by every refresh
 * (the refresh is the same), but no step reads it.  Not combinable with
 * TSR_BLOCK_REEXPRESS_MOMENT. */
typedef enum { TSR_BLOCK_REEXPRESS_MOMENT = 1, TSR_BLOCK_ONE_SIDED = 2 } tsr_block_flags;

/* One matrix block.  Embedding blocks are ordinary blocks with their own (r, K)
 * (Section 3.6); is_embedding only labels them for tsr_embed_step. */
typedef struct {
    int64_t m, n;         /* rows, columns of G and W                                   */
    int64_t ldg, ldw;     /* leading dimensions of G and W in elements (>= n)           */
    int32_t r;            /* rank of the bases                                          */
    int32_t p;            /* oversampling: sketches have k = r + p columns, k <= min(m,n), k <= 1056 */
    int32_t q;            /* power iterations in the refresh (>= 0)                     */
    int32_t K;            /* refresh when step % K == 0; K <= 0 disables in-loop refresh */
    int32_t g_dtype;      /* tsr_dtype of G                                             */
    int32_t w_dtype;      /* tsr_dtype of W: TSR_F32, or TSR_BF16 (updated in FP32, rounded   */
                          /* to nearest even); the same for every block of a context        */
    int32_t is_embedding; /* 0 / 1                                                      */
    int32_t flags;        /* bit set of tsr_block_flags; 0 = Algorithm 1 as printed     */
} tsr_mat_desc;

typedef struct {
    const void *G; /* m x n (ldg), g_dtype                                              */
    void *W;       /* m x n (ldw), FP32, updated in place                               */
    float *U;      /* m x r                                                             */
    float *V;      /* n x r                                                             */
    float *M;      /* r x r first moment (r x n for a TSR_BLOCK_ONE_SIDED block, like Vm and C) */
    float *Vm;     /* r x r second moment (unused by TSR_RULE_SGD, may then be NULL)    */
    float *C;      /* r x r core, written by every projection: the tensor a data-parallel
                      job would all-reduce (Algorithm 1, "C_bar <- AR(C)")              */
} tsr_mat_ptrs;

typedef struct {
    float lr, beta1, beta2, eps, weight_decay;
    float scale;   /* multiplies the lifted update U D V^T only; 1 = Algorithm 1 as printed.
                      TSR_RULE_SGD ignores scale and weight_decay (Algorithm 2 has neither). */
    int64_t step;  /* t >= 1: global step counter used for bias correction and refresh schedule */
    int32_t rule;  /* tsr_rule                                                          */
    int32_t reserved;
} tsr_hyper;

/* ---- library / context management (host only) ------------------------------------------- */

TSR_API int tsr_version(void);
TSR_API const char *tsr_status_string(tsr_status s);
/* Text of the last error recorded on ctx (empty string if none); valid until the next call. */
TSR_API const char *tsr_last_error(const tsr_ctx *ctx);

/* Validates `count` descriptors and builds the plan.  descs is copied.  Returns
 * TSR_ERR_SHAPE / TSR_ERR_UNSUPPORTED / TSR_ERR_INVALID_ARG and sets *ctx = NULL on failure. */
TSR_API tsr_status tsr_create(tsr_ctx **ctx, const tsr_mat_desc *descs, int32_t count);
TSR_API tsr_status tsr_destroy(tsr_ctx *ctx);

/* Bytes of device scratch the context needs.  step_bytes covers projection, core update and
 * back-projection (BF16 operand copies of U and V, the m x r intermediates, device tables);
 * refresh_bytes covers one refresh of all blocks at once.  tsr_bind wants a single buffer of
 * step_bytes + refresh_bytes. */
TSR_API tsr_status tsr_workspace_bytes(const tsr_ctx *ctx, size_t *step_bytes, size_t *refresh_bytes);

/* Attaches the caller's device buffers and the scratch buffer (256-byte aligned), encodes the
 * TMA descriptors and uploads the device tables.  Synchronous; may be called again to re-point
 * the context.  The contents of U, V are not read here: call tsr_init_subspace[_grouped] or,
 * after writing U and V yourself, tsr_bases_changed. */
TSR_API tsr_status tsr_bind(tsr_ctx *ctx, const tsr_mat_ptrs *ptrs, int32_t count, void *workspace,
                            size_t workspace_bytes);

/* Tells the library that the caller overwrote U and/or V of the listed blocks (idx = NULL: all):
 * rebuilds the BF16 operand copies the tensor-core path keeps in the workspace. */
TSR_API tsr_status tsr_bases_changed(tsr_ctx *ctx, const int32_t *idx, int32_t count, void *stream);

/* ---- single-block calls (block index i of the plan) ------------------------------------- */

/* Algorithm 1, initialisation: M <- 0, Vm <- 0 and (U, V) <- one refresh on the bound G.
 * omega: device pointer to an n x (r+p) FP32 Gaussian test matrix, or NULL to draw it from
 * `seed` with the library's counter-based generator (see tsr_generate_omega). */
TSR_API tsr_status tsr_init_subspace(tsr_ctx *ctx, int32_t i, uint64_t seed, const float *omega, void *stream);

/* Section 3.3: C <- U^T G V. */
TSR_API tsr_status tsr_project_core(tsr_ctx *ctx, int32_t i, void *stream);

/* Section 3.4: moments and normalised core D from the (possibly all-reduced) C in place in
 * the C buffer's companion scratch; uses hyper->step for bias correction. */
TSR_API tsr_status tsr_adam_core_step(tsr_ctx *ctx, int32_t i, const tsr_hyper *hyper, void *stream);

/* Section 3.4: W <- W - lr (scale * U D V^T + weight_decay * W) with the D left by the last
 * tsr_adam_core_step of this block.  The lifted update is never written to memory. */
TSR_API tsr_status tsr_backproject_apply(tsr_ctx *ctx, int32_t i, const tsr_hyper *hyper, void *stream);

/* Section 3.5: randomized-SVD refresh of (U, V) from the bound G; moments are left untouched. */
TSR_API tsr_status tsr_rsvd_refresh(tsr_ctx *ctx, int32_t i, uint64_t seed, const float *omega, void *stream);

/* Section 3.6: one full step of an embedding block on its own (r_emb, K_emb): refresh if
 * hyper->step % K == 0, then project, core update, back-project and apply. */
TSR_API tsr_status tsr_embed_step(tsr_ctx *ctx, int32_t i, const tsr_hyper *hyper, uint64_t seed, void *stream);

/* ---- grouped calls: the same operations over a list of blocks in a few launches ---------- */
/* idx: host array of `count` block indices, or NULL for all blocks of the plan (count ignored).
 * omegas: host array with one device pointer per listed block, or NULL (library-drawn). */

TSR_API tsr_status tsr_init_subspace_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, uint64_t seed,
                                             const float *const *omegas, void *stream);
TSR_API tsr_status tsr_project_core_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, void *stream);
TSR_API tsr_status tsr_adam_core_step_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count,
                                              const tsr_hyper *hyper, void *stream);
TSR_API tsr_status tsr_backproject_apply_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count,
                                                 const tsr_hyper *hyper, void *stream);
TSR_API tsr_status tsr_rsvd_refresh_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, uint64_t seed,
                                            const float *const *omegas, void *stream);
TSR_API tsr_status tsr_embed_step_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count,
                                          const tsr_hyper *hyper, uint64_t seed, void *stream);

/* One optimizer step of Algorithm 1 for every block: refresh the blocks whose K divides
 * hyper->step (each block, embeddings included, on its own K), then project, update the core
 * moments and apply.  fuse_adam != 0 runs the core update inside the projection kernel's
 * epilogue (valid when no all-reduce of C is needed between the two); 0 runs the three stages
 * as separate launches.  Both orders give the same result. */
TSR_API tsr_status tsr_step_grouped(tsr_ctx *ctx, const tsr_hyper *hyper, uint64_t seed, int32_t fuse_adam,
                                    void *stream);

/* The same step driven from HOST memory: G_host[i] is a host pointer to block i's gradient,
 * dense m x n in the block's g_dtype; each is copied into the bound device G buffer, the step
 * runs, and the cores of all blocks are copied back, packed block after block (r*r floats
 * each), into C_host (may be NULL).  On steps without a refresh the blocks travel in chunks: while
 * one chunk is stepped, the next one's gradients arrive and the previous one's cores leave on the
 * context's side streams (pinned host memory is needed for that overlap; pageable memory works but
 * serialises).  Results are identical to the plain order.  Returns after everything has finished. */
TSR_API tsr_status tsr_step_grouped_host(tsr_ctx *ctx, const void *const *G_host, float *C_host,
                                         const tsr_hyper *hyper, uint64_t seed, int32_t fuse_adam, void *stream);

/* ---- dense parameters ------------------------------------------------------------------------ */

/* One dense (non-matrix) parameter tensor: biases, normalisation weights.  All DEVICE pointers;
 * param, m, v are FP32 arrays of `count` elements updated in place, grad is FP32 or BF16. */
typedef struct {
    float *param;
    const void *grad;
    float *m, *v;
    int64_t count;
    int32_t g_dtype; /* tsr_dtype of grad */
    int32_t reserved;
} tsr_dense_tensor;

/* Sections 3.1 / 3.4: parameters that are not matrix blocks are updated by dense AdamW,
 *   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g o g;  p <- p - lr (m_hat / (sqrt(v_hat) + eps) + wd p),
 * for all listed tensors in one multi-tensor launch per 48 tensors.  `tensors` is a HOST array;
 * hyper->scale is ignored; hyper->rule must be TSR_RULE_ADAM.  Needs no context and no
 * workspace.  Errors (null pointers, negative counts, bad dtype) are found before any launch. */
TSR_API tsr_status tsr_dense_adamw(const tsr_dense_tensor *tensors, int32_t count, const tsr_hyper *hyper, void *stream);

/* ---- reporting -------------------------------------------------------------------------- */

/* Section 3.2: bytes one worker would hand to the all-reduce in one step, summed over blocks:
 * *core = sum r^2 * bytes_per_elem (every step; r n for a one-sided block, Table 1); *sketch =
 * sum (r+p)(m+n) * bytes_per_elem for the blocks that refresh at `step` (0 if none; step <= 0
 * counts a refresh of every block). */
TSR_API tsr_status tsr_comm_bytes(const tsr_ctx *ctx, int64_t step, int32_t bytes_per_elem, uint64_t *core,
                                  uint64_t *sketch);

/* Optimizer-state elements (U, V, M, Vm) summed over blocks: sum (m+n) r + 2 r^2 (Table 2);
 * a one-sided block counts U and its r x n moments: m r + 2 r n. */
TSR_API tsr_status tsr_state_elems(const tsr_ctx *ctx, uint64_t *elems);

/* Copies the per-block device status words (a tsr_status each; TSR_OK if nothing was detected
 * since the last poll) into the HOST array per_block_status[count] and clears them.
 * Synchronises `stream`. */
TSR_API tsr_status tsr_poll_status(tsr_ctx *ctx, int32_t *per_block_status, int32_t count, void *stream);

/* Fills the DEVICE buffer out (n x k FP32, row-major) with the N(0,1) matrix the library
 * would draw for (seed, block i): entry e = row * k + col comes from a counter-based hash of
 * (seed, i, e) followed by a Box-Muller transform, so the draw does not depend on the launch
 * shape. */
TSR_API tsr_status tsr_generate_omega(tsr_ctx *ctx, int32_t i, uint64_t seed, float *out, void *stream);

/* Stage timing of tsr_step_grouped for profiling (off by default).  When enabled, every
 * tsr_step_grouped / tsr_embed_step records CUDA events at its stage boundaries on the step's
 * stream; tsr_get_stage_ms waits for the last recorded step and returns, in milliseconds,
 * ms[0] refresh (0 when none was due), ms[1] the projection launch (a step over all blocks may
 * run the first contraction -- T = G V, or T = U^T G for a block with m > n -- and the core GEMM
 * with its fused core update as ONE launch; otherwise the first contraction runs here),
 * ms[2] what follows it (the core GEMM when it is a launch of its own; the split-K reduction of
 * tall blocks), ms[3] stand-alone core update (unfused order only),
 * ms[4] P = U D, ms[5] the apply kernel W <- decay W - step_scale P V^T.  count must be 6.
 * Enabling creates the events (a small driver allocation); disabling destroys them. */
TSR_API tsr_status tsr_set_profiling(tsr_ctx *ctx, int32_t enable);
TSR_API tsr_status tsr_get_stage_ms(tsr_ctx *ctx, float *ms, int32_t count);

/* Limits of the device-side loops and waits, and one diagnostic switch.  (No passage of the
 * paper corresponds to this call; it makes the device-detected conditions of this library
 * observable.)  Defaults are in force until the first call; a zero field restores its default.
 *   wait_clocks   bound, in SM clock ticks, of every wait a tensor-core kernel of this context
 *                 performs on an mbarrier (default 4e9, about two seconds).  When it runs out the
 *                 CTA gives up on its remaining tiles, releases its tensor memory and returns;
 *                 every block that owns one of those tiles reads TSR_ERR_TIMEOUT at the next
 *                 tsr_poll_status and its outputs of that call are undefined.
 *   max_sweeps    limit of the small eigen-solver of the refresh (Jacobi sweeps for k < 100,
 *                 QL iterations per eigenvalue above; defaults 40 / 60) for block sweep_block
 *                 (-1: every block).  A solver that stops at the limit flags
 *                 TSR_ERR_NOT_CONVERGED on that block; other blocks are not affected.
 *   starve_block  -1 (off), or a block index: the first projection GEMM (T = G V or U^T G) issues no
 *                 loads for the tiles of that block, so that its consumers run into the bounded
 *                 wait.  Nothing is in flight and no address is touched for those tiles.  It
 *                 exists to exercise the time-out path and requires 0 < wait_clocks <= 1e8.
 *   projection_launches  how a call that covers every two-sided tensor-core block runs the two
 *                 contractions of C = U^T G V: 0 = the library decides (ONE launch, with the
 *                 intermediate T read back from L2, when the T of all blocks together is more than
 *                 twice the L2 cache; TWO launches otherwise, where T stays in L2 between them
 *                 anyway and the tiles need not wait for one another), 1 = one launch whenever
 *                 the device accepts a cooperative launch, 2 = always two.  Tiles, reduction
 *                 order and results are the same either way.
 * Call it between compute calls of the context (it is synchronous).  Host struct. */
typedef struct {
    int64_t wait_clocks;
    int32_t max_sweeps;
    int32_t sweep_block;
    int32_t starve_block;
    int32_t projection_launches;
} tsr_limits;
TSR_API tsr_status tsr_set_limits(tsr_ctx *ctx, const tsr_limits *limits);

/* The Gram step of the refresh on its own: S = X^T X for an X of (side == 0 ? m : n) rows and
 * k = r + p columns, through exactly the kernels the orthonormalisations and the small SVD of
 * Section 3.5 use for block `block` (the integer tensor-core form for a sketch with
 * 2k <= min(m, n), k >= 8 on the tensor-core path; the FP64 tensor path otherwise).  (No passage of
 * the paper defines this call; it exists so that the Gram matrices can be checked against their
 * definition.)  X: device, FP32, row-major, row pitch k.  S: device, FP64, k x k, row pitch k,
 * both triangles written.  The block's refresh work buffers are overwritten; U, V, moments and
 * weights are not touched.  Asynchronous on `stream`; a non-finite X flags TSR_ERR_NONFINITE. */
TSR_API tsr_status tsr_refresh_gram(tsr_ctx *ctx, int32_t block, int32_t side, const float *X, double *S, void *stream);

/* Number of CUDA kernels this context has launched since tsr_create. */
TSR_API tsr_status tsr_launch_count(const tsr_ctx *ctx, uint64_t *count);

/* Core projection C = U^T G V of ONE block without any allocation.  (The paper has no
 * counterpart of this call; it exists for callers that cannot allocate device memory.)
 *
 * Who needs it: code that may neither allocate device memory nor synchronise the device -- a
 * process whose memory is owned by another framework's pool with nothing left to hand out, an
 * allocator that forbids foreign allocations, a region where cudaMalloc's implicit
 * synchronisation is not acceptable -- and that cannot provide the scratch buffer tsr_bind asks
 * for either.  (It still launches kernels, so it is not for use inside a stream host callback,
 * where no CUDA call may be made.)  Here the
 * only scratch the computation needs, the m x r intermediate T = G V, sits in a fixed
 * TSR_STATIC_SCRATCH_FLOATS-element FP32 array inside the library image (4 MiB of device
 * memory per GPU that loads the library, held until the process exits).
 *
 * All pointers are DEVICE pointers: G is m x n (leading dimension ldg, g_dtype TSR_F32 or
 * TSR_BF16), U is m x r, V is n x r, C is r x r (output), all row-major, U / V / C FP32 dense.
 * The call takes no context, calls no cudaMalloc / cudaFree or any allocating routine, and runs
 * on the CUDA-core FP32 path (same kernels and therefore the same bits as tsr_project_core on
 * that path).  Limits and errors: m * r must not exceed TSR_STATIC_SCRATCH_FLOATS, otherwise
 * TSR_ERR_WORKSPACE is returned and nothing is launched; bad pointers / shapes / dtypes give
 * TSR_ERR_INVALID_ARG / TSR_ERR_SHAPE / TSR_ERR_UNSUPPORTED.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress,
 * with that device current); make that first call outside any stream capture.
 * Every call on a device shares the one array and finds the previous call's contents in it;
 * nothing needs clearing because T is fully overwritten before it is read.  Two calls whose
 * kernels may overlap on the GPU (different streams, or different host threads without
 * ordering) race on the array: serialise them on one stream. */
#define TSR_STATIC_SCRATCH_FLOATS (1 << 20)
TSR_API tsr_status tsr_project_core_static(const void *G, int32_t g_dtype, int64_t m, int64_t n, int64_t ldg,
                                           const float *U, const float *V, int32_t r, float *C, void *stream);

/* 1 if block i takes the tensor-core path, 0 if the FP32 CUDA-core path, < 0 on a bad index. */
TSR_API int32_t tsr_block_uses_tensor_cores(const tsr_ctx *ctx, int32_t i);

#ifdef __cplusplus
}
#endif
#endif /* TSR_H_ */
