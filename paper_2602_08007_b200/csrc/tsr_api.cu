// Host side of libtsr: the C ABI declared in tsr.h, plan construction, workspace layout,
// TMA descriptor encoding and the launch sequences of Algorithm 1 (project -> core update ->
// lift and apply, with the randomized-SVD refresh of Section 3.5 when due).
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "tsr_internal.h"

using namespace tsr;

namespace {

// KR*: tall-times-small products of the refresh on tensor cores (three TF32 products): rows of side
// 0 (m) or 1 (n) times R^{-1} into buf[1] / buf[2], and the final U = Q Wu, V = B^T Wv.
// KCM: the core problems encoded for the merged projection launch (its B boxes follow the tile width of KT);
// KM: the merged tile table itself (tiles of KT and KCM problems interleaved; it has no problem table of its own).
// KG0 / KG1: the exact integer Gram matrices of the refresh, of matrices with m / n rows.
enum Kind : int { KT = 0, KC, KP, KA, KY, KZ, KR01, KR02, KR12, KRU, KRV, KO, KOA, KCM, KM, KG0, KG1, NKIND };
constexpr int TSR_NUM_STAGES = 6;  // refresh, G*V, core GEMM, core update, U*D, apply

struct Block {
    tsr_mat_desc d;
    tsr_mat_ptrs p;
    bool fast = false;        // tensor-core path
    int k = 0;                // r + p
    int64_t rl = 0, ml = 0, nl = 0;  // padded leading dimensions of BF16 operand copies
    // step scratch
    bf16 *Ub = nullptr, *Ubt = nullptr, *Vb = nullptr, *Vbt = nullptr, *Tt = nullptr, *Pb = nullptr;
    bf16 *Db = nullptr, *Dbt = nullptr;
    bool one_sided = false;   // C = U^T G (r x n): the comparison arm of Table 1
    bool right_first = false; // the lift goes through Z^T = V D^T (n x r) instead of P = U D (m x r): the smaller intermediate
    bool proj_right = false;  // the projection goes through T = U^T G (r x n) instead of T~ = (G V)^T (r x m): m > n and m short
                              // enough for one pass over it (Section 3.3: the intermediate whose long side is min(m, n))
    int64_t cn = 0;           // columns of C, M, Vm: r, or n for a one-sided block
    float *partial = nullptr;
    int nsplit = 1, kb_per_split = 0;
    float *T32 = nullptr, *P32 = nullptr, *D32 = nullptr;
    // refresh scratch
    bf16 *Xt = nullptr;
    float *Om = nullptr;
    float *buf[3] = {nullptr, nullptr, nullptr};
    double *S = nullptr, *Xw = nullptr, *Wj = nullptr, *gpart = nullptr, *lam = nullptr;
    float *Rinv = nullptr, *Wu = nullptr, *Wv = nullptr;
    double *tau = nullptr, *dvec = nullptr, *evec = nullptr;
    double2 *rot = nullptr;
    int2 *sweeps = nullptr, *groups = nullptr;
    double *dc_z = nullptr, *dc_scal = nullptr;
    int32_t *dc_nd = nullptr, *dc_info = nullptr;
    int2 *dc_rot_idx = nullptr;
    double2 *dc_rot_cs = nullptr;
    float *Xs = nullptr, *Bts = nullptr;   // TF32 operand planes (value truncated to TF32, remainder): rows, small matrix^T
    bool tc_rows = false;                  // tall-times-small products of the refresh run on tensor cores
    int32_t *nsweeps = nullptr, *rank = nullptr;
    int32_t *col_exp = nullptr;            // exact integer Gram: column exponents, digit planes (k x ldp bytes each, six of them)
    int8_t *planes = nullptr;
    int64_t ldp = 0;
    int rot_cap = 0, sweep_cap = 0;
    float *Uold = nullptr, *Vold = nullptr, *Ra = nullptr, *Rb = nullptr, *Rt = nullptr;   // moment re-expression
    int tile_begin[NKIND], tile_end[NKIND];
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Arena {  // bump allocator over the caller's workspace; base == nullptr only measures
    char *base;
    size_t off;
    void *take(size_t bytes)
    {
        off = (off + 255) & ~(size_t)255;
        void *p = base ? (void *)(base + off) : nullptr;
        off += bytes;
        return p;
    }
};

}  // namespace

struct tsr_ctx {
    std::vector<Block> blocks;
    std::vector<int> order;                    // table order: blocks by descending m*n
    std::vector<UmmaTile> tiles[NKIND];        // host copies
    bool bound = false;
    bool any_fast = false;
    size_t step_bytes = 0, refresh_bytes = 0;
    std::string err;
    // device tables (inside the workspace)
    UmmaProblem *d_probs[NKIND] = {};
    UmmaTile *d_tiles[NKIND] = {};
    CoreUpdateArgs *d_cu_all = nullptr, *d_cu_split = nullptr;
    RefreshDev *d_refresh = nullptr;
    int32_t *d_status = nullptr;
    int32_t *d_list = nullptr;                 // scratch: block list of the running call
    int32_t *d_list2 = nullptr;                // scratch: second list (split-K blocks, ...)
    int32_t *d_rlist = nullptr;                // block lists of the refresh groups
    RowItem *d_items[5] = {};                  // [side*2 + 0]: 64-row slabs, [side*2 + 1]: Gram slabs, [4]: eigenvector panels
    size_t items_cap[5] = {};
    EncodeTiledFn encode = nullptr;
    int max_r = 0, max_k = 0;
    uint64_t launches = 0;                     // kernels launched through this context
    int num_sms = 148;
    int bn[NKIND] = {128, 128, 128, 128, 128, 128, 256, 256, 256, 256, 256, 128, 128, 128, 128, 64, 64};   // tile width of each GEMM kind
    int32_t *d_counters = nullptr;             // merged projection launch: one dependency counter per block
    bool merged_ok = true;                     // cleared when the device refuses the cooperative launch
    int proj_mode = 0;                         // tsr_limits::projection_launches
    bool merge_pays = false;                   // the T~ of all blocks is more than twice the L2 cache (set by the layout)
    size_t l2_bytes = 0;
    bool profiling = false;
    cudaEvent_t ev[TSR_NUM_STAGES + 1] = {};   // stage boundaries of the last step (profiling only)
    bool ev_valid = false;
    cudaStream_t stage_stream = nullptr;
    int stage_next = 0;
    // refresh runs as up to NGROUP independent groups of blocks on side streams, so that the
    // latency-bound small-matrix kernels of one group overlap the GEMM-like kernels of another
    static constexpr int NGROUP = 8;
    cudaStream_t aux[NGROUP] = {};
    cudaEvent_t ev_fork = nullptr, ev_join[NGROUP] = {};
    static constexpr int NPIPE = 8;            // chunks of the pipelined host-buffer step
    cudaEvent_t ev_pipe_in[NPIPE] = {}, ev_pipe_done[NPIPE] = {};
    bool aux_ready = false;
    // What the device copies of the refresh tables (block lists, row-slab and panel tables) and of the step lists
    // d_list / d_list2 currently hold, so that a call over the same blocks as the previous one uploads nothing.
    // Cleared by tsr_bind and by any other writer of those tables.
    std::vector<int> refresh_sig;              // the refresh (its groups, in order) those tables were last written for
    std::vector<int> list_cache[2];
    // limits (tsr_set_limits)
    long long wait_clocks = 0;                 // 0: the kernels' default budget
    std::vector<int32_t> max_sweeps;           // per block; 0: the solvers' defaults
    int starve_block = -1;                     // diagnostic: block whose first projection GEMM gets no loads
};

namespace {

tsr_status fail(tsr_ctx *ctx, tsr_status s, const char *fmt, ...)
{
    if (ctx) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        ctx->err = buf;
    }
    return s;
}

#define TSR_CUDA(ctx, call)                                                                            \
    do {                                                                                               \
        cudaError_t e__ = (call);                                                                      \
        if (e__ != cudaSuccess)                                                                        \
            return fail(ctx, TSR_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__));           \
    } while (0)

#define TSR_KERNEL(ctx, n, call)                                                                       \
    do {                                                                                               \
        TSR_CUDA(ctx, call);                                                                           \
        (ctx)->launches += (n);                                                                        \
    } while (0)

bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

int elem_size(int dtype) { return dtype == TSR_BF16 ? 2 : 4; }

// Walks the workspace layout; with a.base == nullptr it only measures.
void layout(tsr_ctx *ctx, Arena &a, bool assign, size_t *step_end)
{
    const int nb = (int)ctx->blocks.size();
    // ---- step area: device tables
    for (int kd = 0; kd < NKIND; ++kd) {
        void *p = a.take(sizeof(UmmaProblem) * (size_t)nb);
        void *t = a.take(sizeof(UmmaTile) * std::max<size_t>(1, ctx->tiles[kd].size()));
        if (assign) { ctx->d_probs[kd] = (UmmaProblem *)p; ctx->d_tiles[kd] = (UmmaTile *)t; }
    }
    void *p1 = a.take(sizeof(CoreUpdateArgs) * (size_t)nb);
    void *p2 = a.take(sizeof(CoreUpdateArgs) * (size_t)nb);
    void *p3 = a.take(sizeof(RefreshDev) * (size_t)nb);
    void *p4 = a.take(sizeof(int32_t) * (size_t)nb);
    void *p5 = a.take(sizeof(int32_t) * (size_t)nb);
    void *p6 = a.take(sizeof(int32_t) * (size_t)nb);
    void *p7 = a.take(sizeof(int32_t) * (size_t)nb);
    void *p8 = a.take(sizeof(int32_t) * (size_t)(nb + 1));
    if (assign) {
        ctx->d_rlist = (int32_t *)p7;
        ctx->d_counters = (int32_t *)p8;
        ctx->d_cu_all = (CoreUpdateArgs *)p1; ctx->d_cu_split = (CoreUpdateArgs *)p2;
        ctx->d_refresh = (RefreshDev *)p3; ctx->d_status = (int32_t *)p4;
        ctx->d_list = (int32_t *)p5; ctx->d_list2 = (int32_t *)p6;
    }
    size_t cap[5] = {0, 0, 0, 0, 0};
    for (const Block &b : ctx->blocks) {
        cap[0] += (size_t)((b.d.m + RG_ROWS - 1) / RG_ROWS);
        cap[1] += (size_t)gram_chunks(b.d.m);
        cap[2] += (size_t)((b.d.n + RG_ROWS - 1) / RG_ROWS);
        cap[3] += (size_t)gram_chunks(b.d.n);
        cap[4] += (size_t)((b.k + 7) / 8);
    }
    for (int i = 0; i < 5; ++i) {
        void *q = a.take(sizeof(RowItem) * cap[i]);
        if (assign) { ctx->d_items[i] = (RowItem *)q; ctx->items_cap[i] = cap[i]; }
    }
    // ---- step area: per-block operands
    for (Block &b : ctx->blocks) {
        const int64_t m = b.d.m, n = b.d.n, r = b.d.r;
        if (b.fast) {
            void *ub = a.take((size_t)(m * b.rl) * 2), *ubt = a.take((size_t)(r * b.ml) * 2);
            void *vb = a.take((size_t)(n * b.rl) * 2), *vbt = a.take((size_t)(r * b.nl) * 2);
            void *tt = a.take((size_t)(r * b.ml) * 2), *pb = a.take((size_t)(m * b.rl) * 2);
            void *db = a.take((size_t)(r * b.rl) * 2), *dbt = a.take((size_t)(b.cn * b.rl) * 2);
            void *part = (b.nsplit > 1 && !b.one_sided) ? a.take((size_t)b.nsplit * r * r * 4) : nullptr;
            if (assign) {
                b.Ub = (bf16 *)ub; b.Ubt = (bf16 *)ubt; b.Vb = (bf16 *)vb; b.Vbt = (bf16 *)vbt;
                b.Tt = (bf16 *)tt; b.Pb = (bf16 *)pb; b.Db = (bf16 *)db; b.Dbt = (bf16 *)dbt;
                b.partial = (float *)part;
            }
        } else {
            void *t = a.take((size_t)(m * r) * 4), *pp = a.take((size_t)(m * r) * 4);
            if (assign) { b.T32 = (float *)t; b.P32 = (float *)pp; }
        }
        void *d32 = a.take((size_t)(r * b.cn) * 4);
        if (assign) b.D32 = (float *)d32;
    }
    a.off = (a.off + 255) & ~(size_t)255;
    *step_end = a.off;
    // ---- refresh area
    for (Block &b : ctx->blocks) {
        const int64_t m = b.d.m, n = b.d.n, r = b.d.r, k = b.k;
        const int64_t mx = std::max(m, n);
        if (b.fast) {
            void *xt = a.take((size_t)(2 * k * std::max(b.ml, b.nl)) * 2);
            if (assign) b.Xt = (bf16 *)xt;
        }
        if (b.tc_rows) {
            void *xs = a.take((size_t)(2 * mx * k) * 4), *bts = a.take((size_t)(2 * k * k) * 4);
            if (assign) { b.Xs = (float *)xs; b.Bts = (float *)bts; }
        }
        if (b.fast) {
            const int64_t ldp = round_up(mx, 128);   // 128-byte lines of a digit plane line up with the 128-row slabs that write them
            void *ce = a.take((size_t)k * 4), *pl = a.take((size_t)(6 * k * ldp));
            if (assign) { b.col_exp = (int32_t *)ce; b.planes = (int8_t *)pl; b.ldp = ldp; }
        }
        void *om = a.take((size_t)(n * k) * 4);
        void *b0 = a.take((size_t)(mx * k) * 4), *b1 = a.take((size_t)(mx * k) * 4), *b2 = a.take((size_t)(mx * k) * 4);
        void *S = a.take((size_t)(k * k) * 8), *Xw = a.take((size_t)(k * k) * 8), *Wj = a.take((size_t)(k * k) * 8);
        void *gp = a.take((size_t)gram_chunks(mx) * k * k * 8);
        void *lam = a.take((size_t)k * 8);
        void *ri = a.take((size_t)(k * k) * 4), *wu = a.take((size_t)(k * r) * 4), *wv = a.take((size_t)(k * r) * 4);
        const int rot_cap = (int)std::min<int64_t>(eig_rot_capacity((int)k), 0x7fffffff), sweep_cap = (int)(64 * k);
        void *tau = a.take((size_t)k * 8), *dv = a.take((size_t)k * 8), *ev = a.take((size_t)k * 8);
        void *rot = a.take((size_t)rot_cap * 16), *sw = a.take((size_t)sweep_cap * 8);
        void *grp = a.take((size_t)(sweep_cap / 32 + 4) * 8);
        void *nsw = a.take(16), *rk = a.take((size_t)k * 4);
        // divide-and-conquer merge: z vector, list of coordinates that take part, deflation rotations, scalars
        void *dcz = a.take((size_t)k * 8), *dcnd = a.take((size_t)k * 4), *dcri = a.take((size_t)k * 8), *dcrc = a.take((size_t)k * 16);
        void *dcs = a.take(64), *dci = a.take(64);
        if (assign) {
            b.tau = (double *)tau; b.dvec = (double *)dv; b.evec = (double *)ev; b.rot = (double2 *)rot;
            b.sweeps = (int2 *)sw; b.groups = (int2 *)grp; b.nsweeps = (int32_t *)nsw; b.rank = (int32_t *)rk;
            b.dc_z = (double *)dcz; b.dc_nd = (int32_t *)dcnd; b.dc_rot_idx = (int2 *)dcri; b.dc_rot_cs = (double2 *)dcrc;
            b.dc_scal = (double *)dcs; b.dc_info = (int32_t *)dci;
            b.rot_cap = rot_cap; b.sweep_cap = sweep_cap;
        }
        if (b.d.flags & TSR_BLOCK_REEXPRESS_MOMENT) {
            void *uo = a.take((size_t)(m * r) * 4), *vo = a.take((size_t)(n * r) * 4);
            void *ra = a.take((size_t)(r * r) * 4), *rb = a.take((size_t)(r * r) * 4), *rt = a.take((size_t)(r * r) * 4);
            if (assign) { b.Uold = (float *)uo; b.Vold = (float *)vo; b.Ra = (float *)ra; b.Rb = (float *)rb; b.Rt = (float *)rt; }
        }
        if (assign) {
            b.Om = (float *)om; b.buf[0] = (float *)b0; b.buf[1] = (float *)b1; b.buf[2] = (float *)b2;
            b.S = (double *)S; b.Xw = (double *)Xw; b.Wj = (double *)Wj; b.gpart = (double *)gp; b.lam = (double *)lam;
            b.Rinv = (float *)ri; b.Wu = (float *)wu; b.Wv = (float *)wv;
        }
    }
    a.off = (a.off + 255) & ~(size_t)255;
}

// tri > 0: B is the transpose of an upper-triangular matrix, so the columns n0 .. of the product only
// need the first n0 + bn entries of the contraction (tri = elements per K block).
void gen_tiles(std::vector<UmmaTile> &v, int bi, int M, int N, int K, int kb_per_split, int bn, bool apply, int tri)
{
    const int bm = apply ? 128 : 256;   // the grouped GEMM runs on CTA pairs: 256-row tiles
    const int nkb = (K + 63) / 64;
    const int nsp = kb_per_split > 0 ? (nkb + kb_per_split - 1) / kb_per_split : 1;
    // Columns: the grouped GEMM takes tiles of any width that is a multiple of 16, so N is cut into equal parts
    // (528 columns: three tiles of 176 instead of 256 + 256 + 16, whose narrow tile would cost a whole pass
    // over the A operand); the apply kernel keeps full-width tiles.
    const int ntn = (N + bn - 1) / bn;
    int wn = bn;
    if (!apply && ntn > 0) wn = std::min(bn, (((N + ntn - 1) / ntn) + 15) & ~15);
    for (int m0 = 0; m0 < M; m0 += bm)
        for (int n0 = 0; n0 < N; n0 += wn)
            for (int s = 0; s < nsp; ++s) {
                UmmaTile t;
                memset(&t, 0, sizeof t);
                t.prob = bi; t.m0 = m0; t.n0 = n0;
                t.kb0 = kb_per_split > 0 ? s * kb_per_split : 0;
                t.kb1 = kb_per_split > 0 ? std::min(nkb, (s + 1) * kb_per_split) : nkb;
                t.nw = apply ? 0 : std::min(wn, ((N - n0) + 15) & ~15);
                if (tri > 0) t.kb1 = std::min(nkb, (n0 + (apply ? bn : t.nw) + tri - 1) / tri);
                t.split = s;
                t.wait_slot = -1; t.signal_slot = -1;
                v.push_back(t);
            }
}

// tri > 0: B is the transpose of an upper-triangular matrix, so the columns n0 .. of the product only
// need the first n0 + bn entries of the contraction (tri = elements per K block).
void add_tiles(tsr_ctx *ctx, int kind, int bi, int M, int N, int K, int kb_per_split, int tri = 0)
{
    Block &b = ctx->blocks[bi];
    std::vector<UmmaTile> &v = ctx->tiles[kind];
    b.tile_begin[kind] = (int)v.size();
    gen_tiles(v, bi, M, N, K, kb_per_split, ctx->bn[kind], kind == KA || kind == KOA, tri);
    b.tile_end[kind] = (int)v.size();
}

// The merged projection table: for the two-sided tensor-core blocks in table order, the tiles of T~ = (G V)^T of a
// block, and -- once at least MERGE_GAP later tiles separate them from the block's last T~ tile -- the tiles of its
// core C = U^T T.  A core tile therefore always sits behind the tiles it depends on (CTA pairs take tiles in table
// order, round-robin, so the wait cannot deadlock), close enough that T~ is still in L2 when it is read back, and far
// enough that its producers have normally finished when a pair reaches it.
constexpr int MERGE_GAP = 128;

void build_merged(tsr_ctx *ctx)
{
    std::vector<UmmaTile> &v = ctx->tiles[KM];
    v.clear();
    struct Pending { int bi; size_t t_end; int n_t; };
    std::vector<Pending> pending;
    size_t head = 0;
    auto emit_core = [&](const Pending &pd) {
        const Block &b = ctx->blocks[pd.bi];
        const size_t first = v.size();
        gen_tiles(v, pd.bi, b.d.r, b.d.r, (int)(b.proj_right ? b.d.n : b.d.m), b.nsplit > 1 ? b.kb_per_split : 0, ctx->bn[KCM], false, 0);
        for (size_t i = first; i < v.size(); ++i) {
            v[i].kind = 1;
            v[i].wait_slot = pd.bi;
            v[i].wait_count = pd.n_t * UMMA_SIGNALS_PER_TILE;
        }
    };
    for (int bi : ctx->order) {
        const Block &b = ctx->blocks[bi];
        if (!b.fast || b.one_sided) continue;
        const size_t first = v.size();
        if (b.proj_right) gen_tiles(v, bi, b.d.r, (int)b.d.n, (int)b.d.m, 0, ctx->bn[KT], false, 0);
        else gen_tiles(v, bi, (int)b.d.m, b.d.r, (int)b.d.n, 0, ctx->bn[KT], false, 0);
        for (size_t i = first; i < v.size(); ++i) { v[i].kind = 0; v[i].signal_slot = bi; }
        pending.push_back({bi, v.size(), (int)(v.size() - first)});
        while (head < pending.size() && v.size() >= pending[head].t_end + MERGE_GAP) emit_core(pending[head++]);
    }
    while (head < pending.size()) emit_core(pending[head++]);
}

void build_tiles(tsr_ctx *ctx)
{
    for (int kd = 0; kd < NKIND; ++kd) ctx->tiles[kd].clear();
    int rmax = 0;
    for (const Block &b : ctx->blocks) if (b.fast) rmax = std::max(rmax, (int)b.d.r);
    for (int kd : {KT, KP}) ctx->bn[kd] = rmax >= 256 ? 256 : 128;
    // the core GEMM has few, long tiles: 256-wide tiles only pay once r reaches 512 (measured)
    ctx->bn[KC] = rmax >= 512 ? 256 : 128;
    // apply: 256-wide tiles halve the P traffic per byte of W, which pays once the operands are as wide
    // as r = 512 (measured 2.28 -> 2.05 ms on the 1B set; at r = 256 the narrow tile is faster)
    ctx->bn[KA] = rmax >= 512 ? 256 : 128;
    // sketches (N = k columns): wide tiles read the gradient rows fewer times
    for (int kd : {KY, KZ}) ctx->bn[kd] = rmax >= 256 ? 256 : 128;
    ctx->bn[KO] = ctx->bn[KT];
    ctx->bn[KOA] = ctx->bn[KA];
    ctx->bn[KCM] = ctx->bn[KT];
    ctx->bn[KM] = ctx->bn[KT];
    for (int bi : ctx->order) {
        Block &b = ctx->blocks[bi];
        for (int kd = 0; kd < NKIND; ++kd) b.tile_begin[kd] = b.tile_end[kd] = (int)ctx->tiles[kd].size();
        if (!b.fast) continue;
        const int m = (int)b.d.m, n = (int)b.d.n, r = b.d.r, k = b.k;
        if (b.one_sided) {   // C = U^T G with the core update in the epilogue, then W -= U D
            add_tiles(ctx, KO, bi, r, n, m, 0);
            add_tiles(ctx, KOA, bi, m, n, r, 0);
        } else {
            if (b.proj_right) add_tiles(ctx, KT, bi, r, n, m, 0);      // T = U^T G
            else add_tiles(ctx, KT, bi, m, r, n, 0);                   // T~ = (G V)^T
            // a block with a long contraction (an embedding) is cut into split-K slabs; its tiles sit in the same
            // table, so that one launch covers every block
            add_tiles(ctx, KC, bi, r, r, b.proj_right ? n : m, b.nsplit > 1 ? b.kb_per_split : 0);
            add_tiles(ctx, KP, bi, b.right_first ? n : m, r, r, 0);
            add_tiles(ctx, KA, bi, m, n, r, 0);
        }
        add_tiles(ctx, KY, bi, m, k, n, 0);
        add_tiles(ctx, KZ, bi, n, k, m, 0);
        if (b.tc_rows) {   // K blocks of 32 FP32 elements: pass 2 k so that the count comes out as ceil(k / 32)
            add_tiles(ctx, KR01, bi, m, k, 2 * k, 0, 32);
            add_tiles(ctx, KR02, bi, m, k, 2 * k, 0, 32);
            add_tiles(ctx, KR12, bi, n, k, 2 * k, 0, 32);
            add_tiles(ctx, KRU, bi, m, r, 2 * k, 0);
            add_tiles(ctx, KRV, bi, n, r, 2 * k, 0);
        }
        // exact integer Gram matrices: 256 x 64 tiles on or above the diagonal, one per chunk of GRAM_ROWS rows
        for (int side = 0; side < 2; ++side) {
            const int kd = KG0 + side, rows = side ? n : m;
            std::vector<UmmaTile> &v = ctx->tiles[kd];
            b.tile_begin[kd] = (int)v.size();
            for (int c = 0; c < gram_chunks(rows); ++c)
                for (int i0 = 0; i0 < k; i0 += 256)
                    for (int j0 = 0; j0 < k; j0 += 64) {
                        if (j0 + 64 <= i0) continue;
                        UmmaTile t;
                        memset(&t, 0, sizeof t);
                        t.prob = bi; t.m0 = i0; t.n0 = j0; t.split = c;
                        t.kb0 = c * (GRAM_ROWS / 64);
                        t.kb1 = (std::min(rows, (c + 1) * GRAM_ROWS) + 63) / 64;
                        t.wait_slot = -1; t.signal_slot = -1;
                        v.push_back(t);
                    }
            b.tile_end[kd] = (int)v.size();
        }
    }
    build_merged(ctx);
}

// BF16 row-major [rows x cols] (ld elements) -> tensor map with a 64 x box_rows box, 128B swizzle.
tsr_status encode_map(tsr_ctx *ctx, CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int64_t ld,
                      int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS)
        return fail(ctx, TSR_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) rows=%lld cols=%lld ld=%lld", (int)rc,
                    (long long)rows, (long long)cols, (long long)ld);
    return TSR_OK;
}

// INT8 row-major [rows x cols] (ld bytes) -> tensor map with a 64-byte x box_rows box, 64B swizzle.
tsr_status encode_map_i8(tsr_ctx *ctx, CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int64_t ld, int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS)
        return fail(ctx, TSR_ERR_CUDA, "cuTensorMapEncodeTiled (digit planes) failed (%d) rows=%lld cols=%lld", (int)rc,
                    (long long)rows, (long long)cols);
    return TSR_OK;
}

// FP32 row-major [rows x cols] (ld elements) -> tensor map with a 32 x box_rows box (128 bytes of K), 128B swizzle.
tsr_status encode_map_f32(tsr_ctx *ctx, CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int64_t ld,
                          int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS)
        return fail(ctx, TSR_ERR_CUDA, "cuTensorMapEncodeTiled (FP32 operand) failed (%d) rows=%lld cols=%lld", (int)rc,
                    (long long)rows, (long long)cols);
    return TSR_OK;
}

// BF16 row-major output [rows x cols] (ld elements) -> tensor map with a 32 x 32 box (64-byte rows), 64B swizzle.
tsr_status encode_map_out_bf16(tsr_ctx *ctx, CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int64_t ld)
{
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return fail(ctx, TSR_ERR_CUDA, "cuTensorMapEncodeTiled (BF16 output) failed (%d)", (int)rc);
    return TSR_OK;
}

// FP32 row-major [rows x cols] (ld elements) -> tensor map with a 32 x 32 box, 128B swizzle.
tsr_status encode_map_w(tsr_ctx *ctx, CUtensorMap *out, const void *base, int64_t rows, int64_t cols, int64_t ld,
                        int w_dtype)
{
    const bool bf = (w_dtype == TSR_BF16);   // BF16 weights: 64-byte box rows, 64-byte swizzle
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * (bf ? 2 : 4)};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = ctx->encode(out, bf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                              const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              bf ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return fail(ctx, TSR_ERR_CUDA, "cuTensorMapEncodeTiled (W) failed (%d)", (int)rc);
    return TSR_OK;
}

StepScalars make_scalars(const tsr_ctx *ctx, const tsr_hyper *h)
{
    StepScalars sc;
    sc.wait_clocks = ctx->wait_clocks;
    sc.beta1 = h->beta1; sc.beta2 = h->beta2; sc.eps = h->eps;
    sc.omb1 = (float)(1.0 - (double)h->beta1);
    sc.omb2 = (float)(1.0 - (double)h->beta2);
    const double t = (double)h->step;
    sc.inv_bc1 = (float)(1.0 / (1.0 - pow((double)h->beta1, t)));
    sc.inv_bc2 = (float)(1.0 / (1.0 - pow((double)h->beta2, t)));
    sc.rule = h->rule;
    if (h->rule == TSR_RULE_SGD) {
        sc.decay = 1.0f;
        sc.step_scale = h->lr;
    } else {
        sc.decay = 1.0f - h->lr * h->weight_decay;
        sc.step_scale = h->lr * h->scale;
    }
    return sc;
}

tsr_status check_hyper(tsr_ctx *ctx, const tsr_hyper *h)
{
    if (!h) return fail(ctx, TSR_ERR_INVALID_ARG, "hyper is NULL");
    if (h->step < 1) return fail(ctx, TSR_ERR_INVALID_ARG, "hyper.step must be >= 1");
    if (h->rule != TSR_RULE_ADAM && h->rule != TSR_RULE_SGD) return fail(ctx, TSR_ERR_INVALID_ARG, "unknown rule");
    if (!(h->beta1 >= 0.f && h->beta1 < 1.f) || !(h->beta2 >= 0.f && h->beta2 < 1.f))
        return fail(ctx, TSR_ERR_INVALID_ARG, "betas must lie in [0, 1)");
    return TSR_OK;
}

// The Adam rule reads and writes the second moment of every listed block: a block bound with
// Vm == NULL (allowed for callers that only ever use TSR_RULE_SGD) is an argument error here,
// found before anything is launched.
tsr_status check_rule_ptrs(tsr_ctx *ctx, const std::vector<int> &list, int rule)
{
    if (rule != TSR_RULE_ADAM) return TSR_OK;
    for (int bi : list)
        if (!ctx->blocks[bi].p.Vm)
            return fail(ctx, TSR_ERR_INVALID_ARG, "block %d: TSR_RULE_ADAM needs a second-moment buffer (Vm is NULL)", bi);
    return TSR_OK;
}

// Profiling: records the stage-boundary events ev[stage_next .. upto] on the step's stream.
void mark_stage(tsr_ctx *ctx, int upto)
{
    if (!ctx->profiling) return;
    for (; ctx->stage_next <= upto; ++ctx->stage_next) cudaEventRecord(ctx->ev[ctx->stage_next], ctx->stage_stream);
}

// Resolves (idx, count) into a validated list of block indices.
tsr_status resolve_list(tsr_ctx *ctx, const int32_t *idx, int32_t count, std::vector<int> &out)
{
    out.clear();
    const int nb = (int)ctx->blocks.size();
    if (!idx) {
        for (int i = 0; i < nb; ++i) out.push_back(i);
        return TSR_OK;
    }
    if (count < 0) return fail(ctx, TSR_ERR_INVALID_ARG, "negative count");
    std::vector<char> seen(nb, 0);
    for (int j = 0; j < count; ++j) {
        if (idx[j] < 0 || idx[j] >= nb) return fail(ctx, TSR_ERR_INVALID_ARG, "block index %d out of range", idx[j]);
        if (seen[idx[j]]) return fail(ctx, TSR_ERR_INVALID_ARG, "block index %d listed twice", idx[j]);
        seen[idx[j]] = 1;
        out.push_back(idx[j]);
    }
    return TSR_OK;
}

tsr_status check_ready(tsr_ctx *ctx)
{
    if (!ctx) return TSR_ERR_INVALID_ARG;
    if (!ctx->bound) return fail(ctx, TSR_ERR_NOT_BOUND, "tsr_bind has not been called");
    return TSR_OK;
}

// Launches one tensor-core GEMM kind over the listed blocks (adjacent table ranges are merged).
tsr_status launch_kind(tsr_ctx *ctx, int kind, const std::vector<int> &list, int epilogue, int planes,
                       const StepScalars &sc, cudaStream_t st)
{
    std::vector<std::pair<int, int>> ranges;
    for (int bi : list) {
        const Block &b = ctx->blocks[bi];
        if (b.tile_end[kind] > b.tile_begin[kind]) ranges.push_back({b.tile_begin[kind], b.tile_end[kind]});
    }
    std::sort(ranges.begin(), ranges.end());
    size_t i = 0;
    while (i < ranges.size()) {
        int lo = ranges[i].first, hi = ranges[i].second;
        size_t j = i + 1;
        while (j < ranges.size() && ranges[j].first == hi) { hi = ranges[j].second; ++j; }
        if (kind == KA || kind == KOA)
            TSR_CUDA(ctx, umma_apply_launch(ctx->d_probs[kind], ctx->d_tiles[kind] + lo, hi - lo, ctx->num_sms, ctx->bn[kind],
                                            elem_size(ctx->blocks[0].d.w_dtype), sc, ctx->d_status, st));
        else
            TSR_CUDA(ctx, umma_gemm_launch(ctx->d_probs[kind], ctx->d_tiles[kind] + lo, hi - lo, ctx->num_sms, ctx->bn[kind],
                                           epilogue, planes, sc, ctx->d_status, st));
        ctx->launches++;
        i = j;
    }
    return TSR_OK;
}

// which: 0 = d_list, 1 = d_list2 (their last contents are remembered, so that a step over the same blocks as the
// previous one uploads nothing), -1 = any other destination, always copied.
tsr_status upload_list(tsr_ctx *ctx, int32_t *dst, const std::vector<int> &v, cudaStream_t st, int which = -1)
{
    if (v.empty()) return TSR_OK;
    if (which >= 0 && ctx->list_cache[which] == v) return TSR_OK;
    TSR_CUDA(ctx, cudaMemcpyAsync(dst, v.data(), v.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    if (which >= 0) ctx->list_cache[which] = v;
    return TSR_OK;
}

// ---- Section 3.3: C = U^T G V (optionally with the fused core update) -------------------
tsr_status do_project(tsr_ctx *ctx, const std::vector<int> &list, bool fuse, const StepScalars &sc, cudaStream_t st)
{
    tsr_status s;
    if (ctx->any_fast) {
        // A call that covers every two-sided tensor-core block of the plan runs both contractions as ONE launch
        // (T~ tiles with the core tiles a few blocks behind them, T~ read back from L2); a partial list, or a
        // device that cannot take the cooperative launch, runs them as two launches.  The tiles, their
        // reduction order and therefore the results are the same either way.
        bool merged = false;
        // One launch saves the trip of T~ to DRAM and back, which only happens when T~ does not fit the L2 cache;
        // where it does (measured on the 60M, 130M and 350M sets: 0.079 / 0.157 / 0.297 ms as two launches against
        // 0.090 / 0.174 / 0.339 ms as one) the tiles of two plain launches need not wait for one another and win.
        const bool want_merged = ctx->proj_mode == 1 || (ctx->proj_mode == 0 && ctx->merge_pays);
        if (want_merged && ctx->merged_ok && !ctx->tiles[KM].empty()) {
            int have = 0, all = 0;
            for (const Block &b : ctx->blocks) all += (b.fast && !b.one_sided) ? 1 : 0;
            for (int bi : list) have += (ctx->blocks[bi].fast && !ctx->blocks[bi].one_sided) ? 1 : 0;
            if (have == all) {
                TSR_CUDA(ctx, cudaMemsetAsync(ctx->d_counters, 0, sizeof(int32_t) * (ctx->blocks.size() + 1), st));
                const cudaError_t e = umma_project_launch(ctx->d_probs[KT], ctx->d_probs[KCM], ctx->d_tiles[KM], (int)ctx->tiles[KM].size(),
                                                          ctx->num_sms, ctx->bn[KM], fuse ? 1 : 0, ctx->d_counters, sc, ctx->d_status, st,
                                                          (int)ctx->blocks.size());
                if (e == cudaSuccess) { merged = true; ctx->launches++; }
                else { (void)cudaGetLastError(); ctx->merged_ok = false; }   // refused: nothing ran; use two launches from now on
            }
        }
        if (!merged && (s = launch_kind(ctx, KT, list, EPI_STORE_BF16_T, 1, sc, st)) != TSR_OK) return s;
        mark_stage(ctx, 2);
        if (!merged && (s = launch_kind(ctx, KC, list, fuse ? EPI_CORE_UPDATE : EPI_STORE_F32, 1, sc, st)) != TSR_OK) return s;
        // one-sided blocks: C = U^T G contracts the gradient over its rows (read MN-major, no transposed copy)
        bool any_one_sided = false;
        for (int bi : list) {
            const Block &b = ctx->blocks[bi];
            if (b.fast && b.one_sided) any_one_sided = true;
        }
        if (any_one_sided && (s = launch_kind(ctx, KO, list, fuse ? EPI_CORE_UPDATE : EPI_STORE_F32, 1, sc, st)) != TSR_OK) return s;
    }
    std::vector<int> split, later;
    int max_r = 1, max_c = 1;
    for (int bi : list) {
        Block &b = ctx->blocks[bi];
        const int m = (int)b.d.m, n = (int)b.d.n, r = b.d.r;
        if (!b.fast && b.one_sided) {
            // C = U^T G on CUDA cores
            TSR_KERNEL(ctx, 1, simt_gemm_bt(r, n, m, b.p.U, 1, r, b.p.G, b.d.g_dtype, b.d.ldg, 1, b.p.C, n, st));
            if (fuse) { later.push_back(bi); max_r = std::max(max_r, r); max_c = std::max(max_c, n); }
        } else if (!b.fast) {
            // T = G V, C = U^T T on CUDA cores
            TSR_KERNEL(ctx, 1, simt_gemm(m, r, n, b.p.G, b.d.g_dtype, b.d.ldg, 1, b.p.V, r, 1, b.T32, r, SIMT_STORE, 0, 0, st));
            TSR_KERNEL(ctx, 1, simt_gemm(r, r, m, b.p.U, TSR_F32, 1, r, b.T32, r, 1, b.p.C, r, SIMT_STORE, 0, 0, st));
            if (fuse) { later.push_back(bi); max_r = std::max(max_r, r); max_c = std::max(max_c, r); }
        } else if (b.nsplit > 1) {
            split.push_back(bi);
            max_r = std::max(max_r, r); max_c = std::max(max_c, r);
        }
    }
    if (!split.empty()) {   // sum the split-K slabs (and, when fused, run the core update on the sum)
        if ((s = upload_list(ctx, ctx->d_list2, split, st, 1)) != TSR_OK) return s;
        TSR_KERNEL(ctx, 1, core_update_launch(ctx->d_cu_split, ctx->d_list2, (int)split.size(), max_r, max_c, sc, fuse ? 0 : 1, st));
    }
    if (!later.empty()) {
        if ((s = upload_list(ctx, ctx->d_list2, later, st, 1)) != TSR_OK) return s;
        TSR_KERNEL(ctx, 1, core_update_launch(ctx->d_cu_all, ctx->d_list2, (int)later.size(), max_r, max_c, sc, 0, st));
    }
    mark_stage(ctx, 3);
    return TSR_OK;
}

// ---- Section 3.4: moments and D from C ----------------------------------------------------
tsr_status do_core_update(tsr_ctx *ctx, const std::vector<int> &list, const StepScalars &sc, cudaStream_t st)
{
    tsr_status s;
    if ((s = check_rule_ptrs(ctx, list, sc.rule)) != TSR_OK) return s;
    int max_r = 1, max_c = 1;
    for (int bi : list) {
        max_r = std::max(max_r, (int)ctx->blocks[bi].d.r);
        max_c = std::max(max_c, (int)ctx->blocks[bi].cn);
    }
    if ((s = upload_list(ctx, ctx->d_list, list, st, 0)) != TSR_OK) return s;
    TSR_KERNEL(ctx, 1, core_update_launch(ctx->d_cu_all, ctx->d_list, (int)list.size(), max_r, max_c, sc, 0, st));
    return TSR_OK;
}

// ---- Section 3.4: W <- decay W - step_scale U D V^T ---------------------------------------
tsr_status do_apply(tsr_ctx *ctx, const std::vector<int> &list, const StepScalars &sc, cudaStream_t st)
{
    tsr_status s;
    if (ctx->any_fast) {
        if ((s = launch_kind(ctx, KP, list, EPI_STORE_BF16, 1, sc, st)) != TSR_OK) return s;
        mark_stage(ctx, 5);
        if ((s = launch_kind(ctx, KA, list, EPI_APPLY, 1, sc, st)) != TSR_OK) return s;
        if ((s = launch_kind(ctx, KOA, list, EPI_APPLY, 1, sc, st)) != TSR_OK) return s;
    }
    for (int bi : list) {
        Block &b = ctx->blocks[bi];
        if (b.fast) continue;
        const int m = (int)b.d.m, n = (int)b.d.n, r = b.d.r;
        if (b.one_sided) {   // W <- decay W - step_scale U D, D being r x n
            TSR_KERNEL(ctx, 1, simt_gemm(m, n, r, b.p.U, TSR_F32, r, 1, b.D32, n, 1, (float *)b.p.W, b.d.ldw,
                                    b.d.w_dtype == TSR_BF16 ? SIMT_APPLY_BF16 : SIMT_APPLY, sc.decay, sc.step_scale, st));
            continue;
        }
        TSR_KERNEL(ctx, 1, simt_gemm(m, r, r, b.p.U, TSR_F32, r, 1, b.D32, r, 1, b.P32, r, SIMT_STORE, 0, 0, st));
        TSR_KERNEL(ctx, 1, simt_gemm(m, n, r, b.P32, TSR_F32, r, 1, b.p.V, 1, r, (float *)b.p.W, b.d.ldw,
                                b.d.w_dtype == TSR_BF16 ? SIMT_APPLY_BF16 : SIMT_APPLY, sc.decay, sc.step_scale, st));
    }
    return TSR_OK;
}

// BF16 operand copies of U and V for the listed blocks.  One launch per block and basis: measured against a
// form that converts all blocks of a refresh group in one launch per stage, the refresh of the 1B set took 141 ms
// this way and 153 ms batched (with the groups on concurrent streams the small launches interleave with the other
// groups' kernels; the batched ones kept the groups in step with one another).
tsr_status do_shadows(tsr_ctx *ctx, const std::vector<int> &list, cudaStream_t st)
{
    for (int bi : list) {
        Block &b = ctx->blocks[bi];
        if (!b.fast) continue;
        TSR_KERNEL(ctx, 1, make_shadows(b.p.U, (int)b.d.m, b.d.r, b.Ub, b.rl, b.Ubt, b.ml, st));
        TSR_KERNEL(ctx, 1, make_shadows(b.p.V, (int)b.d.n, b.d.r, b.Vb, b.rl, b.Vbt, b.nl, st));
    }
    return TSR_OK;
}

// ---- Section 3.5: randomized-SVD refresh ---------------------------------------------------
struct RefreshLists {
    std::vector<int> list;
    int nitems[4];
    int kmax, rmax;
    int32_t *dlist;        // this group's slice of the device list / item tables
    RowItem *ditems[5];
};

// dst = buf[src] * Mat for every block of the list (see rows_gemm_batched for the selectors).  Lists
// whose blocks all qualify run on tensor cores: the rows and the transposed small matrix are split
// into a TF32 plane and a remainder plane, and the product is three TF32 MMAs per K step.
tsr_status rows_product(tsr_ctx *ctx, const RefreshLists &L, int side, int src, int mat, int dst, bool exact_not_needed,
                        cudaStream_t st)
{
    const int nl = (int)L.list.size();
    // The tensor cores accumulate with less than FP32 rounding accuracy (measured: bases came out
    // orthonormal to 2e-4 instead of 1e-6), so the three products whose result is final -- the second
    // Cholesky-QR pass and U, V -- stay on the FP32 CUDA-core kernel.
    bool tc = exact_not_needed;
    for (int bi : L.list) tc = tc && ctx->blocks[bi].tc_rows;
    if (!tc) {
        TSR_KERNEL(ctx, 1, rows_gemm_batched(ctx->d_refresh, L.ditems[side * 2], L.nitems[side * 2], side, src, mat, dst,
                                             mat == 0 ? L.kmax : L.rmax, st));
        return TSR_OK;
    }
    const int kind = (dst == 3) ? KRU : (dst == 4) ? KRV : (side == 1) ? KR12 : (dst == 1 ? KR01 : KR02);
    if (side == 1 && dst != 2 && dst != 4) return fail(ctx, TSR_ERR_INVALID_ARG, "unexpected destination of a row product");
    TSR_KERNEL(ctx, 2, split_operands_batched(ctx->d_refresh, L.ditems[side * 2], L.nitems[side * 2], L.dlist, nl, side, src,
                                              mat, L.kmax, st));
    StepScalars sc;
    memset(&sc, 0, sizeof sc);
    sc.wait_clocks = ctx->wait_clocks;
    return launch_kind(ctx, kind, L.list, EPI_STORE_F32, 3, sc, st);
}

// S = X^T X (X = buf[src], FP64 result) for every block of the group.  Blocks on the tensor-core path whose sketch
// is a genuine sketch (k <= min(m, n) / 2) take the integer form (digit planes, INT8 MMAs, see tsr_gram_i8.cu): it
// carries 42 bits below each column's largest entry, i.e. S to about 5e-11 relative to |x_i| |x_j|, against the
// kappa(X)^2 <= 5e8 of such sketches.  A sketch as wide as the matrix (the exact-SVD arm: kappa(X)^2 up to 1e14)
// needs everything FP64 has, and goes, like any block off the tensor-core path, through the FP64 tensor path.
tsr_status gram(tsr_ctx *ctx, const RefreshLists &L, int side, int src, cudaStream_t st)
{
    const int nl = (int)L.list.size();
    bool i8 = true;
    for (int bi : L.list) {
        const Block &b = ctx->blocks[bi];
        i8 = i8 && b.fast && b.k >= 8 && 2 * (int64_t)b.k <= std::min(b.d.m, b.d.n);   // (k >= 8: the slab maxima fit the partial-sum buffer)
    }
    if (!i8) {
        TSR_KERNEL(ctx, 2, gram_batched(ctx->d_refresh, L.ditems[side * 2 + 1], L.nitems[side * 2 + 1], L.dlist, nl, side, src,
                                        L.kmax, st));
        return TSR_OK;
    }
    TSR_KERNEL(ctx, 3, gram_i8_prepare(ctx->d_refresh, L.ditems[side * 2], L.nitems[side * 2], L.dlist, nl, side, src, L.kmax, st));
    const int kind = KG0 + side;
    std::vector<std::pair<int, int>> ranges;
    for (int bi : L.list) ranges.push_back({ctx->blocks[bi].tile_begin[kind], ctx->blocks[bi].tile_end[kind]});
    std::sort(ranges.begin(), ranges.end());
    for (size_t i = 0; i < ranges.size();) {
        int lo = ranges[i].first, hi = ranges[i].second;
        size_t j = i + 1;
        while (j < ranges.size() && ranges[j].first == hi) { hi = ranges[j].second; ++j; }
        TSR_KERNEL(ctx, 1, gram_i8_launch(ctx->d_probs[kind], ctx->d_tiles[kind] + lo, hi - lo, ctx->num_sms, ctx->wait_clocks,
                                          ctx->d_status, st));
        i = j;
    }
    TSR_KERNEL(ctx, 1, gram_reduce_batched(ctx->d_refresh, L.dlist, nl, side, L.kmax, st));
    return TSR_OK;
}

tsr_status orth_pass(tsr_ctx *ctx, const RefreshLists &L, int side, int src, int dst, bool refined_later, cudaStream_t st)
{
    const int nl = (int)L.list.size();
    tsr_status sg = gram(ctx, L, side, src, st);
    if (sg != TSR_OK) return sg;
    TSR_KERNEL(ctx, 1, chol_inverse_batched(ctx->d_refresh, L.dlist, nl, L.kmax, st));
    return rows_product(ctx, L, side, src, 0, dst, refined_later, st);
}

// orth(buf[0]) -> buf[2] by Cholesky-QR with the Gram matrix accumulated in FP64.
// The basis that enters B = Q^T G and U = Q U~ (final = true) gets a second pass (buf[1] holds the
// first one), which brings Q^T Q to the identity at FP32 rounding level.  The bases inside the
// power iteration only have to span the right subspace and stay well conditioned: one pass
// leaves Q^T Q = I + O(kappa(Y)^2 u) with exactly the same range, so a single pass is used there.
tsr_status orth(tsr_ctx *ctx, const RefreshLists &L, int side, bool final, cudaStream_t st)
{
    tsr_status s;
    if (!final) return orth_pass(ctx, L, side, 0, 2, true, st);
    if ((s = orth_pass(ctx, L, side, 0, 1, true, st)) != TSR_OK) return s;
    return orth_pass(ctx, L, side, 1, 2, false, st);
}

// buf[0] (rows_out x k) = G X  (transposed = false, X = buf[2] or Omega, n x k)
//                      or G^T X (transposed = true,  X = buf[2], m x k)
// planes: 2 = the FP32 operand X as BF16 hi + lo planes (two MMAs into one accumulator); 1 = its BF16 rounding
// alone.  The sketches inside the power iteration take one plane: rounding the test matrix or the intermediate
// basis perturbs it by 2^-9, which acts like a slightly different starting matrix (measured against the oracle: the
// captured energy agrees to seven digits either way, the projector at the spectral gap moves from 2e-5 to 3e-5..6e-5,
// only the ill-determined directions inside the noise bulk differ more).  B = Q^T G, which the singular vectors
// are computed from, keeps both planes.
tsr_status sketch(tsr_ctx *ctx, const RefreshLists &L, bool transposed, bool from_omega,
                  const float *const *omegas, cudaStream_t st, int planes = 2)
{
    StepScalars sc = {};
    sc.wait_clocks = ctx->wait_clocks;
    tsr_status s;
    (void)omegas;   // a caller-given Omega has been copied into the block's own buffer by now
    for (size_t j = 0; j < L.list.size(); ++j) {
        Block &b = ctx->blocks[L.list[j]];
        const int m = (int)b.d.m, n = (int)b.d.n, k = b.k;
        const float *X = from_omega ? b.Om : b.buf[2];
        if (b.fast) {   // X^T as BF16 plane(s): the B operand of the sketch GEMM
            TSR_KERNEL(ctx, 1, split_transpose(X, transposed ? m : n, k, b.Xt, transposed ? b.ml : b.nl, k, planes, st));
        } else if (!transposed) {
            TSR_KERNEL(ctx, 1, simt_gemm(m, k, n, b.p.G, b.d.g_dtype, b.d.ldg, 1, X, k, 1, b.buf[0], k, SIMT_STORE, 0, 0, st));
        } else {
            TSR_KERNEL(ctx, 1, simt_gemm(n, k, m, b.p.G, b.d.g_dtype, 1, b.d.ldg, X, k, 1, b.buf[0], k, SIMT_STORE, 0, 0, st));
        }
    }
    if (ctx->any_fast)
        if ((s = launch_kind(ctx, transposed ? KZ : KY, L.list, EPI_STORE_F32, planes, sc, st)) != TSR_OK) return s;
    return TSR_OK;
}

// One group of blocks through the whole refresh on stream st.  list_off / item_off: where this
// group's slices start inside the context's device list / item tables.
tsr_status do_refresh_group(tsr_ctx *ctx, const std::vector<int> &list, uint64_t seed, const float *const *omegas,
                            cudaStream_t st, size_t list_off, const size_t *item_off, bool reexpress, bool cached)
{
    if (list.empty()) return TSR_OK;
    tsr_status s;
    RefreshLists L;
    L.list = list;
    L.dlist = ctx->d_rlist + list_off;
    for (int i = 0; i < 5; ++i) L.ditems[i] = ctx->d_items[i] + item_off[i];
    L.kmax = 1; L.rmax = 1;
    std::vector<RowItem> items[4];
    int qmax = 0;
    for (int bi : list) {
        const Block &b = ctx->blocks[bi];
        L.kmax = std::max(L.kmax, b.k);
        L.rmax = std::max(L.rmax, (int)b.d.r);
        qmax = std::max(qmax, (int)b.d.q);
        for (int side = 0; side < 2; ++side) {
            const int rows = (int)(side ? b.d.n : b.d.m);
            for (int r0 = 0; r0 < rows; r0 += RG_ROWS) items[side * 2].push_back({bi, r0});
            for (int r0 = 0; r0 < rows; r0 += GRAM_ROWS) items[side * 2 + 1].push_back({bi, r0});
        }
    }
    for (int bi : list)
        if (ctx->blocks[bi].d.q != qmax)
            return fail(ctx, TSR_ERR_UNSUPPORTED, "blocks refreshed in one grouped call must share q");
    // cached: the device tables still hold exactly this refresh (same groups in the same order) from last time
    if (!cached) {
        if ((s = upload_list(ctx, L.dlist, list, st)) != TSR_OK) return s;
        for (int i = 0; i < 4; ++i)
            TSR_CUDA(ctx, cudaMemcpyAsync(L.ditems[i], items[i].data(), items[i].size() * sizeof(RowItem),
                                          cudaMemcpyHostToDevice, st));
    }
    for (int i = 0; i < 4; ++i) L.nitems[i] = (int)items[i].size();
    // Omega (drawn by the library, or the caller's copied into the block's buffer) and the transposed gradients
    for (size_t j = 0; j < list.size(); ++j) {
        Block &b = ctx->blocks[list[j]];
        if (omegas && omegas[j])
            TSR_CUDA(ctx, cudaMemcpyAsync(b.Om, omegas[j], (size_t)b.d.n * b.k * sizeof(float), cudaMemcpyDeviceToDevice, st));
        else
            TSR_KERNEL(ctx, 1, fill_gaussian(b.Om, (int64_t)b.d.n * b.k, seed, (uint64_t)list[j], st));
    }
    // Y = G Omega; Q = orth(Y)
    if ((s = sketch(ctx, L, false, true, omegas, st, 1)) != TSR_OK) return s;
    if ((s = orth(ctx, L, 0, qmax == 0, st)) != TSR_OK) return s;
    for (int it = 0; it < qmax; ++it) {
        // Yrow = G^T Q; Qrow = orth(Yrow); Y = G Qrow; Q = orth(Y)
        if ((s = sketch(ctx, L, true, false, nullptr, st, 1)) != TSR_OK) return s;
        if ((s = orth(ctx, L, 1, false, st)) != TSR_OK) return s;
        if ((s = sketch(ctx, L, false, false, nullptr, st, 1)) != TSR_OK) return s;
        if ((s = orth(ctx, L, 0, it == qmax - 1, st)) != TSR_OK) return s;
    }
    // B^T = G^T Q (n x k) in buf[0]; small SVD through the k x k Gram matrix B B^T
    if ((s = sketch(ctx, L, true, false, nullptr, st)) != TSR_OK) return s;
    const int nl = (int)list.size();
    if ((s = gram(ctx, L, 1, 0, st)) != TSR_OK) return s;
    // From k = 100 on the tridiagonal route is the faster one (k = 136: 11.4 ms of one-CTA Jacobi sweeps against about
    // 3 ms; the refresh of the single-matrix configuration went from 12.4 to 4.8 ms, of the 60M set from 15.9 to 8.0 ms)
    if (L.kmax >= 100) {
        const int pr = eig_panel_rows(L.kmax);
        std::vector<RowItem> panels;
        for (int bi : list)
            for (int r0 = 0; r0 < ctx->blocks[bi].k; r0 += pr) panels.push_back({bi, r0});
        if (!cached)
            TSR_CUDA(ctx, cudaMemcpyAsync(L.ditems[4], panels.data(), panels.size() * sizeof(RowItem), cudaMemcpyHostToDevice, st));
        TSR_KERNEL(ctx, 16, eig_tridiag_batched(ctx->d_refresh, L.dlist, nl, L.ditems[4], (int)panels.size(), L.kmax, st));
    } else {
        TSR_KERNEL(ctx, 1, jacobi_batched(ctx->d_refresh, L.dlist, nl, 40, st));
    }
    // V = B^T Wt / sigma ; U = Q Wt
    if (reexpress)   // keep the outgoing bases of the blocks that asked for moment re-expression
        for (int bi : list) {
            Block &b = ctx->blocks[bi];
            if (!(b.d.flags & TSR_BLOCK_REEXPRESS_MOMENT)) continue;
            TSR_CUDA(ctx, cudaMemcpyAsync(b.Uold, b.p.U, (size_t)b.d.m * b.d.r * 4, cudaMemcpyDeviceToDevice, st));
            TSR_CUDA(ctx, cudaMemcpyAsync(b.Vold, b.p.V, (size_t)b.d.n * b.d.r * 4, cudaMemcpyDeviceToDevice, st));
        }
    if ((s = rows_product(ctx, L, 1, 0, 2, 4, false, st)) != TSR_OK) return s;
    if ((s = rows_product(ctx, L, 0, 2, 1, 3, false, st)) != TSR_OK) return s;
    if (reexpress)   // M <- (Unew^T Uold) M (Vold^T Vnew)
        for (int bi : list) {
            Block &b = ctx->blocks[bi];
            if (!(b.d.flags & TSR_BLOCK_REEXPRESS_MOMENT)) continue;
            const int m = (int)b.d.m, n = (int)b.d.n, r = b.d.r;
            TSR_KERNEL(ctx, 1, simt_gemm(r, r, m, b.p.U, TSR_F32, 1, r, b.Uold, r, 1, b.Ra, r, SIMT_STORE, 0, 0, st));
            TSR_KERNEL(ctx, 1, simt_gemm(r, r, n, b.Vold, TSR_F32, 1, r, b.p.V, r, 1, b.Rb, r, SIMT_STORE, 0, 0, st));
            TSR_KERNEL(ctx, 1, simt_gemm(r, r, r, b.Ra, TSR_F32, r, 1, b.p.M, r, 1, b.Rt, r, SIMT_STORE, 0, 0, st));
            TSR_KERNEL(ctx, 1, simt_gemm(r, r, r, b.Rt, TSR_F32, r, 1, b.Rb, r, 1, b.p.M, r, SIMT_STORE, 0, 0, st));
        }
    return do_shadows(ctx, list, st);
}

// Refresh of a list of blocks (all with the same q).  Large lists are cut into up to NGROUP groups
// of consecutive blocks (in tile-table order) that run concurrently on the context's side streams;
// the caller's stream forks into them and joins afterwards, so the call keeps stream semantics.
tsr_status do_refresh(tsr_ctx *ctx, const std::vector<int> &list, uint64_t seed, const float *const *omegas,
                      cudaStream_t st, bool reexpress)
{
    if (list.empty()) return TSR_OK;
    const size_t zero[5] = {0, 0, 0, 0, 0};
    int ngroup = std::min<int>(tsr_ctx::NGROUP, (int)list.size() / 8);
    if (!ctx->aux_ready || ngroup < 2) {
        std::vector<int> sig = list;
        sig.push_back(-1);
        const bool cached = (sig == ctx->refresh_sig);
        ctx->refresh_sig.clear();
        const tsr_status s1 = do_refresh_group(ctx, list, seed, omegas, st, 0, zero, reexpress, cached);
        if (s1 == TSR_OK) ctx->refresh_sig.swap(sig);
        return s1;
    }
    // order the listed blocks as the tile tables do, remembering each one's omega
    std::vector<int> pos(ctx->blocks.size(), 0);
    for (size_t i = 0; i < ctx->order.size(); ++i) pos[ctx->order[i]] = (int)i;
    std::vector<size_t> perm(list.size());
    for (size_t i = 0; i < perm.size(); ++i) perm[i] = i;
    std::sort(perm.begin(), perm.end(), [&](size_t x, size_t y) { return pos[list[x]] < pos[list[y]]; });
    std::vector<int> sig;
    for (int g = 0; g < ngroup; ++g) {
        const size_t lo = perm.size() * g / ngroup, hi = perm.size() * (g + 1) / ngroup;
        for (size_t i = lo; i < hi; ++i) sig.push_back(list[perm[i]]);
        sig.push_back(-1);
    }
    const bool cached = (sig == ctx->refresh_sig);
    ctx->refresh_sig.clear();
    TSR_CUDA(ctx, cudaEventRecord(ctx->ev_fork, st));
    size_t list_off = 0, item_off[5] = {0, 0, 0, 0, 0};
    tsr_status result = TSR_OK;
    for (int g = 0; g < ngroup && result == TSR_OK; ++g) {
        const size_t lo = perm.size() * g / ngroup, hi = perm.size() * (g + 1) / ngroup;
        std::vector<int> grp;
        std::vector<const float *> om;
        for (size_t i = lo; i < hi; ++i) { grp.push_back(list[perm[i]]); om.push_back(omegas ? omegas[perm[i]] : nullptr); }
        // All groups start together: with eight groups of about twenty blocks the one-CTA-per-matrix
        // kernels of different groups drift apart by themselves, and a forced offset between the
        // groups only lengthened the critical path when it was measured.
        if (cudaStreamWaitEvent(ctx->aux[g], ctx->ev_fork, 0) != cudaSuccess)
            result = fail(ctx, TSR_ERR_CUDA, "cudaStreamWaitEvent failed on a refresh side stream");
        else
            result = do_refresh_group(ctx, grp, seed, omegas ? om.data() : nullptr, ctx->aux[g], list_off, item_off, reexpress, cached);
        // The side stream is joined whether or not its group was issued completely: the caller's
        // stream must not run ahead of (and the caller must not free buffers under) work in flight.
        if (cudaEventRecord(ctx->ev_join[g], ctx->aux[g]) != cudaSuccess ||
            cudaStreamWaitEvent(st, ctx->ev_join[g], 0) != cudaSuccess) {
            cudaStreamSynchronize(ctx->aux[g]);
            if (result == TSR_OK) result = fail(ctx, TSR_ERR_CUDA, "joining a refresh side stream failed");
        }
        list_off += grp.size();
        for (int bi : grp) {
            const Block &b = ctx->blocks[bi];
            item_off[0] += (size_t)((b.d.m + RG_ROWS - 1) / RG_ROWS);
            item_off[1] += (size_t)gram_chunks(b.d.m);
            item_off[2] += (size_t)((b.d.n + RG_ROWS - 1) / RG_ROWS);
            item_off[3] += (size_t)gram_chunks(b.d.n);
            item_off[4] += (size_t)((b.k + 7) / 8);
        }
    }
    if (result == TSR_OK) ctx->refresh_sig.swap(sig);
    return result;
}

tsr_status zero_moments(tsr_ctx *ctx, const std::vector<int> &list, cudaStream_t st)
{
    for (int bi : list) {
        Block &b = ctx->blocks[bi];
        const int64_t rr = (int64_t)b.d.r * b.cn;
        TSR_CUDA(ctx, fill_zero_f32(b.p.M, rr, st));
        if (b.p.Vm) TSR_CUDA(ctx, fill_zero_f32(b.p.Vm, rr, st));
    }
    return TSR_OK;
}

tsr_status do_step(tsr_ctx *ctx, const std::vector<int> &list, const tsr_hyper *h, uint64_t seed, bool fuse,
                   cudaStream_t st)
{
    tsr_status s;
    if ((s = check_rule_ptrs(ctx, list, h->rule)) != TSR_OK) return s;
    if (ctx->profiling) TSR_CUDA(ctx, cudaEventRecord(ctx->ev[0], st));
    std::vector<int> due;
    for (int bi : list) {
        const Block &b = ctx->blocks[bi];
        if (b.d.K > 0 && h->step % b.d.K == 0) due.push_back(bi);
    }
    if (!due.empty()) {
        // blocks with different q refresh in separate groups
        std::vector<int> qs;
        for (int bi : due) if (std::find(qs.begin(), qs.end(), (int)ctx->blocks[bi].d.q) == qs.end()) qs.push_back(ctx->blocks[bi].d.q);
        for (int q : qs) {
            std::vector<int> grp;
            for (int bi : due) if (ctx->blocks[bi].d.q == q) grp.push_back(bi);
            if ((s = do_refresh(ctx, grp, seed ^ ((uint64_t)h->step * 0x9E3779B97F4A7C15ull), nullptr, st, true)) != TSR_OK) return s;
        }
    }
    const StepScalars sc = make_scalars(ctx, h);
    ctx->stage_stream = st;
    ctx->stage_next = 1;
    if (ctx->profiling) {
        ctx->ev_valid = false;
        TSR_CUDA(ctx, cudaEventRecord(ctx->ev[1], st));
        ctx->stage_next = 2;
    }
    if ((s = do_project(ctx, list, fuse, sc, st)) != TSR_OK) return s;
    if (!fuse && (s = do_core_update(ctx, list, sc, st)) != TSR_OK) return s;
    mark_stage(ctx, 4);
    if ((s = do_apply(ctx, list, sc, st)) != TSR_OK) return s;
    mark_stage(ctx, 6);
    if (ctx->profiling) ctx->ev_valid = true;
    return TSR_OK;
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

int tsr_version(void) { return 100; }

const char *tsr_status_string(tsr_status s)
{
    switch (s) {
    case TSR_OK: return "ok";
    case TSR_ERR_INVALID_ARG: return "invalid argument";
    case TSR_ERR_SHAPE: return "bad shape";
    case TSR_ERR_ALIGNMENT: return "bad alignment";
    case TSR_ERR_WORKSPACE: return "workspace missing or too small";
    case TSR_ERR_CUDA: return "CUDA error";
    case TSR_ERR_UNSUPPORTED: return "unsupported";
    case TSR_ERR_NOT_CONVERGED: return "eigen-solver did not converge";
    case TSR_ERR_RANK_DEFICIENT: return "rank-deficient sketch";
    case TSR_ERR_NONFINITE: return "non-finite value";
    case TSR_ERR_TIMEOUT: return "bounded device wait ran out";
    case TSR_ERR_NOT_BOUND: return "context not bound";
    }
    return "unknown status";
}

const char *tsr_last_error(const tsr_ctx *ctx) { return ctx ? ctx->err.c_str() : ""; }

tsr_status tsr_create(tsr_ctx **out, const tsr_mat_desc *descs, int32_t count)
{
    if (!out) return TSR_ERR_INVALID_ARG;
    *out = nullptr;
    if (!descs || count <= 0) return TSR_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) {
        const tsr_mat_desc &d = descs[i];
        if (d.m <= 0 || d.n <= 0 || d.r <= 0 || d.p < 0 || d.q < 0) return TSR_ERR_SHAPE;
        if (d.ldg < d.n || d.ldw < d.n) return TSR_ERR_SHAPE;
        if ((int64_t)d.r + d.p > std::min(d.m, d.n)) return TSR_ERR_SHAPE;
        if (d.m > 0x3fffffff || d.n > 0x3fffffff || d.r + d.p > 1056) return TSR_ERR_SHAPE;
        if (d.g_dtype != TSR_F32 && d.g_dtype != TSR_BF16) return TSR_ERR_UNSUPPORTED;
        if (d.w_dtype != TSR_F32 && d.w_dtype != TSR_BF16) return TSR_ERR_UNSUPPORTED;
        if (d.w_dtype != descs[0].w_dtype) return TSR_ERR_UNSUPPORTED;   // one weight type per context (one apply launch)
        if ((d.flags & ~(int32_t)(TSR_BLOCK_REEXPRESS_MOMENT | TSR_BLOCK_ONE_SIDED)) != 0 || (d.is_embedding != 0 && d.is_embedding != 1)) return TSR_ERR_INVALID_ARG;
        if ((d.flags & TSR_BLOCK_REEXPRESS_MOMENT) && (d.flags & TSR_BLOCK_ONE_SIDED)) return TSR_ERR_UNSUPPORTED;
    }
    tsr_ctx *ctx = new (std::nothrow) tsr_ctx;
    if (!ctx) return TSR_ERR_INVALID_ARG;
    ctx->blocks.resize(count);
    for (int i = 0; i < count; ++i) {
        Block &b = ctx->blocks[i];
        b.d = descs[i];
        memset(&b.p, 0, sizeof b.p);
        b.k = b.d.r + b.d.p;
        b.one_sided = (b.d.flags & TSR_BLOCK_ONE_SIDED) != 0;
        b.cn = b.one_sided ? b.d.n : b.d.r;
        b.right_first = !b.one_sided && b.d.m > b.d.n;
        b.rl = round_up(b.d.r, 8); b.ml = round_up(b.d.m, 8); b.nl = round_up(b.d.n, 8);
        // Candidate for the tensor-core path: BF16 gradient with 16-byte row pitches.  Pointer
        // alignment is checked at bind time.
        b.fast = (b.d.g_dtype == TSR_BF16) && ((b.d.ldg * 2) % 16 == 0) && ((b.d.ldw * elem_size(b.d.w_dtype)) % 16 == 0);
        b.tc_rows = b.fast && (b.k % 4 == 0);   // FP32 rows of k elements as a TMA operand: 16-byte row pitch
        const int nkb = (int)((b.d.m + 63) / 64);
        if (nkb > 128 && !b.one_sided) { b.kb_per_split = 32; b.nsplit = (nkb + 31) / 32; }
        // (an embedding-like block, whose m is a single long contraction for U^T G, keeps T~ = (G V)^T and the split-K core)
        b.proj_right = b.right_first && nkb <= 128;
        ctx->max_r = std::max(ctx->max_r, (int)b.d.r);
        ctx->max_k = std::max(ctx->max_k, b.k);
        ctx->order.push_back(i);
    }
    ctx->max_sweeps.assign(count, 0);
    std::stable_sort(ctx->order.begin(), ctx->order.end(), [&](int a, int b) {
        return ctx->blocks[a].d.m * ctx->blocks[a].d.n > ctx->blocks[b].d.m * ctx->blocks[b].d.n;
    });
    build_tiles(ctx);
    Arena a{nullptr, 0};
    size_t step_end = 0;
    layout(ctx, a, false, &step_end);
    ctx->step_bytes = step_end;
    ctx->refresh_bytes = a.off - step_end;
    *out = ctx;
    return TSR_OK;
}

tsr_status tsr_destroy(tsr_ctx *ctx)
{
    if (!ctx) return TSR_ERR_INVALID_ARG;
    if (ctx->profiling)
        for (cudaEvent_t e : ctx->ev) if (e) cudaEventDestroy(e);
    if (ctx->aux_ready) {
        for (int g = 0; g < tsr_ctx::NGROUP; ++g) { cudaStreamDestroy(ctx->aux[g]); cudaEventDestroy(ctx->ev_join[g]); }
        cudaEventDestroy(ctx->ev_fork);
        for (int c = 0; c < tsr_ctx::NPIPE; ++c) { cudaEventDestroy(ctx->ev_pipe_in[c]); cudaEventDestroy(ctx->ev_pipe_done[c]); }
    }
    delete ctx;
    return TSR_OK;
}

tsr_status tsr_workspace_bytes(const tsr_ctx *ctx, size_t *step_bytes, size_t *refresh_bytes)
{
    if (!ctx || !step_bytes || !refresh_bytes) return TSR_ERR_INVALID_ARG;
    *step_bytes = ctx->step_bytes;
    *refresh_bytes = ctx->refresh_bytes;
    return TSR_OK;
}

tsr_status tsr_bind(tsr_ctx *ctx, const tsr_mat_ptrs *ptrs, int32_t count, void *workspace, size_t workspace_bytes)
{
    if (!ctx) return TSR_ERR_INVALID_ARG;
    if (!ptrs || count != (int32_t)ctx->blocks.size()) return fail(ctx, TSR_ERR_INVALID_ARG, "ptrs/count mismatch");
    if (!workspace || workspace_bytes < ctx->step_bytes + ctx->refresh_bytes)
        return fail(ctx, TSR_ERR_WORKSPACE, "workspace needs %zu bytes", ctx->step_bytes + ctx->refresh_bytes);
    if (((uintptr_t)workspace & 255) != 0) return fail(ctx, TSR_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
    for (int i = 0; i < count; ++i) {
        const tsr_mat_ptrs &p = ptrs[i];
        if (!p.G || !p.W || !p.U || !p.V || !p.M || !p.C) return fail(ctx, TSR_ERR_INVALID_ARG, "block %d: NULL pointer", i);
        if ((((uintptr_t)p.U | (uintptr_t)p.V | (uintptr_t)p.M | (uintptr_t)p.C) & 3) ||
            ((uintptr_t)p.W & (uintptr_t)(elem_size(ctx->blocks[i].d.w_dtype) - 1)))
            return fail(ctx, TSR_ERR_ALIGNMENT, "block %d: FP32 buffer not 4-byte aligned", i);
    }
    int dev_count = 0;
    if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count <= 0)
        return fail(ctx, TSR_ERR_CUDA, "no CUDA device available");
    ctx->bound = false;
    ctx->refresh_sig.clear();
    ctx->list_cache[0].clear(); ctx->list_cache[1].clear();
    bool layout_changed = false;
    for (int i = 0; i < count; ++i) {
        Block &b = ctx->blocks[i];
        b.p = ptrs[i];
        const bool cand = (b.d.g_dtype == TSR_BF16) && ((b.d.ldg * 2) % 16 == 0) && ((b.d.ldw * elem_size(b.d.w_dtype)) % 16 == 0);
        const bool fast = cand && aligned16(b.p.G) && aligned16(b.p.W);
        if (fast != b.fast) { b.fast = fast; b.tc_rows = fast && (b.k % 4 == 0); layout_changed = true; }
    }
    if (layout_changed) {   // a misaligned pointer moved a block to the CUDA-core path
        build_tiles(ctx);
        Arena m{nullptr, 0};
        size_t se = 0;
        layout(ctx, m, false, &se);
        ctx->step_bytes = se;
        ctx->refresh_bytes = m.off - se;
        if (workspace_bytes < m.off) return fail(ctx, TSR_ERR_WORKSPACE, "workspace needs %zu bytes", m.off);
    }
    ctx->any_fast = false;
    for (const Block &b : ctx->blocks) ctx->any_fast = ctx->any_fast || b.fast;
    Arena a{(char *)workspace, 0};
    size_t step_end = 0;
    layout(ctx, a, true, &step_end);

    if (ctx->any_fast) {
        if (!ctx->encode) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            TSR_CUDA(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
            if (!fn || qres != cudaDriverEntryPointSuccess) return fail(ctx, TSR_ERR_CUDA, "cuTensorMapEncodeTiled unavailable");
            ctx->encode = (EncodeTiledFn)fn;
        }
        TSR_CUDA(ctx, umma_configure());
        TSR_CUDA(ctx, umma_apply_configure());
        TSR_CUDA(ctx, gram_i8_configure());
        int dev = 0;
        TSR_CUDA(ctx, cudaGetDevice(&dev));
        TSR_CUDA(ctx, cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, dev));
        int l2 = 0;
        TSR_CUDA(ctx, cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev));
        ctx->l2_bytes = (size_t)l2;
    }
    {   // bytes of the intermediate T~ (BF16, r x m) over the blocks that go through the merged projection launch
        size_t tt = 0;
        for (const Block &b : ctx->blocks)
            if (b.fast && !b.one_sided) tt += (size_t)b.d.r * (size_t)(b.proj_right ? b.nl : b.ml) * 2;
        ctx->merge_pays = ctx->l2_bytes > 0 && tt > 2 * ctx->l2_bytes;
    }

    const int nb = count;
    std::vector<UmmaProblem> probs[NKIND];
    for (int kd = 0; kd < NKIND; ++kd) { probs[kd].resize(nb); memset((void *)probs[kd].data(), 0, sizeof(UmmaProblem) * nb); }
    std::vector<CoreUpdateArgs> cu_all(nb), cu_split(nb);
    std::vector<RefreshDev> rdev(nb);
    tsr_status s;
    for (int i = 0; i < nb; ++i) {
        Block &b = ctx->blocks[i];
        const int64_t m = b.d.m, n = b.d.n, r = b.d.r, k = b.k;
        CoreUpdateArgs &ca = cu_all[i];
        memset(&ca, 0, sizeof ca);
        ca.C = b.p.C; ca.Cout = b.p.C; ca.mom1 = b.p.M; ca.mom2 = b.p.Vm; ca.d_f32 = b.D32;
        ca.d_bf16 = (b.fast && b.right_first) ? b.Db : nullptr; ca.dt_bf16 = b.fast ? b.Dbt : nullptr; ca.ldd = b.rl;
        ca.split_stride = 0; ca.r = (int)r; ca.nc = (int)b.cn; ca.nsplit = 1;
        cu_split[i] = ca;
        cu_split[i].C = b.partial; cu_split[i].nsplit = b.nsplit; cu_split[i].split_stride = r * r;
        RefreshDev &rd = rdev[i];
        memset(&rd, 0, sizeof rd);
        rd.m = (int)m; rd.n = (int)n; rd.k = (int)k; rd.r = (int)r;
        for (int j = 0; j < 3; ++j) rd.buf[j] = b.buf[j];
        rd.S = b.S; rd.Xw = b.Xw; rd.Wj = b.Wj; rd.gpart = b.gpart; rd.lam = b.lam;
        rd.Xs = b.Xs; rd.Bts = b.Bts;
        rd.Rinv = b.Rinv; rd.Wu = b.Wu; rd.Wv = b.Wv; rd.U = b.p.U; rd.V = b.p.V; rd.status = ctx->d_status + i;
        rd.tau = b.tau; rd.dvec = b.dvec; rd.evec = b.evec; rd.rot = b.rot; rd.sweeps = b.sweeps; rd.groups = b.groups; rd.nsweeps = b.nsweeps;
        rd.rank = b.rank; rd.rot_cap = b.rot_cap; rd.sweep_cap = b.sweep_cap;
        rd.max_sweeps = ctx->max_sweeps[i];
        rd.col_exp = b.col_exp; rd.planes = b.planes; rd.ldp = b.ldp;
        rd.dc_z = b.dc_z; rd.dc_nd = b.dc_nd; rd.dc_rot_idx = b.dc_rot_idx; rd.dc_rot_cs = b.dc_rot_cs;
        rd.dc_scal = b.dc_scal; rd.dc_info = b.dc_info;
        if (!b.fast) continue;
        auto base = [&](UmmaProblem &P, int M, int N, int K, int epi) {
            P.M = M; P.N = N; P.K = K; P.planes = 1; P.plane_rows = 0; P.block = i; P.epilogue = epi;
        };
        if (b.one_sided) {
            {   // C = U^T G (+ core update) : A = U^T copy [r x m], B = G itself, contracted over its rows (MN-major)
                UmmaProblem &P = probs[KO][i];
                base(P, (int)r, (int)n, (int)m, EPI_CORE_UPDATE);
                if ((s = encode_map(ctx, &P.tmA, b.Ubt, r, m, b.ml, 128)) != TSR_OK) return s;
                if ((s = encode_map(ctx, &P.tmB, b.p.G, m, n, b.d.ldg, 64)) != TSR_OK) return s;
                P.b_mn = 1;
                P.out = b.p.C; P.ld_out = n; P.split_stride = 0;
                P.mom1 = b.p.M; P.mom2 = b.p.Vm; P.d_bf16 = nullptr; P.dt_bf16 = b.Dbt; P.ldd = b.rl;
            }
            {   // W update : A = U copy [m x r], B = D^T copy [n x r]
                UmmaProblem &P = probs[KOA][i];
                base(P, (int)m, (int)n, (int)r, EPI_APPLY);
                if ((s = encode_map(ctx, &P.tmA, b.Ub, m, r, b.rl, 128)) != TSR_OK) return s;
                if ((s = encode_map(ctx, &P.tmB, b.Dbt, n, r, b.rl, 128)) != TSR_OK) return s;
                if ((s = encode_map_w(ctx, &P.tmW, b.p.W, m, n, b.d.ldw, b.d.w_dtype)) != TSR_OK) return s;
                P.out = b.p.W; P.ld_out = b.d.ldw;
            }
        }
        if (b.proj_right) {   // T = U^T G : A = U^T copy [r x m], B = G itself, [m x n] contracted over its rows (MN-major)
            UmmaProblem &P = probs[KT][i];
            base(P, (int)r, (int)n, (int)m, EPI_STORE_BF16);
            if ((s = encode_map(ctx, &P.tmA, b.Ubt, r, m, b.ml, 128)) != TSR_OK) return s;
            if ((s = encode_map(ctx, &P.tmB, b.p.G, m, n, b.d.ldg, 64)) != TSR_OK) return s;
            P.b_mn = 1;
            P.out = b.Tt; P.ld_out = b.nl;
            P.starve = (ctx->starve_block == i) ? 1 : 0;
        } else {   // T~ = (G V)^T : A = G [m x n], B = V^T copy [r x n]
            UmmaProblem &P = probs[KT][i];
            base(P, (int)m, (int)r, (int)n, EPI_STORE_BF16_T);
            if ((s = encode_map(ctx, &P.tmA, b.p.G, m, n, b.d.ldg, 128)) != TSR_OK) return s;
            if ((s = encode_map(ctx, &P.tmB, b.Vbt, r, n, b.nl, ctx->bn[KT] / 2)) != TSR_OK) return s;
            P.out = b.Tt; P.ld_out = b.ml;
            P.starve = (ctx->starve_block == i) ? 1 : 0;
        }
        {   // C = U^T T : A = U^T copy [r x m], B = T~ [r x m].  A split-K block only stores its slabs
            // (the sum and the core update follow in core_update_kernel), whatever epilogue the launch has.
            UmmaProblem &P = probs[KC][i];
            if (b.proj_right) {   // C = T V : A = T [r x n], B = V^T copy [r x n]
                base(P, (int)r, (int)r, (int)n, EPI_CORE_UPDATE);
                if ((s = encode_map(ctx, &P.tmA, b.Tt, r, n, b.nl, 128)) != TSR_OK) return s;
                if ((s = encode_map(ctx, &P.tmB, b.Vbt, r, n, b.nl, ctx->bn[KC] / 2)) != TSR_OK) return s;
            } else {
                base(P, (int)r, (int)r, (int)m, b.nsplit > 1 ? EPI_STORE_F32 : EPI_CORE_UPDATE);
                if ((s = encode_map(ctx, &P.tmA, b.Ubt, r, m, b.ml, 128)) != TSR_OK) return s;
                if ((s = encode_map(ctx, &P.tmB, b.Tt, r, m, b.ml, ctx->bn[KC] / 2)) != TSR_OK) return s;
            }
            P.out = (b.nsplit > 1) ? (void *)b.partial : (void *)b.p.C;
            P.ld_out = r; P.split_stride = r * r;
            P.mom1 = b.p.M; P.mom2 = b.p.Vm; P.d_bf16 = b.right_first ? b.Db : nullptr; P.dt_bf16 = b.Dbt; P.ldd = b.rl;
        }
        {   // the same core problem for the merged projection launch: B boxes as wide as that launch's tiles
            UmmaProblem &P = probs[KCM][i];
            P = probs[KC][i];
            if (b.proj_right) { if ((s = encode_map(ctx, &P.tmB, b.Vbt, r, n, b.nl, ctx->bn[KCM] / 2)) != TSR_OK) return s; }
            else if ((s = encode_map(ctx, &P.tmB, b.Tt, r, m, b.ml, ctx->bn[KCM] / 2)) != TSR_OK) return s;
        }
        // The lift U D V^T goes through the smaller of the two intermediates: P = U D (m x r) when m <= n,
        // Z^T = V D^T (n x r) when m > n; either one lives in Pb and is the apply kernel's A or B operand.
        if (!b.right_first) {   // P = U D : A = U copy [m x r], B = D^T copy [r x r]
            UmmaProblem &P = probs[KP][i];
            base(P, (int)m, (int)r, (int)r, EPI_STORE_BF16);
            if ((s = encode_map(ctx, &P.tmA, b.Ub, m, r, b.rl, 128)) != TSR_OK) return s;
            if ((s = encode_map(ctx, &P.tmB, b.Dbt, r, r, b.rl, ctx->bn[KP] / 2)) != TSR_OK) return s;
            P.out = b.Pb; P.ld_out = b.rl;
            if ((s = encode_map_out_bf16(ctx, &P.tmW, b.Pb, m, r, b.rl)) != TSR_OK) return s;
            P.out_tma = 1;
        } else {                // Z^T = V D^T : A = V copy [n x r], B = D copy [r x r]
            UmmaProblem &P = probs[KP][i];
            base(P, (int)n, (int)r, (int)r, EPI_STORE_BF16);
            if ((s = encode_map(ctx, &P.tmA, b.Vb, n, r, b.rl, 128)) != TSR_OK) return s;
            if ((s = encode_map(ctx, &P.tmB, b.Db, r, r, b.rl, ctx->bn[KP] / 2)) != TSR_OK) return s;
            P.out = b.Pb; P.ld_out = b.rl;
            if ((s = encode_map_out_bf16(ctx, &P.tmW, b.Pb, n, r, b.rl)) != TSR_OK) return s;
            P.out_tma = 1;
        }
        {   // W update : A = P [m x r], B = V copy [n x r]   (or A = U copy, B = Z^T)
            UmmaProblem &P = probs[KA][i];
            base(P, (int)m, (int)n, (int)r, EPI_APPLY);
            if ((s = encode_map(ctx, &P.tmA, b.right_first ? b.Ub : b.Pb, m, r, b.rl, 128)) != TSR_OK) return s;
            if ((s = encode_map(ctx, &P.tmB, b.right_first ? b.Pb : b.Vb, n, r, b.rl, 128)) != TSR_OK) return s;
            if ((s = encode_map_w(ctx, &P.tmW, b.p.W, m, n, b.d.ldw, b.d.w_dtype)) != TSR_OK) return s;
            P.out = b.p.W; P.ld_out = b.d.ldw;
        }
        {   // Y = G X : A = G, B = X^T planes [2k x n]
            UmmaProblem &P = probs[KY][i];
            base(P, (int)m, (int)k, (int)n, EPI_STORE_F32);
            P.planes = 2; P.plane_rows = (int)k;
            if ((s = encode_map(ctx, &P.tmA, b.p.G, m, n, b.d.ldg, 128)) != TSR_OK) return s;
            if ((s = encode_map(ctx, &P.tmB, b.Xt, 2 * k, n, b.nl, ctx->bn[KY] / 2)) != TSR_OK) return s;
            P.out = b.buf[0]; P.ld_out = k;
        }
        {   // Z = G^T X : A = G itself, contracted over its rows (MN-major), B = X^T planes [2k x m]
            UmmaProblem &P = probs[KZ][i];
            base(P, (int)n, (int)k, (int)m, EPI_STORE_F32);
            P.planes = 2; P.plane_rows = (int)k;
            if ((s = encode_map(ctx, &P.tmA, b.p.G, m, n, b.d.ldg, 64)) != TSR_OK) return s;
            P.a_mn = 1;
            if ((s = encode_map(ctx, &P.tmB, b.Xt, 2 * k, m, b.ml, ctx->bn[KZ] / 2)) != TSR_OK) return s;
            P.out = b.buf[0]; P.ld_out = k;
        }
        for (int side = 0; side < 2; ++side) {   // exact integer Gram: the digit planes as a (6 k) x rows INT8 matrix
            UmmaProblem &P = probs[KG0 + side][i];
            const int64_t rows = side ? n : m;
            base(P, (int)k, (int)k, (int)rows, EPI_STORE_F32);
            if ((s = encode_map_i8(ctx, &P.tmA, b.planes, 6 * k, rows, b.ldp, 128)) != TSR_OK) return s;
            if ((s = encode_map_i8(ctx, &P.tmB, b.planes, 6 * k, rows, b.ldp, 32)) != TSR_OK) return s;
            P.out = b.gpart; P.ld_out = k; P.split_stride = k * k; P.col_exp = b.col_exp;
        }
        if (b.tc_rows) {   // rows [M x k] (planes Xs) times small matrix^T planes Bts [N x k]
            const int64_t mx = std::max(m, n);
            struct { int kd; int64_t M, N; float *out; } rk[5] = {
                {KR01, m, k, b.buf[1]}, {KR02, m, k, b.buf[2]}, {KR12, n, k, b.buf[2]}, {KRU, m, r, b.p.U}, {KRV, n, r, b.p.V}};
            for (const auto &e : rk) {
                UmmaProblem &P = probs[e.kd][i];
                base(P, (int)e.M, (int)e.N, (int)k, EPI_STORE_F32);
                P.planes = 3; P.plane_rows = (int)k; P.a_plane_rows = (int)mx;
                if ((s = encode_map_f32(ctx, &P.tmA, b.Xs, 2 * mx, k, k, 128)) != TSR_OK) return s;
                if ((s = encode_map_f32(ctx, &P.tmB, b.Bts, 2 * k, k, k, ctx->bn[e.kd] / 2)) != TSR_OK) return s;
                P.out = e.out; P.ld_out = e.N;
            }
        }
    }
    for (int kd = 0; kd < NKIND; ++kd) {
        TSR_CUDA(ctx, cudaMemcpy(ctx->d_probs[kd], probs[kd].data(), sizeof(UmmaProblem) * nb, cudaMemcpyHostToDevice));
        if (!ctx->tiles[kd].empty())
            TSR_CUDA(ctx, cudaMemcpy(ctx->d_tiles[kd], ctx->tiles[kd].data(), sizeof(UmmaTile) * ctx->tiles[kd].size(),
                                     cudaMemcpyHostToDevice));
    }
    TSR_CUDA(ctx, cudaMemcpy(ctx->d_cu_all, cu_all.data(), sizeof(CoreUpdateArgs) * nb, cudaMemcpyHostToDevice));
    TSR_CUDA(ctx, cudaMemcpy(ctx->d_cu_split, cu_split.data(), sizeof(CoreUpdateArgs) * nb, cudaMemcpyHostToDevice));
    TSR_CUDA(ctx, cudaMemcpy(ctx->d_refresh, rdev.data(), sizeof(RefreshDev) * nb, cudaMemcpyHostToDevice));
    TSR_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(int32_t) * nb));
    if (!ctx->aux_ready) {
        for (int g = 0; g < tsr_ctx::NGROUP; ++g) {
            TSR_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->aux[g], cudaStreamNonBlocking));
            TSR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_join[g], cudaEventDisableTiming));
        }
        TSR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming));
        for (int c = 0; c < tsr_ctx::NPIPE; ++c) {
            TSR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_pipe_in[c], cudaEventDisableTiming));
            TSR_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_pipe_done[c], cudaEventDisableTiming));
        }
        ctx->aux_ready = true;
    }
    ctx->bound = true;
    ctx->err.clear();
    return TSR_OK;
}

tsr_status tsr_bases_changed(tsr_ctx *ctx, const int32_t *idx, int32_t count, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    std::vector<int> list;
    if ((s = resolve_list(ctx, idx, count, list)) != TSR_OK) return s;
    return do_shadows(ctx, list, (cudaStream_t)stream);
}

static tsr_status refresh_listed(tsr_ctx *ctx, const int32_t *idx, int32_t count, uint64_t seed,
                                 const float *const *omegas, void *stream, bool reexpress);

// ---- grouped calls ------------------------------------------------------------------------
tsr_status tsr_init_subspace_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, uint64_t seed,
                                     const float *const *omegas, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    std::vector<int> list;
    if ((s = resolve_list(ctx, idx, count, list)) != TSR_OK) return s;
    if ((s = zero_moments(ctx, list, (cudaStream_t)stream)) != TSR_OK) return s;
    return refresh_listed(ctx, idx, count, seed, omegas, stream, false);   // moments are zero: nothing to re-express
}

static tsr_status refresh_listed(tsr_ctx *ctx, const int32_t *idx, int32_t count, uint64_t seed,
                                 const float *const *omegas, void *stream, bool reexpress)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    std::vector<int> list;
    if ((s = resolve_list(ctx, idx, count, list)) != TSR_OK) return s;
    // group by q, keeping each block's omega with it
    std::vector<int> qs;
    for (int bi : list) if (std::find(qs.begin(), qs.end(), (int)ctx->blocks[bi].d.q) == qs.end()) qs.push_back(ctx->blocks[bi].d.q);
    for (int q : qs) {
        std::vector<int> grp;
        std::vector<const float *> om;
        for (size_t j = 0; j < list.size(); ++j)
            if (ctx->blocks[list[j]].d.q == q) { grp.push_back(list[j]); om.push_back(omegas ? omegas[j] : nullptr); }
        if ((s = do_refresh(ctx, grp, seed, omegas ? om.data() : nullptr, (cudaStream_t)stream, reexpress)) != TSR_OK) return s;
    }
    return TSR_OK;
}

tsr_status tsr_rsvd_refresh_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, uint64_t seed,
                                    const float *const *omegas, void *stream)
{
    return refresh_listed(ctx, idx, count, seed, omegas, stream, true);
}

tsr_status tsr_project_core_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    std::vector<int> list;
    if ((s = resolve_list(ctx, idx, count, list)) != TSR_OK) return s;
    StepScalars sc = {};
    sc.wait_clocks = ctx->wait_clocks;
    return do_project(ctx, list, false, sc, (cudaStream_t)stream);
}

tsr_status tsr_adam_core_step_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, const tsr_hyper *hyper,
                                      void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    if ((s = check_hyper(ctx, hyper)) != TSR_OK) return s;
    std::vector<int> list;
    if ((s = resolve_list(ctx, idx, count, list)) != TSR_OK) return s;
    return do_core_update(ctx, list, make_scalars(ctx, hyper), (cudaStream_t)stream);
}

tsr_status tsr_backproject_apply_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, const tsr_hyper *hyper,
                                         void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    if ((s = check_hyper(ctx, hyper)) != TSR_OK) return s;
    std::vector<int> list;
    if ((s = resolve_list(ctx, idx, count, list)) != TSR_OK) return s;
    return do_apply(ctx, list, make_scalars(ctx, hyper), (cudaStream_t)stream);
}

tsr_status tsr_embed_step_grouped(tsr_ctx *ctx, const int32_t *idx, int32_t count, const tsr_hyper *hyper,
                                  uint64_t seed, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    if ((s = check_hyper(ctx, hyper)) != TSR_OK) return s;
    std::vector<int> list;
    if (!idx) {
        for (int i = 0; i < (int)ctx->blocks.size(); ++i) if (ctx->blocks[i].d.is_embedding) list.push_back(i);
    } else if ((s = resolve_list(ctx, idx, count, list)) != TSR_OK) {
        return s;
    }
    for (int bi : list)
        if (!ctx->blocks[bi].d.is_embedding) return fail(ctx, TSR_ERR_INVALID_ARG, "block %d is not an embedding", bi);
    return do_step(ctx, list, hyper, seed, true, (cudaStream_t)stream);
}

tsr_status tsr_step_grouped(tsr_ctx *ctx, const tsr_hyper *hyper, uint64_t seed, int32_t fuse_adam, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    if ((s = check_hyper(ctx, hyper)) != TSR_OK) return s;
    std::vector<int> list;
    resolve_list(ctx, nullptr, 0, list);
    return do_step(ctx, list, hyper, seed, fuse_adam != 0, (cudaStream_t)stream);
}

tsr_status tsr_step_grouped_host(tsr_ctx *ctx, const void *const *G_host, float *C_host, const tsr_hyper *hyper,
                                 uint64_t seed, int32_t fuse_adam, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    if (!G_host) return fail(ctx, TSR_ERR_INVALID_ARG, "G_host is NULL");
    if ((s = check_hyper(ctx, hyper)) != TSR_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    const int nb = (int)ctx->blocks.size();
    {
        std::vector<int> all;
        resolve_list(ctx, nullptr, 0, all);
        if ((s = check_rule_ptrs(ctx, all, hyper->rule)) != TSR_OK) return s;
    }
    bool refresh_due = false;
    for (int i = 0; i < nb; ++i) {
        const Block &b = ctx->blocks[i];
        if (!G_host[i]) return fail(ctx, TSR_ERR_INVALID_ARG, "G_host[%d] is NULL", i);
        if (b.d.K > 0 && hyper->step % b.d.K == 0) refresh_due = true;
    }
    auto copy_in = [&](int i, cudaStream_t cs) -> cudaError_t {
        const Block &b = ctx->blocks[i];
        const size_t es = (size_t)elem_size(b.d.g_dtype);
        return cudaMemcpy2DAsync(const_cast<void *>(b.p.G), (size_t)b.d.ldg * es, G_host[i], (size_t)b.d.n * es,
                                 (size_t)b.d.n * es, (size_t)b.d.m, cudaMemcpyHostToDevice, cs);
    };
    std::vector<size_t> c_off(nb, 0);
    {
        size_t off = 0;
        for (int i = 0; i < nb; ++i) { c_off[i] = off; off += (size_t)ctx->blocks[i].d.r * (size_t)ctx->blocks[i].cn; }
    }
    auto copy_out = [&](int i, cudaStream_t cs) -> cudaError_t {
        const Block &b = ctx->blocks[i];
        return cudaMemcpyAsync(C_host + c_off[i], b.p.C, (size_t)b.d.r * (size_t)b.cn * sizeof(float), cudaMemcpyDeviceToHost, cs);
    };
    constexpr int NCHUNK = tsr_ctx::NPIPE;
    if (refresh_due || !ctx->aux_ready || nb < 2 * NCHUNK) {
        // plain order: all gradients in, the step, all cores out
        cudaError_t e = cudaSuccess;
        for (int i = 0; i < nb && e == cudaSuccess; ++i) e = copy_in(i, st);
        s = (e == cudaSuccess) ? tsr_step_grouped(ctx, hyper, seed, fuse_adam, stream) : TSR_OK;
        if (C_host && s == TSR_OK)
            for (int i = 0; i < nb && e == cudaSuccess; ++i) e = copy_out(i, st);
        const cudaError_t es = cudaStreamSynchronize(st);   // also on failure: nothing stays in flight on the host buffers
        if (s != TSR_OK) return s;
        if (e != cudaSuccess || es != cudaSuccess)
            return fail(ctx, TSR_ERR_CUDA, "host-buffer step failed: %s", cudaGetErrorString(e != cudaSuccess ? e : es));
        return TSR_OK;
    }
    // Pipelined order (no refresh in this step): the blocks go in chunks of about equal gradient bytes;
    // while chunk c is stepped on the caller's stream, chunk c + 1 arrives on one side stream and the
    // cores of chunk c - 1 leave on another, so the step hides behind the host link.
    size_t total_bytes = 0;
    for (const Block &b : ctx->blocks) total_bytes += (size_t)b.d.m * b.d.n * elem_size(b.d.g_dtype);
    std::vector<std::vector<int>> chunks(NCHUNK);
    {
        size_t acc = 0;
        for (int bi : ctx->order) {
            const Block &b = ctx->blocks[bi];
            const int c = (int)std::min<size_t>(NCHUNK - 1, acc * NCHUNK / std::max<size_t>(1, total_bytes));
            chunks[c].push_back(bi);
            acc += (size_t)b.d.m * b.d.n * elem_size(b.d.g_dtype);
        }
    }
    cudaStream_t s_in = ctx->aux[0], s_out = ctx->aux[1];
    // After the fork every exit, the failing ones included, waits for the side streams and the
    // caller's stream: copies from G_host or into C_host must not be in flight when the call returns.
    tsr_status result = TSR_OK;
    auto cuda_ok = [&](cudaError_t e, const char *what) {
        if (e != cudaSuccess && result == TSR_OK) result = fail(ctx, TSR_ERR_CUDA, "%s failed: %s", what, cudaGetErrorString(e));
        return e == cudaSuccess;
    };
    bool go = cuda_ok(cudaEventRecord(ctx->ev_fork, st), "cudaEventRecord") &&
              cuda_ok(cudaStreamWaitEvent(s_in, ctx->ev_fork, 0), "cudaStreamWaitEvent") &&
              cuda_ok(cudaStreamWaitEvent(s_out, ctx->ev_fork, 0), "cudaStreamWaitEvent");
    for (int c = 0; c < NCHUNK && go; ++c) {
        for (int bi : chunks[c]) go = go && cuda_ok(copy_in(bi, s_in), "gradient copy");
        go = go && cuda_ok(cudaEventRecord(ctx->ev_pipe_in[c], s_in), "cudaEventRecord");
    }
    for (int c = 0; c < NCHUNK && go; ++c) {
        if (chunks[c].empty()) continue;
        go = cuda_ok(cudaStreamWaitEvent(st, ctx->ev_pipe_in[c], 0), "cudaStreamWaitEvent");
        if (!go) break;
        if ((s = do_step(ctx, chunks[c], hyper, seed, fuse_adam != 0, st)) != TSR_OK) {
            if (result == TSR_OK) result = s;
            break;
        }
        if (C_host) {
            go = cuda_ok(cudaEventRecord(ctx->ev_pipe_done[c], st), "cudaEventRecord") &&
                 cuda_ok(cudaStreamWaitEvent(s_out, ctx->ev_pipe_done[c], 0), "cudaStreamWaitEvent");
            for (int bi : chunks[c]) go = go && cuda_ok(copy_out(bi, s_out), "core copy");
        }
    }
    cuda_ok(cudaStreamSynchronize(s_in), "cudaStreamSynchronize");
    cuda_ok(cudaStreamSynchronize(s_out), "cudaStreamSynchronize");
    cuda_ok(cudaStreamSynchronize(st), "cudaStreamSynchronize");
    return result;
}

// ---- single-block calls ---------------------------------------------------------------------
tsr_status tsr_init_subspace(tsr_ctx *ctx, int32_t i, uint64_t seed, const float *omega, void *stream)
{
    const float *om[1] = {omega};
    return tsr_init_subspace_grouped(ctx, &i, 1, seed, omega ? om : nullptr, stream);
}
tsr_status tsr_rsvd_refresh(tsr_ctx *ctx, int32_t i, uint64_t seed, const float *omega, void *stream)
{
    const float *om[1] = {omega};
    return tsr_rsvd_refresh_grouped(ctx, &i, 1, seed, omega ? om : nullptr, stream);
}
tsr_status tsr_project_core(tsr_ctx *ctx, int32_t i, void *stream) { return tsr_project_core_grouped(ctx, &i, 1, stream); }
tsr_status tsr_adam_core_step(tsr_ctx *ctx, int32_t i, const tsr_hyper *hyper, void *stream)
{
    return tsr_adam_core_step_grouped(ctx, &i, 1, hyper, stream);
}
tsr_status tsr_backproject_apply(tsr_ctx *ctx, int32_t i, const tsr_hyper *hyper, void *stream)
{
    return tsr_backproject_apply_grouped(ctx, &i, 1, hyper, stream);
}
tsr_status tsr_embed_step(tsr_ctx *ctx, int32_t i, const tsr_hyper *hyper, uint64_t seed, void *stream)
{
    return tsr_embed_step_grouped(ctx, &i, 1, hyper, seed, stream);
}

// ---- reporting --------------------------------------------------------------------------------
tsr_status tsr_comm_bytes(const tsr_ctx *ctx, int64_t step, int32_t bytes_per_elem, uint64_t *core, uint64_t *sketch)
{
    if (!ctx || !core || !sketch || bytes_per_elem <= 0) return TSR_ERR_INVALID_ARG;
    uint64_t c = 0, sk = 0;
    for (const Block &b : ctx->blocks) {
        c += (uint64_t)b.d.r * (uint64_t)b.cn * (uint64_t)bytes_per_elem;
        const bool refresh = step <= 0 || (b.d.K > 0 && step % b.d.K == 0);
        if (refresh) sk += (uint64_t)b.k * (uint64_t)(b.d.m + b.d.n) * (uint64_t)bytes_per_elem;
    }
    *core = c;
    *sketch = sk;
    return TSR_OK;
}

tsr_status tsr_state_elems(const tsr_ctx *ctx, uint64_t *elems)
{
    if (!ctx || !elems) return TSR_ERR_INVALID_ARG;
    uint64_t e = 0;
    for (const Block &b : ctx->blocks)
        e += b.one_sided ? (uint64_t)b.d.m * b.d.r + 2ull * b.d.r * b.d.n : (uint64_t)(b.d.m + b.d.n) * b.d.r + 2ull * b.d.r * b.d.r;
    *elems = e;
    return TSR_OK;
}

tsr_status tsr_poll_status(tsr_ctx *ctx, int32_t *per_block_status, int32_t count, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    if (!per_block_status || count != (int32_t)ctx->blocks.size()) return fail(ctx, TSR_ERR_INVALID_ARG, "bad status array");
    cudaStream_t st = (cudaStream_t)stream;
    TSR_CUDA(ctx, cudaMemcpyAsync(per_block_status, ctx->d_status, sizeof(int32_t) * count, cudaMemcpyDeviceToHost, st));
    TSR_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(int32_t) * count, st));
    TSR_CUDA(ctx, cudaStreamSynchronize(st));
    return TSR_OK;
}

tsr_status tsr_generate_omega(tsr_ctx *ctx, int32_t i, uint64_t seed, float *out, void *stream)
{
    if (!ctx) return TSR_ERR_INVALID_ARG;
    if (i < 0 || i >= (int32_t)ctx->blocks.size() || !out) return fail(ctx, TSR_ERR_INVALID_ARG, "bad block index or NULL out");
    int dev_count = 0;
    if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count <= 0) return fail(ctx, TSR_ERR_CUDA, "no CUDA device available");
    const Block &b = ctx->blocks[i];
    TSR_KERNEL(ctx, 1, fill_gaussian(out, (int64_t)b.d.n * b.k, seed, (uint64_t)i, (cudaStream_t)stream));
    return TSR_OK;
}

tsr_status tsr_refresh_gram(tsr_ctx *ctx, int32_t block, int32_t side, const float *X, double *S, void *stream)
{
    tsr_status s = check_ready(ctx);
    if (s != TSR_OK) return s;
    if (block < 0 || block >= (int)ctx->blocks.size() || (side != 0 && side != 1) || !X || !S)
        return fail(ctx, TSR_ERR_INVALID_ARG, "tsr_refresh_gram: bad argument");
    cudaStream_t st = (cudaStream_t)stream;
    Block &b = ctx->blocks[block];
    const int rows = (int)(side ? b.d.n : b.d.m);
    // the device tables of the refresh are rewritten for this one block: a cached refresh is no longer valid
    ctx->refresh_sig.clear();
    RefreshLists L;
    L.list = {block};
    L.dlist = ctx->d_rlist;
    for (int i = 0; i < 5; ++i) L.ditems[i] = ctx->d_items[i];
    L.kmax = b.k; L.rmax = (int)b.d.r;
    std::vector<RowItem> items[4];
    for (int sd = 0; sd < 2; ++sd) {
        const int rr = (int)(sd ? b.d.n : b.d.m);
        for (int r0 = 0; r0 < rr; r0 += RG_ROWS) items[sd * 2].push_back({block, r0});
        for (int r0 = 0; r0 < rr; r0 += GRAM_ROWS) items[sd * 2 + 1].push_back({block, r0});
    }
    if ((s = upload_list(ctx, L.dlist, L.list, st)) != TSR_OK) return s;
    for (int i = 0; i < 4; ++i) {
        TSR_CUDA(ctx, cudaMemcpyAsync(L.ditems[i], items[i].data(), items[i].size() * sizeof(RowItem), cudaMemcpyHostToDevice, st));
        L.nitems[i] = (int)items[i].size();
    }
    TSR_CUDA(ctx, cudaMemcpyAsync(b.buf[0], X, (size_t)rows * b.k * sizeof(float), cudaMemcpyDeviceToDevice, st));
    if ((s = gram(ctx, L, side, 0, st)) != TSR_OK) return s;
    TSR_CUDA(ctx, cudaMemcpyAsync(S, b.S, (size_t)b.k * b.k * sizeof(double), cudaMemcpyDeviceToDevice, st));
    // the host vectors above feed asynchronous copies from pageable memory, which the runtime stages before it
    // returns, so they may go out of scope here
    return TSR_OK;
}

tsr_status tsr_set_limits(tsr_ctx *ctx, const tsr_limits *lim)
{
    if (!ctx) return TSR_ERR_INVALID_ARG;
    if (!lim) return fail(ctx, TSR_ERR_INVALID_ARG, "limits is NULL");
    const int nb = (int)ctx->blocks.size();
    if (lim->wait_clocks < 0 || lim->max_sweeps < 0 || lim->sweep_block < -1 || lim->sweep_block >= nb ||
        lim->starve_block < -1 || lim->starve_block >= nb || lim->projection_launches < 0 || lim->projection_launches > 2)
        return fail(ctx, TSR_ERR_INVALID_ARG, "limit out of range");
    if (lim->starve_block >= 0 && (lim->wait_clocks <= 0 || lim->wait_clocks > 100000000ll))
        return fail(ctx, TSR_ERR_INVALID_ARG, "starve_block needs a wait budget of at most 1e8 clock ticks");
    ctx->wait_clocks = lim->wait_clocks;
    for (int i = 0; i < nb; ++i)
        if (lim->sweep_block < 0 || lim->sweep_block == i) ctx->max_sweeps[i] = lim->max_sweeps;
    ctx->starve_block = lim->starve_block;
    ctx->proj_mode = lim->projection_launches;
    if (!ctx->bound) return TSR_OK;   // tsr_bind writes the device tables from these values
    // refresh the two fields inside the device tables (the device is idle with respect to this
    // context by contract: limits are set between calls, and the copies below are synchronous)
    for (int i = 0; i < nb; ++i) {
        TSR_CUDA(ctx, cudaMemcpy(&ctx->d_refresh[i].max_sweeps, &ctx->max_sweeps[i], sizeof(int32_t), cudaMemcpyHostToDevice));
        if (ctx->blocks[i].fast) {
            const int32_t sv = (ctx->starve_block == i) ? 1 : 0;
            TSR_CUDA(ctx, cudaMemcpy(&ctx->d_probs[KT][i].starve, &sv, sizeof(int32_t), cudaMemcpyHostToDevice));
        }
    }
    return TSR_OK;
}

tsr_status tsr_set_profiling(tsr_ctx *ctx, int32_t enable)
{
    if (!ctx) return TSR_ERR_INVALID_ARG;
    if (enable && !ctx->profiling) {
        for (cudaEvent_t &e : ctx->ev) TSR_CUDA(ctx, cudaEventCreate(&e));
        ctx->profiling = true;
        ctx->ev_valid = false;
    } else if (!enable && ctx->profiling) {
        for (cudaEvent_t &e : ctx->ev) { if (e) cudaEventDestroy(e); e = nullptr; }
        ctx->profiling = false;
        ctx->ev_valid = false;
    }
    return TSR_OK;
}

tsr_status tsr_get_stage_ms(tsr_ctx *ctx, float *ms, int32_t count)
{
    if (!ctx || !ms || count != TSR_NUM_STAGES) return TSR_ERR_INVALID_ARG;
    if (!ctx->profiling || !ctx->ev_valid) return fail(ctx, TSR_ERR_INVALID_ARG, "no profiled step recorded");
    TSR_CUDA(ctx, cudaEventSynchronize(ctx->ev[TSR_NUM_STAGES]));
    for (int i = 0; i < TSR_NUM_STAGES; ++i) TSR_CUDA(ctx, cudaEventElapsedTime(&ms[i], ctx->ev[i], ctx->ev[i + 1]));
    return TSR_OK;
}

tsr_status tsr_launch_count(const tsr_ctx *ctx, uint64_t *count)
{
    if (!ctx || !count) return TSR_ERR_INVALID_ARG;
    *count = ctx->launches;
    return TSR_OK;
}

int32_t tsr_block_uses_tensor_cores(const tsr_ctx *ctx, int32_t i)
{
    if (!ctx || i < 0 || i >= (int32_t)ctx->blocks.size()) return -1;
    return ctx->blocks[i].fast ? 1 : 0;
}

}  // extern "C"
