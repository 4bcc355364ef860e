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
#include "tsr_pdl.cuh"
#include <type_traits>

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
    static constexpr int SCHED_SLOTS = 4;                            // ring of tile indices (dynamic tile order)
    static constexpr int NBARS = 2 * STAGES + 4 + 2 * SCHED_SLOTS;
    static constexpr int TOTAL = BAR_OFFSET + NBARS * 8 + 64 + 1024;  // + slack for 1024-byte alignment
};

template <int BN, int EPI, int PLANES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(UG_THREADS, 1)
umma_gemm_kernel(const UmmaProblem *__restrict__ probs, const UmmaTile *__restrict__ tiles, int num_tiles,
                 StepScalars sc, int32_t *__restrict__ status, const UmmaProblem *__restrict__ probs2, int32_t *counters,
                 int fuse, int nslots)
{
    // counters (merged projection launch): [0, nslots) dependency counters, [nslots] the tile counter
    using SM = UmmaSmem<BN, PLANES>;
    constexpr int STAGES = SM::STAGES;
    constexpr uint32_t TMEM_COLS = 2 * BN;   // 256 or 512

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = (uint64_t *)(smem + SM::BAR_OFFSET);
    uint64_t *bar_full = bars, *bar_empty = bars + STAGES;
    uint64_t *bar_acc_full = bars + 2 * STAGES, *bar_acc_empty = bar_acc_full + 2;
    uint32_t *tmem_slot = (uint32_t *)(bars + SM::NBARS);
    __shared__ int s_timeout;   // 0, or 1 + the first tile (table index) this CTA gave up on (INT_MAX: a wait outside any tile)
    __shared__ int s_fetched, s_done[UG_EPI_WARPS];   // dynamic order: tiles this CTA's producer saw / each epilogue warp finished
    // Tile order.  Fixed instantiations: static round-robin, pair p takes tiles p, p + pairs, ...  The merged
    // projection launch (DYN): tiles are handed out in table order by a global counter, so a pair that draws short
    // tiles simply draws more of them, and a tile is never started before every earlier tile has been (which bounds
    // how long a core tile waits for the T~ tiles it depends on).  The leader's producer thread draws the index and
    // publishes it through a ring of SCHED_SLOTS slots (sched_tile, "full" barriers in both CTAs, one "empty" barrier
    // in the leader) to the other roles of the pair: the peer's producer, the MMA thread, the sixteen epilogue warps.
    constexpr bool DYN = (EPI == EPI_RUNTIME);
    constexpr int SR = SM::SCHED_SLOTS;
    uint64_t *bar_sfull = bar_acc_empty + 2, *bar_sempty = bar_sfull + SR;
    volatile int *sched_tile = (volatile int *)(tmem_slot + 1);     // [SR]

    pdl_trigger();   // the next kernel of the stream may set itself up on SMs this grid does not (or no longer) use
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long budget = wait_budget(sc);
    const uint32_t rank = cluster_ctarank();          // 0 = leader of the CTA pair
    const int pair = blockIdx.x >> 1;
    const int stride = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        s_timeout = 0;
        s_fetched = 0;
        for (int w = 0; w < UG_EPI_WARPS; ++w) s_done[w] = 0;
        for (int s = 0; s < SR; ++s) sched_tile[s] = -1;
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(bar_full + s), 1); mbar_init(smem_u32(bar_empty + s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(bar_acc_full + b), 1); mbar_init(smem_u32(bar_acc_empty + b), 2 * UG_EPI_WARPS); }
        // readers of a slot: MMA thread, B loader and 8 epilogue warps of the leader; both loaders and 8 epilogue warps of the peer
        for (int s = 0; s < SR; ++s) { mbar_init(smem_u32(bar_sfull + s), 1); mbar_init(smem_u32(bar_sempty + s), 2 * UG_EPI_WARPS + 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs allocates the pair's tensor memory
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();      // the peer's barriers are initialised before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The permit to allocate is given up only now, when BOTH CTAs of the pair hold their tensor memory (the
    // cluster barrier above): under cta_group::2 the permit belongs to the pair, and a CTA that relinquished it
    // while its peer had not yet allocated left the peer waiting in tcgen05.alloc for ever (seen when other
    // kernels on the same SMs delayed one of the two warps).
    if (warp == 1) asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    pdl_wait();      // set-up done; from here on the kernel reads what its predecessors wrote

    // i-th tile of this pair, for a reader of the ring (every role but the leader's producer): false when the wait ran
    // out; t < 0 when the table is exhausted.  `arrive`: this thread releases the slot (one lane per epilogue warp).
    // `whole_warp`: all 32 lanes call together (the epilogue warps); the slot is released only after every lane has read it.
    auto next_tile = [&](uint32_t i, int &t, bool arrive, bool whole_warp = false) -> bool {
        if (!DYN) {
            t = pair + (int)i * stride;
            if (t >= num_tiles) t = -1;
            return true;
        }
        const int s = (int)(i % SR);
        bool got = mbar_wait_cluster(smem_u32(bar_sfull + s), (i / SR) & 1u, budget);
        if (whole_warp) got = __all_sync(0xffffffffu, got);   // a warp gives up as a whole
        if (!got) return false;
        t = sched_tile[s];
        if (whole_warp) __syncwarp();
        if (arrive) mbar_arrive_leader(smem_u32(bar_sempty + s));
        return true;
    };

    if (warp == 0) {
        if (lane == 0) {
            int p_stage = 0;             // stage and phase of the operand ring this thread fills next
            uint32_t p_phase = 0;
            bool ok = true;
            for (uint32_t ti = 0; ok; ++ti) {
                int t;
                if (DYN && rank == 0) {
                    // draw the next tile of the table and publish it to both CTAs
                    const int s = (int)(ti % SR);
                    if (!mbar_wait(smem_u32(bar_sempty + s), ((ti / SR) & 1u) ^ 1u, budget)) { note_timeout(&s_timeout, 0x7ffffffe); break; }
                    t = atomicAdd(counters + nslots, 1);
                    if (t >= num_tiles) t = -1;
                    sched_tile[s] = t;
                    st_shared_peer(smem_u32((const void *)(sched_tile + s)), 1, t);
                    mbar_arrive_rank(smem_u32(bar_sfull + s), 0);
                    mbar_arrive_rank(smem_u32(bar_sfull + s), 1);
                } else if (!next_tile(ti, t, true)) { note_timeout(&s_timeout, 0x7ffffffe); break; }
                if (t < 0) break;
                if (DYN) s_fetched = (int)ti + 1;
                const UmmaTile tile = tiles[t];
                const UmmaProblem *P = ((EPI == EPI_RUNTIME && tile.kind) ? probs2 : probs) + tile.prob;
                if (EPI == EPI_RUNTIME && tile.kind && tile.wait_slot >= 0) {
                    // the tile's B operand is T~, written by earlier tiles of this launch (on other SMs): wait until all
                    // of them have published their stores, then order the TMA (async proxy) reads behind the acquire
                    if (!counter_wait(counters + tile.wait_slot, tile.wait_count, budget)) { note_timeout(&s_timeout, t); break; }
                    asm volatile("fence.proxy.async;" ::: "memory");
                }
                if (P->starve) {   // diagnostic: nothing is loaded for this tile, so every consumer's bounded wait runs out
                    note_timeout(&s_timeout, t);
                    break;
                }
                // Everything the K loop needs is fetched once per tile: the loop itself is on the critical path of the
                // pipeline (a stage is refilled the moment its MMAs retire), and every dependent global access in it --
                // a flag of the problem record, a plane offset -- showed up as lost operand bandwidth (a tenth of the
                // kernel's time for two flags read per K block).
                const bool a_mn = PLANES != 3 && P->a_mn;
                const int a_row = tile.m0 + (int)rank * UM_BM;
                const int a_plane_rows = P->a_plane_rows;
                const CUtensorMap *tmA = &P->tmA;
                auto k_loop = [&](auto mn_any) {
                    constexpr bool MN = decltype(mn_any)::value;   // false: both operands K-major, no branch in the loop
                    for (int kb = tile.kb0; kb < tile.kb1; ++kb) {
                        if (!mbar_wait(smem_u32(bar_empty + p_stage), p_phase ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                        // both CTAs' copies report their bytes to the leader's "full" barrier
                        const uint32_t full = leader_addr(smem_u32(bar_full + p_stage));
                        if (rank == 0) mbar_expect_tx(smem_u32(bar_full + p_stage), 2u * (uint32_t)SM::STAGE_BYTES);
                        const uint32_t st = smem_u32(smem + p_stage * SM::STAGE_BYTES);
                        const int kx = kb * SM::BK_ELEMS;
                        if (MN && a_mn) {
                            // A = a row-major [K x M] matrix: two boxes of 64 columns x 64 rows, this CTA's 128 columns
#pragma unroll
                            for (int j = 0; j < 2; ++j) tma_load_2d_pair(st + j * 8192, tmA, full, a_row + 64 * j, kx);
                        } else {
#pragma unroll
                            for (int pl = 0; pl < SM::A_PLANES; ++pl)
                                tma_load_2d_pair(st + pl * SM::A_BYTES, tmA, full, kx, a_row + pl * a_plane_rows);
                        }
                        if (++p_stage == STAGES) { p_stage = 0; p_phase ^= 1u; }
                    }
                };
                if (a_mn) k_loop(std::true_type{});
                else k_loop(std::false_type{});
            }
        }
    } else if (warp == 2) {
        // The B operand has a loader of its own: one thread issuing the copies of both operands was what bounded the K loop
        // (every instruction added to it showed up in the kernel's time), and the two threads issue side by side.  It
        // follows the tile sequence like the other readers of the ring and waits for the same "empty" barriers.
        if (lane == 0) {
            int p_stage = 0;
            uint32_t p_phase = 0;
            bool ok = true;
            for (uint32_t ti = 0; ok; ++ti) {
                int t;
                if (!next_tile(ti, t, true)) { note_timeout(&s_timeout, 0x7ffffffe); break; }
                if (t < 0) break;
                const UmmaTile tile = tiles[t];
                const UmmaProblem *P = ((EPI == EPI_RUNTIME && tile.kind) ? probs2 : probs) + tile.prob;
                if (EPI == EPI_RUNTIME && tile.kind && tile.wait_slot >= 0) {
                    if (!counter_wait(counters + tile.wait_slot, tile.wait_count, budget)) { note_timeout(&s_timeout, t); break; }
                    asm volatile("fence.proxy.async;" ::: "memory");
                }
                if (P->starve) { note_timeout(&s_timeout, t); break; }
                int n_eff = P->N - tile.n0;
                n_eff = tile.nw > 0 ? tile.nw : (n_eff >= BN ? BN : ((n_eff + 15) & ~15));
                const int b_row = tile.n0 + (int)rank * (n_eff / 2);   // this CTA's half of the B rows
                const bool b_mn = PLANES == 1 && P->b_mn;
                const int b_plane_rows = P->plane_rows;
                const CUtensorMap *tmB = &P->tmB;
                auto k_loop = [&](auto mn_any) {
                    constexpr bool MN = decltype(mn_any)::value;
                    for (int kb = tile.kb0; kb < tile.kb1; ++kb) {
                        if (!mbar_wait(smem_u32(bar_empty + p_stage), p_phase ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                        const uint32_t full = leader_addr(smem_u32(bar_full + p_stage));
                        const uint32_t st = smem_u32(smem + p_stage * SM::STAGE_BYTES) + SM::A_PLANES * SM::A_BYTES;
                        const int kx = kb * SM::BK_ELEMS;
                        if (MN) {
                            // B = a row-major [K x N] matrix: boxes of 64 columns x 64 rows, this CTA's half of the columns
#pragma unroll
                            for (int j = 0; j < BN / 128; ++j) tma_load_2d_pair(st + j * 8192, tmB, full, b_row + 64 * j, kx);
                        } else {
#pragma unroll
                            for (int pl = 0; pl < SM::B_PLANES; ++pl)
                                tma_load_2d_pair(st + pl * SM::B_BYTES, tmB, full, kx, b_row + pl * b_plane_rows);
                        }
                        if (++p_stage == STAGES) { p_stage = 0; p_phase ^= 1u; }
                    }
                };
                if (b_mn) k_loop(std::true_type{});
                else k_loop(std::false_type{});
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {   // the leader issues the pair's MMAs (256 x N x 16 each)
            uint32_t tc = 0;
            int c_stage = 0;             // stage and phase of the operand ring this thread consumes next
            uint32_t c_phase = 0;
            bool ok = true;
            for (; ok; ++tc) {
                int t;
                if (!next_tile(tc, t, true)) { note_timeout(&s_timeout, 0x7ffffffe); break; }
                if (t < 0) break;
                const UmmaTile tile = tiles[t];
                const UmmaProblem *Pm = ((EPI == EPI_RUNTIME && tile.kind) ? probs2 : probs) + tile.prob;
                int n_eff = Pm->N - tile.n0;
                n_eff = tile.nw > 0 ? tile.nw : (n_eff >= BN ? BN : ((n_eff + 15) & ~15));
                const bool b_mn = PLANES == 1 && Pm->b_mn, a_mn = PLANES != 3 && Pm->a_mn;
                // (the operand forms are fixed per tile: the MMA loop below only adds addresses)
                const uint64_t a_hi = a_mn ? UMMA_DESC_HI_MN : UMMA_DESC_HI_K, b_hi = b_mn ? UMMA_DESC_HI_MN : UMMA_DESC_HI_K;
                const uint32_t a_step = a_mn ? 2048u : 32u, b_step = b_mn ? 2048u : 32u;
                const uint32_t idesc = PLANES == 3 ? umma_idesc_pair_tf32(n_eff)
                                                   : (umma_idesc_pair(n_eff) | (b_mn ? UMMA_IDESC_B_MN_MAJOR : 0u) | (a_mn ? UMMA_IDESC_A_MN_MAJOR : 0u));
                const uint32_t buf = tc & 1u;
                if (!mbar_wait(smem_u32(bar_acc_empty + buf), ((tc >> 1) & 1u) ^ 1u, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = tile.kb0; kb < tile.kb1; ++kb) {
                    const int s = c_stage;
                    if (!mbar_wait(smem_u32(bar_full + s), c_phase, budget)) { note_timeout(&s_timeout, t); ok = false; break; }
                    if (++c_stage == STAGES) { c_stage = 0; c_phase ^= 1u; }
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
                                tc_mma_bf16_pair(d_tmem, umma_desc_at(a_hi, a_base + k4 * a_step), umma_desc_at(b_hi, b_base + k4 * b_step),
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
        for (; ok; ++tc) {
            int t;
            if (!next_tile(tc, t, lane == 0, true)) { note_timeout(&s_timeout, 0x7ffffffe); break; }
            if (t < 0) break;
            const UmmaTile tile = tiles[t];
            const UmmaProblem *__restrict__ P = ((EPI == EPI_RUNTIME && tile.kind) ? probs2 : probs) + tile.prob;
            // the tile's epilogue: fixed by the instantiation, or (merged projection launch) by the tile's kind
            // (a problem of the first contraction stores T~ transposed, or -- where it forms T = U^T G -- as it comes)
            const int epi = (EPI == EPI_STORE_BF16_T) ? P->epilogue
                            : (EPI != EPI_RUNTIME) ? EPI
                            : (tile.kind == 0 ? P->epilogue : (fuse ? P->epilogue : (int)EPI_STORE_F32));
            const uint32_t buf = tc & 1u;
            const int N = P->N, M = P->M;
            const int Nt = tile.nw > 0 ? min(N, tile.n0 + tile.nw) : N;   // first column past this tile
            const int row0 = tile.m0 + (int)rank * UM_BM + q * 32;   // this CTA holds rows 128 rank .. of the tile
            // a split-K problem inside a core-update launch only stores its slab
            const bool store_f32 = (epi == EPI_STORE_F32) || (epi == EPI_CORE_UPDATE && P->epilogue == EPI_STORE_F32);
            if (epi == EPI_CORE_UPDATE && !store_f32) {
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
            // (the warp gives up as a whole: the tensor-memory loads below need all 32 lanes)
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(bar_acc_full + buf), (tc >> 1) & 1u, budget))) { note_timeout(&s_timeout, t); ok = false; break; }
            tc_fence_after();
            const int nrows = min(32, M - row0);        // may be <= 0
            const int c_begin = half * (BN / 2), c_end = c_begin + BN / 2;
            if (tile.n0 + c_begin >= Nt) {   // this warp's column half lies outside the tile
                tc_fence_before();
                if (lane == 0) mbar_arrive_leader(smem_u32(bar_acc_empty + buf));
                if (EPI == EPI_RUNTIME && tile.signal_slot >= 0 && lane == 0) counter_signal(counters + tile.signal_slot);
                if (DYN && lane == 0) s_done[warp - 4] = (int)tc + 1;
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
                if (epi == EPI_STORE_BF16_T) {
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
                if (epi == EPI_STORE_BF16 && P->out_tma) {
                    if (ncols < 32 && Nt != N) {
                        // A box is always 32 columns wide and is clipped only at the matrix edge.  Where the tile ends before
                        // the matrix does, a box of its last, narrower chunk would also cover the first columns of the
                        // neighbouring tile (and race with that tile's own store): such a chunk is stored from the registers.
                        if (lane < nrows) {
                            bf16 *out = (bf16 *)P->out + (int64_t)(row0 + lane) * P->ld_out + col0;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < ncols) out[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
                        }
                        continue;
                    }
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
                if (epi == EPI_STORE_BF16 && ncols == 32 && (P->ld_out & 7) == 0 && (col0 & 7) == 0 &&
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
                if (full_chunk && epi == EPI_CORE_UPDATE && !store_f32) {
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
                } else if (epi == EPI_STORE_BF16) {
                    bf16 *out = (bf16 *)P->out + (int64_t)row0 * P->ld_out + col;
                    if (col_ok)
                        for (int i = 0; i < nrows; ++i) out[(int64_t)i * P->ld_out] = __float2bfloat16_rn(patch[i * 33 + lane]);
                } else if (epi == EPI_CORE_UPDATE && !store_f32) {
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
            if (EPI == EPI_RUNTIME && tile.signal_slot >= 0) {
                // this warp's part of the T~ tile is stored: publish it (every lane's stores, then one arrival)
                __threadfence();
                __syncwarp();
                if (lane == 0) counter_signal(counters + tile.signal_slot);
            }
            if (DYN && lane == 0) s_done[warp - 4] = (int)tc + 1;
        }
        // TMA stores read their boxes asynchronously: they must have done so before the CTA goes away
        if ((EPI == EPI_STORE_BF16 || EPI == EPI_RUNTIME) && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    if (s_timeout) __nanosleep(2000000);   // let copies in flight land before the CTA goes away
    tc_fence_before();
    __syncthreads();
    cluster_sync();      // neither CTA may leave while the peer still uses its shared or tensor memory
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    // Every block that owns a tile this CTA did not finish is flagged: with the static order, the tile it gave up
    // on and all its later ones; with the dynamic order (other pairs draw the remaining tiles), the tiles its
    // producer had drawn that not every epilogue warp has finished (they are still in the ring).
    if (threadIdx.x == 0 && s_timeout && status) {
        if (!DYN) {
            for (int t = s_timeout - 1; t < num_tiles; t += stride) atomicMax(status + probs[tiles[t].prob].block, (int)TSR_ERR_TIMEOUT);
        } else {
            if (s_timeout - 1 < num_tiles) atomicMax(status + probs[tiles[s_timeout - 1].prob].block, (int)TSR_ERR_TIMEOUT);
            int done = s_done[0];
            for (int w = 1; w < UG_EPI_WARPS; ++w) done = min(done, s_done[w]);
            for (int i = max(done, s_fetched - SR); i < s_fetched; ++i) {
                const int t = sched_tile[i % SR];
                if (t >= 0 && t < num_tiles) atomicMax(status + probs[tiles[t].prob].block, (int)TSR_ERR_TIMEOUT);
            }
        }
    }
}

template <int BN, int EPI, int PLANES>
static cudaError_t launch_one(const UmmaProblem *probs, const UmmaTile *tiles, int num_tiles, int num_sms,
                              const StepScalars &sc, int32_t *status, cudaStream_t stream)
{
    using SM = UmmaSmem<BN, PLANES>;
    const int pairs = num_tiles < num_sms / 2 ? num_tiles : num_sms / 2;
    return launch_dependent(umma_gemm_kernel<BN, EPI, PLANES>, dim3(2 * pairs), dim3(UG_THREADS), (size_t)SM::TOTAL, stream, 1, probs,
                            tiles, num_tiles, sc, status, (const UmmaProblem *)nullptr, (int32_t *)nullptr, 0, 0);
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
    if ((e = configure_one<128, EPI_RUNTIME, 1>()) != cudaSuccess) return e;
    if ((e = configure_one<256, EPI_RUNTIME, 1>()) != cudaSuccess) return e;
    return cudaSuccess;
}

// The merged projection launch.  Its core tiles wait on counters that other CTAs of the same grid advance, so
// every CTA has to be resident: the launch is cooperative (the driver refuses it, instead of letting it
// deadlock, when the grid does not fit), and the grid is one CTA pair per two SMs at most.
template <int BN>
static cudaError_t project_launch_one(const UmmaProblem *probs_t, const UmmaProblem *probs_c, const UmmaTile *tiles, int num_tiles,
                                      int num_sms, int fuse, int32_t *counters, const StepScalars &sc, int32_t *status,
                                      cudaStream_t stream, int nslots)
{
    using SM = UmmaSmem<BN, 1>;
    static int max_clusters = -1;      // clusters of this kernel the device holds at once (queried once)
    if (max_clusters < 0) {
        cudaLaunchConfig_t q = {};
        q.gridDim = dim3(num_sms & ~1, 1, 1);
        q.blockDim = dim3(UG_THREADS, 1, 1);
        q.dynamicSmemBytes = SM::TOTAL;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, (const void *)umma_gemm_kernel<BN, EPI_RUNTIME, 1>, &q) != cudaSuccess) n = 0;
        max_clusters = n;
    }
    int pairs = num_tiles < num_sms / 2 ? num_tiles : num_sms / 2;
    if (pairs > max_clusters) pairs = max_clusters;
    if (pairs <= 0) return cudaErrorNotSupported;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(UG_THREADS, 1, 1);
    cfg.dynamicSmemBytes = SM::TOTAL;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, umma_gemm_kernel<BN, EPI_RUNTIME, 1>, probs_t, tiles, num_tiles, sc, status, probs_c, counters,
                              fuse, nslots);
}

cudaError_t umma_project_launch(const UmmaProblem *probs_t, const UmmaProblem *probs_c, const UmmaTile *tiles, int num_tiles,
                                int num_sms, int bn, int fuse, int32_t *counters, const StepScalars &sc, int32_t *status,
                                cudaStream_t stream, int nslots)
{
    if (num_tiles <= 0) return cudaSuccess;
    if (bn == 256) return project_launch_one<256>(probs_t, probs_c, tiles, num_tiles, num_sms, fuse, counters, sc, status, stream, nslots);
    if (bn == 128) return project_launch_one<128>(probs_t, probs_c, tiles, num_tiles, num_sms, fuse, counters, sc, status, stream, nslots);
    return cudaErrorInvalidValue;
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
