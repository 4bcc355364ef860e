// Symmetric eigen-decomposition of the k x k Gram matrix S = B B^T of the refresh (Section 3.5:
// "compute a small SVD") for ranks too large for a shared-memory Jacobi solver.
//
// Batched over blocks, FP64 throughout:
//   1. Householder reduction to tridiagonal form T = Q^T S Q (one CTA per matrix; the
//      reflectors are kept in the rows of S above the first superdiagonal);
//   2. divide and conquer on T: it is torn in the middle, T = diag(T1', T2') + rho u u^T, and each
//      half runs an implicit-shift QL iteration on (d, e) alone, one thread per half, which LOGS
//      every plane rotation instead of applying it;
//   3. the merge: eigen-decomposition of D + rho z z^T (D = eigenvalues of the halves, z = Z^T u)
//      through the secular equation, one root per thread;
//   4. the eigenvectors W = Q diag(Z1, Z2) G Uhat: Q = I - V T V^T comes out of tiled products on the
//      FP64 tensor path (compact WY form of all reflectors at once); a second kernel streams every
//      row of Q through the two rotation logs as a systolic pipeline over the lanes of a warp (32
//      sweeps advance per step) and through the deflation rotations G (rows are independent under
//      right-multiplication); a last tiled product multiplies by the merged eigenvector matrix Uhat
//      and writes the leading r columns in descending eigenvalue order: Wu = W[:, :r],
//      Wv = W[:, :r] / sqrt(lambda).
// Failure to converge within the iteration or log budget flags TSR_ERR_NOT_CONVERGED.
#include "tsr_internal.h"

namespace tsr {

constexpr int TR_THREADS = 512;
constexpr int TR_NB = 8;          // columns per panel

// D (8 x 8, two entries per lane) += A (8 x 4) B (4 x 8) on the FP64 tensor path
__device__ __forceinline__ void dmma_f64(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c0), "+d"(c1)
                 : "d"(a), "d"(b));
}

// Tiled FP64 tensor-path products below: 64 x 64 tiles, operands staged 16 deep, 68 doubles per staged row
// (68 = 4 mod 16: the 64-bit fragment loads are conflict-free).
constexpr int MG_T = 64, MG_K = 16, MG_PITCH = 68;

// ---- stage 1: tridiagonalisation -----------------------------------------------------------
// Panels of TR_NB columns with the rank-2 updates deferred (the scheme of LAPACK's blocked
// reduction): inside a panel the trailing matrix T0 is left as it was at the start of the panel
// and the reflector pairs (v_i, w_i) found so far are kept in shared memory; the current matrix
// is T0 - sum_i (v_i w_i^T + w_i v_i^T).  A column step reads T0 once (the matrix-vector
// product); the trailing matrix is rewritten once per panel instead of once per column, which
// cuts the traffic per column from three passes to 1 + 2 / TR_NB.  The matrix is symmetric and
// stored in full; row j is used where the textbook takes column j.  Indices s, t below are
// relative to the first row / column j0 of the panel.
__global__ void __launch_bounds__(TR_THREADS)
tridiag_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int kpad)
{
    extern __shared__ double tr_smem[];          // vs, ps : 2 x kpad;  Vp, Wp : 2 x TR_NB x kpad
    double *vs = tr_smem, *ps = tr_smem + kpad;
    double *Vp = tr_smem + 2 * kpad, *Wp = Vp + TR_NB * kpad;
    __shared__ double red[32];
    __shared__ double dots[2 * TR_NB];           // dots[2 i] = w_i . v, dots[2 i + 1] = v_i . v
    const RefreshDev d = rd[list[blockIdx.x]];
    const int k = d.k;
    double *__restrict__ A = d.S;
    const int tid = threadIdx.x, nt = blockDim.x, warp = tid >> 5, lane = tid & 31, nwarps = nt >> 5;

    auto block_sum = [&](double x) -> double {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
        __syncthreads();
        if (lane == 0) red[warp] = x;
        __syncthreads();
        double t = (lane < nwarps) ? red[lane] : 0.0;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
        return t;   // every thread of every warp holds the total
    };

    for (int j0 = 0; j0 + 2 < k; j0 += TR_NB) {
        const int L0 = k - j0;
        const int nbc = min(TR_NB, k - 2 - j0);  // columns of this panel that get a reflector
        for (int c = 0; c < nbc; ++c) {
            const int j = j0 + c;
            const int len = k - j - 1;           // x = current row j, columns j+1 .. k-1  (t = c+1 .. L0-1)
            double *xrow = A + (int64_t)j * k + j + 1;
            double part = 0.0;
            for (int i = tid; i < len; i += nt) {
                double x = xrow[i];
                for (int u = 0; u < c; ++u)
                    x -= Vp[u * kpad + c] * Wp[u * kpad + c + 1 + i] + Wp[u * kpad + c] * Vp[u * kpad + c + 1 + i];
                vs[i] = x;
                part += x * x;
            }
            double dj = A[(int64_t)j * k + j];   // current diagonal entry (every thread computes it)
            for (int u = 0; u < c; ++u) dj -= 2.0 * Vp[u * kpad + c] * Wp[u * kpad + c];
            const double nrm2 = block_sum(part);
            const double x0 = vs[0];
            const double nrm = sqrt(nrm2);
            const double tail2 = nrm2 - x0 * x0;
            if (!(tail2 > 0.0) || nrm == 0.0) {  // nothing to annihilate: H_j = I
                if (tid == 0) { d.tau[j] = 0.0; d.dvec[j] = dj; d.evec[j] = x0; }
                for (int t = tid; t < L0; t += nt) { Vp[c * kpad + t] = 0.0; Wp[c * kpad + t] = 0.0; }
                __syncthreads();
                continue;
            }
            const double alpha = (x0 >= 0.0) ? -nrm : nrm;
            const double v0 = x0 - alpha;
            const double tau = -v0 / alpha;
            __syncthreads();
            for (int i = tid; i < len; i += nt) {
                const double v = (i == 0) ? 1.0 : vs[i] / v0;
                vs[i] = v;
                if (i > 0) xrow[i] = v;          // keep the reflector for stage 3
            }
            if (tid == 0) { d.tau[j] = tau; d.dvec[j] = dj; d.evec[j] = alpha; }
            __syncthreads();
            // ps = T0[c+1.., c+1..] v   (row-wise dot products; a warp takes four rows at a time and four
            // 32-column segments of each per trip, so that sixteen loads are in flight per lane; the four
            // sums are then reduced together: two exchange steps leave one sum per group of eight lanes)
            for (int a0 = 4 * warp; a0 < len; a0 += 4 * nwarps) {
                const double *row0 = A + (int64_t)(j + 1 + a0) * k + j + 1;
                const int na = min(4, len - a0);
                double acc[4] = {0.0, 0.0, 0.0, 0.0};
                for (int b0 = 0; b0 < len; b0 += 128) {
                    double x[4][4], vb[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int b = b0 + 32 * q + lane;
                        const bool ok = b < len;
                        vb[q] = ok ? vs[b] : 0.0;
#pragma unroll
                        for (int u = 0; u < 4; ++u) x[u][q] = (ok && u < na) ? row0[(int64_t)u * k + b] : 0.0;
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q)
#pragma unroll
                        for (int u = 0; u < 4; ++u) acc[u] += x[u][q] * vb[q];
                }
                // lanes with bit 4 set keep sums 2, 3, the others 0, 1; then bit 3 picks one of the two
                {
                    const bool hi4 = (lane & 16) != 0;
                    const double s0 = hi4 ? acc[0] : acc[2], s1 = hi4 ? acc[1] : acc[3];
                    const double k0 = hi4 ? acc[2] : acc[0], k1 = hi4 ? acc[3] : acc[1];
                    const double t0 = k0 + __shfl_xor_sync(0xffffffffu, s0, 16);
                    const double t1 = k1 + __shfl_xor_sync(0xffffffffu, s1, 16);
                    const bool hi3 = (lane & 8) != 0;
                    const double snd = hi3 ? t0 : t1, keep = hi3 ? t1 : t0;
                    double t = keep + __shfl_xor_sync(0xffffffffu, snd, 8);
#pragma unroll
                    for (int off = 4; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
                    // lanes 0..7 hold sum 0, 8..15 sum 1, 16..23 sum 2, 24..31 sum 3
                    const int u = lane >> 3;
                    if ((lane & 7) == 0 && u < na) ps[a0 + u] = t;
                }
            }
            // the earlier pairs of the panel against v: one warp per dot product
            if (warp < 2 * c) {
                const double *vec = ((warp & 1) ? Vp : Wp) + (warp >> 1) * kpad + c + 1;
                double acc = 0.0;
                for (int b = lane; b < len; b += 32) acc += vec[b] * vs[b];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (lane == 0) dots[warp] = acc;
            }
            __syncthreads();
            // p = tau (T0 v - sum_i (v_i (w_i . v) + w_i (v_i . v)))
            part = 0.0;
            for (int a = tid; a < len; a += nt) {
                double acc = ps[a];
                for (int u = 0; u < c; ++u)
                    acc -= Vp[u * kpad + c + 1 + a] * dots[2 * u] + Wp[u * kpad + c + 1 + a] * dots[2 * u + 1];
                acc *= tau;
                ps[a] = acc;
                part += acc * vs[a];
            }
            const double pv = block_sum(part);
            const double kk = 0.5 * tau * pv;
            for (int t = tid; t < L0; t += nt) {   // the new pair, zero where the reflector does not act
                const int a = t - c - 1;
                Vp[c * kpad + t] = (a >= 0) ? vs[a] : 0.0;
                Wp[c * kpad + t] = (a >= 0) ? ps[a] - kk * vs[a] : 0.0;
            }
            __syncthreads();
        }
        // T0[s][t] -= sum_i (v_i[s] w_i[t] + w_i[s] v_i[t]) for s, t >= nbc: a rank-16 update [V W] [W V]^T on
        // the FP64 tensor path (mma m8n8k4, four steps), 8 x 8 tiles, a row of tiles per warp, eight tiles
        // of T0 in flight per lane as 16-byte accesses and the next eight already requested: the update
        // is bound by the latency of those loads and by the cache lines a warp visits.
        if (nbc == TR_NB) {
            const int g = lane >> 2, q = lane & 3;
            const bool k_even = (k & 1) == 0;      // then L0 is even and every pair (t, t + 1), t even, is aligned
            const int ntile = (L0 - TR_NB + 7) >> 3;
            for (int si = warp; si < ntile; si += nwarps) {
                const int srow = TR_NB + si * 8 + g;
                const bool s_ok = srow < L0;
                const int sc = min(srow, L0 - 1);
                const double af[4] = {Vp[q * kpad + sc], Vp[(4 + q) * kpad + sc], Wp[q * kpad + sc], Wp[(4 + q) * kpad + sc]};
                double *trow = A + (int64_t)(j0 + sc) * k + j0;
                double cv[8][2], nv[8][2];
                auto cload = [&](int tj0, double (&v)[8][2]) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int t = TR_NB + (tj0 + u) * 8 + 2 * q;
                        if (k_even) {
                            const double2 x = (s_ok && t < L0) ? *(const double2 *)(trow + t) : make_double2(0.0, 0.0);
                            v[u][0] = x.x; v[u][1] = x.y;
                        } else {
                            v[u][0] = (s_ok && t < L0) ? trow[t] : 0.0;
                            v[u][1] = (s_ok && t + 1 < L0) ? trow[t + 1] : 0.0;
                        }
                    }
                };
                cload(0, cv);
                for (int tj0 = 0; tj0 < ntile; tj0 += 8) {
                    cload(tj0 + 8, nv);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (tj0 + u < ntile) {
                            const int tc = min(TR_NB + (tj0 + u) * 8 + g, L0 - 1);
                            double a0 = 0.0, a1 = 0.0, b0 = 0.0, b1 = 0.0;    // two chains of two products
                            dmma_f64(a0, a1, af[0], Wp[q * kpad + tc]);
                            dmma_f64(b0, b1, af[1], Wp[(4 + q) * kpad + tc]);
                            dmma_f64(a0, a1, af[2], Vp[q * kpad + tc]);
                            dmma_f64(b0, b1, af[3], Vp[(4 + q) * kpad + tc]);
                            const int t = TR_NB + (tj0 + u) * 8 + 2 * q;
                            if (k_even) {
                                if (s_ok && t < L0) *(double2 *)(trow + t) = make_double2(cv[u][0] - (a0 + b0), cv[u][1] - (a1 + b1));
                            } else {
                                if (s_ok && t < L0) trow[t] = cv[u][0] - (a0 + b0);
                                if (s_ok && t + 1 < L0) trow[t + 1] = cv[u][1] - (a1 + b1);
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) { cv[u][0] = nv[u][0]; cv[u][1] = nv[u][1]; }
                }
            }
        } else {
            // the last, narrower panel: a few entries, straight from shared memory
            for (int s1 = nbc + warp; s1 < L0; s1 += nwarps)
                for (int t = nbc + lane; t < L0; t += 32) {
                    double acc = 0.0;
                    for (int u = 0; u < nbc; ++u) acc += Vp[u * kpad + s1] * Wp[u * kpad + t] + Wp[u * kpad + s1] * Vp[u * kpad + t];
                    A[(int64_t)(j0 + s1) * k + j0 + t] -= acc;
                }
        }
        __syncthreads();
    }
    if (tid == 0) {
        if (k >= 2) {
            d.dvec[k - 2] = A[(int64_t)(k - 2) * k + (k - 2)];
            d.evec[k - 2] = A[(int64_t)(k - 2) * k + (k - 1)];
            d.tau[k - 2] = 0.0;
        }
        d.dvec[k - 1] = A[(int64_t)(k - 1) * k + (k - 1)];
        d.evec[k - 1] = 0.0;
        d.tau[k - 1] = 0.0;
    }
}

// ---- stage 2: implicit QL on the tridiagonal matrix, logging the rotations ------------------
// e[i] couples d[i] and d[i+1].  Sweep header: x = index of the first rotation (m - 1), y = count;
// rotation t of a sweep acts on columns (x - t, x - t + 1).
//
// The log is written in the layout the systolic eigenvector kernel reads.  Sweeps are taken in groups of 32 (sweep s is lane
// s % 32 of group s / 32).  A group streams the columns k-1, k-2, ..., lg of a row through the 32
// lanes, lane t two steps behind lane t-1, so lane t meets column j at step (k-1-j) + 2t; the
// rotation of sweep t on columns (j, j+1) is stored at rot[(base + (k-1-j) + 2t) * 32 + t], i.e. the
// 32 rotations a warp needs at one step are contiguous.  lg is the l of the group's first sweep
// (l never decreases).  groups[g] = (base row, E = k - lg + 1 stream elements); entries that no
// sweep writes are never used (the reader tests each lane's column against its sweep's range).
// Deflation threshold: an off-diagonal entry below QL_TOL (|d[m]| + |d[m+1]|) is set aside.  The
// eigenvectors leave this stage as FP32 numbers, and the rotations are orthogonal whatever the
// threshold, so a threshold of 1e-13 instead of the unit roundoff only perturbs the eigenvalues by
// 1e-13 ||T|| and saves the last, already converged, sweep of many eigenvalues.
constexpr double QL_TOL = 1e-13;
constexpr int SYS_LAG = 2;                        // steps between neighbouring lanes
constexpr int SYS_FILL = SYS_LAG * 31;            // steps until the last lane sees the first column
constexpr int SYS_PF = 8;                         // steps of rotations the reader fetches ahead

// 1 / sqrt(x) for a positive, normal x: hardware estimate (about 22 bits) and one third-order
// correction, which leaves an error of a few units of 2^-53; no special-case branches.
__device__ __forceinline__ double rsqrt_nocheck(double x)
{
    double y;
    asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
    const double e = fma(-x * y, y, 1.0);
    return fma(y * e, fma(0.375, e, 0.5), y);
}

// One QL problem: d[0..n), e[0..n) (e[n-1] is not used) in shared memory, run by one thread.
// Returns the number of sweeps logged, or -1 when a budget ran out.
__device__ int ql_run(double *d, double *e, int n, double2 *__restrict__ rot, int64_t rot_cap, int2 *__restrict__ sweeps,
                      int sweep_cap, int2 *__restrict__ groups, int iter_limit)
{
    int nrot = 0, nsw = 0;
    int64_t next_row = 0;                     // first free row of the skewed log
    double2 *lane_rot = rot;                  // rot + (base * 32 + t) + 32 * SYS_LAG * t
    for (int l = 0; l < n; ++l) {
        int iter = 0;
        while (true) {
            int m = l;
            for (; m < n - 1; ++m) {
                const double dd = fabs(d[m]) + fabs(d[m + 1]);
                if (fabs(e[m]) <= QL_TOL * dd) break;
            }
            if (m == l) break;
            if (++iter > iter_limit || nsw >= sweep_cap) return -1;
            {
                const int t = nsw & 31;
                if (t == 0) {                 // a new group starts with this sweep
                    const int E = n - l + 1;
                    if ((next_row + E + SYS_FILL + 2 * SYS_PF) * 32 > rot_cap) return -1;
                    groups[nsw >> 5] = make_int2((int)next_row, E);
                    next_row += E + SYS_FILL;
                }
                const int2 gr = groups[nsw >> 5];
                lane_rot = rot + ((int64_t)gr.x + SYS_LAG * t) * 32 + t;
            }
            double g = (d[l + 1] - d[l]) / (2.0 * e[l]);
            double r = sqrt(g * g + 1.0);
            g = d[m] - d[l] + e[l] / (g + (g >= 0.0 ? r : -r));
            double s = 1.0, c = 1.0, p = 0.0;
            const int first = nrot;
            int i = m - 1;
            bool early = false;
            // The loop is one dependent chain g -> r2 -> 1/sqrt(r2) -> g.  Everything that does not need
            // the reciprocal square root is formed before it: with rinv = 1/sqrt(f^2 + g^2),
            // s = f rinv, c = g rinv, (d[i] - g1) s + 2 c b = u rinv with u = (d[i] - g1) f + 2 g b,
            // so p = s (u rinv) = f u rinv^2 and the next g = c (u rinv) - b = g u rinv^2 - b.
            // d[i+1] and the next d[i], e[i] travel in registers (fetched ahead of the stores).
            double e_nx = e[i], d_nx = d[i], dprev = d[m];
            double2 *lr = lane_rot + (int64_t)(n - 1 - i) * 32;
            for (; i >= l; --i) {
                const double ei = e_nx, di = d_nx;
                if (i > l) { e_nx = e[i - 1]; d_nx = d[i - 1]; }
                const double f = s * ei, b = c * ei;
                // r = hypot(f, g).  The entries are bounded by the eigenvalues of a Gram matrix of FP32
                // data, so the squares stay far inside the FP64 range and no rescaling is needed.
                const double r2 = fma(f, f, g * g);
                if (r2 == 0.0) { e[i + 1] = 0.0; d[i + 1] = dprev - p; e[m] = 0.0; early = true; break; }
                const double g1 = dprev - p;
                const double u = fma(di - g1, f, 2.0 * g * b);
                const double gu = g * u, fu = f * u;
                const double rinv = rsqrt_nocheck(r2);
                const double rinv2 = rinv * rinv;
                const double gn = fma(gu, rinv2, -b);     // the chain continues here
                p = fu * rinv2;
                s = f * rinv;
                c = g * rinv;
                g = gn;
                e[i + 1] = r2 * rinv;
                d[i + 1] = g1 + p;
                *lr = make_double2(c, s);
                lr += 32;
                ++nrot;
                dprev = di;
            }
            if (nrot > first) sweeps[nsw++] = make_int2(m - 1, nrot - first);
            if (early) continue;
            d[l] -= p;
            e[l] = g;
            e[m] = 0.0;
        }
    }
    return nsw;
}

// dc = 0: one problem of size k, run by warp 0.  dc = 1 (divide and conquer, Cuppen): the matrix is
// torn at s = k / 2, T = diag(T1', T2') + rho u u^T with rho = e[s-1], u = e_{s-1} + e_s and the two
// diagonal entries next to the tear reduced by rho; warp h runs the QL iteration of half h with its
// own half of the log buffers, which takes a quarter of the serial chain of the whole problem.
// The merge is done by dc_secular_kernel.  nsweeps[h] = sweeps of half h.
__global__ void __launch_bounds__(64)
ql_log_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int dc)
{
    extern __shared__ double ql_smem[];           // d[n], e[n]
    const RefreshDev D = rd[list[blockIdx.x]];
    const int n = D.k;
    double *d = ql_smem, *e = ql_smem + n;
    for (int i = threadIdx.x; i < n; i += 64) { d[i] = D.dvec[i]; e[i] = D.evec[i]; }
    __syncthreads();
    const int s = dc ? n / 2 : n;
    if (dc && threadIdx.x == 0) {
        const double rho = e[s - 1];
        D.dc_scal[0] = rho;
        d[s - 1] -= rho;
        d[s] -= rho;
        e[s - 1] = 0.0;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0 && (warp == 0 || dc)) {
        const int off = warp ? s : 0, nh = warp ? n - s : s;
        const int64_t rcap = dc ? (int64_t)(D.rot_cap / 64) * 32 : (int64_t)D.rot_cap;   // entries per half
        const int scap = dc ? D.sweep_cap / 2 : D.sweep_cap;
        const int gcap = D.sweep_cap / 64 + 2;                                           // group slots per half
        const int nsw = ql_run(d + off, e + off, nh, D.rot + (warp ? rcap : 0), rcap, D.sweeps + (warp ? scap : 0), scap,
                               D.groups + (warp ? gcap : 0), D.max_sweeps > 0 ? D.max_sweeps : 60);
        D.nsweeps[warp] = nsw < 0 ? 0 : nsw;
        if (!dc) D.nsweeps[1] = 0;
        if (nsw < 0) atomicMax(D.status, (int)TSR_ERR_NOT_CONVERGED);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += 64) D.dvec[i] = d[i];
}

// Bit 30 of rank[c] marks a coordinate that takes part in the secular problem (dc only): its column of the
// eigenvector matrix comes out of the merge product, the other columns are final after the rotations.
constexpr int RANK_MERGED = 1 << 30;

__global__ void eig_rank_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int dc)
{
    const RefreshDev D = rd[list[blockIdx.x]];
    const int k = D.k, r = D.r;
    int flag = 0;
    for (int j = threadIdx.x; j < k; j += blockDim.x) {
        const double lj = D.dvec[j];
        if (!(lj == lj)) flag = TSR_ERR_NONFINITE;
        int rank = 0;
        for (int l = 0; l < k; ++l) {
            const double ll = D.dvec[l];
            rank += (ll > lj || (ll == lj && l < j)) ? 1 : 0;
        }
        D.rank[j] = rank;
        D.lam[rank] = lj;
        if (rank < r && !(lj > 1e-300) && flag == 0) flag = TSR_ERR_RANK_DEFICIENT;
    }
    if (flag) atomicMax(D.status, flag);
    if (dc) {
        __syncthreads();
        const int K = D.dc_info[0];
        for (int j = threadIdx.x; j < K; j += blockDim.x) D.rank[D.dc_nd[j]] |= RANK_MERGED;
    }
}

// ---- stage 3: the eigenvectors (k <= SYS_KMAX) -------------------------------------------------
constexpr int SYS_KMAX = 1056;
constexpr int DC_MIN_K = 200;    // the tridiagonal problem is torn in two from this size on
constexpr int SYS_WARPS = 12;    // warps of the rotation kernel (three per scheduler)

// 3a: Q = H_0 H_1 ... H_{k-3} = I - V T V^T with V = (v_0 .. v_{k-3}) and T upper
// triangular (the compact WY representation of all reflectors at once), every step a tiled product on the FP64
// tensor path (mma m8n8k4; 64 x 64 tiles, eight warps of 32 x 16, operands staged 16 deep):
//   G  = V^T V (above the diagonal)                                      -> Xw
//   T  : 64 x 64 diagonal blocks by the column recurrence T[0:i, i] = -tau_i T[0:i, 0:i] G[0:i, i], then
//        blocks of 64, 128, 256 ... merged pairwise, T_AB = -T_A (G_AB T_B)  -> gpart (X = G_AB T_B in Wj)
//   M  = T V^T                                                             -> Xw (G is no longer needed)
//   Q  = I - V M                                                           -> Wj
// v_j = (0 .. 0, 1 at j + 1, S[j][j + 2 ..]); a reflector with tau_j = 0 has a zero row and column in T and
// drops out whatever its row of S holds.  About 2.5 k^3 multiply-adds instead of k^3, but as products that
// run near the rate of the tensor path instead of dependent reduce-and-update rounds.
enum WyMode : int { WY_G = 0, WY_X, WY_T12, WY_M, WY_Q, WY_W };
constexpr int WY_NB = 64;      // base block of T

__device__ __forceinline__ double wy_vt(const double *__restrict__ S, int k, int nr, int j, int c)
{
    // V^T[j][c]: entry c of reflector j
    if (j >= nr || c <= j || c >= k) return 0.0;
    return (c == j + 1) ? 1.0 : S[(int64_t)j * k + c];
}

template <int MODE>
__global__ void __launch_bounds__(256)
eig_wy_gemm_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int s)
{
    const RefreshDev D = rd[list[blockIdx.z]];
    const int k = D.k, nr = k - 2;
    const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
    const double *__restrict__ S = D.S;
    double *__restrict__ G = D.Xw;       // G, later M
    double *__restrict__ T = D.gpart;
    double *__restrict__ X = D.Wj;       // X during the merges, Q at the end
    // extent of this tile's product: rows < Mr, columns < Nc, contraction index in [kb, ke)
    int Mr, Nc, kb, ke;
    if (MODE == WY_G) {                  // G[a][b] = sum_c V^T[a][c] V^T[b][c], tiles on or above the diagonal
        if (c0 < r0) return;
        Mr = nr; Nc = nr; kb = c0 & ~15; ke = k;      // v_b is zero up to column b >= c0
    } else if (MODE == WY_X || MODE == WY_T12) {
        // pair of blocks A = [pa, pa + s), B = [pa + s, pa + 2 s): the tile must lie in rows A, columns B
        const int pa = (r0 / (2 * s)) * (2 * s), pb = pa + s;
        if (r0 >= pb || c0 < pb || c0 >= pb + s) return;
        Mr = min(pb, nr); Nc = min(pb + s, nr);
        if (MODE == WY_X) { kb = pb; ke = min(c0 + 64, Nc); }        // X[a][j] = sum_{l in B, l <= j} G[a][l] T[l][j]
        else { kb = r0; ke = Mr; }                                    // T[a][j] = -sum_{l in A, l >= a} T[a][l] X[l][j]
    } else if (MODE == WY_M) {           // M[i][c] = sum_{l >= i} T[i][l] V^T[l][c]; V^T[l][c] = 0 for l >= c
        Mr = nr; Nc = k; kb = r0; ke = min(nr, c0 + 64);
    } else if (MODE == WY_Q) {           // Q[c][c'] = delta - sum_j V^T[j][c] M[j][c'], j < c
        Mr = k; Nc = k; kb = 0; ke = min(nr, r0 + 64);
    } else {                             // W = Q Ztot (Q in Wj, Ztot in gpart): the eigenvectors of S
        Mr = k; Nc = k; kb = 0; ke = k;
    }
    if (r0 >= Mr || c0 >= Nc) return;
    __shared__ __align__(16) double As[MG_K][MG_PITCH];     // As[kk][row]
    __shared__ __align__(16) double Bs[MG_K][MG_PITCH];     // Bs[kk][col]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wi = warp >> 2, wj = warp & 3;
    const int g = lane >> 2, q = lane & 3;
    double acc[4][2][2];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
    // element maps: the index that is contiguous in memory goes to consecutive threads
    constexpr bool A_KFAST = (MODE != WY_Q);                 // A(i, kk) contiguous in kk, except V (= V^T transposed)
    const int r_out = D.r;
    constexpr bool B_KFAST = (MODE == WY_G);                 // B(kk, j) contiguous in j, except V^T[b][c] over c
    double ra[4], rb[4];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = tid + l * 256;
            {
                const int row = r0 + (A_KFAST ? (e >> 4) : (e & 63)), kk = k0 + (A_KFAST ? (e & 15) : (e >> 6));
                double v = 0.0;
                if (row < Mr && kk < ke) {
                    if (MODE == WY_G) v = wy_vt(S, k, nr, row, kk);
                    else if (MODE == WY_X) v = G[(int64_t)row * k + kk];
                    else if (MODE == WY_T12 || MODE == WY_M) v = (kk >= row) ? T[(int64_t)row * k + kk] : 0.0;
                    else if (MODE == WY_Q) v = wy_vt(S, k, nr, kk, row);
                    else v = X[(int64_t)row * k + kk];
                }
                ra[l] = v;
            }
            {
                const int col = c0 + (B_KFAST ? (e >> 4) : (e & 63)), kk = k0 + (B_KFAST ? (e & 15) : (e >> 6));
                double v = 0.0;
                if (col < Nc && kk < ke) {
                    if (MODE == WY_G) v = wy_vt(S, k, nr, col, kk);
                    else if (MODE == WY_X) v = (kk <= col) ? T[(int64_t)kk * k + col] : 0.0;
                    else if (MODE == WY_T12) v = X[(int64_t)kk * k + col];
                    else if (MODE == WY_M) v = wy_vt(S, k, nr, kk, col);
                    else if (MODE == WY_Q) v = G[(int64_t)kk * k + col];
                    else v = T[(int64_t)kk * k + col];
                }
                rb[l] = v;
            }
        }
    };
    kb &= ~15;
    if (kb < ke) fetch(kb);
    for (int k0 = kb; k0 < ke; k0 += MG_K) {
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = tid + l * 256;
            if (A_KFAST) As[e & 15][e >> 4] = ra[l]; else As[e >> 6][e & 63] = ra[l];
            if (B_KFAST) Bs[e & 15][e >> 4] = rb[l]; else Bs[e >> 6][e & 63] = rb[l];
        }
        __syncthreads();
        if (k0 + MG_K < ke) fetch(k0 + MG_K);
#pragma unroll
        for (int st = 0; st < MG_K / 4; ++st) {
            double af[4], bf[2];
#pragma unroll
            for (int a = 0; a < 4; ++a) af[a] = As[st * 4 + q][wi * 32 + a * 8 + g];
#pragma unroll
            for (int b = 0; b < 2; ++b) bf[b] = Bs[st * 4 + q][wj * 16 + b * 8 + g];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 2; ++b) dmma_f64(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int row = r0 + wi * 32 + a * 8 + g, col = c0 + wj * 16 + b * 8 + 2 * q + h;
                if (row >= Mr || col >= Nc) continue;
                const double v = acc[a][b][h];
                if (MODE == WY_G) G[(int64_t)row * k + col] = v;
                else if (MODE == WY_X) X[(int64_t)row * k + col] = v;
                else if (MODE == WY_T12) T[(int64_t)row * k + col] = -v;
                else if (MODE == WY_M) G[(int64_t)row * k + col] = v;
                else if (MODE == WY_Q) X[(int64_t)row * k + col] = ((row == col) ? 1.0 : 0.0) - v;
                else {
                    // the leading r columns in descending eigenvalue order: Wu = W[:, :r], Wv = W[:, :r] / sqrt(lambda)
                    const int rk = D.rank[col] & (RANK_MERGED - 1);
                    if (rk < r_out) {
                        const double lj = D.dvec[col];
                        const double inv = (lj > 1e-300) ? 1.0 / sqrt(lj) : 0.0;
                        D.Wu[(int64_t)row * r_out + rk] = (float)v;
                        D.Wv[(int64_t)row * r_out + rk] = (float)(v * inv);
                    }
                }
            }
}

// The 64 x 64 diagonal blocks of T: thread rr owns row rr of a block (T[rr][i] needs T[rr][rr .. i-1] only),
// with the block of G and the rows of T in shared memory.
__global__ void __launch_bounds__(WY_NB)
eig_wy_base_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list)
{
    extern __shared__ double wb_smem[];        // Gs[64][65], Ts[64][65]
    double *Gs = wb_smem, *Ts = wb_smem + WY_NB * (WY_NB + 1);
    const RefreshDev D = rd[list[blockIdx.y]];
    const int k = D.k, nr = k - 2, b0 = blockIdx.x * WY_NB;
    if (b0 >= nr) return;
    const double *__restrict__ G = D.Xw;
    double *__restrict__ T = D.gpart;
    const int rr = threadIdx.x;
    const int nb = min(WY_NB, nr - b0);
    __shared__ double taus[WY_NB];
    taus[rr] = (rr < nb) ? D.tau[b0 + rr] : 0.0;
    for (int l = 0; l < nb; ++l) Gs[l * (WY_NB + 1) + rr] = (rr < nb) ? G[(int64_t)(b0 + l) * k + b0 + rr] : 0.0;
    __syncthreads();
    if (rr >= nb) return;
    double *trow = Ts + rr * (WY_NB + 1);
    for (int i = rr; i < nb; ++i) {
        double v;
        if (i == rr) v = taus[i];
        else {
            double sacc = 0.0;
            for (int l = rr; l < i; ++l) sacc += trow[l] * Gs[l * (WY_NB + 1) + i];
            v = -taus[i] * sacc;
        }
        trow[i] = v;
        T[(int64_t)(b0 + rr) * k + b0 + i] = v;
    }
}

// 3b: the logged rotations as a systolic pipeline.  A warp owns R rows of Q in shared memory.
// Per group of 32 sweeps the columns kh-1 ... lg of each row enter at lane 0, one per step; lane t
// applies its sweep's rotation to the incoming column and the value it holds, passes the finished
// column on to lane t+1 (one shuffle) and keeps the other; lane 31 writes the finished columns
// back.  All 32 sweeps of a group advance in every step and the R rows are independent chains.
// z: the warp's rows (row stride zs), already offset to the first of the kh columns the log acts on.
template <int R>
__device__ __forceinline__ void systolic_apply(double *z, int zs, int kh, const double2 *__restrict__ rot,
                                               const int2 *__restrict__ groups, const int2 *__restrict__ sweeps, int nsw,
                                               int lane)
{
    const int ngroups = (nsw + 31) >> 5;
    for (int g = 0; g < ngroups; ++g) {
        const int2 gr = groups[g];
        const int E = gr.y, T = E + SYS_FILL;
        const int sidx = 32 * g + lane;
        int hi = -1, lo = 0;                      // this lane's sweep acts on columns lo .. hi
        if (sidx < nsw) { const int2 sw = sweeps[sidx]; hi = sw.x; lo = sw.x - sw.y + 1; }
        const double2 *__restrict__ rp = rot + (int64_t)gr.x * 32 + lane;
        double held[R], out[R];
#pragma unroll
        for (int q = 0; q < R; ++q) { held[q] = 0.0; out[q] = 0.0; }
        int j = kh - 1 + SYS_LAG * lane;          // column this lane consumes at step tau
        // the rotations of the next SYS_PF steps are fetched while the current ones are applied
        double2 nxt[SYS_PF];
#pragma unroll
        for (int u = 0; u < SYS_PF; ++u) nxt[u] = __ldg(rp + (int64_t)u * 32);
        for (int tau0 = 0; tau0 < T; tau0 += SYS_PF) {
            double2 cur[SYS_PF];
#pragma unroll
            for (int u = 0; u < SYS_PF; ++u) cur[u] = nxt[u];
#pragma unroll
            for (int u = 0; u < SYS_PF; ++u) nxt[u] = __ldg(rp + (int64_t)(tau0 + SYS_PF + u) * 32);
#pragma unroll
            for (int u = 0; u < SYS_PF; ++u, --j) {
                const int tau = tau0 + u;
                if (tau >= T) break;
                const bool act = (j <= hi) && (j >= lo);
                const double c = act ? cur[u].x : 1.0, s = act ? cur[u].y : 0.0;
                const int cin = max(kh - 1 - tau, 0);     // column entering lane 0 (all lanes read it: a broadcast)
                const int cout = kh - (tau - SYS_FILL);   // column leaving lane 31
                const bool feed = (lane == 0), real = (tau < E - 1);
                const bool emit = (lane == 31) && (tau > SYS_FILL);
                double zin[R];
#pragma unroll
                for (int q = 0; q < R; ++q) zin[q] = z[q * zs + cin];
#pragma unroll
                for (int q = 0; q < R; ++q) {
                    const double up = __shfl_up_sync(0xffffffffu, out[q], 1);
                    const double in = feed ? (real ? zin[q] : 0.0) : up;
                    const double ch = c * held[q], sh = s * held[q];
                    const double o = fma(s, in, ch);
                    held[q] = fma(c, in, -sh);
                    out[q] = o;
                    if (emit) z[q * zs + cout] = o;
                }
            }
        }
        __syncwarp();
    }
}

// Offsets of half 1's share of the log buffers (see ql_log_kernel).
__device__ __forceinline__ int64_t dc_rot_off(const RefreshDev &D) { return (int64_t)(D.rot_cap / 64) * 32; }
__device__ __forceinline__ int dc_sweep_off(const RefreshDev &D) { return D.sweep_cap / 2; }
__device__ __forceinline__ int dc_group_off(const RefreshDev &D) { return D.sweep_cap / 64 + 2; }

// Divide and conquer, step 2: z = Z^T u = (last row of Z1, first row of Z2), i.e. the logs of the
// two halves applied to one unit row vector each (warp h = half h).
__global__ void __launch_bounds__(64)
dc_zrows_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list)
{
    extern __shared__ double zr_smem[];          // k
    const RefreshDev D = rd[list[blockIdx.x]];
    const int k = D.k, s = k / 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int off = warp ? s : 0, kh = warp ? k - s : s;
    double *z = zr_smem + off;
    const int one = warp ? 0 : s - 1;            // e_{s-1} of half 0, e_0 of half 1
    for (int c = lane; c < kh; c += 32) z[c] = (c == one) ? 1.0 : 0.0;
    __syncwarp();
    systolic_apply<1>(z, k, kh, D.rot + (warp ? dc_rot_off(D) : 0), D.groups + (warp ? dc_group_off(D) : 0),
                      D.sweeps + (warp ? dc_sweep_off(D) : 0), D.nsweeps[warp], lane);
    for (int c = lane; c < kh; c += 32) D.dc_z[off + c] = z[c];
}

// Divide and conquer, step 3: eigen-decomposition of D + rho z z^T (D = eigenvalues of the halves),
// one CTA per matrix.  Sort, deflate (negligible z_i; nearly equal d_i, by a plane rotation), solve the
// secular equation 1 + rho sum_i z_i^2 / (d_i - lambda) = 0 for one root per thread by bisection on
// the distance tau from the nearer pole (so that all differences d_i - lambda keep full relative
// accuracy), recompute z from the roots (Gu and Eisenstat's formula, which makes the eigenvectors
// orthogonal to working precision however close the roots are), and write the eigenvector matrix
// Uhat (K x K, row pitch k, in Xw), the coordinate list nd, the deflation rotations and the
// eigenvalues of all k coordinates (dvec).
constexpr int DC_THREADS = 1024;

__global__ void __launch_bounds__(DC_THREADS)
dc_secular_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list, int kpad)
{
    extern __shared__ double sc_smem[];          // ds, zs, dk, zk, tk, zh : 6 x kpad doubles; perm, org, state : 3 x kpad ints
    const RefreshDev D = rd[list[blockIdx.x]];
    const int n = D.k;
    double *ds = sc_smem, *zs = ds + kpad, *dk = zs + kpad, *zk = dk + kpad, *tk = zk + kpad, *zh = tk + kpad;
    int *perm = (int *)(zh + kpad), *org = perm + kpad, *state = org + kpad;
    __shared__ int s_K, s_nr;
    __shared__ double s_rho, s_flip;
    const int tid = threadIdx.x, nt = blockDim.x;
    double rho = D.dc_scal[0];
    const double flip = (rho < 0.0) ? -1.0 : 1.0;   // solve for -T when rho < 0
    rho = fabs(rho) * 2.0;                       // ||u||^2 = 2: z is normalised below
    // sort ascending (rank sort); dk / zk serve as staging for the unsorted values
    for (int i = tid; i < n; i += nt) { dk[i] = flip * D.dvec[i]; zk[i] = D.dc_z[i] * 0.70710678118654752440; }
    __syncthreads();
    for (int i = tid; i < n; i += nt) {
        const double di = dk[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (dk[j] < di || (dk[j] == di && j < i)) ? 1 : 0;
        ds[rank] = di; zs[rank] = zk[i]; perm[rank] = i;
    }
    __syncthreads();
    if (tid == 0) {
        double dmax = 0.0, zmax = 0.0;
        for (int p = 0; p < n; ++p) { dmax = fmax(dmax, fabs(ds[p])); zmax = fmax(zmax, fabs(zs[p])); }
        const double tol = 8.0 * 2.220446049250313e-16 * fmax(dmax, zmax);
        int K = 0, nr = 0, prev = -1;
        if (!(rho * zmax > tol)) {               // the halves do not interact at working precision
            for (int p = 0; p < n; ++p) state[p] = 0;
        } else {
            for (int p = 0; p < n; ++p) {
                if (rho * fabs(zs[p]) <= tol) { state[p] = 0; continue; }
                if (prev < 0) { prev = p; continue; }
                double sN = zs[prev], cN = zs[p];
                const double tauN = sqrt(cN * cN + sN * sN);
                const double t = ds[p] - ds[prev];
                cN /= tauN; sN = -sN / tauN;
                if (fabs(t * cN * sN) <= tol) {  // rotate z[prev] into z[p]: prev deflates
                    zs[p] = tauN; zs[prev] = 0.0;
                    D.dc_rot_idx[nr] = make_int2(perm[prev], perm[p]);
                    D.dc_rot_cs[nr] = make_double2(cN, sN);
                    ++nr;
                    const double tt = ds[prev] * cN * cN + ds[p] * sN * sN;
                    ds[p] = ds[prev] * sN * sN + ds[p] * cN * cN;
                    ds[prev] = tt;
                    state[prev] = 0;
                } else {
                    state[prev] = 1; dk[K] = ds[prev]; zk[K] = zs[prev]; D.dc_nd[K] = perm[prev]; ++K;
                }
                prev = p;
            }
            if (prev >= 0) { state[prev] = 1; dk[K] = ds[prev]; zk[K] = zs[prev]; D.dc_nd[K] = perm[prev]; ++K; }
        }
        // dk is ascending except where a rotation moved a value: restore the order (insertion, rarely needed)
        for (int a = 1; a < K; ++a) {
            int bq = a;
            while (bq > 0 && dk[bq - 1] > dk[bq]) {
                const double td = dk[bq]; dk[bq] = dk[bq - 1]; dk[bq - 1] = td;
                const double tz = zk[bq]; zk[bq] = zk[bq - 1]; zk[bq - 1] = tz;
                const int ti = D.dc_nd[bq]; D.dc_nd[bq] = D.dc_nd[bq - 1]; D.dc_nd[bq - 1] = ti;
                --bq;
            }
        }
        s_K = K; s_nr = nr; s_rho = rho; s_flip = flip;
        D.dc_info[0] = K; D.dc_info[1] = nr;
    }
    __syncthreads();
    const int K = s_K;
    // eigenvalues of the deflated coordinates
    for (int p = tid; p < n; p += nt)
        if (state[p] == 0) D.dvec[perm[p]] = flip * ds[p];
    if (K == 0) return;
    double z2sum = 0.0;
    for (int i = 0; i < K; ++i) z2sum += zk[i] * zk[i];
    // secular roots: lambda_j = dk[org[j]] + tk[j]
    for (int j = tid; j < K; j += nt) {
        int o;
        double hi;        // |tau| lies in (0, hi]
        double sgn;       // tau = sgn * sigma
        if (j == K - 1) { o = j; hi = rho * z2sum; sgn = 1.0; }
        else {
            const double gap = dk[j + 1] - dk[j];
            double f = 1.0;                       // f at the midpoint
            for (int i = 0; i < K; ++i) f += rho * zk[i] * zk[i] / ((dk[i] - dk[j]) - 0.5 * gap);
            if (f > 0.0) { o = j; sgn = 1.0; } else { o = j + 1; sgn = -1.0; }
            hi = 0.5 * gap;
        }
        const double dorg = dk[o];
        // h(sigma) = sgn f(dorg + sgn sigma) increases from -inf at sigma = 0+ to h(hi) >= 0; its derivative
        // is rho sum_i z_i^2 / (d_i - lambda)^2 > 0.  Both come out of one pass over the poles.
        auto h = [&](double sigma, double &dh) -> double {
            double f = 1.0, df = 0.0;
            const double t = sgn * sigma;
            for (int i = 0; i < K; ++i) {
                const double inv = 1.0 / ((dk[i] - dorg) - t);
                const double w = rho * zk[i] * zk[i] * inv;
                f += w;
                df += w * inv;
            }
            dh = df;
            return sgn * f;
        };
        // 1. a bracket [lo, hi] with lo > 0.  Components of z can be tiny (eigenvectors of a graded matrix
        //    decay towards the ends), and the root then sits many binades below the gap.  Near the pole
        //    h(sigma) ~ sgn R(0) - rho z_o^2 / sigma, R being the sum over the other poles, so
        //    sigma ~ rho z_o^2 / (sgn R(0)) is the right binade; a few doublings or halvings from there
        //    make the bracket.  When the estimate is unusable, halve down from hi instead.
        double lo = 0.0, dh = 0.0;
        {
            double R0 = 1.0;
            for (int i = 0; i < K; ++i)
                if (i != o) R0 += rho * zk[i] * zk[i] / (dk[i] - dorg);
            const double est = rho * zk[o] * zk[o] / (sgn * R0);
            if (est > 0.0 && est < hi) {
                if (h(est, dh) > 0.0) {
                    hi = est;
                    double sg = est;
                    for (int it = 0; it < 6; ++it) {
                        sg *= 0.25;
                        if (!(sg > 0.0)) break;
                        if (h(sg, dh) > 0.0) hi = sg; else { lo = sg; break; }
                    }
                } else {
                    lo = est;
                    double sg = est;
                    for (int it = 0; it < 6; ++it) {
                        sg *= 4.0;
                        if (!(sg < hi)) break;
                        if (h(sg, dh) > 0.0) { hi = sg; break; } else lo = sg;
                    }
                }
            }
        }
        if (!(lo > 0.0)) {
            for (int it = 0; it < 1100; ++it) {
                const double mid = 0.5 * hi;
                if (!(mid > 0.0)) break;
                if (h(mid, dh) > 0.0) hi = mid; else { lo = mid; break; }
            }
        }
        // 2. Newton's iteration kept inside the bracket [lo, hi] (a step that leaves it is replaced by
        //    bisection); the bracket shrinks at every step, so the loop ends by itself
        double x = 0.5 * (lo + hi);
        for (int it = 0; it < 80 && lo > 0.0; ++it) {
            const double hx = h(x, dh);
            if (hx > 0.0) hi = x; else lo = x;
            double xn = x - hx / dh;
            if (!(xn > lo && xn < hi)) xn = 0.5 * (lo + hi);
            if (!(xn > lo && xn < hi)) break;            // the bracket is two neighbouring numbers
            if (fabs(xn - x) <= 4.0e-16 * xn) { x = xn; break; }
            x = xn;
        }
        if (!(lo > 0.0)) x = 0.5 * (lo + hi);
        org[j] = o;
        tk[j] = sgn * x;
    }
    __syncthreads();
    // z recomputed from the roots: zh_i^2 = prod_j (lambda_j - d_i) / (rho prod_{j != i} (d_j - d_i))
    for (int i = tid; i < K; i += nt) {
        double pr = ((dk[org[i]] - dk[i]) + tk[i]) / rho;
        for (int j = 0; j < K; ++j) {
            if (j == i) continue;
            pr *= ((dk[org[j]] - dk[i]) + tk[j]) / (dk[j] - dk[i]);
        }
        const double mag = sqrt(fabs(pr));
        zh[i] = (zk[i] < 0.0) ? -mag : mag;
    }
    __syncthreads();
    // eigenvectors: column j = zh_i / (d_i - lambda_j), normalised; eigenvalues
    double *__restrict__ Uh = D.Xw;
    for (int j = tid; j < K; j += nt) {
        const double dorg = dk[org[j]], tj = tk[j];
        double nrm2 = 0.0;
        for (int i = 0; i < K; ++i) { const double v = zh[i] / ((dk[i] - dorg) - tj); nrm2 += v * v; }
        const double inv = rsqrt(nrm2);
        for (int i = 0; i < K; ++i) Uh[(int64_t)i * n + j] = zh[i] / ((dk[i] - dorg) - tj) * inv;
        D.dvec[D.dc_nd[j]] = flip * (dorg + tj);
    }
}

template <int R>
__global__ void __launch_bounds__(SYS_WARPS * 32)
eig_rot_systolic_kernel(const RefreshDev *__restrict__ rd, const RowItem *__restrict__ items, int dc)
{
    extern __shared__ double zs[];                // [SYS_WARPS][R][k]
    const RowItem it = items[blockIdx.x];
    const RefreshDev D = rd[it.block];
    const int k = D.k, r = D.r;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row0 = it.row0 + warp * R;
    if (row0 >= k) return;                        // warps never synchronise with one another
    double *z = zs + (size_t)warp * R * k;
#pragma unroll
    for (int q = 0; q < R; ++q) {
        const int row = min(row0 + q, k - 1);     // rows past the end shadow the last row, never stored
        // dc: rows of the identity (the kernel forms diag(Z1, Z2) G; Q is multiplied in afterwards); else rows of Q
        for (int c = lane; c < k; c += 32) z[q * k + c] = dc ? ((c == row) ? 1.0 : 0.0) : D.Wj[(int64_t)row * k + c];
    }
    __syncwarp();
    if (!dc) {
        systolic_apply<R>(z, k, k, D.rot, D.groups, D.sweeps, D.nsweeps[0], lane);
    } else {
        // rows of diag(Z1, Z2): a unit row lies in one half of the columns and only that half's log changes it
        // (a group of rows that straddles the middle goes through both: zeros stay zeros)
        const int s = k / 2;
        if (row0 < s) systolic_apply<R>(z, k, s, D.rot, D.groups, D.sweeps, D.nsweeps[0], lane);
        if (row0 + R > s)
            systolic_apply<R>(z + s, k, k - s, D.rot + dc_rot_off(D), D.groups + dc_group_off(D), D.sweeps + dc_sweep_off(D),
                              D.nsweeps[1], lane);
        // deflation rotations (few), one row per lane
        const int nr = D.dc_info[1];
        if (lane < R) {
            double *zr = z + lane * k;
            for (int t = 0; t < nr; ++t) {
                const int2 ab = D.dc_rot_idx[t];
                const double2 cs = D.dc_rot_cs[t];
                const double xa = zr[ab.x], xb = zr[ab.y];
                zr[ab.x] = cs.x * xa + cs.y * xb;
                zr[ab.y] = cs.x * xb - cs.y * xa;
            }
        }
        __syncwarp();
        // Z = diag(Z1, Z2) G is done for this row.  The coordinates of the secular problem still have to be
        // multiplied by Uhat: their values, gathered in the order of the secular problem, go to row `row` of S
        // (free since Q was formed) for eig_merge_kernel; the other columns are final and go to Ztot (gpart).
        const int K = D.dc_info[0];
        const int32_t *__restrict__ nd = D.dc_nd;
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const int row = row0 + q;
            if (row >= k) continue;
            for (int i = lane; i < K; i += 32) D.S[(int64_t)row * k + i] = z[q * k + nd[i]];
            for (int c = lane; c < k; c += 32)
                if (!(D.rank[c] & RANK_MERGED)) D.gpart[(int64_t)row * k + c] = z[q * k + c];
        }
        return;
    }
    // rank the eigenvalues (descending, ties by index) and emit the leading r columns
    const double *__restrict__ lam = D.dvec;
    for (int jj = lane; jj < k; jj += 32) {
        const int rank = D.rank[jj];
        if (rank >= r) continue;
        const double lj = lam[jj];
        const double inv = (lj > 1e-300) ? 1.0 / sqrt(lj) : 0.0;
#pragma unroll
        for (int q = 0; q < R; ++q) {
            const int row = row0 + q;
            if (row < k) {
                const double w = z[q * k + jj];
                D.Wu[(int64_t)row * r + rank] = (float)w;
                D.Wv[(int64_t)row * r + rank] = (float)(w * inv);
            }
        }
    }
}

// Divide and conquer, step 4b: the coordinates of the secular problem times the merged eigenvector matrix,
// Y = Zg Uhat (Zg: k x K, the rows the rotation kernel left in S; Uhat: K x K in Xw), on the FP64 tensor
// path.  A CTA owns a 64 x 64 tile of Y, its eight warps 32 x 16 regions of it as 4 x 2 sub-tiles of 8 x 8
// (mma m8n8k4); operands are staged 16 columns of Zg / rows of Uhat at a time.  Column j of Y is column
// nd[j] of Ztot = diag(Z1, Z2) G Uhat (in gpart), whose other columns the rotation kernel wrote.

__global__ void __launch_bounds__(256)
eig_merge_kernel(const RefreshDev *__restrict__ rd, const int32_t *__restrict__ list)
{
    const RefreshDev D = rd[list[blockIdx.z]];
    const int k = D.k, r = D.r, K = D.dc_info[0];
    const int r0 = blockIdx.y * MG_T, c0 = blockIdx.x * MG_T;
    if (r0 >= k || c0 >= K) return;
    const double *__restrict__ Zg = D.S;
    const double *__restrict__ Uh = D.Xw;
    __shared__ __align__(16) double As[MG_K][MG_PITCH];     // As[i][row] = Zg[r0 + row][i0 + i]
    __shared__ __align__(16) double Bs[MG_K][MG_PITCH];     // Bs[i][col] = Uhat[i0 + i][c0 + col]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wi = warp >> 2, wj = warp & 3;
    const int g = lane >> 2, q = lane & 3;
    double acc[4][2][2];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
    double ra[4], rb[4];
    auto fetch = [&](int i0) {
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = tid + l * 256;
            {
                const int row = r0 + (e >> 4), i = i0 + (e & 15);
                ra[l] = (row < k && i < K) ? Zg[(int64_t)row * k + i] : 0.0;
            }
            {
                const int i = i0 + (e >> 6), col = c0 + (e & 63);
                rb[l] = (i < K && col < K) ? Uh[(int64_t)i * k + col] : 0.0;
            }
        }
    };
    fetch(0);
    for (int i0 = 0; i0 < K; i0 += MG_K) {
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int e = tid + l * 256;
            As[e & 15][e >> 4] = ra[l];
            Bs[e >> 6][e & 63] = rb[l];
        }
        __syncthreads();
        if (i0 + MG_K < K) fetch(i0 + MG_K);
#pragma unroll
        for (int st = 0; st < MG_K / 4; ++st) {
            double af[4], bf[2];
#pragma unroll
            for (int a = 0; a < 4; ++a) af[a] = As[st * 4 + q][wi * 32 + a * 8 + g];
#pragma unroll
            for (int b = 0; b < 2; ++b) bf[b] = Bs[st * 4 + q][wj * 16 + b * 8 + g];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 2; ++b) dmma_f64(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int b = 0; b < 2; ++b)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int j = c0 + wj * 16 + b * 8 + 2 * q + h;
            if (j >= K) continue;
            const int cj = D.dc_nd[j];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int row = r0 + wi * 32 + a * 8 + g;
                if (row < k) D.gpart[(int64_t)row * k + cj] = acc[a][b][h];
            }
        }
}

static int sys_rows_per_warp(int kmax) { return kmax <= 544 ? 4 : 2; }

int eig_panel_rows(int kmax)
{
    return SYS_WARPS * sys_rows_per_warp(kmax);
}

int64_t eig_rot_capacity(int k)
{
    // rows of the skewed log (typical need: 0.03 k^2 + 4 k), 32 entries each
    const int64_t rows = (int64_t)k * k / 10 + 12 * (int64_t)k + 512;
    return rows * 32;
}

template <typename F>
static cudaError_t raise_smem(F *fn, size_t bytes, size_t *configured)
{
    if (bytes <= *configured) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) *configured = bytes;
    return e;
}

cudaError_t eig_tridiag_batched(const RefreshDev *rd, const int32_t *list, int nlist, const RowItem *panel_items,
                                int npanels, int kmax, cudaStream_t stream)
{
    if (nlist <= 0) return cudaSuccess;
    const int kpad = kmax + 8;
    const size_t tr_bytes = (size_t)(2 + 2 * TR_NB) * kpad * sizeof(double);
    static size_t tr_cfg = 0, sys4_cfg = 0, sys2_cfg = 0, sec_cfg = 0;
    cudaError_t e;
    if ((e = raise_smem(tridiag_kernel, tr_bytes, &tr_cfg)) != cudaSuccess) return e;
    tridiag_kernel<<<nlist, TR_THREADS, tr_bytes, stream>>>(rd, list, kpad);
    const size_t ql_bytes = (size_t)2 * kmax * sizeof(double);
    if (kmax <= SYS_KMAX) {
        const int threads = SYS_WARPS * 32;
        {   // Q = I - V T V^T, every step a tiled product (see eig_wy_gemm_kernel)
            const int t = (kmax + 63) / 64;
            const dim3 grid(t, t, nlist);
            const size_t wb_bytes = (size_t)2 * WY_NB * (WY_NB + 1) * sizeof(double);
            static size_t wb_cfg = 0;
            if ((e = raise_smem(eig_wy_base_kernel, wb_bytes, &wb_cfg)) != cudaSuccess) return e;
            eig_wy_gemm_kernel<WY_G><<<grid, 256, 0, stream>>>(rd, list, 0);
            eig_wy_base_kernel<<<dim3(t, nlist), WY_NB, wb_bytes, stream>>>(rd, list);
            for (int sz = WY_NB; sz < kmax - 2; sz *= 2) {
                eig_wy_gemm_kernel<WY_X><<<grid, 256, 0, stream>>>(rd, list, sz);
                eig_wy_gemm_kernel<WY_T12><<<grid, 256, 0, stream>>>(rd, list, sz);
            }
            eig_wy_gemm_kernel<WY_M><<<grid, 256, 0, stream>>>(rd, list, 0);
            eig_wy_gemm_kernel<WY_Q><<<grid, 256, 0, stream>>>(rd, list, 0);
        }
        const int dc = kmax >= DC_MIN_K ? 1 : 0;
        ql_log_kernel<<<nlist, 64, ql_bytes, stream>>>(rd, list, dc);
        if (dc) {
            dc_zrows_kernel<<<nlist, 64, (size_t)kmax * sizeof(double), stream>>>(rd, list);
            const size_t sec_bytes = (size_t)kpad * (6 * sizeof(double) + 3 * sizeof(int));
            if ((e = raise_smem(dc_secular_kernel, sec_bytes, &sec_cfg)) != cudaSuccess) return e;
            dc_secular_kernel<<<nlist, DC_THREADS, sec_bytes, stream>>>(rd, list, kpad);
        }
        eig_rank_kernel<<<nlist, 256, 0, stream>>>(rd, list, dc);
        const int R = sys_rows_per_warp(kmax);
        const size_t sys_bytes = (size_t)SYS_WARPS * R * kmax * sizeof(double);
        if (R == 4) {
            if ((e = raise_smem(eig_rot_systolic_kernel<4>, sys_bytes, &sys4_cfg)) != cudaSuccess) return e;
            eig_rot_systolic_kernel<4><<<npanels, threads, sys_bytes, stream>>>(rd, panel_items, dc);
        } else {
            if ((e = raise_smem(eig_rot_systolic_kernel<2>, sys_bytes, &sys2_cfg)) != cudaSuccess) return e;
            eig_rot_systolic_kernel<2><<<npanels, threads, sys_bytes, stream>>>(rd, panel_items, dc);
        }
        if (dc) {   // Ztot = diag(Z1, Z2) G Uhat, then W = Q Ztot
            const int t = (kmax + MG_T - 1) / MG_T;
            eig_merge_kernel<<<dim3(t, t, nlist), 256, 0, stream>>>(rd, list);
            eig_wy_gemm_kernel<WY_W><<<dim3(t, t, nlist), 256, 0, stream>>>(rd, list, 0);
        }
        return cudaGetLastError();
    }
    return cudaErrorInvalidValue;   // k is limited to SYS_KMAX when a context is created
}

}  // namespace tsr
