/*
 * tsr_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, FP64 CPU statement of what the TSR-Adam optimizer hot path
 * computes (two-sided low-rank Adam: Algorithm 1 and Sections 3.3-3.5 of the
 * paper; Algorithm 2 for the momentum-SGD variant).  It exists only so that the
 * tests, the smoke check and the CPU-baseline leg of the benchmark have
 * something independent to compare the CUDA library with.  It shares no code,
 * header, table or helper with the CUDA path and the product never calls it.
 *
 * Every routine is the definition written out: triple loops for the matrix
 * products, Householder reflections for `orth`, one-sided (Hestenes) Jacobi
 * rotations for the small SVD.  No blocking, no fusion, no BLAS/LAPACK.
 * OpenMP only splits an outermost loop whose iterations are independent.
 *
 * Conventions: all matrices are row-major FP64 with explicit leading
 * dimensions where the caller may pad (G, W); everything else is dense.
 * Inputs in reduced precision are widened exactly to FP64 by the caller.
 *
 * Parity pins (tests/test_oracle_pins.py): every routine below is pinned by at
 * least one check that does not come from this file -- torch.optim.AdamW,
 * numpy.linalg.qr / svd, exact-recovery identities, orthonormality invariants,
 * closed forms and the byte counts the paper's tables print.  The only thing
 * left unpinned is a full multi-step trajectory on the LLaMA-shaped synthetic
 * gradient sets (nothing external fixes those numbers).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define IDX(i, j, ld) ((size_t)(i) * (size_t)(ld) + (size_t)(j))

/* ------------------------------------------------------------------------- */
/* Two-sided core projection, Algorithm 1 "C <- U^T G V" (Section 3.3).      */
/* T = G V (m x r), then C = U^T T (r x r).                                  */
/* ------------------------------------------------------------------------- */
int tsro_project_core(int64_t m, int64_t n, int64_t r, const double *G, int64_t ldg,
                      const double *U, const double *V, double *C)
{
    double *T = (double *)calloc((size_t)m * (size_t)r, sizeof(double));
    if (!T) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < n; ++j) {
            const double g = G[IDX(i, j, ldg)];
            for (int64_t a = 0; a < r; ++a) T[IDX(i, a, r)] += g * V[IDX(j, a, r)];
        }
#pragma omp parallel for schedule(static)
    for (int64_t a = 0; a < r; ++a)
        for (int64_t b = 0; b < r; ++b) {
            double s = 0.0;
            for (int64_t i = 0; i < m; ++i) s += U[IDX(i, a, r)] * T[IDX(i, b, r)];
            C[IDX(a, b, r)] = s;
        }
    free(T);
    return 0;
}

/* One-sided core C = U^T G (r x n): the ablation arm of Section 5 / Table 1. */
int tsro_project_one_sided(int64_t m, int64_t n, int64_t r, const double *G, int64_t ldg,
                           const double *U, double *C)
{
#pragma omp parallel for schedule(static)
    for (int64_t a = 0; a < r; ++a)
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            for (int64_t i = 0; i < m; ++i) s += U[IDX(i, a, r)] * G[IDX(i, j, ldg)];
            C[IDX(a, j, n)] = s;
        }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Core-space Adam, Algorithm 1 lines "m <- ...", "v <- ...", bias           */
/* correction and D = m_hat / (sqrt(v_hat) + eps)  (Section 3.4).            */
/* `count` = r*r entries; t is the 1-based global step.                      */
/* ------------------------------------------------------------------------- */
int tsro_adam_core(int64_t count, const double *Cbar, double *M, double *Vm, double *D,
                   double beta1, double beta2, double eps, int64_t t)
{
    const double bc1 = 1.0 - pow(beta1, (double)t);
    const double bc2 = 1.0 - pow(beta2, (double)t);
    for (int64_t e = 0; e < count; ++e) {
        const double c = Cbar[e];
        M[e] = beta1 * M[e] + (1.0 - beta1) * c;
        Vm[e] = beta2 * Vm[e] + (1.0 - beta2) * (c * c);
        const double mh = M[e] / bc1;
        const double vh = Vm[e] / bc2;
        D[e] = mh / (sqrt(vh) + eps);
    }
    return 0;
}

/* Momentum-SGD core update of Algorithm 2: m <- beta m + (1-beta) C; D <- m. */
int tsro_sgd_core(int64_t count, const double *Cbar, double *M, double *D, double beta)
{
    for (int64_t e = 0; e < count; ++e) {
        M[e] = beta * M[e] + (1.0 - beta) * Cbar[e];
        D[e] = M[e];
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Dense AdamW for parameters that are not matrix blocks (Section 3.1, the    */
/* dense update; Section 3.4 "all non-matrix parameters ... are updated in    */
/* dense form"): moments, bias correction, decoupled weight decay.            */
/* ------------------------------------------------------------------------- */
int tsro_dense_adamw(int64_t count, double *P, const double *G, double *M, double *Vm, double lr,
                     double beta1, double beta2, double eps, double weight_decay, int64_t t)
{
    const double bc1 = 1.0 - pow(beta1, (double)t);
    const double bc2 = 1.0 - pow(beta2, (double)t);
    for (int64_t e = 0; e < count; ++e) {
        const double g = G[e];
        M[e] = beta1 * M[e] + (1.0 - beta1) * g;
        Vm[e] = beta2 * Vm[e] + (1.0 - beta2) * (g * g);
        const double upd = (M[e] / bc1) / (sqrt(Vm[e] / bc2) + eps);
        P[e] = P[e] - lr * (upd + weight_decay * P[e]);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Lift and AdamW apply, Algorithm 1: dW = U D V^T; W <- W - eta(dW + lam W). */
/* `scale` multiplies the lifted update only (the experiments' "scaling       */
/* factor"; 1 reproduces Algorithm 1 as printed).                             */
/* ------------------------------------------------------------------------- */
int tsro_backproject_apply(int64_t m, int64_t n, int64_t r, const double *U, const double *D,
                           const double *V, double *W, int64_t ldw, double lr, double weight_decay,
                           double scale)
{
    double *P = (double *)calloc((size_t)m * (size_t)r, sizeof(double)); /* P = U D */
    if (!P) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i)
        for (int64_t a = 0; a < r; ++a) {
            const double u = U[IDX(i, a, r)];
            for (int64_t b = 0; b < r; ++b) P[IDX(i, b, r)] += u * D[IDX(a, b, r)];
        }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < n; ++j) {
            double dw = 0.0;
            for (int64_t b = 0; b < r; ++b) dw += P[IDX(i, b, r)] * V[IDX(j, b, r)];
            const double w = W[IDX(i, j, ldw)];
            W[IDX(i, j, ldw)] = w - lr * (scale * dw + weight_decay * w);
        }
    free(P);
    return 0;
}

/* One-sided arm of the comparison (Table 1, "One-sided": the synchronized object is C = U^T G,   */
/* r x n; Section 5 ablation): the update lives in the left subspace only, dW = U D with D the    */
/* r x n normalised core, and the weights move as in Algorithm 1:                                 */
/* W <- W - lr (scale * U D + weight_decay * W).                                                  */
int tsro_backproject_one_sided(int64_t m, int64_t n, int64_t r, const double *U, const double *D,
                               double *W, int64_t ldw, double lr, double weight_decay, double scale)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < n; ++j) {
            double dw = 0.0;
            for (int64_t a = 0; a < r; ++a) dw += U[IDX(i, a, r)] * D[IDX(a, j, n)];
            const double w = W[IDX(i, j, ldw)];
            W[IDX(i, j, ldw)] = w - lr * (scale * dw + weight_decay * w);
        }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* orth(Y): thin QR by Householder reflections (Section 3.5, "implemented by  */
/* thin QR").  Y is M x k, M >= k.  Q (M x k) = first k columns of            */
/* H_1 ... H_k.  A column that is already zero below the diagonal gets        */
/* H_j = I, so Q is orthonormal even when Y is rank-deficient.  R (k x k,     */
/* upper triangular) is returned when Rout != NULL.                           */
/* ------------------------------------------------------------------------- */
int tsro_orth(int64_t M, int64_t k, const double *Y, double *Q, double *Rout)
{
    if (M < k) return -2;
    double *A = (double *)malloc((size_t)M * (size_t)k * sizeof(double));
    double *tau = (double *)calloc((size_t)k, sizeof(double));
    if (!A || !tau) { free(A); free(tau); return -1; }
    memcpy(A, Y, (size_t)M * (size_t)k * sizeof(double));

    for (int64_t j = 0; j < k; ++j) {
        /* reflector for column j, rows j..M-1: v = x + sign(x0)|x| e0, stored with v0 = 1 */
        double nrm2 = 0.0;
        for (int64_t i = j; i < M; ++i) nrm2 += A[IDX(i, j, k)] * A[IDX(i, j, k)];
        const double nrm = sqrt(nrm2);
        if (nrm == 0.0) { tau[j] = 0.0; continue; }
        const double x0 = A[IDX(j, j, k)];
        const double alpha = (x0 >= 0.0) ? -nrm : nrm; /* R_jj */
        const double v0 = x0 - alpha;
        tau[j] = -v0 / alpha; /* = 2 / (v^T v) with v scaled so v0 = 1 */
        for (int64_t i = j + 1; i < M; ++i) A[IDX(i, j, k)] /= v0;
        A[IDX(j, j, k)] = alpha;
        /* apply H_j = I - tau v v^T to the trailing columns */
#pragma omp parallel for schedule(static)
        for (int64_t c = j + 1; c < k; ++c) {
            double s = A[IDX(j, c, k)];
            for (int64_t i = j + 1; i < M; ++i) s += A[IDX(i, j, k)] * A[IDX(i, c, k)];
            s *= tau[j];
            A[IDX(j, c, k)] -= s;
            for (int64_t i = j + 1; i < M; ++i) A[IDX(i, c, k)] -= s * A[IDX(i, j, k)];
        }
    }
    if (Rout) {
        for (int64_t i = 0; i < k; ++i)
            for (int64_t j = 0; j < k; ++j) Rout[IDX(i, j, k)] = (j >= i) ? A[IDX(i, j, k)] : 0.0;
    }
    /* Q = H_1 ... H_k [I_k; 0]: start from the identity block and apply H_k ... H_1 */
    for (int64_t i = 0; i < M; ++i)
        for (int64_t c = 0; c < k; ++c) Q[IDX(i, c, k)] = (i == c) ? 1.0 : 0.0;
    for (int64_t j = k - 1; j >= 0; --j) {
        if (tau[j] == 0.0) continue;
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < k; ++c) {
            double s = Q[IDX(j, c, k)];
            for (int64_t i = j + 1; i < M; ++i) s += A[IDX(i, j, k)] * Q[IDX(i, c, k)];
            s *= tau[j];
            Q[IDX(j, c, k)] -= s;
            for (int64_t i = j + 1; i < M; ++i) Q[IDX(i, c, k)] -= s * A[IDX(i, j, k)];
        }
    }
    free(A);
    free(tau);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Small SVD B = Ut * diag(S) * Vt^T of a k x n matrix (k <= n), Section 3.5  */
/* "compute a small SVD".  One-sided Jacobi on A = B^T (n x k): plane         */
/* rotations from the right make the columns of A mutually orthogonal;        */
/* then S_j = |A_j|, Vt_j = A_j / S_j and the accumulated rotations are Ut.   */
/* Singular values are sorted in descending order.  Columns of Vt that        */
/* belong to a zero singular value are completed to an orthonormal set.       */
/* Returns the number of sweeps used, or a negative error.                    */
/* ------------------------------------------------------------------------- */
int tsro_svd_jacobi(int64_t k, int64_t n, const double *B, double *Ut, double *S, double *Vt,
                    int max_sweeps)
{
    if (k > n) return -2;
    double *A = (double *)malloc((size_t)n * (size_t)k * sizeof(double)); /* n x k, column j = row j of B */
    double *J = (double *)calloc((size_t)k * (size_t)k, sizeof(double));
    int64_t *ord = (int64_t *)malloc((size_t)k * sizeof(int64_t));
    double *nrm = (double *)malloc((size_t)k * sizeof(double));
    if (!A || !J || !ord || !nrm) { free(A); free(J); free(ord); free(nrm); return -1; }
    for (int64_t i = 0; i < k; ++i)
        for (int64_t j = 0; j < n; ++j) A[IDX(j, i, k)] = B[IDX(i, j, n)];
    for (int64_t i = 0; i < k; ++i) J[IDX(i, i, k)] = 1.0;

    const double tol = 1e-15;
    int sweeps = 0, rotated = 1;
    while (rotated && sweeps < max_sweeps) {
        rotated = 0;
        ++sweeps;
        for (int64_t p = 0; p < k - 1; ++p)
            for (int64_t q = p + 1; q < k; ++q) {
                double app = 0.0, aqq = 0.0, apq = 0.0;
                for (int64_t i = 0; i < n; ++i) {
                    const double x = A[IDX(i, p, k)], y = A[IDX(i, q, k)];
                    app += x * x; aqq += y * y; apq += x * y;
                }
                if (fabs(apq) <= tol * sqrt(app * aqq) || apq == 0.0) continue;
                rotated = 1;
                /* rotation that zeroes the (p,q) entry of A^T A */
                const double zeta = (aqq - app) / (2.0 * apq);
                const double tt = ((zeta >= 0.0) ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                const double cs = 1.0 / sqrt(1.0 + tt * tt), sn = cs * tt;
                for (int64_t i = 0; i < n; ++i) {
                    const double x = A[IDX(i, p, k)], y = A[IDX(i, q, k)];
                    A[IDX(i, p, k)] = cs * x - sn * y;
                    A[IDX(i, q, k)] = sn * x + cs * y;
                }
                for (int64_t i = 0; i < k; ++i) {
                    const double x = J[IDX(i, p, k)], y = J[IDX(i, q, k)];
                    J[IDX(i, p, k)] = cs * x - sn * y;
                    J[IDX(i, q, k)] = sn * x + cs * y;
                }
            }
    }
    for (int64_t j = 0; j < k; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < n; ++i) s += A[IDX(i, j, k)] * A[IDX(i, j, k)];
        nrm[j] = sqrt(s);
        ord[j] = j;
    }
    /* descending selection sort of the column order (stable for ties) */
    for (int64_t a = 0; a < k; ++a)
        for (int64_t b = a + 1; b < k; ++b)
            if (nrm[ord[b]] > nrm[ord[a]]) { int64_t tmp = ord[a]; ord[a] = ord[b]; ord[b] = tmp; }
    const double smax = nrm[ord[0]];
    for (int64_t c = 0; c < k; ++c) {
        const int64_t j = ord[c];
        S[c] = nrm[j];
        for (int64_t i = 0; i < k; ++i) Ut[IDX(i, c, k)] = J[IDX(i, j, k)];
        if (nrm[j] > 1e-300 && nrm[j] > 1e-14 * smax) {
            for (int64_t i = 0; i < n; ++i) Vt[IDX(i, c, k)] = A[IDX(i, j, k)] / nrm[j];
        } else {
            /* zero singular value: any unit vector orthogonal to the columns already placed */
            S[c] = (nrm[j] > 1e-300) ? nrm[j] : 0.0;
            int done = 0;
            for (int64_t e = 0; e < n && !done; ++e) {
                for (int64_t i = 0; i < n; ++i) Vt[IDX(i, c, k)] = (i == e) ? 1.0 : 0.0;
                for (int pass = 0; pass < 2; ++pass)
                    for (int64_t d = 0; d < c; ++d) {
                        double dot = 0.0;
                        for (int64_t i = 0; i < n; ++i) dot += Vt[IDX(i, d, k)] * Vt[IDX(i, c, k)];
                        for (int64_t i = 0; i < n; ++i) Vt[IDX(i, c, k)] -= dot * Vt[IDX(i, d, k)];
                    }
                double s = 0.0;
                for (int64_t i = 0; i < n; ++i) s += Vt[IDX(i, c, k)] * Vt[IDX(i, c, k)];
                if (s > 0.25) {
                    s = sqrt(s);
                    for (int64_t i = 0; i < n; ++i) Vt[IDX(i, c, k)] /= s;
                    done = 1;
                }
            }
            if (!done) { free(A); free(J); free(ord); free(nrm); return -3; }
        }
    }
    free(A); free(J); free(ord); free(nrm);
    return rotated ? -4 : sweeps; /* -4: not converged within max_sweeps */
}

/* Y (m x k) = G (m x n) * X (n x k) */
static void mul_G_X(int64_t m, int64_t n, int64_t k, const double *G, int64_t ldg, const double *X, double *Y)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i) {
        for (int64_t c = 0; c < k; ++c) Y[IDX(i, c, k)] = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            const double g = G[IDX(i, j, ldg)];
            for (int64_t c = 0; c < k; ++c) Y[IDX(i, c, k)] += g * X[IDX(j, c, k)];
        }
    }
}

/* Z (n x k) = G^T (n x m) * Q (m x k) */
static void mul_Gt_Q(int64_t m, int64_t n, int64_t k, const double *G, int64_t ldg, const double *Q, double *Z)
{
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        for (int64_t c = 0; c < k; ++c) Z[IDX(j, c, k)] = 0.0;
        for (int64_t i = 0; i < m; ++i) {
            const double g = G[IDX(i, j, ldg)];
            for (int64_t c = 0; c < k; ++c) Z[IDX(j, c, k)] += g * Q[IDX(i, c, k)];
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Randomized-SVD subspace refresh (Algorithm 1, the "t mod K = 0" branch;    */
/* Section 3.5) for one worker (all-reduce averages are the identity):        */
/*   Y = G Omega; Q = orth(Y);                                                */
/*   q times: Yrow = G^T Q; Qrow = orth(Yrow); Y = G Qrow; Q = orth(Y);       */
/*   B = Q^T G; B = Ut S Vt^T; U = Q Ut[:, :r]; V = Vt[:, :r].                */
/* Omega is n x k with k = r + p.  sigma (k values, descending) is optional.  */
/* Returns Jacobi sweeps used (>0) or a negative error.                       */
/* ------------------------------------------------------------------------- */
int tsro_rsvd_refresh(int64_t m, int64_t n, int64_t r, int64_t p, int64_t q, const double *G,
                      int64_t ldg, const double *Omega, double *U, double *V, double *sigma)
{
    const int64_t k = r + p;
    if (k > m || k > n || r < 1 || p < 0 || q < 0) return -2;
    double *Y = (double *)malloc((size_t)m * k * sizeof(double));
    double *Q = (double *)malloc((size_t)m * k * sizeof(double));
    double *Yr = (double *)malloc((size_t)n * k * sizeof(double));
    double *Qr = (double *)malloc((size_t)n * k * sizeof(double));
    double *B = (double *)malloc((size_t)k * n * sizeof(double));
    double *Ut = (double *)malloc((size_t)k * k * sizeof(double));
    double *S = (double *)malloc((size_t)k * sizeof(double));
    double *Vt = (double *)malloc((size_t)n * k * sizeof(double));
    int rc = -1;
    if (!Y || !Q || !Yr || !Qr || !B || !Ut || !S || !Vt) goto done;

    mul_G_X(m, n, k, G, ldg, Omega, Y);
    if ((rc = tsro_orth(m, k, Y, Q, NULL)) != 0) goto done;
    for (int64_t it = 0; it < q; ++it) {
        mul_Gt_Q(m, n, k, G, ldg, Q, Yr);
        if ((rc = tsro_orth(n, k, Yr, Qr, NULL)) != 0) goto done;
        mul_G_X(m, n, k, G, ldg, Qr, Y);
        if ((rc = tsro_orth(m, k, Y, Q, NULL)) != 0) goto done;
    }
    /* B = Q^T G (k x n) */
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < k; ++c)
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            for (int64_t i = 0; i < m; ++i) s += Q[IDX(i, c, k)] * G[IDX(i, j, ldg)];
            B[IDX(c, j, n)] = s;
        }
    rc = tsro_svd_jacobi(k, n, B, Ut, S, Vt, 60);
    if (rc < 0) goto done;
    /* U = Q Ut[:, :r]; V = Vt[:, :r] */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i)
        for (int64_t a = 0; a < r; ++a) {
            double s = 0.0;
            for (int64_t c = 0; c < k; ++c) s += Q[IDX(i, c, k)] * Ut[IDX(c, a, k)];
            U[IDX(i, a, r)] = s;
        }
    for (int64_t j = 0; j < n; ++j)
        for (int64_t a = 0; a < r; ++a) V[IDX(j, a, r)] = Vt[IDX(j, a, k)];
    if (sigma) memcpy(sigma, S, (size_t)k * sizeof(double));
done:
    free(Y); free(Q); free(Yr); free(Qr); free(B); free(Ut); free(S); free(Vt);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* Moment re-expression at a refresh (the "refresh alignment" assumption of   */
/* the convergence analysis, Appendix): the core moment is replaced by the    */
/* one whose lifted matrix is the old lifted moment projected onto the new    */
/* subspaces,  M' = Unew^T (Uold M Vold^T) Vnew.  Algorithm 1 itself leaves   */
/* M untouched; this is an option.                                            */
/* ------------------------------------------------------------------------- */
int tsro_reexpress_moment(int64_t m, int64_t n, int64_t r, const double *Uold, const double *Vold,
                          const double *Unew, const double *Vnew, double *M)
{
    double *L = (double *)calloc((size_t)m * (size_t)n, sizeof(double));   /* lifted old moment */
    double *UM = (double *)calloc((size_t)m * (size_t)r, sizeof(double));
    if (!L || !UM) { free(L); free(UM); return -1; }
    for (int64_t i = 0; i < m; ++i)
        for (int64_t a = 0; a < r; ++a)
            for (int64_t b = 0; b < r; ++b) UM[IDX(i, b, r)] += Uold[IDX(i, a, r)] * M[IDX(a, b, r)];
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            for (int64_t b = 0; b < r; ++b) s += UM[IDX(i, b, r)] * Vold[IDX(j, b, r)];
            L[IDX(i, j, n)] = s;
        }
    int rc = tsro_project_core(m, n, r, L, n, Unew, Vnew, M);
    free(L); free(UM);
    return rc;
}

/* Exact-SVD refresh (the "naive" arm of Section 3.5): top-r singular vectors of G itself. */
int tsro_exact_svd_refresh(int64_t m, int64_t n, int64_t r, const double *G, int64_t ldg, double *U,
                           double *V, double *sigma)
{
    /* work on whichever orientation has rows <= cols */
    const int tall = (m > n);
    const int64_t kk = tall ? n : m, nn = tall ? m : n;
    if (r > kk) return -2;
    double *B = (double *)malloc((size_t)kk * nn * sizeof(double));
    double *Ut = (double *)malloc((size_t)kk * kk * sizeof(double));
    double *S = (double *)malloc((size_t)kk * sizeof(double));
    double *Vt = (double *)malloc((size_t)nn * kk * sizeof(double));
    int rc = -1;
    if (!B || !Ut || !S || !Vt) goto done;
    for (int64_t i = 0; i < kk; ++i)
        for (int64_t j = 0; j < nn; ++j) B[IDX(i, j, nn)] = tall ? G[IDX(j, i, ldg)] : G[IDX(i, j, ldg)];
    rc = tsro_svd_jacobi(kk, nn, B, Ut, S, Vt, 60);
    if (rc < 0) goto done;
    for (int64_t a = 0; a < r; ++a) {
        if (!tall) {
            for (int64_t i = 0; i < m; ++i) U[IDX(i, a, r)] = Ut[IDX(i, a, kk)];
            for (int64_t j = 0; j < n; ++j) V[IDX(j, a, r)] = Vt[IDX(j, a, kk)];
        } else {
            for (int64_t i = 0; i < m; ++i) U[IDX(i, a, r)] = Vt[IDX(i, a, kk)];
            for (int64_t j = 0; j < n; ++j) V[IDX(j, a, r)] = Ut[IDX(j, a, kk)];
        }
    }
    if (sigma) memcpy(sigma, S, (size_t)kk * sizeof(double));
done:
    free(B); free(Ut); free(S); free(Vt);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* Communicated-bytes accounting (Section 3.2): what one worker would hand to */
/* the all-reduce for one block.  Non-refresh step: the r x r core.  Refresh  */
/* step: additionally Q (m x k) and B (k x n).                                */
/* ------------------------------------------------------------------------- */
uint64_t tsro_core_bytes(int64_t r, int64_t bytes_per_elem)
{
    return (uint64_t)r * (uint64_t)r * (uint64_t)bytes_per_elem;
}

uint64_t tsro_sketch_bytes(int64_t m, int64_t n, int64_t r, int64_t p, int64_t bytes_per_elem)
{
    const uint64_t k = (uint64_t)(r + p);
    return k * ((uint64_t)m + (uint64_t)n) * (uint64_t)bytes_per_elem;
}

/* Optimizer-state entries of one block (Table 2): U, V and the two core moments. */
uint64_t tsro_state_elems(int64_t m, int64_t n, int64_t r)
{
    return (uint64_t)(m + n) * (uint64_t)r + 2ull * (uint64_t)r * (uint64_t)r;
}

int tsro_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
