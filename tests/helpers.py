"""Shared helpers for the GPU parity tests (CUDA library vs the FP64 CPU oracle)."""
import numpy as np
import torch

import oracle
import tsr_inputs as ti

TOL_F32 = 1e-4      # max relative Frobenius error, FP32-gradient path
TOL_BF16 = 2e-2     # max relative Frobenius error, BF16-gradient path
TOL_SUBSPACE = 1e-3  # || P - P' ||_F of projectors at a spectral gap
TOL_ORTHO = 1e-4    # || U^T U - I ||_F after a refresh
# Element-wise companion of TOL_F32: max |x_gpu - x_oracle| <= TOL_F32_MAXABS * max |x_oracle|.  A relative
# Frobenius norm can hide one bad tile edge among 10^5 good entries; this bound cannot.  FP32 products of
# length <= 1376 accumulate about sqrt(K) * 2^-24 ~ 2e-6 relative to the largest entry (measured 1.2e-6 on
# C, M, Vm; W moves by lr per step, so its error is far smaller); the bound leaves a factor of eight.
TOL_F32_MAXABS = 1e-5
# Off-diagonal part of U^T G V after a refresh, relative to sigma_1.  U = Q U~ and V = B^T U~ / sigma come from
# the same eigenvectors, so U^T G V = U~^T (B B^T) U~ / sigma is diagonal up to the rounding of the FP32 bases
# and of the eigen-solver: measured 3e-8 ... 1.5e-5 over every block of the five configurations (FP32 bases carry
# 2^-24 ~ 6e-8 per entry, times sqrt(k)); the bound leaves a factor of three above the worst block.
TOL_OFFDIAG = 5e-5


def to64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def rel_fro(a, b) -> float:
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (den if den > 0 else 1.0))


def max_abs_err(a, b) -> float:
    """max |a - b| relative to max |b| (element-wise gate next to the Frobenius one)."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    den = np.abs(b).max()
    return float(np.abs(a - b).max() / (den if den > 0 else 1.0))


def proj(X: np.ndarray) -> np.ndarray:
    return X @ X.T


def fill_gradient(plan, i, seed, signal_rank=None, noise_std=ti.NOISE_STD):
    """Writes a seeded low-rank-plus-noise gradient into block i's bound G buffer; returns FP64 copy."""
    G = plan.G[i]
    m, n = G.shape
    sr = min(ti.SIGNAL_RANK, min(m, n) // 2) if signal_rank is None else signal_rank
    g = ti.gradient(m, n, seed, dtype=G.dtype, device="cpu", signal_rank=sr, noise_std=noise_std)
    G.copy_(g.to(G.device))
    return to64(g)


def fill_weights(plan, i, seed):
    W = plan.W[i]
    w = ti.weights(W.shape[0], W.shape[1], seed)
    W.copy_(w.to(W.device))
    return to64(w)


def set_bases(plan, i, U, V):
    plan.U[i].copy_(U.to(plan.U[i].device))
    plan.V[i].copy_(V.to(plan.V[i].device))


class RefreshChecks:
    """Oracle-side checks of refreshed bases, run on background host threads.  The oracle's refresh spends most of
    its time in a serial Jacobi loop (minutes for a 1B-shaped block), and nothing downstream waits for its result:
    the parity protocol hands the LIBRARY's bases to the oracle after a refresh.  So the checks of all blocks run
    side by side while the test goes on stepping, and `join` re-raises the first failed assertion at the end.
    (ctypes releases the interpreter lock during the oracle's calls.)"""

    def __init__(self, workers=None):
        import os
        from concurrent.futures import ThreadPoolExecutor
        # a few checks at a time, each with the oracle's full OpenMP team: its matrix products and Householder
        # sweeps scale with the cores (one thread each was tried and is several times slower on 1B-shaped blocks)
        self.pool = ThreadPoolExecutor(max_workers=workers or 3)
        self.futures = []

    def submit(self, U, V, G64, Om64, r, q, gap, tol_sub=TOL_SUBSPACE):
        self.futures.append(self.pool.submit(check_refresh_uv, U, V, G64, Om64, r, q, gap, tol_sub))

    def join(self):
        try:
            for f in self.futures:
                f.result()
        finally:
            self.pool.shutdown(wait=True)


def check_refresh_invariants(U, V, G64, r):
    """The part of the refresh check that needs no oracle: orthonormal bases, and U^T G V diagonal, non-negative and
    descending.  Returns (orthonormality, off-diagonal / sigma_1)."""
    ortho = max(np.linalg.norm(U.T @ U - np.eye(r)), np.linalg.norm(V.T @ V - np.eye(r)))
    assert ortho < TOL_ORTHO, ortho
    core = U.T @ G64 @ V
    d = np.diag(core)
    offdiag = float(np.abs(core - np.diag(d)).max() / d[0])
    assert offdiag < TOL_OFFDIAG, offdiag
    assert np.all(d > 0) and np.all(np.diff(d) < 1e-5 * d[0])
    return float(ortho), offdiag


REFRESH_MEASURED = []   # one record per check_refresh call, printed by the tests that want a table


def check_refresh(plan, i, G64, Om64, r, q, gap, tol_sub=TOL_SUBSPACE):
    """Invariants and subspace agreement of block i's refreshed bases against the oracle's refresh
    of the same (G, Omega) bits.  Returns the oracle's (U, V, sigma)."""
    return check_refresh_uv(to64(plan.U[i]), to64(plan.V[i]), G64, Om64, r, q, gap, tol_sub)


def check_refresh_uv(U, V, G64, Om64, r, q, gap, tol_sub=TOL_SUBSPACE):
    """check_refresh for bases given as FP64 arrays (a snapshot: the plan's may have moved on)."""
    import time
    t_start = time.perf_counter()
    ortho = max(np.linalg.norm(U.T @ U - np.eye(r)), np.linalg.norm(V.T @ V - np.eye(r)))
    assert ortho < TOL_ORTHO, ortho
    Uo, Vo, sig = oracle.rsvd_refresh(G64, Om64, r, q)
    core = U.T @ G64 @ V
    d = np.diag(core)
    # U^T G V is diag(sigma), descending and non-negative, up to rounding relative to sigma_1
    offdiag = float(np.abs(core - np.diag(d)).max() / sig[0])
    assert offdiag < TOL_OFFDIAG, offdiag
    assert np.all(d > -1e-3 * sig[0])
    assert np.all(np.diff(d) < 1e-5 * sig[0])           # descending
    lead = float(np.abs(d[:gap] / sig[:gap] - 1).max())
    assert lead < 1e-3, lead
    # energy captured
    energy = float(abs(np.linalg.norm(core) / np.linalg.norm(Uo.T @ G64 @ Vo) - 1))
    assert energy < 1e-4, energy
    # leading `gap` directions agree
    pu = float(np.linalg.norm(proj(U[:, :gap]) - proj(Uo[:, :gap])))
    pv = float(np.linalg.norm(proj(V[:, :gap]) - proj(Vo[:, :gap])))
    assert pu < tol_sub and pv < tol_sub, (pu, pv)
    REFRESH_MEASURED.append(dict(m=G64.shape[0], n=G64.shape[1], r=r, ortho=float(ortho), offdiag=offdiag, lead=lead,
                                 energy=energy, proj=max(pu, pv), seconds=time.perf_counter() - t_start))
    return Uo, Vo, sig


def f32(x: float) -> float:
    """The value an FP32 field of tsr_hyper holds for x, widened exactly to FP64 (the oracle is
    given the same bits the library receives)."""
    return float(np.float32(x))


HYPER = dict(lr=f32(1e-3), beta1=f32(0.9), beta2=f32(0.999), eps=f32(1e-8))


def update_err(w_gpu_before, w_gpu_after, w_ref_before, w_ref_after):
    """Error of one step's update W_t - W_{t-1} of the library against the reference's, relative to the reference's
    update (FP64 arrays).  The weights dwarf one step's update, so a gate on W alone cannot see a wrong update."""
    d_ref = w_ref_after - w_ref_before
    return float(np.linalg.norm((w_gpu_after - w_gpu_before) - d_ref) / np.linalg.norm(d_ref))


def update_bound(bf16, first_adam_step=False, after_refresh=False):
    """Bound on update_err.  BF16 path: the tolerance of the core (2e-2) from the second step on, 0.25 on the first Adam
    step (D = sign(C): every sign the operand rounding flips costs 2; measured 0.05 .. 0.153, the largest on a 32 x 32 core), three times the tolerance
    from an in-loop refresh on (moments of the old basis amplify the rounding of the new core; measured up to 0.037).
    FP32 path: 1e-2 throughout (measured 2e-5 .. 2e-4)."""
    if not bf16:
        return 100 * TOL_F32
    if first_adam_step:
        return 0.25
    return 3 * TOL_BF16 if after_refresh else TOL_BF16
