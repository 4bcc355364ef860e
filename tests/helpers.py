"""Shared helpers for the GPU parity tests (CUDA library vs the FP64 CPU oracle)."""
import numpy as np
import torch

import oracle
import tsr_inputs as ti

TOL_F32 = 1e-4      # max relative Frobenius error, FP32-gradient path
TOL_BF16 = 2e-2     # max relative Frobenius error, BF16-gradient path
TOL_SUBSPACE = 1e-3  # || P - P' ||_F of projectors at a spectral gap
TOL_ORTHO = 1e-4    # || U^T U - I ||_F after a refresh


def to64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def rel_fro(a, b) -> float:
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (den if den > 0 else 1.0))


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


def check_refresh(plan, i, G64, Om64, r, q, gap, tol_sub=TOL_SUBSPACE):
    """Invariants and subspace agreement of block i's refreshed bases against the oracle's refresh
    of the same (G, Omega) bits.  Returns the oracle's (U, V, sigma)."""
    U, V = to64(plan.U[i]), to64(plan.V[i])
    assert np.linalg.norm(U.T @ U - np.eye(r)) < TOL_ORTHO
    assert np.linalg.norm(V.T @ V - np.eye(r)) < TOL_ORTHO
    Uo, Vo, sig = oracle.rsvd_refresh(G64, Om64, r, q)
    core = U.T @ G64 @ V
    d = np.diag(core)
    # U^T G V is diag(sigma), descending and non-negative, up to rounding relative to sigma_1
    assert np.abs(core - np.diag(d)).max() < 2e-3 * sig[0]
    assert np.all(d > -1e-3 * sig[0])
    assert np.abs(d[:gap] / sig[:gap] - 1).max() < 1e-3
    # energy captured
    assert abs(np.linalg.norm(core) / np.linalg.norm(Uo.T @ G64 @ Vo) - 1) < 1e-4
    # leading `gap` directions agree
    assert np.linalg.norm(proj(U[:, :gap]) - proj(Uo[:, :gap])) < tol_sub
    assert np.linalg.norm(proj(V[:, :gap]) - proj(Vo[:, :gap])) < tol_sub
    return Uo, Vo, sig


def f32(x: float) -> float:
    """The value an FP32 field of tsr_hyper holds for x, widened exactly to FP64 (the oracle is
    given the same bits the library receives)."""
    return float(np.float32(x))


HYPER = dict(lr=f32(1e-3), beta1=f32(0.9), beta2=f32(0.999), eps=f32(1e-8))
