"""Pins for the FP64 CPU oracle: each check ties an oracle routine to something that does
not come from the oracle itself -- a library routine (torch.optim.AdamW, numpy.linalg),
an exact identity, a closed form, a brute-force result, or a number the paper prints."""
import os

import numpy as np
import pytest
import torch

import oracle
import tsr_inputs as ti

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_bytes_tables.txt")


def _rand_orth(m, r, seed):
    return np.linalg.qr(np.random.default_rng(seed).standard_normal((m, r)))[0]


def _lowrank(m, n, rank, seed, noise=0.0, decay=True):
    rng = np.random.default_rng(seed)
    a, b = rng.standard_normal((m, rank)), rng.standard_normal((n, rank))
    s = 1.0 / np.arange(1, rank + 1) if decay else np.ones(rank)
    g = (a * s) @ b.T
    if noise:
        g = g + noise * rng.standard_normal((m, n))
    return g


def _proj(X):
    return X @ X.T


# ---- Algorithm 1 with U = I, V = I is textbook AdamW (library routine) -------------------
@pytest.mark.parametrize("wd,scale", [(0.0, 1.0), (0.1, 1.0)])
def test_identity_bases_reduce_to_torch_adamw(wd, scale):
    n = 12
    rng = np.random.default_rng(1)
    W0 = rng.standard_normal((n, n)) * 0.02
    blk = oracle.OracleBlock(W0, r=n, p=0, q=0, K=0)
    blk.set_bases(np.eye(n), np.eye(n))
    w = torch.tensor(W0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([w], lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
    for t in range(10):
        G = rng.standard_normal((n, n))
        blk.step(G, lr=1e-2, weight_decay=wd, scale=scale)
        w.grad = torch.tensor(G, dtype=torch.float64)
        opt.step()
        assert np.abs(blk.W - w.detach().numpy()).max() < 1e-14
    assert blk.t == 11


# ---- the one-sided arm (Table 1) with U = I is the same textbook AdamW; rectangular on purpose
@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_one_sided_arm_with_identity_basis_reduces_to_torch_adamw(wd):
    m, n = 7, 12
    rng = np.random.default_rng(21)
    W = rng.standard_normal((m, n)) * 0.02
    M, Vm = np.zeros((m, n)), np.zeros((m, n))
    w = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([w], lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
    for t in range(1, 9):
        G = rng.standard_normal((m, n))
        C = oracle.project_one_sided(G, np.eye(m))
        D = oracle.adam_core(C, M, Vm, 0.9, 0.999, 1e-8, t)
        oracle.backproject_one_sided(np.eye(m), D, W, lr=1e-2, weight_decay=wd)
        w.grad = torch.tensor(G, dtype=torch.float64)
        opt.step()
        assert np.abs(W - w.detach().numpy()).max() < 1e-14


def test_one_sided_lift_invariants_and_closed_form():
    m, n, r = 30, 44, 6
    U = _rand_orth(m, r, 31)
    rng = np.random.default_rng(32)
    D = rng.standard_normal((r, n))
    W0 = rng.standard_normal((m, n))
    W = np.zeros((m, n))
    oracle.backproject_one_sided(U, D, W, lr=1.0)               # W = -U D
    assert np.abs(U.T @ (-W) - D).max() < 1e-12                  # U^T dW = D
    assert np.abs(U @ U.T @ W - W).max() < 1e-12                 # dW lives in range(U)
    W = W0.copy()
    oracle.backproject_one_sided(U, D, W, lr=0.3, weight_decay=0.2, scale=0.5)
    assert np.allclose(W, (1 - 0.3 * 0.2) * W0 - 0.3 * 0.5 * (U @ D), atol=1e-13)
    # a two-sided step whose right basis spans everything is the one-sided step: V = I_n needs the
    # square core D V^T = D, which the two-sided routine takes when r = n
    Usq = _rand_orth(n, n, 33)
    Dsq = rng.standard_normal((n, n))
    Wa, Wb = rng.standard_normal((n, n)), None
    Wb = Wa.copy()
    oracle.backproject_apply(Usq, Dsq, np.eye(n), Wa, lr=0.1, weight_decay=0.05, scale=2.0)
    oracle.backproject_one_sided(Usq, Dsq, Wb, lr=0.1, weight_decay=0.05, scale=2.0)
    assert np.abs(Wa - Wb).max() < 1e-12


def test_scale_multiplies_lifted_update_only():
    # with U = V = I the step is W - lr*(scale*D + wd*W); check against AdamW run with lr*scale
    # for the update part and decoupled decay lr*wd for the decay part (t = 1, closed form).
    n = 6
    rng = np.random.default_rng(2)
    W0 = rng.standard_normal((n, n))
    G = rng.standard_normal((n, n))
    blk = oracle.OracleBlock(W0, r=n, p=0, q=0, K=0)
    blk.set_bases(np.eye(n), np.eye(n))
    blk.step(G, lr=0.1, eps=0.0, weight_decay=0.5, scale=0.25)
    # at t = 1 with eps = 0, D = sign(G)
    expect = W0 - 0.1 * (0.25 * np.sign(G) + 0.5 * W0)
    assert np.abs(blk.W - expect).max() < 1e-14


def test_dense_adamw_matches_torch_adamw():
    rng = np.random.default_rng(12)
    p0 = rng.standard_normal(257)
    P, M, Vm = p0.copy(), np.zeros(257), np.zeros(257)
    w = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([w], lr=3e-3, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.1)
    for t in range(1, 9):
        g = rng.standard_normal(257)
        oracle.dense_adamw(P, g, M, Vm, 3e-3, 0.9, 0.95, 1e-8, 0.1, t)
        w.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        assert np.abs(P - w.detach().numpy()).max() < 1e-14


# ---- core Adam: closed forms ------------------------------------------------------------
def test_adam_constant_core_closed_form():
    # constant core c: m_t = (1-b1^t)c, v_t = (1-b2^t)c^2  =>  D = c / (|c| + eps) at every t
    C = np.array([[0.5, -2.0], [1e-3, 7.0]])
    M, Vm = np.zeros((2, 2)), np.zeros((2, 2))
    for t in range(1, 8):
        D = oracle.adam_core(C, M, Vm, 0.9, 0.999, 1e-8, t)
        assert np.allclose(M, (1 - 0.9 ** t) * C, rtol=1e-13, atol=0)
        assert np.allclose(Vm, (1 - 0.999 ** t) * C * C, rtol=1e-12, atol=0)
        assert np.allclose(D, C / (np.abs(C) + 1e-8), rtol=1e-12, atol=0)


def test_adam_first_step_and_scale_invariance():
    rng = np.random.default_rng(3)
    C = rng.standard_normal((5, 5))
    D1 = oracle.adam_core(C, np.zeros((5, 5)), np.zeros((5, 5)), 0.9, 0.999, 1e-8, 1)
    assert np.allclose(D1, C / (np.abs(C) + 1e-8), rtol=1e-12)
    # G -> cG leaves D unchanged when eps = 0
    Ma, Va, Mb, Vb = (np.zeros((5, 5)) for _ in range(4))
    for t in range(1, 5):
        Ct = rng.standard_normal((5, 5))
        Da = oracle.adam_core(Ct, Ma, Va, 0.9, 0.999, 0.0, t)
        Db = oracle.adam_core(37.0 * Ct, Mb, Vb, 0.9, 0.999, 0.0, t)
        assert np.allclose(Da, Db, rtol=1e-12)


def test_adam_moments_match_unrolled_ema_sum():
    # m_T = (1-b1) sum_s b1^(T-s) C_s ; v_T likewise with squares (geometric-sum closed form)
    rng = np.random.default_rng(4)
    Cs = [rng.standard_normal((3, 3)) for _ in range(9)]
    M, Vm = np.zeros((3, 3)), np.zeros((3, 3))
    for t, C in enumerate(Cs, 1):
        oracle.adam_core(C, M, Vm, 0.8, 0.95, 1e-8, t)
    T = len(Cs)
    m_ref = sum((1 - 0.8) * 0.8 ** (T - s) * Cs[s - 1] for s in range(1, T + 1))
    v_ref = sum((1 - 0.95) * 0.95 ** (T - s) * Cs[s - 1] ** 2 for s in range(1, T + 1))
    assert np.allclose(M, m_ref, rtol=1e-12) and np.allclose(Vm, v_ref, rtol=1e-12)


def test_sgd_variant_identity_bases_is_momentum_sgd():
    # Algorithm 2 with U = V = I: torch SGD with momentum b and dampening b gives
    # buf <- b*buf + (1-b)*g from the second step on; its first step uses buf = g, so compare
    # against the EMA recursion started from zero through the closed-form sum instead.
    n = 5
    rng = np.random.default_rng(5)
    W0 = rng.standard_normal((n, n))
    blk = oracle.OracleBlock(W0, r=n, p=0, q=0, K=0, sgd=True)
    blk.set_bases(np.eye(n), np.eye(n))
    Gs = [rng.standard_normal((n, n)) for _ in range(6)]
    W = W0.copy()
    for T, G in enumerate(Gs, 1):
        blk.step(G, lr=0.05, beta1=0.9)
        m_T = sum(0.1 * 0.9 ** (T - s) * Gs[s - 1] for s in range(1, T + 1))
        W = W - 0.05 * m_T
        assert np.abs(blk.W - W).max() < 1e-14


# ---- projection / lift: exact identities -------------------------------------------------
def test_project_recovers_core_exactly():
    m, n, r = 40, 56, 7
    U, V = _rand_orth(m, r, 11), _rand_orth(n, r, 12)
    C0 = np.random.default_rng(6).standard_normal((r, r))
    G = U @ C0 @ V.T
    assert np.abs(oracle.project_core(G, U, V) - C0).max() < 1e-12


def test_project_matches_numpy_and_is_not_transposed():
    m, n, r = 23, 31, 5
    rng = np.random.default_rng(7)
    G, U, V = rng.standard_normal((m, n)), rng.standard_normal((m, r)), rng.standard_normal((n, r))
    assert np.allclose(oracle.project_core(G, U, V), U.T @ G @ V, rtol=1e-12, atol=1e-12)
    assert np.allclose(oracle.project_one_sided(G, U), U.T @ G, rtol=1e-12, atol=1e-12)


def test_lift_invariants():
    m, n, r = 30, 44, 6
    U, V = _rand_orth(m, r, 13), _rand_orth(n, r, 14)
    D = np.random.default_rng(8).standard_normal((r, r))
    W = np.zeros((m, n))
    oracle.backproject_apply(U, D, V, W, lr=1.0)          # W = -U D V^T
    dW = -W
    assert np.abs(U.T @ dW @ V - D).max() < 1e-12            # U^T dW V = D
    assert np.abs(U @ U.T @ dW @ V @ V.T - dW).max() < 1e-12  # dW lives in the two subspaces
    assert np.allclose(dW, U @ D @ V.T, atol=1e-13)


def test_apply_decoupled_weight_decay_closed_form():
    m, n, r = 9, 11, 3
    rng = np.random.default_rng(9)
    U, V, D = rng.standard_normal((m, r)), rng.standard_normal((n, r)), rng.standard_normal((r, r))
    W0 = rng.standard_normal((m, n))
    W = W0.copy()
    oracle.backproject_apply(U, D, V, W, lr=0.3, weight_decay=0.2, scale=0.5)
    assert np.allclose(W, (1 - 0.3 * 0.2) * W0 - 0.3 * 0.5 * (U @ D @ V.T), atol=1e-13)


def test_metamorphic_sign_flip_and_permutation():
    # flipping column j of U together with row j of the moments, or permuting columns of U with
    # rows of the moments, must leave the weight trajectory unchanged
    m, n, r = 20, 26, 4
    rng = np.random.default_rng(10)
    U, V = _rand_orth(m, r, 15), _rand_orth(n, r, 16)
    W0 = rng.standard_normal((m, n)) * 0.02
    Gs = [rng.standard_normal((m, n)) for _ in range(4)]
    perm = np.array([2, 0, 3, 1])
    sgn = np.array([1.0, -1.0, 1.0, -1.0])
    a = oracle.OracleBlock(W0, r, 0, 0, 0)
    b = oracle.OracleBlock(W0, r, 0, 0, 0)
    a.set_bases(U, V)
    b.set_bases(U[:, perm] * sgn, V)
    for G in Gs:
        a.step(G, lr=1e-2)
        b.step(G, lr=1e-2)
    assert np.abs(a.W - b.W).max() < 1e-13
    assert np.allclose(b.M, (a.M[perm, :].T * sgn).T, atol=1e-14)


# ---- orth and the small SVD against numpy.linalg -----------------------------------------
def test_orth_matches_numpy_qr_up_to_signs():
    rng = np.random.default_rng(20)
    Y = rng.standard_normal((60, 9))
    Q, R = oracle.orth(Y, return_r=True)
    Qn, Rn = np.linalg.qr(Y)
    s = np.sign(np.sum(Q * Qn, axis=0))
    assert np.abs(Q - Qn * s).max() < 1e-12
    assert np.abs(R - (Rn.T * s).T).max() < 1e-12
    assert np.abs(Q @ R - Y).max() < 1e-12
    assert np.abs(np.tril(R, -1)).max() == 0.0


def test_orth_rank_deficient_still_orthonormal_and_spans_range():
    rng = np.random.default_rng(21)
    Y = rng.standard_normal((40, 3)) @ rng.standard_normal((3, 8))    # rank 3, 8 columns
    Y[:, 5] = 0.0
    Q = oracle.orth(Y)
    assert np.abs(Q.T @ Q - np.eye(8)).max() < 1e-12
    assert np.abs(_proj(Q) @ Y - Y).max() < 1e-10


def test_svd_jacobi_matches_numpy_svd():
    rng = np.random.default_rng(22)
    B = rng.standard_normal((10, 37)) * np.logspace(0, -6, 10)[:, None]
    Ut, S, Vt = oracle.svd_jacobi(B)
    Sn = np.linalg.svd(B, compute_uv=False)
    assert np.all(np.diff(S) <= 0) and np.all(S >= 0)
    assert np.abs(S / Sn - 1).max() < 1e-12
    assert np.abs(Ut @ np.diag(S) @ Vt.T - B).max() < 1e-12
    assert np.abs(Ut.T @ Ut - np.eye(10)).max() < 1e-12
    assert np.abs(Vt.T @ Vt - np.eye(10)).max() < 1e-12


def test_svd_jacobi_rank_deficient_completes_basis():
    rng = np.random.default_rng(23)
    B = rng.standard_normal((6, 2)) @ rng.standard_normal((2, 15))
    Ut, S, Vt = oracle.svd_jacobi(B)
    assert S[2] < 1e-12 * S[0]
    assert np.abs(Vt.T @ Vt - np.eye(6)).max() < 1e-10
    assert np.abs(Ut.T @ Ut - np.eye(6)).max() < 1e-12
    assert np.abs(Ut @ np.diag(S) @ Vt.T - B).max() < 1e-12


# ---- refresh: invariants, brute force, exact-rank recovery ------------------------------
def test_refresh_invariants_and_interlacing():
    m, n, r, p, q = 48, 72, 10, 4, 1
    G = _lowrank(m, n, 6, 30, noise=1e-3)
    Om = np.random.default_rng(31).standard_normal((n, r + p))
    U, V, sig = oracle.rsvd_refresh(G, Om, r, q)
    assert np.abs(U.T @ U - np.eye(r)).max() < 1e-12
    assert np.abs(V.T @ V - np.eye(r)).max() < 1e-12
    core = U.T @ G @ V
    assert np.abs(core - np.diag(sig[:r])).max() < 1e-10         # U^T G V = diag(sigma(B))
    assert np.all(np.diff(sig) <= 1e-15) and np.all(sig >= 0)
    sG = np.linalg.svd(G, compute_uv=False)
    assert np.all(sig <= sG[: r + p] * (1 + 1e-12))              # sigma_i(B) <= sigma_i(G)
    # leading 6 directions (the gap) agree with the exact SVD
    Un, _, Vnt = np.linalg.svd(G)
    assert np.linalg.norm(_proj(U[:, :6]) - _proj(Un[:, :6])) < 1e-5
    assert np.linalg.norm(_proj(V[:, :6]) - _proj(Vnt.T[:, :6])) < 1e-5


def test_refresh_recovers_exact_rank_r_subspace():
    m, n, r, p = 40, 52, 8, 4
    for rho in (8, 5):                                            # rank = r and rank < r
        G = _lowrank(m, n, rho, 32 + rho, noise=0.0)
        Om = np.random.default_rng(33).standard_normal((n, r + p))
        U, V, sig = oracle.rsvd_refresh(G, Om, r, 1)
        assert np.abs(U.T @ U - np.eye(r)).max() < 1e-10
        assert np.abs(V.T @ V - np.eye(r)).max() < 1e-10
        assert np.abs(_proj(U) @ G @ _proj(V) - G).max() < 1e-10 * np.abs(G).max()
        Un, sn, Vnt = np.linalg.svd(G)
        assert np.linalg.norm(_proj(U[:, :rho]) - _proj(Un[:, :rho])) < 1e-8
        assert np.linalg.norm(_proj(V[:, :rho]) - _proj(Vnt.T[:, :rho])) < 1e-8
        assert np.abs(sig[:rho] / sn[:rho] - 1).max() < 1e-10


@pytest.mark.parametrize("m,n", [(12, 20), (24, 16), (9, 9)])
def test_refresh_with_full_sketch_is_dense_svd(m, n):
    # k = min(m, n): the sketch spans everything, so rSVD must equal the brute-force SVD
    k = min(m, n)
    r = k - 2
    rng = np.random.default_rng(40 + m)
    G = rng.standard_normal((m, n)) * 1.0
    Om = rng.standard_normal((n, k))
    U, V, sig = oracle.rsvd_refresh(G, Om, r, 2)
    Un, sn, Vnt = np.linalg.svd(G)
    assert np.abs(sig / sn[:k] - 1).max() < 1e-10
    for j in range(r):       # singular values are distinct here: vectors agree up to a joint sign
        s = np.sign(U[:, j] @ Un[:, j])
        assert np.abs(U[:, j] - s * Un[:, j]).max() < 1e-8
        assert np.abs(V[:, j] - s * Vnt[j, :]).max() < 1e-8


def test_exact_svd_refresh_matches_numpy():
    for (m, n) in ((14, 22), (22, 14)):
        G = np.random.default_rng(50 + m).standard_normal((m, n))
        U, V, sig = oracle.exact_svd_refresh(G, 4)
        Un, sn, Vnt = np.linalg.svd(G)
        assert np.abs(sig / sn - 1).max() < 1e-12
        assert np.linalg.norm(_proj(U) - _proj(Un[:, :4])) < 1e-9
        assert np.linalg.norm(_proj(V) - _proj(Vnt.T[:, :4])) < 1e-9
        assert np.abs(np.diag(U.T @ G @ V) - sn[:4]).max() < 1e-10


def test_refresh_on_config_generator_finds_signal_subspace():
    # the benchmark's gradient recipe at a reduced size: 16 signal directions, r = 32
    g = ti.gradient(96, 160, ti.seed_for(0, 0, 0, ti.ROLE_INIT_GRAD), signal_rank=16).double().numpy()
    Om = ti.omega(160, 40, ti.seed_for(0, 0, 0, ti.ROLE_INIT_OMEGA)).double().numpy()
    U, V, sig = oracle.rsvd_refresh(g, Om, 32, 1)
    Un, sn, Vnt = np.linalg.svd(g)
    assert np.linalg.norm(_proj(U[:, :16]) - _proj(Un[:, :16])) < 1e-5
    assert np.linalg.norm(_proj(V[:, :16]) - _proj(Vnt.T[:, :16])) < 1e-5
    assert np.abs(sig[:16] / sn[:16] - 1).max() < 1e-8


def test_step_refreshes_before_projecting_and_keeps_moments():
    # refresh is due when t mod K == 0, runs before the projection of the same gradient, and
    # leaves m, v untouched: after the refresh step the core of that step is diag(sigma)
    m, n, r, p, K = 30, 36, 5, 3, 3
    rng = np.random.default_rng(60)
    blk = oracle.OracleBlock(rng.standard_normal((m, n)) * 0.02, r, p, 1, K)
    blk.init_subspace(_lowrank(m, n, 4, 61, 1e-3), rng.standard_normal((n, r + p)))
    for t in (1, 2):
        assert not blk.refresh_due()
        blk.step(_lowrank(m, n, 4, 62 + t, 1e-3), lr=1e-3)
    M_before = blk.M.copy()
    assert blk.refresh_due() and blk.t == 3
    G3 = _lowrank(m, n, 4, 70, 1e-3)
    blk.step(G3, lr=1e-3, Omega=rng.standard_normal((n, r + p)))
    assert np.abs(blk.C - np.diag(np.diag(blk.C))).max() < 1e-10 * np.abs(blk.C).max()
    assert np.allclose(blk.M, 0.9 * M_before + 0.1 * blk.C, atol=1e-14)


def test_moment_reexpression_is_the_double_projection():
    m, n, r = 18, 25, 4
    rng = np.random.default_rng(70)
    Uo, Vo, Un, Vn = _rand_orth(m, r, 71), _rand_orth(n, r, 72), _rand_orth(m, r, 73), _rand_orth(n, r, 74)
    M0 = rng.standard_normal((r, r))
    M = M0.copy()
    oracle.reexpress_moment(M, Uo, Vo, Un, Vn)
    lifted_old = Uo @ M0 @ Vo.T
    # the new lifted moment is the old one projected onto the new subspaces from both sides
    assert np.abs(Un @ M @ Vn.T - _proj(Un) @ lifted_old @ _proj(Vn)).max() < 1e-13
    # unchanged subspaces, rotated bases: M' = Ru^T M Rv; identical bases: M' = M
    Ru, Rv = _rand_orth(r, r, 75), _rand_orth(r, r, 76)
    M = M0.copy()
    oracle.reexpress_moment(M, Uo, Vo, Uo @ Ru, Vo @ Rv)
    assert np.abs(M - Ru.T @ M0 @ Rv).max() < 1e-13
    M = M0.copy()
    oracle.reexpress_moment(M, Uo, Vo, Uo, Vo)
    assert np.abs(M - M0).max() < 1e-13


# ---- byte and state accounting against the numbers the paper prints ---------------------
def _golden_rows():
    rows = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def _blocks(layers, hidden, ffn):
    return [(hidden, hidden)] * (4 * layers) + [(ffn, hidden)] * (2 * layers) + [(hidden, ffn)] * layers


def test_dense_bytes_match_paper_table3():
    for row in _golden_rows():
        if row[0] != "dense":
            continue
        layers, hidden, ffn, vocab = map(int, row[2:6])
        printed = float(row[6])
        elems = sum(m * n for m, n in _blocks(layers, hidden, ffn)) + vocab * hidden
        assert round(4 * elems / 1e9, 2) == printed


def test_tsr_peak_and_core_bytes_against_paper_tables():
    for row in _golden_rows():
        if row[0] != "tsr":
            continue
        layers, hidden, ffn, vocab, r, r_emb = map(int, row[2:8])
        per_step, peak = float(row[8]), float(row[9])
        blocks = _blocks(layers, hidden, ffn)
        core = sum(oracle.core_bytes(r, 4) for _ in blocks) + oracle.core_bytes(r_emb, 4)
        sketch = sum(oracle.sketch_bytes(m, n, r, 0, 4) for m, n in blocks) + oracle.sketch_bytes(vocab, hidden, r_emb, 0, 4)
        assert abs((core + sketch) / 1e9 / peak - 1) < 0.08       # the paper's oversampling is not stated
        assert core / 1e9 <= per_step                             # printed average also carries refresh traffic


def test_state_elems_formula_table2():
    # Table 2: a linear layer keeps U (m r), V (n r) and two r x r moments
    assert oracle.state_elems(512, 1376, 128) == 512 * 128 + 1376 * 128 + 2 * 128 * 128
    assert oracle.state_elems(32000, 512, 64) == 32000 * 64 + 64 * 512 + 2 * 64 * 64
    assert oracle.core_bytes(128, 4) == 128 * 128 * 4
    assert oracle.sketch_bytes(512, 1376, 128, 8, 4) == 136 * (512 + 1376) * 4


def test_workload_shapes_and_seeds():
    w = ti.workload(4)
    assert len(w.blocks) == 169 and w.blocks[-1].is_embedding and w.blocks[-1].r == 256
    assert sum(b.m * b.n for b in w.blocks) == 1273446400
    assert ti.seed_for(1, 2, 3, 0) != ti.seed_for(1, 2, 4, 0)
    a = ti.gradient(32, 48, 5, torch.bfloat16)
    b = ti.gradient(32, 48, 5, torch.bfloat16)
    assert torch.equal(a, b)
    assert ti.padded_ld(5461, 2) == 5464 and ti.padded_ld(5461, 4) == 5464 and ti.padded_ld(512, 2) == 512
