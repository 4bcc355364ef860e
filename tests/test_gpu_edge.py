"""Edge and degenerate cases of the CUDA path: tiny and extreme shapes, q = 0 / p = 0, exactly
rank-deficient and non-finite gradients (flagged per block, never a fault), run-to-run
determinism and checkpoint / resume."""
import numpy as np
import pytest
import torch

import oracle
import tsr_inputs as ti
from helpers import HYPER, TOL_BF16, TOL_F32, check_refresh, fill_gradient, fill_weights, proj, rel_fro, set_bases, to64

pytestmark = pytest.mark.gpu


def _tsr():
    import paper_2602_08007_b200 as tsr
    return tsr


@pytest.mark.parametrize("dtype,shape,gap", [
    (torch.float32, dict(m=24, n=17, r=5, p=2, q=1), 3),        # tiny, nothing a multiple of any tile
    (torch.bfloat16, dict(m=64, n=48, r=8, p=0, q=0), 4),       # no oversampling, no power iteration
    (torch.bfloat16, dict(m=40, n=136, r=32, p=8, q=1), 8),     # k = min(m, n): the sketch spans everything
    (torch.float32, dict(m=150, n=90, r=30, p=6, q=3), 12),     # three power iterations
    (torch.bfloat16, dict(m=320, n=304, r=250, p=5, q=1), 16),  # odd k = 255: tridiagonal eigen-solver, no TMA row products
    (torch.bfloat16, dict(m=640, n=704, r=560, p=8, q=1), 16),  # k = 568: the wide variants of the eigenvector kernels
])
def test_refresh_small_and_extreme_shapes(dtype, shape, gap):
    tsr = _tsr()
    plan = tsr.Plan([shape], g_dtype=dtype)
    G64 = fill_gradient(plan, 0, 31, signal_rank=gap)
    Om = ti.omega(shape["n"], shape["r"] + shape["p"], 32).cuda()
    plan.init_subspace(omegas=[Om])
    torch.cuda.synchronize()
    assert plan.poll_status() == [0]
    tol_sub = 1e-3 if shape["q"] > 0 else 2e-2     # without a power iteration the sketch itself is less accurate
    check_refresh(plan, 0, G64, to64(Om), shape["r"], shape["q"], gap, tol_sub=tol_sub)


@pytest.mark.parametrize("dtype,shape", [
    (torch.float32, dict(m=200, n=176, r=32)),
    (torch.bfloat16, dict(m=288, n=320, r=48)),
])
def test_exact_svd_arm_matches_the_dense_svd(dtype, shape):
    """The exact-SVD refresh arm of the ablation (Section 3.5 names it as the costly alternative the
    randomized refresh replaces) is the same refresh with a sketch as wide as the matrix is small
    (k = min(m, n), no power iteration): the sketch then spans the whole range of G, B = Q^T G loses
    nothing, and U, V are the leading singular vectors of G itself.  Checked against the oracle's
    dense SVD of G: singular values, and the projectors on the signal directions."""
    tsr = _tsr()
    r = shape["r"]
    k = min(shape["m"], shape["n"])
    full = dict(shape, p=k - r, q=0)
    plan = tsr.Plan([full], g_dtype=dtype)
    G64 = fill_gradient(plan, 0, 57, signal_rank=r)
    Om = ti.omega(shape["n"], k, 58).cuda()
    plan.init_subspace(omegas=[Om])
    torch.cuda.synchronize()
    assert plan.poll_status() == [0]
    Ue, Ve, Se = oracle.exact_svd_refresh(G64, r)
    U, V = to64(plan.U[0]), to64(plan.V[0])
    core = U.T @ G64 @ V
    assert np.abs(np.diag(core) / Se[:r] - 1).max() < 1e-4
    assert np.abs(core - np.diag(np.diag(core))).max() < 1e-4 * Se[0]
    assert np.linalg.norm(proj(U) - proj(Ue)) < 1e-3
    assert np.linalg.norm(proj(V) - proj(Ve)) < 1e-3
    assert np.linalg.norm(U.T @ U - np.eye(r)) < 1e-4 and np.linalg.norm(V.T @ V - np.eye(r)) < 1e-4


def test_refresh_with_repeated_singular_values():
    """Groups of equal singular values and a flat tail: the Gram matrix of the sketch has repeated
    eigenvalues, which the divide-and-conquer eigen-solver must deflate (rotations between nearly
    equal poles, negligible components of the rank-one vector).  Any orthonormal basis of an
    eigenspace is correct, so the check is on orthonormality, the diagonal core, the singular values
    and the projector at the boundary between distinct groups."""
    tsr = _tsr()
    shape = dict(m=320, n=288, r=250, p=6, q=1)
    rng = np.random.default_rng(11)
    A, _ = np.linalg.qr(rng.standard_normal((shape["m"], 64)))
    B, _ = np.linalg.qr(rng.standard_normal((shape["n"], 64)))
    sig = np.array([10.0] * 4 + [7.0] * 4 + [5.0] * 8 + [1e-2] * 48)
    G = torch.from_numpy((A * sig) @ B.T).float()
    plan = tsr.Plan([shape], g_dtype=torch.float32)
    plan.G[0].copy_(G.cuda())
    Om = ti.omega(shape["n"], shape["r"] + shape["p"], 77).cuda()
    plan.init_subspace(omegas=[Om])
    torch.cuda.synchronize()
    # the gradient has rank 64 < k: the sketch is rank deficient by construction and is flagged as such
    assert plan.poll_status()[0] in (0, 8)
    U, V = to64(plan.U[0]), to64(plan.V[0])
    G64 = to64(G)
    core = U.T @ G64 @ V
    d = np.diag(core)
    assert np.abs(core - np.diag(d)).max() < 2e-3 * sig[0]
    assert np.abs(d[:16] / sig[:16] - 1).max() < 1e-4
    for cols in (4, 8, 16):                       # boundaries between the groups of equal values
        assert np.linalg.norm(proj(U[:, :cols]) - proj(A[:, :cols])) < 1e-3
        assert np.linalg.norm(proj(V[:, :cols]) - proj(B[:, :cols])) < 1e-3
    lead = 64                                     # directions that carry any signal stay orthonormal
    assert np.linalg.norm(U[:, :lead].T @ U[:, :lead] - np.eye(lead)) < 1e-4
    assert np.linalg.norm(V[:, :lead].T @ V[:, :lead] - np.eye(lead)) < 1e-4


def test_tiny_step_matches_oracle():
    tsr = _tsr()
    shapes = [dict(m=9, n=7, r=3), dict(m=33, n=65, r=8)]
    plan = tsr.Plan(shapes, g_dtype=torch.float32)
    blks = []
    for i, s in enumerate(shapes):
        set_bases(plan, i, ti.orthonormal(s["m"], s["r"], 40 + i), ti.orthonormal(s["n"], s["r"], 50 + i))
        W0 = fill_weights(plan, i, 60 + i)
        ob = oracle.OracleBlock(W0, s["r"], 0, 0, 0)
        ob.set_bases(to64(plan.U[i]), to64(plan.V[i]))
        blks.append(ob)
    plan.bases_changed()
    for t in (1, 2, 3):
        G64 = [fill_gradient(plan, i, 70 + 10 * t + i, signal_rank=2) for i in range(2)]
        plan.step(tsr.make_hyper(t))
        torch.cuda.synchronize()
        for i, ob in enumerate(blks):
            ob.step(G64[i], **HYPER)
            assert rel_fro(to64(plan.W[i]), ob.W) < TOL_F32 and rel_fro(to64(plan.C[i]), ob.C) < TOL_F32


def test_exactly_rank_deficient_gradient_is_flagged_not_fatal():
    tsr = _tsr()
    shape = dict(m=256, n=320, r=32, p=8, q=1)
    plan = tsr.Plan([shape, shape], g_dtype=torch.float32)
    # block 0: exact rank 12 < k = 40 (no noise); block 1: an ordinary full-rank gradient
    G0 = fill_gradient(plan, 0, 81, signal_rank=12, noise_std=0.0)
    G1 = fill_gradient(plan, 1, 82, signal_rank=12)
    oms = [ti.omega(320, 40, 83).cuda(), ti.omega(320, 40, 84).cuda()]
    plan.init_subspace(omegas=oms)
    torch.cuda.synchronize()
    st = plan.poll_status()
    assert st[0] == 8 and st[1] == 0                      # TSR_ERR_RANK_DEFICIENT on block 0 only
    U0, V0 = to64(plan.U[0]), to64(plan.V[0])
    assert np.isfinite(U0).all() and np.isfinite(V0).all()
    # the rank-12 range of G is still captured by the leading directions
    Un, sn, Vnt = np.linalg.svd(G0)
    assert np.linalg.norm(proj(U0[:, :12]) - proj(Un[:, :12])) < 1e-3
    assert np.linalg.norm(proj(V0[:, :12]) - proj(Vnt.T[:, :12])) < 1e-3
    check_refresh(plan, 1, G1, to64(oms[1]), 32, 1, 12)   # the healthy block is untouched by its neighbour
    assert plan.poll_status() == [0, 0]                   # polling clears the words


def test_nonfinite_gradient_flags_its_block_only():
    tsr = _tsr()
    shape = dict(m=192, n=256, r=16, p=8, q=1)
    res = []
    for poison in (False, True):
        plan = tsr.Plan([shape, shape], g_dtype=torch.bfloat16)
        for i in range(2):
            fill_gradient(plan, i, 90 + i, signal_rank=8)
            fill_weights(plan, i, 92 + i)
        if poison:
            plan.G[0][5, 7] = float("nan")
        oms = [ti.omega(256, 24, 94).cuda(), ti.omega(256, 24, 95).cuda()]
        plan.init_subspace(omegas=oms)
        plan.step(tsr.make_hyper(1))
        torch.cuda.synchronize()
        st = plan.poll_status()
        res.append((st, plan.W[1].clone(), plan.U[1].clone()))
    assert res[0][0] == [0, 0]
    assert res[1][0][0] == 9 and res[1][0][1] == 0        # TSR_ERR_NONFINITE on the poisoned block only
    assert torch.equal(res[0][1], res[1][1]) and torch.equal(res[0][2], res[1][2])


@pytest.mark.parametrize("shape", [dict(m=192, n=256, r=16, p=8, q=1),       # k = 24: Jacobi solver
                                   dict(m=320, n=384, r=200, p=8, q=1)])     # k = 208: tridiagonal + QL solver
def test_sweep_limit_flags_not_converged_on_that_block_only(shape):
    """The eigen-solver of one block is given a limit of one sweep (one QL iteration per
    eigenvalue): it stops there, the block reads TSR_ERR_NOT_CONVERGED, and its neighbour, whose
    limit is the default, comes out bit for bit as in a run without any limit."""
    tsr = _tsr()
    res = []
    for limited in (False, True):
        plan = tsr.Plan([shape, shape], g_dtype=torch.bfloat16)
        for i in range(2):
            fill_gradient(plan, i, 120 + i, signal_rank=8)
        if limited:
            plan.set_limits(max_sweeps=1, sweep_block=0)
        oms = [ti.omega(shape["n"], shape["r"] + shape["p"], 124 + i).cuda() for i in range(2)]
        plan.init_subspace(omegas=oms)
        torch.cuda.synchronize()
        st = plan.poll_status()
        res.append((st, plan.U[1].clone(), plan.V[1].clone(), plan.U[0].clone()))
        if limited:
            assert torch.isfinite(plan.U[0]).all() and torch.isfinite(plan.V[0]).all()
            # lifting the limit makes the same context converge again
            plan.set_limits()
            plan.rsvd_refresh(omegas=oms)
            torch.cuda.synchronize()
            assert plan.poll_status() == [0, 0]
            assert torch.equal(plan.U[0], res[0][3])
    assert res[0][0] == [0, 0]
    assert res[1][0] == [7, 0]                            # TSR_ERR_NOT_CONVERGED on block 0 only
    assert torch.equal(res[0][1], res[1][1]) and torch.equal(res[0][2], res[1][2])


@pytest.mark.parametrize("launches", [1, 2])
def test_bounded_wait_that_runs_out_reports_timeout_and_the_context_recovers(launches):
    """A wait inside a tensor-core kernel is made to run out in the only safe way: the library is
    told (tsr_set_limits) to issue no loads for the tiles of one block in the first projection
    GEMM and to bound every wait by 2e6 clock ticks (about a millisecond).  Nothing is in flight
    for those tiles and no address is touched; the warps that wait for the data give up at the
    bound, the CTAs release their tensor memory and return, and the block reads TSR_ERR_TIMEOUT.
    The other block finishes normally, and after the switch is cleared the same context steps
    cleanly and matches the oracle."""
    tsr = _tsr()
    shapes = [dict(m=640, n=768, r=64), dict(m=256, n=384, r=64)]     # block 1 is the smaller: its tiles come last
    plan = tsr.Plan(shapes, g_dtype=torch.bfloat16)
    for i, s in enumerate(shapes):
        set_bases(plan, i, ti.orthonormal(s["m"], s["r"], 140 + i), ti.orthonormal(s["n"], s["r"], 150 + i))
    plan.bases_changed()
    with pytest.raises(tsr.TsrError):                     # the switch is refused without a short budget
        plan.set_limits(starve_block=1)
    with pytest.raises(tsr.TsrError) as ei:               # so is a launch mode that does not exist
        plan.set_limits(projection_launches=3)
    assert ei.value.status == 1                           # TSR_ERR_INVALID_ARG
    G64 = [fill_gradient(plan, i, 160 + i) for i in range(2)]
    # (both forms of the projection: one launch with tiles in dynamic order, two plain launches)
    plan.set_limits(wait_clocks=2_000_000, starve_block=1, projection_launches=launches)
    plan.project_core()
    torch.cuda.synchronize()
    assert plan.poll_status() == [0, 10]                  # TSR_ERR_TIMEOUT on the starved block only
    assert rel_fro(to64(plan.C[0]), oracle.project_core(G64[0], to64(plan.U[0]), to64(plan.V[0]))) < TOL_BF16
    # back to the defaults: the same context works as if nothing had happened
    plan.set_limits(projection_launches=launches)
    blks = []
    for i, s in enumerate(shapes):
        W0 = fill_weights(plan, i, 170 + i)
        ob = oracle.OracleBlock(W0, s["r"], 0, 0, 0)
        ob.set_bases(to64(plan.U[i]), to64(plan.V[i]))
        plan.M[i].zero_(); plan.Vm[i].zero_()
        blks.append(ob)
    for t in (1, 2):
        G64 = [fill_gradient(plan, i, 180 + 10 * t + i) for i in range(2)]
        plan.step(tsr.make_hyper(t))
        torch.cuda.synchronize()
        for i, ob in enumerate(blks):
            ob.step(G64[i], **HYPER)
            assert rel_fro(to64(plan.C[i]), ob.C) < TOL_BF16 and rel_fro(to64(plan.W[i]), ob.W) < TOL_BF16
    assert plan.poll_status() == [0, 0]


def test_runs_are_bitwise_reproducible_and_resumable():
    tsr = _tsr()
    w = ti.workload(1)
    shapes = [dict(m=b.m, n=b.n, r=b.r, p=b.p, q=b.q, K=3, is_embedding=b.is_embedding) for b in (w.blocks[0], w.blocks[4], w.blocks[6])]
    shapes.append(dict(m=9000, n=512, r=64, p=8, q=1, K=3, is_embedding=True))     # split-K core GEMM

    def run(steps_a, steps_b):
        plan = tsr.Plan(shapes, g_dtype=torch.bfloat16)
        for i, s in enumerate(shapes):
            fill_gradient(plan, i, 200 + i)
            fill_weights(plan, i, 210 + i)
        plan.init_subspace(seed=11)
        for t in range(1, steps_a + 1):
            for i in range(len(shapes)):
                fill_gradient(plan, i, 1000 * t + i)
            plan.step(tsr.make_hyper(t), seed=11)
        if steps_b:
            # checkpoint: the state is the caller's tensors plus the step counter; resume in a new plan
            torch.cuda.synchronize()
            plan2 = tsr.Plan(shapes, g_dtype=torch.bfloat16)
            for i in range(len(shapes)):
                for a, b in ((plan2.W, plan.W), (plan2.U, plan.U), (plan2.V, plan.V), (plan2.M, plan.M), (plan2.Vm, plan.Vm)):
                    a[i].copy_(b[i])
            plan2.bases_changed()
            plan = plan2
            for t in range(steps_a + 1, steps_a + steps_b + 1):
                for i in range(len(shapes)):
                    fill_gradient(plan, i, 1000 * t + i)
                plan.step(tsr.make_hyper(t), seed=11)
        torch.cuda.synchronize()
        assert plan.poll_status() == [0] * len(shapes)
        return [(plan.W[i].clone(), plan.U[i].clone(), plan.M[i].clone(), plan.Vm[i].clone()) for i in range(len(shapes))]

    a = run(7, 0)
    b = run(7, 0)
    c = run(4, 3)          # refreshes at t = 3 and t = 6 fall on either side of the checkpoint
    for x, y, z in zip(a, b, c):
        for p_, q_, r_ in zip(x, y, z):
            assert torch.equal(p_, q_) and torch.equal(p_, r_)


def test_bind_rejects_bad_arguments_without_touching_buffers():
    tsr = _tsr()
    import ctypes
    plan = tsr.Plan([dict(m=64, n=64, r=8)], g_dtype=torch.bfloat16)
    w_before = plan.W[0].clone()
    L = tsr.lib()
    h = tsr.make_hyper(0)                                  # step must be >= 1
    assert L.tsr_step_grouped(plan.ctx, ctypes.byref(h), 0, 1, None) == 1
    h = tsr.make_hyper(1, beta1=1.5)
    assert L.tsr_step_grouped(plan.ctx, ctypes.byref(h), 0, 1, None) == 1
    idx = (ctypes.c_int32 * 2)(0, 0)                       # duplicate index
    assert L.tsr_project_core_grouped(plan.ctx, idx, 2, None) == 1
    idx = (ctypes.c_int32 * 1)(3)                          # out of range
    assert L.tsr_project_core_grouped(plan.ctx, idx, 1, None) == 1
    assert b"out of range" in L.tsr_last_error(plan.ctx)
    torch.cuda.synchronize()
    assert torch.equal(w_before, plan.W[0])


def test_dense_adamw_matches_oracle():
    """Parameters that are not matrix blocks: multi-tensor dense AdamW against the oracle's."""
    tsr = _tsr()
    sizes = [1, 257, 70000, 0, 2048] + [33] * 60            # more than one batch of 48 tensors, one empty
    gens = torch.Generator().manual_seed(5)
    P = [torch.randn(n, generator=gens).cuda() for n in sizes]
    M = [torch.zeros(n).cuda() for n in sizes]
    V = [torch.zeros(n).cuda() for n in sizes]
    Po = [to64(p).copy() for p in P]
    Mo = [np.zeros(n) for n in sizes]
    Vo = [np.zeros(n) for n in sizes]
    from helpers import f32
    for t in range(1, 6):
        G = [(torch.randn(n, generator=gens).to(torch.bfloat16 if i % 2 else torch.float32)).cuda() for i, n in enumerate(sizes)]
        tsr.dense_adamw(P, G, M, V, tsr.make_hyper(t, lr=3e-3, beta2=0.95, weight_decay=0.1))
        torch.cuda.synchronize()
        for i in range(len(sizes)):
            oracle.dense_adamw(Po[i], to64(G[i]), Mo[i], Vo[i], f32(3e-3), f32(0.9), f32(0.95), f32(1e-8), f32(0.1), t)
            if sizes[i]:
                assert rel_fro(to64(P[i]), Po[i]) < 1e-6 and rel_fro(to64(M[i]), Mo[i]) < 1e-6 and rel_fro(to64(V[i]), Vo[i]) < 1e-6
    with pytest.raises(tsr.TsrError):
        tsr.dense_adamw(P[:1], G[:1], M[:1], V[:1], tsr.make_hyper(1, rule=1))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_optional_moment_reexpression_at_refresh(dtype):
    """TSR_BLOCK_REEXPRESS_MOMENT: M' = Unew^T (Uold M Vold^T) Vnew at an explicit refresh; the
    unflagged neighbour keeps Algorithm 1's behaviour (M untouched)."""
    tsr = _tsr()
    base = dict(m=192, n=256, r=24, p=8, q=1)
    plan = tsr.Plan([dict(base, flags=tsr.TSR_BLOCK_REEXPRESS_MOMENT), dict(base)], g_dtype=dtype)
    for i in range(2):
        fill_gradient(plan, i, 300 + i, signal_rank=12)
        fill_weights(plan, i, 310 + i)
    plan.init_subspace(seed=3)
    for t in (1, 2):
        for i in range(2):
            fill_gradient(plan, i, 320 + 10 * t + i, signal_rank=12)
        plan.step(tsr.make_hyper(t))
    torch.cuda.synchronize()
    Uo, Vo, Mo = [to64(plan.U[i]) for i in range(2)], [to64(plan.V[i]) for i in range(2)], [to64(plan.M[i]) for i in range(2)]
    Vm_before = plan.Vm[0].clone()
    for i in range(2):
        fill_gradient(plan, i, 390 + i, signal_rank=12)
    plan.rsvd_refresh(seed=4)
    torch.cuda.synchronize()
    assert plan.poll_status() == [0, 0]
    M_expect = Mo[0].copy()
    oracle.reexpress_moment(M_expect, Uo[0], Vo[0], to64(plan.U[0]), to64(plan.V[0]))
    assert rel_fro(to64(plan.M[0]), M_expect) < 1e-5
    assert rel_fro(to64(plan.M[0]), Mo[0]) > 1e-2            # it did change
    assert torch.equal(plan.Vm[0], Vm_before)                # the second moment is never re-expressed
    assert np.array_equal(to64(plan.M[1]), Mo[1])            # unflagged block: Algorithm 1 as printed


def _gram_reference(X):
    """X^T X of an FP32 matrix in extended precision (the products of FP32 numbers are exact in it and the sums carry
    64 bits), returned as FP64."""
    Xl = X.astype(np.longdouble)
    return (Xl.T @ Xl).astype(np.float64)


@pytest.mark.parametrize("shape,side", [
    (dict(m=700, n=520, r=64, p=8), 0),        # integer tensor-core form (k = 72 <= min / 2), ragged rows, one 2048-row chunk
    (dict(m=700, n=520, r=64, p=8), 1),
    (dict(m=4500, n=600, r=264, p=8), 0),      # k = 272: several 64-column tiles, tiles off the diagonal, three row chunks
    (dict(m=300, n=260, r=128, p=8), 0),       # k = 136 > min / 2: the FP64 tensor path
])
def test_gram_step_of_the_refresh_against_its_definition(shape, side):
    """S = X^T X as the refresh computes it, against the definition evaluated in extended precision, on columns whose
    scales span forty binary orders of magnitude, with a zero column, exact powers of two and entries that are tiny
    next to their column's largest.  The integer form cuts every column, scaled by a power of two to |y| <= 1/2, into
    six signed 7-bit digits (42 bits below the column's largest entry) and keeps the digit products down to 2^-42:
    per entry of S the error is bounded by rows * 2^-41 * 2^(e_i + e_j), e_j the exponent of column j's largest
    entry (what the digits and the digit products below 2^-42 leave out, all with the same sign), and comes to about
    5e-12 of |x_i| |x_j| for columns without outliers (gated at 2e-11: a level of digit products from the fifth up that
    went missing or landed in the wrong accumulator would show as 1e-9 and more).  The result must also be symmetric bit for bit
    and the same on a second call."""
    tsr = _tsr()
    plan = tsr.Plan([shape], g_dtype=torch.bfloat16)
    rows = shape["n"] if side else shape["m"]
    k = shape["r"] + shape["p"]
    rng = np.random.default_rng(77 + rows + k)
    X = rng.standard_normal((rows, k)).astype(np.float32)
    X *= np.exp2(rng.integers(-20, 21, size=k)).astype(np.float32)[None, :]      # column scales 2^-20 .. 2^20
    X[:, 3] = 0.0                                                                 # a zero column
    X[:, 5] = np.exp2(rng.integers(-3, 4, size=rows)).astype(np.float32)          # exact powers of two
    X[1:, 7] *= np.float32(2.0 ** -30)                                            # one entry dwarfs the rest of its column
    X[rows // 2, 9] = np.float32(0.5) * np.abs(X[:, 9]).max()                     # a tie in the column maximum's binade
    Xd = torch.from_numpy(X).cuda()
    S1 = plan.refresh_gram(0, side, Xd)
    S2 = plan.refresh_gram(0, side, Xd)
    torch.cuda.synchronize()
    assert plan.poll_status() == [0]
    S = S1.cpu().numpy()
    assert torch.equal(S1, S2)
    assert np.array_equal(S, S.T)
    ref = _gram_reference(X)
    cmax = np.abs(X).max(axis=0).astype(np.float64)
    e = np.where(cmax > 0, np.ceil(np.log2(np.maximum(cmax, 1e-300))) + 1, 0.0)   # cmax <= 2^(e - 1)
    bound = rows * 2.0 ** -41 * np.exp2(e[:, None] + e[None, :])
    err = np.abs(S - ref)
    assert np.all(err <= bound), float((err / bound).max())
    assert np.all(S[3, :] == 0) and np.all(S[:, 3] == 0)
    norms = np.sqrt(np.diag(ref))
    rel = err / np.maximum(norms[:, None] * norms[None, :], 1e-300)
    well = np.ones(k, bool); well[[3, 7]] = False                                 # columns without an outlier entry
    print("Gram against its definition: worst error %.1e of |x_i||x_j| (columns without outliers), %.2f of the bound"
          % (rel[np.ix_(well, well)].max(), (err / bound).max()))
    assert rel[np.ix_(well, well)].max() < 2e-11
