"""Full-size parity in the benchmark's launch configuration: the grouped fused step over all 169
blocks of the LLaMA-1B-shaped set (and all 57 of the 60M set), checked on sampled outputs the
oracle computes one by one.

The oracle cannot afford a whole 1B step (about 3 TFLOP of FP64 plain loops), so the chain is cut
into links, each checked against the oracle's own routine on a sub-problem:
  * C[A, B] = U[:, A]^T G V[:, B]   -- oracle.project_core on column subsets of the bases;
  * M, Vm                           -- oracle.adam_core, elementwise, on the complete core;
  * W[I, J]                         -- oracle.backproject_apply on row subsets U[I, :], V[J, :].
"""
import numpy as np
import pytest
import torch

import oracle
import tsr_inputs as ti
from helpers import HYPER, TOL_BF16, rel_fro, to64

pytestmark = pytest.mark.gpu


def _run(config_id, sample_blocks):
    import paper_2602_08007_b200 as tsr
    w = ti.workload(config_id)
    dev = torch.device("cuda")
    plan = tsr.Plan(list(w.blocks), g_dtype=torch.bfloat16, device=dev)
    for i, b in enumerate(w.blocks):
        plan.G[i].copy_(ti.gradient(b.m, b.n, ti.seed_for(config_id, i, 0, ti.ROLE_INIT_GRAD), dtype=torch.bfloat16, device=dev))
        plan.W[i].copy_(ti.weights(b.m, b.n, ti.seed_for(config_id, i, 0, ti.ROLE_WEIGHT), device=dev))
    plan.init_subspace(seed=ti.BASE_SEED)
    torch.cuda.synchronize()
    assert plan.poll_status() == [0] * len(w.blocks)
    W0 = {i: plan.W[i].clone() for i in sample_blocks}
    for i, b in enumerate(w.blocks):
        plan.G[i].copy_(ti.gradient(b.m, b.n, ti.seed_for(config_id, i, 1, ti.ROLE_GRAD), dtype=torch.bfloat16, device=dev))
    lr = 1e-3
    plan.step(tsr.make_hyper(1, lr=lr), seed=ti.BASE_SEED, fuse_adam=True)
    torch.cuda.synchronize()
    assert plan.poll_status() == [0] * len(w.blocks)
    rng = np.random.default_rng(7)
    for i in sample_blocks:
        b = w.blocks[i]
        U, V = to64(plan.U[i]), to64(plan.V[i])
        assert np.linalg.norm(U.T @ U - np.eye(b.r)) < 1e-4 and np.linalg.norm(V.T @ V - np.eye(b.r)) < 1e-4
        G = to64(plan.G[i])
        Cg = to64(plan.C[i])
        # sampled core entries, the oracle's projection on column subsets (include the ragged tail columns)
        A = np.sort(np.concatenate([rng.choice(np.arange(1, b.r - 1), 6, replace=False), [0, b.r - 1]]))
        B = np.sort(np.concatenate([rng.choice(np.arange(1, b.r - 1), 6, replace=False), [0, b.r - 1]]))
        Co = oracle.project_core(G, np.ascontiguousarray(U[:, A]), np.ascontiguousarray(V[:, B]))
        assert rel_fro(Cg[np.ix_(A, B)], Co) < TOL_BF16, (b.name, rel_fro(Cg[np.ix_(A, B)], Co))
        # moments: the oracle's core Adam on the complete core (t = 1, zero moments before)
        Mo, Vo = np.zeros_like(Cg), np.zeros_like(Cg)
        Do = oracle.adam_core(Cg, Mo, Vo, HYPER["beta1"], HYPER["beta2"], HYPER["eps"], 1)
        assert rel_fro(to64(plan.M[i]), Mo) < 1e-6 and rel_fro(to64(plan.Vm[i]), Vo) < 1e-6
        # sampled weights: rows / columns from the first, last (ragged) and random tiles
        I = np.unique(np.concatenate([rng.integers(0, b.m, 5), [0, b.m - 1]]))
        J = np.unique(np.concatenate([rng.integers(0, b.n, 5), [0, b.n - 1]]))
        Wsub = to64(W0[i])[np.ix_(I, J)].copy()
        oracle.backproject_apply(np.ascontiguousarray(U[I, :]), Do, np.ascontiguousarray(V[J, :]), Wsub, HYPER["lr"])
        Wg = to64(plan.W[i])[np.ix_(I, J)]
        upd_o = Wsub - to64(W0[i])[np.ix_(I, J)]
        upd_g = Wg - to64(W0[i])[np.ix_(I, J)]
        assert rel_fro(Wg, Wsub) < TOL_BF16
        assert rel_fro(upd_g, upd_o) < 5e-2, (b.name, rel_fro(upd_g, upd_o))   # the update itself, not hidden behind W
    return plan


def test_llama60m_full_set_sampled_outputs():
    w = ti.workload(1)
    _run(1, [0, 4, 6, len(w.blocks) - 1])       # attention, gate, down, embedding


def test_llama1b_full_set_sampled_outputs():
    w = ti.workload(4)
    _run(4, [0, 4, 6, len(w.blocks) - 1])


def test_llama1b_layer_with_bf16_weights():
    """One layer of the 1B set plus the embedding (r = 512: the 256-wide tiles of the apply kernel)
    with weights stored in BF16; sampled weights against the oracle's update rounded to BF16."""
    import paper_2602_08007_b200 as tsr
    w = ti.workload(4)
    blocks = list(w.blocks[:7]) + [w.blocks[-1]]
    dev = torch.device("cuda")
    plan = tsr.Plan(blocks, g_dtype=torch.bfloat16, w_dtype=torch.bfloat16, device=dev)
    W0 = []
    for i, b in enumerate(blocks):
        plan.G[i].copy_(ti.gradient(b.m, b.n, ti.seed_for(4, i, 1, ti.ROLE_GRAD), dtype=torch.bfloat16, device=dev))
        plan.W[i].copy_(ti.weights(b.m, b.n, ti.seed_for(4, i, 0, ti.ROLE_WEIGHT), device=dev).to(torch.bfloat16))
        plan.U[i].copy_(ti.orthonormal(b.m, b.r, 300 + 2 * i).to(dev))
        plan.V[i].copy_(ti.orthonormal(b.n, b.r, 301 + 2 * i).to(dev))
        W0.append(plan.W[i].clone())
    plan.bases_changed()
    plan.step(tsr.make_hyper(1, lr=1e-3), fuse_adam=True)
    torch.cuda.synchronize()
    assert plan.poll_status() == [0] * len(blocks)
    rng = np.random.default_rng(9)
    for i, b in enumerate(blocks):
        U, V, Cg = to64(plan.U[i]), to64(plan.V[i]), to64(plan.C[i])
        Mo, Vo = np.zeros_like(Cg), np.zeros_like(Cg)
        Do = oracle.adam_core(Cg, Mo, Vo, HYPER["beta1"], HYPER["beta2"], HYPER["eps"], 1)
        I = np.unique(np.concatenate([rng.integers(0, b.m, 6), [0, b.m - 1]]))
        J = np.unique(np.concatenate([rng.integers(0, b.n, 6), [0, b.n - 1]]))
        before = W0[i].double().cpu().numpy()[np.ix_(I, J)]
        Wsub = before.copy()
        oracle.backproject_apply(np.ascontiguousarray(U[I, :]), Do, np.ascontiguousarray(V[J, :]), Wsub, HYPER["lr"])
        step_size = np.abs(Wsub - before).max()
        Wo = torch.from_numpy(Wsub).float().to(torch.bfloat16).double().numpy()
        Wg = plan.W[i].double().cpu().numpy()[np.ix_(I, J)]
        assert np.all(np.abs(Wg - Wo) <= 2.0 ** -7 * np.abs(Wo) + 0.1 * step_size), b.name
        assert rel_fro(Wg, Wo) < TOL_BF16
        assert not np.array_equal(Wg, before)     # the weights did move
