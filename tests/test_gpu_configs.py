"""The five benchmark configurations, protocol as the task states it: bases initialised by a
randomized-SVD refresh on a separate seeded gradient, then 10 optimizer steps on freshly drawn
gradients, the CUDA library and the FP64 oracle in lock-step on the same bits (after every
refresh the library's bases are handed to the oracle, because singular vectors inside the noise
bulk are not unique).  Gated on C, M, Vm and W; the error of the accumulated update W_t - W_0 is reported as well.

Config 1 runs as it is.  For the LLaMA-shaped sets the FP64 plain-loop oracle cannot afford every
block (about 3 TFLOP per step at 1B), so a subset fixed in advance is run: one block of every
distinct shape of the first layer (attention, gate, down) and the embedding -- all ranks, tile
widths, ragged edges and the split-K core of the full set occur in it.  The whole sets, in the
benchmark's launch configuration, are covered by test_gpu_fullsize.py on sampled outputs."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
import tsr_inputs as ti
from helpers import HYPER, TOL_BF16, TOL_F32, check_refresh, rel_fro, to64

pytestmark = pytest.mark.gpu

SUBSET = {0: [0], 1: [0, 4, 6, -1], 2: [0, 4, 6, -1], 3: [0, 4, 6, -1], 4: [0, 6, -1]}   # 1B: the gate shape is sampled in test_gpu_fullsize.py
REFRESH_AT = {0: None, 1: 5, 2: 5, 3: 5, 4: None}     # in-loop refresh inside the 10 steps (1B: init only, oracle cost)


@pytest.mark.parametrize("cid", [0, 1, 2, 3, 4])
def test_config_protocol_matches_oracle(cid):
    import paper_2602_08007_b200 as tsr
    w = ti.workload(cid)
    blocks = [w.blocks[i] for i in SUBSET[cid]]
    dt = torch.float32 if w.g_dtype == "f32" else torch.bfloat16
    tol = TOL_F32 if w.g_dtype == "f32" else TOL_BF16
    plan = tsr.Plan([dict(m=b.m, n=b.n, r=b.r, p=b.p, q=b.q, K=0, is_embedding=b.is_embedding) for b in blocks], g_dtype=dt)
    nb = len(blocks)
    assert all(plan.uses_tensor_cores(i) == (w.g_dtype == "bf16") for i in range(nb))

    def draw(step, role):
        out = []
        for i, b in enumerate(blocks):
            g = ti.gradient(b.m, b.n, ti.seed_for(cid, SUBSET[cid][i] % len(w.blocks), step, role), dtype=dt, device="cuda")
            plan.G[i].copy_(g)
            out.append(to64(g))
        return out

    def omegas(step, role):
        return [ti.omega(b.n, b.r + b.p, ti.seed_for(cid, SUBSET[cid][i] % len(w.blocks), step, role), device="cuda")
                for i, b in enumerate(blocks)]

    gap = min(ti.SIGNAL_RANK, min(min(b.m, b.n) for b in blocks) // 2)
    G0, Om0 = draw(0, ti.ROLE_INIT_GRAD), omegas(0, ti.ROLE_INIT_OMEGA)
    plan.init_subspace(omegas=Om0)
    torch.cuda.synchronize()
    assert plan.poll_status() == [0] * nb
    obs, W0 = [], []
    for i, b in enumerate(blocks):
        check_refresh(plan, i, G0[i], to64(Om0[i]), b.r, b.q, gap)
        wt = ti.weights(b.m, b.n, ti.seed_for(cid, i, 0, ti.ROLE_WEIGHT), device="cuda")
        plan.W[i].copy_(wt)
        W0.append(to64(wt))
        ob = oracle.OracleBlock(W0[i], b.r, b.p, b.q, 0)
        ob.set_bases(to64(plan.U[i]), to64(plan.V[i]))
        obs.append(ob)
    worst = {k: 0.0 for k in ("C", "M", "Vm", "W", "dW")}
    for t in range(1, 11):
        G = draw(t, ti.ROLE_GRAD)
        if REFRESH_AT[cid] == t:
            Om = omegas(t, ti.ROLE_OMEGA)
            plan.rsvd_refresh(omegas=Om)
            torch.cuda.synchronize()
            for i, b in enumerate(blocks):
                check_refresh(plan, i, G[i], to64(Om[i]), b.r, b.q, gap)
                obs[i].set_bases(to64(plan.U[i]), to64(plan.V[i]))
        plan.step(tsr.make_hyper(t), fuse_adam=(t % 2 == 1))
        torch.cuda.synchronize()
        for i, ob in enumerate(obs):
            ob.step(G[i], skip_refresh=True, **HYPER)
            worst["C"] = max(worst["C"], rel_fro(to64(plan.C[i]), ob.C))
            worst["M"] = max(worst["M"], rel_fro(to64(plan.M[i]), ob.M))
            worst["Vm"] = max(worst["Vm"], rel_fro(to64(plan.Vm[i]), ob.Vm))
            worst["W"] = max(worst["W"], rel_fro(to64(plan.W[i]), ob.W))
            worst["dW"] = max(worst["dW"], rel_fro(to64(plan.W[i]) - W0[i], ob.W - W0[i]))
    assert plan.poll_status() == [0] * nb
    out_dir = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "gpurun_out")
    if os.path.isdir(out_dir):
        with open(os.path.join(out_dir, "parity_config%d.json" % cid), "w") as fh:
            json.dump({"config": w.name, "blocks": [b.name for b in blocks], "tolerance": tol, "worst": worst}, fh)
    for key in ("C", "M", "Vm", "W"):
        assert worst[key] < tol, (w.name, worst)
