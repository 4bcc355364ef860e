"""tsr_project_core_static -- the entry point for callers that may not allocate device memory
(its scratch is a fixed array inside the library) -- must give what the FP64 oracle gives for
C = U^T G V, and the same bits as tsr_project_core on the CUDA-core path, without allocating.

Runs last (file name) so that a run stopping at the first failure has already run everything
else; it passes alone in a fresh process as well as after the other tests."""
import numpy as np
import pytest
import torch

import oracle
import tsr_inputs as ti
from helpers import TOL_F32, TOL_F32_MAXABS, max_abs_err, rel_fro, to64

pytestmark = pytest.mark.gpu


def test_static_scratch_projection_matches_oracle_and_context_path_twice_in_a_row():
    import paper_2602_08007_b200 as tsr
    shapes = [dict(m=512, n=1376, r=128), dict(m=200, n=330, r=24)]
    plan = tsr.Plan(shapes, g_dtype=torch.float32)          # FP32 gradients: the CUDA-core path
    for i, s in enumerate(shapes):
        plan.U[i].copy_(ti.orthonormal(s["m"], s["r"], 900 + i).cuda())
        plan.V[i].copy_(ti.orthonormal(s["n"], s["r"], 910 + i).cuda())
    plan.bases_changed()
    for call in range(2):                                   # two calls in a row share the fixed array
        for i, s in enumerate(shapes):
            plan.G[i].copy_(ti.gradient(s["m"], s["n"], 920 + 10 * call + i).cuda())
        plan.project_core()
        for i, s in enumerate(shapes):
            C = torch.full((s["r"], s["r"]), float("nan"), device="cuda")
            torch.cuda.synchronize()
            held = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
            free_before = torch.cuda.mem_get_info()[0]
            tsr.project_core_static(plan.G[i], plan.U[i], plan.V[i], C)
            torch.cuda.synchronize()
            # nothing was allocated through torch, and -- once the first call on the device has made the CUDA
            # runtime load the library's image with its fixed array -- the free device memory does not move
            assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == held
            if call > 0:
                assert torch.cuda.mem_get_info()[0] >= free_before
            want = oracle.project_core(to64(plan.G[i]), to64(plan.U[i]), to64(plan.V[i]))
            assert rel_fro(to64(C), want) < TOL_F32, (call, i)
            assert max_abs_err(to64(C), want) < TOL_F32_MAXABS, (call, i)
            ref = plan.C[i]
            err = float((C - ref).norm() / ref.norm())
            assert err <= 1e-6, (call, i, err)             # same kernels: in practice identical bits


def test_static_scratch_rejects_what_does_not_fit():
    import paper_2602_08007_b200 as tsr
    m, r = 4096, 512                                        # m * r = 2 Mi floats > the 1 Mi-float array
    G = torch.zeros(m, 512, device="cuda")
    U = torch.zeros(m, r, device="cuda")
    V = torch.zeros(512, r, device="cuda")
    C = torch.zeros(r, r, device="cuda")
    with pytest.raises(tsr.TsrError) as ei:
        tsr.project_core_static(G, U, V, C)
    assert ei.value.status == 4                             # TSR_ERR_WORKSPACE
    assert m * r > tsr.STATIC_SCRATCH_FLOATS
    with pytest.raises(ValueError):                         # the wrapper refuses mismatched shapes before the C call
        tsr.project_core_static(G, U, V[:, :8].contiguous(), C)
