"""CPU-side checks of the CUDA library: it loads, exports every symbol the header declares,
validates arguments on the host, and its byte / state accounting matches the oracle's."""
import ctypes
import os
import re

import pytest

import oracle
import tsr_inputs as ti

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tsr():
    import paper_2602_08007_b200 as t
    from paper_2602_08007_b200 import build as b
    b.build()
    return t


def _create(tsr, descs):
    arr = (tsr.MatDesc * len(descs))(*descs)
    ctx = ctypes.c_void_p()
    rc = tsr.lib().tsr_create(ctypes.byref(ctx), arr, len(descs))
    return rc, ctx


def test_library_exports_every_declared_symbol(tsr):
    header = open(os.path.join(ROOT, "include", "tsr.h")).read()
    declared = set(re.findall(r"\b(tsr_[a-z_]+)\s*\(", header))
    declared -= {"tsr_status", "tsr_dtype", "tsr_rule"}
    assert declared == set(tsr.EXPORTS)
    L = tsr.lib()
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert L.tsr_version() >= 100
    assert L.tsr_status_string(0) == b"ok"


def test_create_validates_shapes(tsr):
    D = tsr.MatDesc
    good = D(512, 1376, 1376, 1376, 128, 8, 1, 100, tsr.TSR_BF16, tsr.TSR_F32, 0, 0)
    rc, ctx = _create(tsr, [good])
    assert rc == 0 and ctx.value
    assert tsr.lib().tsr_destroy(ctx) == 0
    bad = [
        D(0, 8, 8, 8, 2, 0, 0, 0, 0, 0, 0, 0),                      # m = 0
        D(16, 16, 8, 16, 4, 0, 0, 0, 0, 0, 0, 0),                    # ldg < n
        D(16, 16, 16, 16, 12, 8, 0, 0, 0, 0, 0, 0),                  # r + p > min(m, n)
        D(16, 16, 16, 16, 4, 0, -1, 0, 0, 0, 0, 0),                  # q < 0
        D(2048, 2048, 2048, 2048, 1050, 8, 1, 0, 0, 0, 0, 0),        # r + p beyond the eigen-solver's limit of 1056
    ]
    for d in bad:
        rc, ctx = _create(tsr, [d])
        assert rc == 2 and not ctx.value
    rc, ctx = _create(tsr, [D(16, 16, 16, 16, 4, 0, 0, 0, 0, 1, 0, 0)])  # BF16 weights
    assert rc == 0 and ctx.value
    assert tsr.lib().tsr_destroy(ctx) == 0
    rc, _ = _create(tsr, [D(16, 16, 16, 16, 4, 0, 0, 0, 0, 1, 0, 0), D(16, 16, 16, 16, 4, 0, 0, 0, 0, 0, 0, 0)])
    assert rc == 6                                                      # one weight type per context
    rc, _ = _create(tsr, [D(16, 16, 16, 16, 4, 0, 0, 0, 7, 0, 0, 0)])
    assert rc == 6
    assert tsr.lib().tsr_create(None, None, 0) == 1


def test_block_flags_are_validated_and_sized(tsr):
    D = tsr.MatDesc
    rc, ctx = _create(tsr, [D(64, 64, 64, 64, 8, 0, 0, 0, 0, 0, 0, 4)])          # unknown flag bit
    assert rc == 1
    rc, ctx = _create(tsr, [D(64, 64, 64, 64, 8, 0, 0, 0, 0, 0, 0, 3)])          # one-sided with re-expressed moments
    assert rc == 6
    sizes = []
    for flags in (0, tsr.TSR_BLOCK_REEXPRESS_MOMENT):
        rc, ctx = _create(tsr, [D(256, 320, 320, 320, 32, 8, 1, 0, 0, 0, 0, flags)])
        assert rc == 0
        sb, rb = ctypes.c_size_t(), ctypes.c_size_t()
        tsr.lib().tsr_workspace_bytes(ctx, ctypes.byref(sb), ctypes.byref(rb))
        sizes.append(rb.value)
        tsr.lib().tsr_destroy(ctx)
    assert sizes[1] - sizes[0] >= 4 * ((256 + 320) * 32 + 3 * 32 * 32)             # old bases + three r x r scratch


def test_one_sided_block_accounting(tsr):
    """Table 1: a one-sided block synchronizes C = U^T G, r n elements instead of r^2, and keeps
    U plus two r x n moments."""
    D = tsr.MatDesc
    m, n, r = 256, 320, 32
    rc, ctx = _create(tsr, [D(m, n, n, n, r, 8, 1, 0, 1, 0, 0, tsr.TSR_BLOCK_ONE_SIDED), D(m, n, n, n, r, 8, 1, 0, 1, 0, 0, 0)])
    assert rc == 0
    L = tsr.lib()
    core, sk, el = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
    assert L.tsr_comm_bytes(ctx, 1, 4, ctypes.byref(core), ctypes.byref(sk)) == 0
    assert core.value == 4 * (r * n + r * r)
    assert L.tsr_state_elems(ctx, ctypes.byref(el)) == 0
    assert el.value == (m * r + 2 * r * n) + ((m + n) * r + 2 * r * r)
    L.tsr_destroy(ctx)


def test_compute_before_bind_is_refused(tsr):
    rc, ctx = _create(tsr, [tsr.MatDesc(64, 64, 64, 64, 8, 0, 0, 0, 0, 0, 0, 0)])
    assert rc == 0
    L = tsr.lib()
    assert L.tsr_project_core(ctx, 0, None) == 11
    h = tsr.make_hyper(1)
    assert L.tsr_step_grouped(ctx, ctypes.byref(h), 0, 1, None) == 11
    assert b"tsr_bind" in L.tsr_last_error(ctx)
    ptrs = (tsr.MatPtrs * 1)()
    assert L.tsr_bind(ctx, ptrs, 1, None, 0) == 4          # no workspace
    L.tsr_destroy(ctx)


def test_comm_bytes_and_state_match_oracle_accounting(tsr):
    for cid in range(5):
        w = ti.workload(cid)
        es = 2 if w.g_dtype == "bf16" else 4
        descs = [tsr.MatDesc(b.m, b.n, ti.padded_ld(b.n, es), ti.padded_ld(b.n, 4), b.r, b.p, b.q, b.K,
                             tsr.TSR_BF16 if w.g_dtype == "bf16" else tsr.TSR_F32, 0, int(b.is_embedding), 0)
                 for b in w.blocks]
        rc, ctx = _create(tsr, descs)
        assert rc == 0
        L = tsr.lib()
        core, sk, el = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
        assert L.tsr_comm_bytes(ctx, 0, 4, ctypes.byref(core), ctypes.byref(sk)) == 0
        assert core.value == sum(oracle.core_bytes(b.r, 4) for b in w.blocks)
        assert sk.value == sum(oracle.sketch_bytes(b.m, b.n, b.r, b.p, 4) for b in w.blocks)
        assert L.tsr_state_elems(ctx, ctypes.byref(el)) == 0
        assert el.value == sum(oracle.state_elems(b.m, b.n, b.r) for b in w.blocks)
        # a step that is not a refresh step carries the cores only
        assert L.tsr_comm_bytes(ctx, 1, 4, ctypes.byref(core), ctypes.byref(sk)) == 0
        assert sk.value == 0
        if cid > 0:
            K = w.blocks[0].K
            assert L.tsr_comm_bytes(ctx, K, 2, ctypes.byref(core), ctypes.byref(sk)) == 0
            assert sk.value == sum(oracle.sketch_bytes(b.m, b.n, b.r, b.p, 2) for b in w.blocks)
        sb, rb = ctypes.c_size_t(), ctypes.c_size_t()
        assert L.tsr_workspace_bytes(ctx, ctypes.byref(sb), ctypes.byref(rb)) == 0
        assert sb.value > 0 and rb.value > 0
        for i in (0, len(descs) - 1):
            assert L.tsr_block_uses_tensor_cores(ctx, i) == (1 if w.g_dtype == "bf16" else 0)
        assert L.tsr_block_uses_tensor_cores(ctx, len(descs)) < 0
        L.tsr_destroy(ctx)
