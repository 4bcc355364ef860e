#!/usr/bin/env python
"""Benchmark of the TSR-Adam optimizer hot path (libtsr) on synthetic LLaMA-shaped gradient sets.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 4] [--impl ours|reference]

A "step" is one full optimizer step over every matrix block of the model: core projection
C = U^T G V, core-space Adam, lift and in-place weight update, plus the randomized-SVD refresh
on the steps where the schedule asks for one (t mod K == 0).  The default workload is the
LLaMA-1B-shaped set (169 blocks, r = 512, embedding rank 256, BF16 gradients, FP32 weights);
its gradients (2.5 GB) and weights (5.1 GB) are far larger than the 126 MB L2, so no explicit
flush is needed between steps.  Prints ONE JSON line (rank 0).

The path does not shard across GPUs (no collective on the data path): with N > 1 every rank
runs an independent replica on its own GPU and the line reports the slowest rank.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import tsr_inputs as ti  # noqa: E402

METRIC = "tsr_adam_step_ms"
UNIT = "ms/step"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def step_work(w: ti.Workload, w_bytes: int = 4):
    """Algorithmic flops and bytes of one non-refresh step, per stage (w_bytes: bytes per weight)."""
    ges = 2 if w.g_dtype == "bf16" else 4
    rmw = 2.0 * w_bytes
    out = {"proj_flops": 0.0, "proj_bytes": 0.0, "apply_flops": 0.0, "apply_bytes": 0.0,
           "apply_kernel_flops": 0.0, "apply_kernel_bytes": 0.0}
    for b in w.blocks:
        m, n, r = b.m, b.n, b.r
        small = 2.0 * min(m, n) * r * r
        out["proj_flops"] += 2.0 * m * n * r + small
        out["proj_bytes"] += ges * m * n + 2.0 * (m + n) * r + 24.0 * r * r
        out["apply_flops"] += 2.0 * m * n * r + small
        out["apply_bytes"] += rmw * m * n + 2.0 * (m + n) * r
        # the apply kernel proper: W <- decay W - step_scale P V^T with P = U D (m x r) given
        out["apply_kernel_flops"] += 2.0 * m * n * r
        out["apply_kernel_bytes"] += rmw * m * n + 2.0 * (m + n) * r
    out["step_flops"] = out["proj_flops"] + out["apply_flops"]
    out["step_bytes"] = out["proj_bytes"] + out["apply_bytes"]
    return out


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index = index
        self.stop_flag = threading.Event()
        self.sm, self.reasons, self.max_sm = [], set(), None
        self.ok = False

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            }
            self.ok = True
            while not self.stop_flag.is_set():
                self.sm.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
                time.sleep(0.05)
        except Exception:
            self.ok = False

    def summary(self):
        if not self.ok or not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_sm, "reasons": ["nvml_unavailable"]}
        return {"sm_mhz": statistics.median(self.sm), "sm_max_mhz": self.max_sm, "reasons": sorted(self.reasons)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# --------------------------------------------------------------------------------------------
# reference arm / cpu baseline: the FP64 oracle on the host cores, on a bounded sample
# --------------------------------------------------------------------------------------------
def distinct_shapes(w: ti.Workload):
    """One representative block per distinct (m, n, r) with its multiplicity, in workload order."""
    seen = {}
    for blk in w.blocks:
        key = (blk.m, blk.n, blk.r)
        if key not in seen:
            seen[key] = [blk, 0]
        seen[key][1] += 1
    return list(seen.values())


def oracle_step_time(w: ti.Workload, blk, reps: int = 1):
    """Seconds the oracle needs for one optimizer step (project, core Adam, lift+apply) of `blk`."""
    import numpy as np

    import oracle
    dt = torch.bfloat16 if w.g_dtype == "bf16" else torch.float32
    G = ti.gradient(blk.m, blk.n, 1, dtype=dt).double().numpy()
    ob = oracle.OracleBlock(ti.weights(blk.m, blk.n, 2).double().numpy(), blk.r, blk.p, blk.q, 0)
    ob.set_bases(ti.orthonormal(blk.m, blk.r, 3).double().numpy(), ti.orthonormal(blk.n, blk.r, 4).double().numpy())
    times = []
    for rep in range(reps):
        t0 = time.perf_counter()
        ob.step(G, lr=1e-3)
        times.append(time.perf_counter() - t0)
    assert np.isfinite(ob.W).all()
    return min(times)


def refresh_flops(b) -> float:
    """Rough flop count of one rSVD refresh of a block (sketches, orthonormalisations, small SVD), used only
    to scale the oracle's time on one sampled block to the other shapes."""
    k = b.r + b.p
    return (2 * b.q + 2) * 2.0 * b.m * b.n * k + (2 * b.q + 2) * 2.0 * (b.m + b.n) * k * k + 20.0 * k ** 3


def oracle_refresh_time(w: ti.Workload, blk):
    """Seconds the oracle needs for one refresh (Section 3.5) of `blk`."""
    import oracle
    dt = torch.bfloat16 if w.g_dtype == "bf16" else torch.float32
    G = ti.gradient(blk.m, blk.n, 1, dtype=dt).double().numpy()
    Om = ti.omega(blk.n, blk.r + blk.p, 5).double().numpy()
    t0 = time.perf_counter()
    oracle.rsvd_refresh(G, Om, blk.r, blk.q)
    return time.perf_counter() - t0


def cpu_baseline(w: ti.Workload, refreshes_per_step: float = 0.0):
    """The oracle, as it stands, on one block of every distinct shape of the workload (one step
    each); the whole-set figure multiplies each time by the number of blocks of that shape.  When
    the timed region holds refreshes, one refresh of the first block is timed as well, scaled to
    the whole set by a flop count and amortised like the GPU figure."""
    import oracle
    total, sampled, parts = 0.0, 0.0, []
    for blk, count in distinct_shapes(w):
        sec = oracle_step_time(w, blk)
        total += sec * count
        sampled += sec
        parts.append("%dx%d r=%d x%d: %.2f s" % (blk.m, blk.n, blk.r, count, sec))
    out = {"unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "step_ms": total * 1e3}
    sample = "one step of one block per distinct shape (%s), each multiplied by its block count" % "; ".join(parts)
    refresh_total = 0.0
    if refreshes_per_step > 0:
        blk = w.blocks[0]
        sec = oracle_refresh_time(w, blk)
        sampled += sec
        refresh_total = sec * sum(refresh_flops(b) for b in w.blocks) / refresh_flops(blk)
        out["refresh_ms"] = refresh_total * 1e3
        sample += "; one refresh of a %dx%d r=%d block (%.1f s), scaled to all blocks by flops and counted %.3f times " \
                  "per step" % (blk.m, blk.n, blk.r, sec, refreshes_per_step)
    out["value"] = (total + refresh_total * refreshes_per_step) * 1e3
    out["sample"] = "%.1f s of CPU work in all: %s" % (sampled, sample)
    return out


def oracle_sample(w: ti.Workload):
    """The reference arm's per-step sample: the first block of the workload (an attention-shaped
    square block for the LLaMA sets), small enough that K + W steps end within a few minutes."""
    return w.blocks[0]


def run_reference(args, w: ti.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    blk = oracle_sample(w)
    work = step_work(w)
    sample = step_work(ti.Workload("sample", w.config_id, w.g_dtype, 1, (blk,)))
    scale = work["step_flops"] / sample["step_flops"]
    # size the per-step sample so the whole run stays within a few minutes
    for _ in range(args.warmup):
        oracle_step_time(w, blk)
    t = [oracle_step_time(w, blk) for _ in range(args.steps)]
    ms = statistics.mean(t) * scale * 1e3
    line = {
        "impl": "reference", "metric": METRIC, "value": ms, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "blocks": len(w.blocks)},
        "cpu_baseline": {"value": ms, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": "each step = one %dx%d r=%d block through the FP64 oracle, scaled by algorithmic "
                                   "flops x%.1f to the whole set" % (blk.m, blk.n, blk.r, scale)},
        "e2e": {"value": ms, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group).
    The path has no collective of its own: replicas only meet here, to report the slowest."""
    if dist is None:
        return [float(v) for v in values]
    tens = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(tens, op=dist.ReduceOp.MAX)
    return [float(x) for x in tens]


def apply_traffic(w: ti.Workload, algorithmic_bytes: float):
    """DRAM bytes per launch of the apply kernel as ncu measured them (dram__bytes_read.sum +
    dram__bytes_write.sum), read from the table profiles/dram_traffic.json keeps per workload together
    with the commit it was captured at.  A capture of a slice of the workload is scaled to the full
    launch by the algorithmic bytes (traffic grows in proportion to the weights streamed).  None when
    the table has no entry for this workload."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as fh:
            table = json.load(fh)
        e = table["umma_apply_kernel"][w.name]
        return {"bytes": float(e["dram_bytes"]) * algorithmic_bytes / float(e["algorithmic_bytes"]),
                "captured_on": e["captured_on"], "commit": e["commit"]}
    except Exception:
        return None


def build_plan(w: ti.Workload, device, bf16_weights: bool = False):
    import paper_2602_08007_b200 as tsr
    dt = torch.bfloat16 if w.g_dtype == "bf16" else torch.float32
    plan = tsr.Plan(list(w.blocks), g_dtype=dt, device=device, w_dtype=torch.bfloat16 if bf16_weights else torch.float32)
    for i, b in enumerate(w.blocks):
        plan.G[i].copy_(ti.gradient(b.m, b.n, ti.seed_for(w.config_id, i, 0, ti.ROLE_INIT_GRAD), dtype=dt, device=device))
        plan.W[i].copy_(ti.weights(b.m, b.n, ti.seed_for(w.config_id, i, 0, ti.ROLE_WEIGHT), device=device).to(plan.W[i].dtype))
    return tsr, plan


def fresh_gradients(plan, w, t, device):
    dt = plan.g_dtype
    for i, b in enumerate(w.blocks):
        plan.G[i].copy_(ti.gradient(b.m, b.n, ti.seed_for(w.config_id, i, t, ti.ROLE_GRAD), dtype=dt, device=device))


def quick_config(cid: int, device, peaks, steps: int = 20):
    """A compact measurement of one of the other benchmark configurations: ms per step with L2 flushed
    between steps (cold) and not (warm), one refresh, and the roofline fractions of the apply and
    projection stages.  About two seconds each; the numbers of the headline workload come from the main run."""
    w = ti.workload(cid)
    tsr, plan = build_plan(w, device)
    work = step_work(w)
    plan.init_subspace(seed=ti.BASE_SEED)
    fresh_gradients(plan, w, 1, device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    for _ in range(3):
        plan.step(tsr.make_hyper(1), seed=ti.BASE_SEED, fuse_adam=True)
    torch.cuda.synchronize()

    def timed(cold):
        ev = []
        for j in range(steps):
            if cold:
                flush.fill_(j & 0xFF)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            plan.step(tsr.make_hyper(j + 1), seed=ti.BASE_SEED, fuse_adam=True)
            b.record()
            ev.append((a, b))
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in ev)

    launches0 = plan.launch_count()
    cold_ms = timed(True)
    launches = (plan.launch_count() - launches0) // steps
    warm_ms = timed(False)
    plan.set_profiling(True)
    rows = []
    for rep in range(7):
        flush.fill_(rep)
        plan.step(tsr.make_hyper(1), seed=ti.BASE_SEED, fuse_adam=True)
        rows.append(plan.stage_ms())
    st = [statistics.median(r[i] for r in rows) for i in range(6)]
    plan.set_profiling(False)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush.fill_(1)
    a.record()
    plan.rsvd_refresh(seed=ti.BASE_SEED + 1)
    b.record()
    torch.cuda.synchronize()
    refresh_ms = a.elapsed_time(b)
    status = sorted(set(plan.poll_status()))
    hbm, tc = peaks["hbm_gbs"], peaks["bf16_tflops"]
    proj_ms, apply_ms = st[1] + st[2], st[4] + st[5]
    proj_roof = max(work["proj_flops"] / (tc * 1e12), work["proj_bytes"] / (hbm * 1e9)) * 1e3
    apply_roof = max(work["apply_flops"] / (tc * 1e12), work["apply_bytes"] / (hbm * 1e9)) * 1e3
    out = {"workload": w.name, "blocks": len(w.blocks), "dtype": w.g_dtype, "step_ms_cold_l2": cold_ms, "step_ms_warm_l2": warm_ms,
           "step_roof_ms": proj_roof + apply_roof, "refresh_ms": refresh_ms, "launches_per_step": launches,
           "projection": {"ms": proj_ms, "roof_ms": proj_roof, "frac": proj_roof / proj_ms if proj_ms > 0 else None},
           "backprojection": {"ms": apply_ms, "roof_ms": apply_roof, "frac": apply_roof / apply_ms if apply_ms > 0 else None},
           "device_status": status}
    plan.close()
    del plan, flush
    torch.cuda.empty_cache()
    return out


def oracle_one_thread(cid: int):
    """The oracle's step time on ONE host thread for a small configuration (a child process, because the
    OpenMP thread count is fixed when the oracle's library loads): one step of one block per distinct
    shape, each multiplied by its block count."""
    import subprocess
    code = ("import sys; sys.path.insert(0, %r); import bench, tsr_inputs as ti; w = ti.workload(%d); "
            "print(sum(bench.oracle_step_time(w, blk) * cnt for blk, cnt in bench.distinct_shapes(w)) * 1e3)" % (ROOT, cid))
    env = dict(os.environ, OMP_NUM_THREADS="1")
    try:
        out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
        return float(out.stdout.strip().splitlines()[-1])
    except Exception:
        return None


def run_ours(args, w: ti.Workload):
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=device)
        dist = dist_mod

    tsr, plan = build_plan(w, device, args.bf16_weights)
    peaks = measured_peaks()
    work = step_work(w, 2 if args.bf16_weights else 4)
    nb = len(w.blocks)
    seed = ti.BASE_SEED

    if args.random_bases:
        # profiling aid: skip the initial refresh, use random (not orthonormal) bases; timings of the
        # step kernels do not depend on the values
        for i, b in enumerate(w.blocks):
            plan.U[i].normal_(0.0, b.m ** -0.5)
            plan.V[i].normal_(0.0, b.n ** -0.5)
        plan.bases_changed()
    else:
        plan.init_subspace(seed=seed)        # Algorithm 1 initialisation: one refresh on G_0
    torch.cuda.synchronize()
    fresh_gradients(plan, w, 1, device)
    flush = None
    if args.flush_l2:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)

    def one_step(t):
        if flush is not None:
            flush.fill_(t & 0xFF)
        plan.step(tsr.make_hyper(t), seed=seed, fuse_adam=True)

    # warm-up on steps that are not refresh steps
    for wstep in range(args.warmup):
        one_step(1)
    torch.cuda.synchronize()
    status = plan.poll_status()

    # stage events only when they are read inside the loop: an event between two kernels keeps the second one from
    # setting itself up under the first one's tail (programmatic dependent launch)
    plan.set_profiling(bool(args.stage_times))
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    stage = []
    sampler = ClockSampler(physical_gpu_index(local_rank))
    launches0 = plan.launch_count()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    wall0 = time.perf_counter()
    for j in range(args.steps):
        t = j + 1
        if flush is not None:
            flush.fill_(t & 0xFF)
        ev[j][0].record()
        plan.step(tsr.make_hyper(t), seed=seed, fuse_adam=True)
        ev[j][1].record()
        if args.stage_times:
            stage.append(plan.stage_ms())     # waits for this step; only with --stage-times
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    wall = time.perf_counter() - wall0
    sampler.stop_flag.set()
    sampler.join(timeout=2)
    launches = plan.launch_count() - launches0
    step_ms = [a.elapsed_time(b) for a, b in ev]
    refresh_steps = [j for j in range(args.steps) if any(b.K > 0 and (j + 1) % b.K == 0 for b in w.blocks)]
    plain = [step_ms[j] for j in range(args.steps) if j not in refresh_steps] or step_ms
    total_ms = sum(step_ms)
    ms_per_step = total_ms / args.steps
    status2 = plan.poll_status()

    # stage breakdown and the dominant kernel (apply), measured with CUDA events on plain steps
    plan.set_profiling(True)
    st_rows = []
    for rep in range(max(5, min(20, args.steps))):
        if flush is not None:
            flush.fill_(rep)
        plan.step(tsr.make_hyper(1), seed=seed, fuse_adam=not args.unfused)
        st_rows.append(plan.stage_ms())
    st_med = [statistics.median(r[i] for r in st_rows) for i in range(6)]
    apply_ms = st_med[5]
    proj_ms = st_med[1] + st_med[2]

    # refresh alone
    refresh_ms, refresh_all_ms = None, []
    if args.refresh_reps > 0:
        rts = []
        for rep in range(args.refresh_reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            plan.rsvd_refresh(seed=seed + 1 + rep)
            b.record()
            torch.cuda.synchronize()
            rts.append(a.elapsed_time(b))
        refresh_ms = min(rts)
        refresh_all_ms = rts
    status3 = plan.poll_status()

    # end to end from host buffers: H2D of every gradient, the step, D2H of the packed cores
    e2e = None
    if args.e2e_steps > 0:
        dt = plan.g_dtype
        g_host = [torch.empty(b.m, b.n, dtype=dt).pin_memory() for b in w.blocks]
        for i in range(nb):
            g_host[i].copy_(plan.G[i])
        c_host = torch.empty(sum(b.r * b.r for b in w.blocks), dtype=torch.float32).pin_memory()
        plan.step_host(g_host, c_host, tsr.make_hyper(1), seed=seed)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for j in range(args.e2e_steps):
            plan.step_host(g_host, c_host, tsr.make_hyper(1), seed=seed)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3 / args.e2e_steps
        e2e = {"value": e2e_ms, "unit": UNIT, "h2d_bytes_per_step": sum(g.numel() * g.element_size() for g in g_host),
               "d2h_bytes_per_step": c_host.numel() * 4}

    # dense AdamW for non-matrix parameters (Section 3.4): HBM-bound, 28 bytes per FP32 parameter
    dense = None
    if args.dense_params > 0:
        n = args.dense_params
        dp = [torch.randn(n, device=device) for _ in range(1)]
        dg = [torch.randn(n, device=device) for _ in range(1)]
        dm = [torch.zeros(n, device=device) for _ in range(1)]
        dv = [torch.zeros(n, device=device) for _ in range(1)]
        for t in range(1, 4):
            tsr.dense_adamw(dp, dg, dm, dv, tsr.make_hyper(t))
        a, bb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for t in range(4, 9):
            tsr.dense_adamw(dp, dg, dm, dv, tsr.make_hyper(t))
        bb.record()
        torch.cuda.synchronize()
        dms = a.elapsed_time(bb) / 5
        dense = {"params": n, "ms": dms, "achieved_gbs": 28.0 * n / (dms * 1e-3) / 1e9,
                 "frac_of_hbm": 28.0 * n / (dms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        del dp, dg, dm, dv

    # max over ranks
    ms_per_step, wall_ms_per_step, apply_ms, proj_ms = max_over_ranks(
        [ms_per_step, wall * 1e3 / args.steps, apply_ms, proj_ms], dist, device)

    if rank == 0:
        hbm = peaks["hbm_gbs"]
        tc = peaks["bf16_tflops_sustained"]
        apply_gbs = work["apply_kernel_bytes"] / (apply_ms * 1e-3) / 1e9
        proj_tflops = work["proj_flops"] / (proj_ms * 1e-3) / 1e12
        proj_roof_ms = max(work["proj_flops"] / (tc * 1e12), work["proj_bytes"] / (hbm * 1e9)) * 1e3
        apply_roof_ms = max(work["apply_kernel_flops"] / (tc * 1e12), work["apply_kernel_bytes"] / (hbm * 1e9)) * 1e3
        plain_ms = statistics.median(plain)
        core_b, sketch_b = plan.comm_bytes(0, 4)
        traffic = apply_traffic(w, work["apply_kernel_bytes"])
        tc_burst = peaks["bf16_tflops"]
        proj_roof_burst_ms = max(work["proj_flops"] / (tc_burst * 1e12), work["proj_bytes"] / (hbm * 1e9)) * 1e3
        line = {
            "metric": METRIC, "value": ms_per_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.g_dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "blocks": nb, "rank": w.blocks[0].r, "embedding_rank": w.blocks[-1].r,
                       "refresh_interval": w.blocks[0].K, "refresh_steps_in_timed_region": len(refresh_steps),
                       "l2": "flushed between steps" if flush is not None else "inputs (G %.2f GB + W %.2f GB) exceed L2"
                       % (sum(b.m * b.n for b in w.blocks) * (2 if w.g_dtype == "bf16" else 4) / 1e9,
                          sum(b.m * b.n for b in w.blocks) * (2 if args.bf16_weights else 4) / 1e9),
                       "weights": "bf16" if args.bf16_weights else "f32",
                       "parallelism": "replicas only" if world > 1 else "single gpu"},
            "step_ms_no_refresh": plain_ms,
            "wall_ms_per_step": wall_ms_per_step,
            "refresh_ms": refresh_ms, "refresh_ms_each": refresh_all_ms,
            "step_tflops": work["step_flops"] / (plain_ms * 1e-3) / 1e12,
            "stage_ms": {"refresh": st_med[0], "projection_launch": st_med[1], "after_projection": st_med[2], "core_update": st_med[3],
                         "gemm_UD": st_med[4], "apply": st_med[5]},
            "roofline": {"kernel": "umma_apply_kernel (W <- decay W - lr P V^T)", "bound": "hbm",
                         "achieved": apply_gbs, "peak": hbm, "unit": "GB/s", "frac": apply_gbs / hbm,
                         "traffic": None if (args.bf16_weights or traffic is None) else traffic["bytes"],
                         "traffic_source": None if traffic is None else "ncu capture on %s at commit %s (profiles/dram_traffic.json)"
                         % (traffic["captured_on"], traffic["commit"]),
                         "algorithmic_bytes": work["apply_kernel_bytes"],
                         "peak_source": peaks["source"] + " copy bandwidth", "ms": apply_ms, "roof_ms": apply_roof_ms},
            "roofline_projection": {"kernels": "umma_gemm_kernel<EPI_RUNTIME>: tiles of the first contraction (T~ = (G V)^T, or T = U^T G where m > n) and core tiles (+ Adam) in one launch"
                                    if st_med[2] < 0.1 * st_med[1] else "umma_gemm_kernel<EPI_STORE_BF16_T> + <EPI_CORE_UPDATE>",
                                    "bound": "tensor" if work["proj_flops"] / (tc * 1e12) > work["proj_bytes"] / (hbm * 1e9) else "hbm",
                                    "achieved_tflops": proj_tflops, "ms": proj_ms, "roof_ms": proj_roof_ms,
                                    "frac": proj_roof_ms / proj_ms, "peak": "sustained BF16 %.0f TFLOP/s" % tc,
                                    "roof_ms_burst_peak": proj_roof_burst_ms, "frac_of_burst_peak": proj_roof_burst_ms / proj_ms},
            "peaks": {"hbm_gbs": hbm, "bf16_tflops_burst": tc_burst, "bf16_tflops_sustained": tc, "source": peaks["source"],
                      "nominal_b200": {"hbm_gbs": 7700.0, "bf16_tflops_dense": 2250.0},
                      "apply_frac_of_nominal_hbm": apply_gbs / 7700.0,
                      "projection_frac_of_nominal": (work["proj_flops"] / 2250e12 * 1e3) / proj_ms},
            "comm_bytes": {"core_per_step": core_b, "sketch_per_refresh": sketch_b,
                           "dense_fp32_per_step": 4 * sum(b.m * b.n for b in w.blocks)},
            "dense_adamw": dense,
            "device_status": sorted(set(status + status2 + status3)),
            "clocks": sampler.summary(),
            "e2e": e2e,
            "gpu_launches": launches,
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(w, len(refresh_steps) / float(args.steps))
        if args.all_configs and world == 1:
            # the other four benchmark configurations, compactly (the headline workload's numbers are the line's own)
            plan.close()
            torch.cuda.empty_cache()
            others = {}
            for cid in range(5):
                if cid == w.config_id:
                    continue
                entry = quick_config(cid, device, peaks)
                if cid <= 1 and not args.no_cpu_baseline:
                    entry["oracle_step_ms_1_thread"] = oracle_one_thread(cid)
                others["config%d" % (cid + 1)] = entry
            line["configs"] = others
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------
# ablation arms (Section 5, "Two-Sidedness, Randomized SVD"): kernel times and bytes
# --------------------------------------------------------------------------------------------
def run_ablation(args, w: ti.Workload):
    """The comparison arms of the paper's ablation on synthetic gradients of the chosen set, one
    JSON line: optimizer step and synchronized bytes of the two-sided method against the one-sided
    arm (C = U^T G, r x n), and the randomized refresh against the exact-SVD arm (the same refresh
    with a sketch as wide as the smaller side of the block and no power iteration, which spans the
    whole range of G).  Not the headline benchmark: a diagnostic report."""
    import paper_2602_08007_b200 as tsr
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    dt = torch.bfloat16 if w.g_dtype == "bf16" else torch.float32
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)

    def spec(b, **over):
        d = dict(m=b.m, n=b.n, r=b.r, p=b.p, q=b.q, K=0, is_embedding=b.is_embedding, flags=0)
        d.update(over)
        return d

    def make(specs):
        plan = tsr.Plan(specs, g_dtype=dt, device=device)
        for i, b in enumerate(w.blocks):
            plan.G[i].copy_(ti.gradient(b.m, b.n, ti.seed_for(w.config_id, i, 0, ti.ROLE_INIT_GRAD), dtype=dt, device=device))
            plan.W[i].copy_(ti.weights(b.m, b.n, ti.seed_for(w.config_id, i, 0, ti.ROLE_WEIGHT), device=device))
        return plan

    def time_refresh(plan, reps=3):
        best = float("inf")
        for rep in range(reps + 1):     # the first call is the warm-up
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.fill_(rep)
            e0.record()
            plan.init_subspace(seed=ti.BASE_SEED + rep)
            e1.record()
            torch.cuda.synchronize()
            if rep > 0:
                best = min(best, e0.elapsed_time(e1))
        return best

    def time_steps(plan, steps):
        times = []
        for t in range(1, steps + args.warmup + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.fill_(t & 0xFF)
            e0.record()
            plan.step(tsr.make_hyper(t), seed=ti.BASE_SEED, fuse_adam=True)
            e1.record()
            torch.cuda.synchronize()
            if t > args.warmup:
                times.append(e0.elapsed_time(e1))
        return statistics.median(times)

    out = {"mode": "ablation", "config": {"workload": w.name, "blocks": len(w.blocks)}, "data": "synthetic",
           "steps": args.steps, "warmup": args.warmup, "l2": "256 MB written before every timed call"}
    arms = {}
    for name, flags in (("two_sided", 0), ("one_sided", tsr.TSR_BLOCK_ONE_SIDED)):
        plan = make([spec(b, flags=flags) for b in w.blocks])
        refresh_ms = time_refresh(plan)
        step_ms = time_steps(plan, args.steps)
        core, sketch = plan.comm_bytes(0, 4)
        arms[name] = {"step_ms": step_ms, "refresh_ms": refresh_ms, "core_bytes_per_step": core,
                      "sketch_bytes_per_refresh": sketch, "state_elems": plan.state_elems(),
                      "device_status": sorted(set(plan.poll_status()))}
        plan.close()
        del plan
        torch.cuda.empty_cache()
    out["arms"] = arms
    out["one_sided_over_two_sided"] = {
        "core_bytes": arms["one_sided"]["core_bytes_per_step"] / arms["two_sided"]["core_bytes_per_step"],
        "step_ms": arms["one_sided"]["step_ms"] / arms["two_sided"]["step_ms"]}
    if max(min(b.m, b.n) for b in w.blocks) <= 1056:
        plan = make([spec(b, p=min(b.m, b.n) - b.r, q=0) for b in w.blocks])
        exact_ms = time_refresh(plan)
        _, exact_sketch = plan.comm_bytes(0, 4)
        out["refresh"] = {"rsvd_ms": arms["two_sided"]["refresh_ms"], "exact_svd_ms": exact_ms,
                          "rsvd_over_exact_ms": arms["two_sided"]["refresh_ms"] / exact_ms,
                          "rsvd_sketch_bytes": arms["two_sided"]["sketch_bytes_per_refresh"],
                          "exact_sketch_bytes": exact_sketch,
                          "device_status": sorted(set(plan.poll_status()))}
        plan.close()
    else:
        out["refresh"] = {"rsvd_ms": arms["two_sided"]["refresh_ms"], "exact_svd_ms": None,
                          "why": "the exact arm needs a sketch as wide as min(m, n), above the library's limit of 1056"}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, help="0..4: the five benchmark configurations")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--flush-l2", action="store_true", help="write a 256 MB buffer before every step")
    ap.add_argument("--stage-times", action="store_true", help="also read stage timings inside the timed loop")
    ap.add_argument("--refresh-reps", type=int, default=3, help="refreshes of all blocks timed alone; refresh_ms is their minimum")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dense-params", type=int, default=1 << 26,
                    help="size of the dense-AdamW micro-measurement (0 = skip)")
    ap.add_argument("--all-configs", dest="all_configs", action="store_true", default=None,
                    help="add a compact measurement of the other four configurations (default: on for the default workload)")
    ap.add_argument("--no-all-configs", dest="all_configs", action="store_false")
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: truncate the model to this many layers")
    ap.add_argument("--unfused", action="store_true", help="diagnostic: run the core update as its own launch")
    ap.add_argument("--bf16-weights", action="store_true",
                    help="variant: weights stored in BF16 (4 instead of 8 bytes of read-modify-write per weight)")
    ap.add_argument("--random-bases", action="store_true",
                    help="profiling aid: random bases instead of the initial refresh (numbers not for reporting)")
    ap.add_argument("--ablation", action="store_true",
                    help="report the one-sided and exact-SVD comparison arms of the chosen set instead of the benchmark")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: start the N replica processes (one per GPU) ourselves
        import socket
        import subprocess
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    w = ti.workload(args.config)
    if args.layers > 0 and args.config > 0:
        # profiling aid: keep the first `layers` transformer layers (7 blocks each) and the embedding
        keep = tuple(w.blocks[:7 * args.layers]) + (w.blocks[-1],)
        w = ti.Workload(w.name + "-first%dlayers" % args.layers, w.config_id, w.g_dtype, w.steps, keep)
    if args.config < 3:
        args.flush_l2 = True
    if args.all_configs is None:
        args.all_configs = (args.config == 4 and args.layers == 0 and not args.bf16_weights)
    if args.ablation:
        run_ablation(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
