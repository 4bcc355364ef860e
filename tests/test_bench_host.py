"""Host-side pieces of bench.py that need no GPU: the workload arithmetic, and the only place
where replicas meet -- the max-over-ranks reduction -- run with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
vals = bench.max_over_ranks([1.0 + rank, 10.0 - rank, 5.0], dist, torch.device("cpu"))
if rank == 0:
    print("RESULT", vals)
dist.destroy_process_group()
""" % ROOT


def test_max_over_ranks_two_gloo_processes(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29531", WORLD_SIZE="2")
    procs = []
    for rank in range(2):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    line = [l for l in outs[0][0].splitlines() if l.startswith("RESULT")][0]
    assert line == "RESULT [2.0, 10.0, 5.0]"


def test_step_work_matches_hand_count():
    import bench
    import tsr_inputs as ti
    w = ti.workload(4)
    work = bench.step_work(w)
    mn = sum(b.m * b.n for b in w.blocks)
    assert mn == 1273446400
    # apply kernel: 8 bytes per weight (FP32 read + write) plus the BF16 operands P (m x r) and V (n x r)
    assert work["apply_kernel_bytes"] == 8.0 * mn + sum(2.0 * (b.m + b.n) * b.r for b in w.blocks)
    assert abs(work["apply_kernel_bytes"] / 1e9 - 11.16) < 0.05
    assert abs(work["proj_flops"] / 1e12 - 1.45) < 0.02
    shapes = bench.distinct_shapes(w)
    assert [c for _, c in shapes] == [96, 48, 24, 1]


def test_reference_arm_prints_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "tsr_adam_step_ms" and line["higher_is_better"] is False
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["value"] > 0
