"""The N > 1 path of the benchmark on CPU: GEMM calls are independent, so ranks are replicas and the only
cross-rank step is the max-over-ranks of the measured times (gloo backend here, NCCL on GPUs).  Also checks the
reference arm under a 2-rank launch: rank 0 prints the one JSON line, rank 1 exits 0 without output."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch.distributed as dist
import bench
rank, world, local = bench.rank_info()
dist.init_process_group("gloo")
# rank r pretends its step took (10 + 5 r) ms and its end-to-end step (30 - r) ms
step_ms, e2e_ms = bench.max_over_ranks([10.0 + 5.0 * rank, 30.0 - rank])
value = bench.aggregate_throughput(2.0e12, step_ms, world)
if rank == 0:
    print(json.dumps({"world": world, "step_ms": step_ms, "e2e_ms": e2e_ms, "value": value}))
dist.barrier()
dist.destroy_process_group()
"""


def torchrun(args, extra_env=None, timeout=300):
    env = dict(os.environ, REPO_ROOT=ROOT, OMP_NUM_THREADS="2")
    env.update(extra_env or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000)] + args
    return subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT, timeout=timeout)


def test_max_over_ranks_and_aggregate_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    r = torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["world"] == 2 and d["step_ms"] == 15.0 and d["e2e_ms"] == 30.0
    # two replicas of 2 TFLOP each in 15 ms
    assert abs(d["value"] - 2 * 2.0 / 15e-3) < 1e-9


def test_reference_arm_under_two_ranks_prints_one_line():
    r = torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1",
                  "--workload", "cfg1_fp32_512"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


def test_single_process_helpers_are_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.aggregate_throughput(1e12, 1000.0, 1) == 1.0
