"""Host logic of the benchmark that needs no GPU: the reference arm and the multi-process
aggregation (replicas: max of the per-rank times, sum of the work), over gloo with two ranks."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "seq-steps/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")       # rank 1 is the slow one
value = bench.job_value(world, 1000, ms)
if rank == 0:
    print("RESULT", ms, value)
dist.destroy_process_group()
"""


def test_two_rank_aggregation_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, REPO_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    res = [l for l in out.stdout.splitlines() if l.startswith("RESULT")]
    assert len(res) == 1
    _, ms, value = res[0].split()
    assert float(ms) == 15.0                       # max over ranks
    assert abs(float(value) - 2 * 1000 / 15e-3) < 1e-6   # both replicas' steps over the slowest time
