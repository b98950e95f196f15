"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas with no
data-path collective, barrier + max-over-ranks timing, rank 0 reports; and the
reference arm under a 2-process launch (rank 0 alone works and prints)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
from paper_2607_15810_b200 import dist_util as D
world, rank = D.init("gloo")
assert world == 2
D.barrier()
ms = D.max_over_ranks(1.0 + rank * 0.5)           # rank 1 is the slow one
rate = D.whole_job_rate(world, 100, ms)
if rank == 0:
    print(json.dumps({"ms": ms, "rate": rate, "world": world}))
D.shutdown()
"""


def _torchrun(args, timeout):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29613"] + args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_take_the_slowest_rank_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    r = _torchrun([str(script)], 240)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                            # only rank 0 reports
    out = json.loads(lines[0])
    assert out["world"] == 2 and out["ms"] == 1.5
    assert abs(out["rate"] - 2 * 100 / 1.5e-3) < 1e-6


def test_reference_arm_under_two_ranks_prints_one_line():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--ref-budget-s", "1.5", "--workload", "decode"], 600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["cpu_baseline"]["kind"] == "oracle"
    assert out["value"] > 0 and out["e2e"]["h2d_bytes_per_step"] == 0
