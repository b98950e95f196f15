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


EP_WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch
from paper_2607_15810_b200 import dist_util as D
from paper_2607_15810_b200 import ep
world, rank = D.init("gloo")
E, T, H = 10, 6, 8
ranges = [ep.expert_range(r, world, E) for r in range(world)]


class FakeBinding:
    # stands in for the CUDA library on CPU: the partial sum of a rank is the sum of its experts' ids
    def moe_w4a4_rac(self, x, logits, w13, w2, topk, n13, n2, a2, expert_range=None, out_f32=None, **kw):
        lo, hi = expert_range
        assert w13["q"].shape[0] == hi - lo and w2["q"].shape[0] == hi - lo
        out_f32.fill_(float(sum(range(lo, hi))))

w = {"q": torch.zeros(E, 2), "sf": torch.zeros(E, 2), "gs": torch.zeros(E)}
lo, hi = ranges[rank]
out = ep.moe_w4a4_rac_expert_parallel(FakeBinding(), torch.zeros(T, H), torch.zeros(T, E), ep.shard_weights(w, lo, hi),
                                      ep.shard_weights(w, lo, hi), 2, 0, 0, None, rank, world)
if rank == 0:
    print(json.dumps({"ranges": ranges, "value": float(out[0, 0]), "shape": list(out.shape), "dtype": str(out.dtype)}))
D.shutdown()
"""


def test_expert_parallel_helper_partitions_the_experts_and_sums_the_partials(tmp_path):
    """Host logic of expert-parallel execution on two gloo ranks: a balanced contiguous split of the
    experts, each rank called with its own weights and range, one all-reduce of the partial sums."""
    from paper_2607_15810_b200 import ep
    for world in (1, 2, 3, 8):
        for E in (1, 8, 10, 128):
            parts = [ep.expert_range(r, world, E) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == E
            assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1
    script = tmp_path / "ep_worker.py"
    script.write_text(EP_WORKER % ROOT)
    r = _torchrun([str(script)], 240)
    assert r.returncode == 0, r.stderr[-2000:]
    out = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][0])
    assert out["ranges"] == [[0, 5], [5, 10]] and out["value"] == float(sum(range(10)))
    assert out["shape"] == [6, 8] and out["dtype"] == "torch.bfloat16"
