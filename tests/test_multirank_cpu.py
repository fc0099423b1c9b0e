"""The benchmark's multi-rank plumbing on CPU (gloo, world size 2): the path itself has no
collective -- ranks run independent replicas -- so what is shared is the barrier, the
max-over-ranks timing reduction and the rank-0-only reporting of the reference arm."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
import torch.distributed as dist
sys.path.insert(0, %r)
import bench                         # the benchmark's own reduction and aggregation, on the gloo backend
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# every rank holds its own replica's step time; the reported time is the max over ranks and the
# reported throughput the sum of the replicas' work over that time
dist.barrier()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)
value = bench.aggregate_value(1000, ms, world)
if rank == 0:
    print(json.dumps({"ms": ms, "value": value, "world": world}))
dist.destroy_process_group()
""" % ROOT


def _torchrun(args, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29517"] + args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_timing_with_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = _torchrun([str(script)])
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["world"] == 2 and line["ms"] == 15.0
    assert abs(line["value"] - 2 * 1000 / 15e-3) < 1e-6


def test_reference_arm_reports_from_rank_zero_only():
    out = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                     "--workload", "c1", "--ref-scale", "0.2"])
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["value"] > 0
    assert lines[0]["cpu_baseline"]["kind"] == "oracle" and lines[0]["e2e"]["h2d_bytes_per_step"] == 0
