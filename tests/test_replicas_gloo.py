"""The path has no exchange step, so N GPUs run N independent replicas and only the timing is
reduced (max over ranks).  This checks that reduction with two CPU ranks over gloo, and that a
plain `python bench.py --gpus 2` starts its two ranks itself."""
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
ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
agg = bench.aggregate_value(per_replica_work=3.0e12, world=dist.get_world_size(), ms=ms)
assert ms == 15.0, ms
assert abs(agg - 2 * 3.0e12 / 15.0e-3 / 1e12) < 1e-9, agg
dist.barrier()
print("rank", rank, "ok")
"""


def test_two_replicas_report_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29613")
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                        "--master-addr", "127.0.0.1", "--master-port", "29613", str(script)],
                       capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.count("ok") == 2


def test_bench_gpus_n_starts_its_own_ranks():
    """No launcher, no WORLD_SIZE in the environment: bench.py --gpus 2 must come back as a two-replica job whose
    time is the slower rank's (the replica self-test needs no GPU: gloo ranks with made-up times)."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--replica-selftest"],
                       capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stdout + r.stderr
    line = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(line) == 1, r.stdout
    out = json.loads(line[0])
    assert out["n_gpus"] == 2 and out["ms"] == 15.0
    assert abs(out["value"] - 2 * 3.0e12 / 15.0e-3 / 1e12) < 1e-9
