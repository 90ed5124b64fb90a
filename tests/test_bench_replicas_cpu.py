"""Host-side logic of the multi-GPU benchmark path, run as two gloo ranks on the CPU: the step time is the
max over ranks, the value is the whole job's tokens per second, and the reference arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench, uoe_inputs as gen
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = gen.WORKLOADS["cfg2_lm"]
ms, e2e = bench.max_over_ranks([1.0 + rank, 5.0 - rank], world)
out = {"rank": rank, "ms": ms, "e2e": e2e, "value": bench.job_throughput(w, world, ms)}
with open(os.path.join(sys.argv[2], "rank%d.json" % rank), "w") as f:   # one file per rank: stdout of two ranks can interleave
    json.dump(out, f)
dist.barrier()
dist.destroy_process_group()
"""


def _torchrun(args, timeout=300):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29653"] + args
    return subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, env=env, cwd=ROOT)


def test_max_over_ranks_and_job_throughput(tmp_path):
    worker = tmp_path / "worker.py"
    worker.write_text(WORKER)
    r = _torchrun([str(worker), ROOT, str(tmp_path)])
    assert r.returncode == 0, r.stderr[-2000:]
    res = [json.loads((tmp_path / ("rank%d.json" % i)).read_text()) for i in range(2)]
    for d in res:
        assert d["ms"] == 2.0 and d["e2e"] == 5.0                 # slowest rank decides
        assert d["value"] == pytest.approx(2 * 16 * 512 / 2e-3)    # both replicas' tokens over that time


def test_reference_arm_runs_on_rank_zero_only():
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--workload", "cfg1_small_f32"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0
