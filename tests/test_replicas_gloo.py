"""The N > 1 path of the benchmark is "replicas only": no collective on the data path, a barrier
and a max-over-ranks reduction of the step time.  Checked here with two gloo ranks on CPU."""
from __future__ import annotations

import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent(
    """
    import os, sys, json
    sys.path.insert(0, os.environ["REPO_ROOT"])
    import torch, torch.distributed as dist
    from workloads import configs
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    w = bench.workload("tiny")
    # every replica derives the same workload and the same per-step byte count on its own
    ct = bench.class_tokens(w["g"], w["T"], w["agents"], w["n_new"])
    moved = 2 * sum(ct.values()) * w["g"].bpt
    t = torch.tensor([float(moved)])
    dist.all_reduce(t)
    assert t.item() == world * moved
    # the benchmark's own control plane: barrier, then the slowest rank's time is the job's time
    cl = bench.Cluster(torch, dist, "cpu", world, "gloo")
    cl.barrier()
    ms = cl.max_ms(10.0 + rank)              # rank-dependent step time: the job reports the slowest
    assert ms == 10.0 + world - 1
    value = world * moved / (ms * 1e-3) / 1e9
    if rank == 0:
        print(json.dumps({"value": value, "n_gpus": world, "scaling": "weak"}))
    dist.destroy_process_group()
    """
)


def test_two_replicas_reduce_time_by_max_and_sum_bytes(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, REPO_ROOT=ROOT)
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr",
         "127.0.0.1", "--master-port", "29631", str(script)],
        env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    import json

    d = json.loads(line)
    assert d["n_gpus"] == 2 and d["scaling"] == "weak" and d["value"] > 0


def test_reference_arm_prints_one_json_line_only_on_rank0():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "2", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    import json

    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
