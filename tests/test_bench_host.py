"""Host-side logic of bench.py that needs no GPU: the reference arm's JSON line, and the
multi-rank aggregation (slowest rank's time, sum of units) on two gloo ranks."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group(backend="gloo")
secs, units = bench.aggregate_over_ranks(dist, 1.0 + rank, 100 * (rank + 1), torch.device("cpu"))
dist.barrier()
dist.destroy_process_group()
print(json.dumps({{"rank": rank, "secs": secs, "units": units}}))
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_aggregate_over_two_gloo_ranks():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER.format(root=ROOT)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
        rec = json.loads(o.strip().splitlines()[-1])
        assert rec["secs"] == 2.0 and rec["units"] == 300.0      # max over ranks, sum over ranks


def test_reference_arm_prints_one_line_on_rank0_only():
    env = dict(os.environ, RANK="0", WORLD_SIZE="2")
    r0 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr
    lines = [l for l in r0.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["unit"] == "node-params/s" and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] >= 1
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["value"] == rec["value"]
    assert rec["config"]["workload"] == "cfg2" and rec["higher_is_better"] is True
    # the config object is the one the GPU arm prints for the same arguments, and exactly `steps` steps were timed
    import argparse

    import bench
    from paper_2104_11981_b200 import inputs
    w = inputs.WORKLOADS["cfg2"]
    ours = bench.workload_config(argparse.Namespace(workload="cfg2", columns=0, tuning=""), w, w.n, w.d, 2, 4)
    assert rec["config"] == ours
    assert rec["steps"] == 1 and rec["cpu_baseline"]["sample"].startswith("cfg2: 1 DecentLaM steps")
    env["RANK"] = "1"
    r1 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""


def test_ours_arm_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        return
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1"], capture_output=True,
                       text=True, timeout=300)
    assert r.returncode != 0 and "no CUDA device" in (r.stderr + r.stdout)
