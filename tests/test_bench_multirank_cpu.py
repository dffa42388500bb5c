"""The multi-rank side of bench.py on CPU (gloo, world size 2): replicas only, so the only cross-rank
logic is the aggregation (time = max over ranks, work = sum over ranks) and rank-dependent seeding; the
reference arm must run on rank 0 alone."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo")
ms, pairs = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100 + rank, dist, "cpu")
wl = bench.WORKLOADS["ring64_d1m_b4"]
sched = bench.PairSchedule(wl, None)
first = sched.next().tolist()
dist.barrier()
print(json.dumps({{"rank": rank, "ms": ms, "pairs": pairs, "first": first}}), flush=True)
dist.destroy_process_group()
"""


def test_aggregate_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29517", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["ms"] == 15.0            # max over ranks
        assert o["pairs"] == 201.0        # sum over ranks
        pairs = np.array(o["first"])
        assert pairs.shape == (32, 2) and len(set(pairs.reshape(-1).tolist())) == 64   # a perfect matching


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--workload", "complete8_d4096_b8_lsq"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                        "--workload", "complete8_d4096_b8_lsq"], env=env, capture_output=True, text=True, timeout=120)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
