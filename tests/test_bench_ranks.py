"""The benchmark's multi-rank plumbing on CPU: two gloo ranks.  Units never interact, so
N > 1 is weak scaling with no data-path collective; what has to be right is the rendezvous,
the per-rank sequences, the max-over-ranks time and the whole-job aggregate."""
import json
import os
import socket
import subprocess
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

PROBE = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import bench, workloads as wl
world, rank, local = bench.dist_setup(2)
w = bench.rank_workload(wl.C1, rank)
q, k, v = wl.decode_inputs(w, 0)
ms_local = 10.0 * (rank + 1)                      # rank 1 is the slow one
bench.barrier(world)
value, ms_total = bench.whole_job_throughput(ms_local, 7 * 100, world)
print("PROBE " + json.dumps(dict(rank=rank, world=world, seed=w.seed, q0=float(q.flatten()[0]),
                                 value=value, ms_total=ms_total)), flush=True)
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_aggregate_by_the_slowest():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", PROBE.format(root=ROOT)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=180)
        assert p.returncode == 0, se[-2000:]
        outs.append(json.loads([l for l in so.splitlines() if l.startswith("PROBE ")][0][6:]))
    outs.sort(key=lambda d: d["rank"])
    assert [d["world"] for d in outs] == [2, 2]
    assert outs[0]["seed"] != outs[1]["seed"] and outs[0]["q0"] != outs[1]["q0"]
    for d in outs:                                   # both ranks agree on the aggregate
        assert d["ms_total"] == 20.0                 # the slower rank's time
        assert abs(d["value"] - 2 * 700 / 20e-3) < 1e-6


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", RANK="1", LOCAL_RANK="1", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "1"], env=env,
                       capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_single_process_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_throughput(2.0, 10, 1) == (10 / 2e-3, 2.0)
    assert not torch.distributed.is_initialized()
