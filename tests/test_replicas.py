"""The N > 1 plumbing of the benchmark (replicas only: no data-path collective) on CPU: two gloo ranks."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
from paper_2509_09679_b200.replicas import Replicas
r = Replicas(device=None, backend="gloo")
r.barrier()
ms = r.max_over_ranks(1.0 + 2.0 * r.rank)          # rank 0 measured 1 ms, rank 1 measured 3 ms
out = dict(rank=r.rank, world=r.world, ms=ms, seed=r.seed(1000), rate=r.whole_job_rate(4096, ms))
r.barrier()
r.close()
print(json.dumps(out))
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER.format(root=ROOT)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=120)
        assert p.returncode == 0, se[-2000:]
        outs.append(json.loads(so.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert [o["world"] for o in outs] == [2, 2]
    assert all(o["ms"] == 3.0 for o in outs)                      # the slowest rank sets the step time
    assert outs[0]["seed"] == 1000 and outs[1]["seed"] == 1100     # every replica draws its own rows
    assert all(abs(o["rate"] - 2 * 4096 / 3e-3) < 1e-6 for o in outs)  # whole-job rate: both ranks' rows / max time


def test_single_process_needs_no_process_group():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    so = subprocess.run([sys.executable, "-c", WORKER.format(root=ROOT)], env=env, capture_output=True, text=True,
                        timeout=120, check=True).stdout
    o = json.loads(so.strip().splitlines()[-1])
    assert o["world"] == 1 and o["ms"] == 1.0 and o["rate"] == 4096 / 1e-3


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
