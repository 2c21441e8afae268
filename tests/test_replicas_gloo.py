"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The path does not shard (replicas
only), so what N > 1 adds is the aggregation -- every rank's kept tokens over the slowest rank's
time -- and the rule that the reference arm runs on rank 0 alone."""
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["SKIPFFN_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%s" % os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
# rank 0: 1472 kept tokens, 10 steps in 20 ms; rank 1: 1000 kept tokens, 10 steps in 40 ms
units, ms = (1472, 20.0) if rank == 0 else (1000, 40.0)
value, ms_step = bench.job_throughput(units, ms, 10)
print(json.dumps({"rank": rank, "value": value, "ms_step": ms_step,
                  "max": bench.max_over_ranks(ms), "sum": bench.sum_over_ranks(units)}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_rank_aggregation_gloo():
    import json
    port = str(_free_port())
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", PORT=port, SKIPFFN_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", _WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    for o in outs:          # both ranks agree on the whole-job figures
        assert o["max"] == 40.0 and o["sum"] == 2472
        assert o["ms_step"] == 4.0
        assert o["value"] == pytest.approx(2472 / 4.0e-3)


def test_single_process_aggregation_is_identity():
    import bench
    assert bench.max_over_ranks(12.5) == 12.5 and bench.sum_over_ranks(7) == 7
    v, ms = bench.job_throughput(1472, 25.0, 20)
    assert ms == 1.25 and v == pytest.approx(1472 / 1.25e-3)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""
