"""The N > 1 path of the benchmark is N independent replicas (the method's hot path exchanges
nothing between devices): what the ranks share is the host-side timing protocol -- a barrier,
the maximum over ranks of the timed region, the whole-job throughput -- and the rule that the
reference arm runs on rank 0 only.  Exercised here as two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["KGE_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + os.environ["KGE_PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
dist.barrier()
mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
worst = bench.max_over_ranks(mine)
value = bench.whole_job_value(world, 1024, worst / 4)
print(json.dumps({"rank": rank, "worst": worst, "value": value, "seed": bench.replica_seed(rank)}), flush=True)
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_aggregate():
    port = str(_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", KGE_PORT=port, KGE_ROOT=str(ROOT))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0
        outs.append(json.loads(out.strip().splitlines()[-1]))
    assert [o["worst"] for o in outs] == [15.0, 15.0]                 # max over ranks, seen by both
    assert outs[0]["value"] == outs[1]["value"] == pytest.approx(2 * 1024 / (15.0 / 4 * 1e-3))
    assert sorted(o["seed"] for o in outs) == [0, 1]                   # replicas draw different batches


def test_single_rank_is_the_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(1, 1024, 0.1) == pytest.approx(1.024e7)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
