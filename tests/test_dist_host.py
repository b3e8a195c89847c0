"""The benchmark's multi-process plumbing with two gloo ranks on the CPU: rendezvous, barrier,
max-over-ranks timing and the whole-job aggregate (replicas only: no data-path collective)."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch
from paper_2609_25442_b200 import dist as wbdist
rank, local_rank, world = wbdist.rank_info()
d = wbdist.init("gloo")
assert d is not None and world == 2
wbdist.barrier(d, cuda=False)
mine = 5.0 + 3.0 * rank                      # rank 1 is the slow one
slowest = wbdist.max_over_ranks(d, mine, torch.device("cpu"))
agg = wbdist.aggregate_gbs(world, 32_000_000_000, slowest)
if rank == 0:
    print(json.dumps({"slowest": slowest, "agg": agg}))
d.destroy_process_group()
"""


def test_two_gloo_ranks_report_the_slowest_time_and_the_aggregate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29611", WORLD_SIZE="2")
    procs = []
    for r in range(2):
        e = dict(env, RANK=str(r), LOCAL_RANK=str(r))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, err) in zip(procs, outs):
        assert p.returncode == 0, err
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["slowest"] == 8.0
    assert abs(res["agg"] - 2 * 32.0 / 8e-3) < 1e-6          # 2 replicas x 32 GB in 8 ms


def test_single_process_defaults():
    from paper_2609_25442_b200 import dist as wbdist
    import torch
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert wbdist.rank_info() == (0, 0, 1)
    assert wbdist.init("gloo") is None
    assert wbdist.max_over_ranks(None, 4.5, torch.device("cpu")) == 4.5
