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


SHARDED_WORKER = r"""
import os, sys, json
sys.path.insert(0, %(root)r)
sys.path.insert(0, %(tests)r)
import numpy as np
import torch
from paper_2609_25442_b200 import binding as wb
from paper_2609_25442_b200 import dist as wbdist
from plan_interp import run_table
from helpers import ckpt_shapes
from oracle import remap_oracle
from wb_workloads import WB_F32, make_workload

rank, local_rank, world = wbdist.rank_info()
d = wbdist.init("gloo")
result = {}
for name, scale, budget in %(cases)r:
    wl = make_workload(name, scale)
    plan = wb.Plan(wb.Layout(wl.trainer.tensors, wl.trainer.slices), wb.Layout(wl.rollout.tensors, wl.rollout.slices),
                   bucket_budget_bytes=budget)
    plan.verify()
    nt, nr = plan.num_ranks()
    t_owner, r_owner = wbdist.block_owner(nt, world), wbdist.block_owner(nr, world)
    bits_s = np.uint32 if wl.src_dtype == WB_F32 else np.uint16
    bits_d = np.uint32 if wl.dst_dtype == WB_F32 else np.uint16
    # every process can compute the trainer tensors, but only reads those of the ranks it owns: the rest
    # is poisoned so that a tile which strays into another process's shard shows in the result
    full = [t.numpy().view(bits_s).copy() for t in wl.load_side_to_list("trainer", lambda i: wl.ckpt_values(i).view(
        torch.int32 if wl.src_dtype == WB_F32 else torch.int16))]
    src = [a if t_owner[int(td["rank"])] == rank else np.full(a.size, 0x7FC1, bits_s)
           for a, td in zip(full, wl.trainer.tensors)]
    fill = 0xCDCD if bits_d == np.uint16 else 0xCDCDCDCD
    dst = [np.full(int(t["numel"]), fill, bits_d) for t in wl.rollout.tensors]
    wrote = [np.zeros(int(t["numel"]), np.int64) for t in wl.rollout.tensors]
    sent = 0
    assert plan.num_rounds() > 1
    for r in range(plan.num_rounds()):
        nb = plan.bucket_bytes(r)
        bucket = torch.full((nb,), 0x5A, dtype=torch.uint8)
        view = bucket.numpy().view(bits_d)
        for v in range(nt):
            if t_owner[v] == rank:
                run_table(plan.rank_tiles(wb.WB_TABLE_PACK, r, v), src, None, view, wl.src_dtype, wl.dst_dtype)
        sent += wbdist.exchange_regions(d, bucket, plan.bucket_regions(r), t_owner, r_owner, rank)
        for v in range(nr):
            if r_owner[v] == rank:
                run_table(plan.rank_tiles(wb.WB_TABLE_UNPACK, r, v), None, dst, view, wl.dst_dtype, wl.dst_dtype,
                          write_counts=wrote)
    # replicas on ranks of the other process were written here on their behalf (a peer store on GPUs):
    # fold the processes' writes together; every described element must have been written exactly once
    ok = True
    for k in range(len(dst)):
        cnt = torch.from_numpy(wrote[k].copy())
        val = torch.from_numpy(np.where(wrote[k] > 0, dst[k].astype(np.int64), 0))
        d.all_reduce(cnt); d.all_reduce(val)
        dst[k] = np.where(cnt.numpy() > 0, val.numpy(), fill).astype(bits_d)
        wrote[k] = cnt.numpy()
    want = remap_oracle(ckpt_shapes(wl), wl.trainer.tensors, wl.trainer.slices, wl.rollout.tensors, wl.rollout.slices,
                        full, [np.full(int(t["numel"]), fill, bits_d) for t in wl.rollout.tensors])
    described = [np.zeros(int(t["numel"]), bool) for t in wl.rollout.tensors]
    for s in wl.rollout.slices:
        i = np.arange(int(s["nr"]))[:, None]; j = np.arange(int(s["nc"]))[None, :]
        described[int(s["tensor"])][int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])] = True
    for k in range(len(dst)):
        ok = ok and np.array_equal(dst[k], want.dst[k]) and np.array_equal(wrote[k] == 1, described[k]) \
            and int(wrote[k].max()) <= 1
    result[name] = {"ok": bool(ok), "sent": sent, "rounds": plan.num_rounds()}
print(json.dumps(result))
d.destroy_process_group()
"""


def test_rank_sharded_transfer_on_two_gloo_processes(tmp_path):
    """Section 3.2's receive stage with the virtual ranks split over two processes: each packs only its own
    trainer ranks' slabs (the other ranks' tensors are poisoned), the (receiver, sender) regions are
    exchanged, each assembles only its own rollout ranks' payloads; the result is the oracle's."""
    cases = [("cfg1b", "full", 1 << 20), ("cfg3", "small", 1 << 20), ("cfg5", "small", 1 << 18)]
    script = tmp_path / "sharded.py"
    script.write_text(SHARDED_WORKER % {"root": ROOT, "tests": os.path.join(ROOT, "tests"), "cases": cases})
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29613", WORLD_SIZE="2")
    procs = []
    for r in range(2):
        e = dict(env, RANK=str(r), LOCAL_RANK=str(r))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=600) for p in procs]
    for p, (o, err) in zip(procs, outs):
        assert p.returncode == 0, err[-3000:]
    import json
    total_sent = {}
    for o, _ in outs:
        res = json.loads(o.strip().splitlines()[-1])
        for name, v in res.items():
            assert v["ok"], name
            total_sent[name] = total_sent.get(name, 0) + v["sent"]
    # cfg3 (8 trainer ranks -> 2 rollout ranks, 4 + 1 each side of the cut): something must cross
    assert total_sent["cfg3"] > 0 and total_sent["cfg5"] > 0
