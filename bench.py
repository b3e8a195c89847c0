#!/usr/bin/env python
"""Benchmark of the weight remap: full-model GB/s moved (read + write) on B200.

A step is one pass of the whole hot path over one model: wb_remap on a bound plan (one
persistent launch).  Layout description and planning happen once before the timed region,
as in the paper (plan once in `connect`, execute every update); their wall time is reported
in `config.plan_build_s`.  Prints one JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg4|cfg5]
  python bench.py --impl reference ...      # the CPU oracle on a bounded sample, same metric
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from wb_workloads import TENSOR_DTYPE, SLICE_DTYPE, make_workload  # noqa: E402

METRIC = "full-model weight remap GB/s (read+write)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one wb_remap launch: the ratio traffic / algorithmic
# bytes measured by ncu on the `large` scale of the same layout (profiles/wb_exec_kernel_large_scale_ncu_full.md),
# times the full-size algorithmic bytes (traffic grows in proportion to the bytes moved); cfg4 moves through
# the same direct bulk-copy path as cfg2 and takes its ratio
NCU_TRAFFIC_RATIO = {"cfg2": 0.988, "cfg3": 0.994, "cfg4": 0.988, "cfg5": 1.060}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--scale", default="full")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tile-bytes", type=int, default=0)
    ap.add_argument("--grid-ctas", type=int, default=0)
    ap.add_argument("--path", default="remap",
                    choices=["remap", "pack_unpack", "rounds", "rounds_serial", "rounds_fp8", "rounds_fp8_pipelined", "rounds_fp8_fused", "extract",
                             "extract_chunks"],
                    help="remap: fused launch; pack_unpack: wb_pack + wb_unpack per round on one stream; "
                         "rounds: wb_transfer_rounds (depth-2 buckets, two streams); rounds_serial: its "
                         "unpipelined baseline; rounds_fp8: amax pass, then per round pack, quantise the bucket to FP8, "
                         "dequantise, unpack; extract: source-map extraction kernel; extract_chunks: Algorithm 1's 8-bit chunk "
                         "passes with carries (entries shipped per pass with and without them)")
    ap.add_argument("--cuda-graph", action="store_true",
                    help="remap path: replay the launch from a captured CUDA graph (for the launch-bound tiny model)")
    ap.add_argument("--budget-mib", type=int, default=0, help="bucket budget per round (0: the 4 GiB default)")
    ap.add_argument("--budget-sweep", default="",
                    help="comma-separated bucket budgets in MiB: time the pipelined and the serial rounds "
                         "path for each and add the list to the JSON line (the buffer-size sensitivity "
                         "experiment of the paper's Appendix D, on the kernels alone)")
    ap.add_argument("--static-schedule", action="store_true",
                    help="fixed per-block tile ranges instead of run-time batches")
    ap.add_argument("--also", default="cfg4,cfg3,cfg5",
                    help="default run (cfg2, fused remap, one GPU): after the headline measurement, time these "
                         "workloads too through the same wb_remap call and list them in config.workloads "
                         "(empty string: none)")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) every few milliseconds
    while the timed region runs."""

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.stop_flag = False
        self.thread = None
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def start(self):
        if self.nv is None:
            return
        self.thread = threading.Thread(target=self._poll, daemon=True)
        self.thread.start()

    def _poll(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                self.samples.append((float(mhz), int(reasons)))
            except Exception:
                break
            time.sleep(0.002)

    def stop(self):
        if self.nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.stop_flag = True
        self.thread.join(timeout=2)
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        seen = set()
        for _, r in self.samples:
            for n, bit in names.items():
                if r & bit:
                    seen.add(n)
        sm = [m for m, _ in self.samples]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(seen), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# the CPU baseline: the oracle, as it stands, on a bounded sample of the same workload
# ------------------------------------------------------------------------------------------------
def oracle_sample(wl, fetch_src, budget_elems=60_000_000):
    """Run the oracle on the first checkpoint tensors of the workload (in order) up to about
    `budget_elems` elements.  Only the local tensors those touch are materialised on the host.
    Returns (seconds, bytes moved, description)."""
    from oracle import remap_oracle

    picked, total = [], 0
    for i, c in enumerate(wl.ckpt):      # in order, skipping tensors that would overshoot
        if total + c.numel > budget_elems:
            continue
        picked.append(i)
        total += c.numel
        if total >= 0.9 * budget_elems:
            break
    pick = np.array(picked)

    def restrict(layout):
        keep = np.isin(layout.slices["ckpt"], pick)
        sl = layout.slices[keep].copy()
        used = np.unique(sl["tensor"])
        remap = {int(t): k for k, t in enumerate(used)}
        sl["tensor"] = np.array([remap[int(t)] for t in sl["tensor"]], dtype=np.uint32)
        return layout.tensors[used].copy(), sl, [int(t) for t in used]

    t_t, t_s, t_used = restrict(wl.trainer)
    r_t, r_s, _ = restrict(wl.rollout)
    if fetch_src is not None:
        src = [fetch_src(k) for k in t_used]
    else:
        # seeded checkpoint values for the sampled tensors, put into the trainer buffers through the
        # trainer's own slice list (so replicas agree, as after a real load_weights)
        bits_dt = np.uint32 if wl.src_dtype == 0 else np.uint16
        src = [np.zeros(int(t["numel"]), bits_dt) for t in t_t]
        vals = {}
        for sl in t_s:
            c = int(sl["ckpt"])
            if c not in vals:
                vals[c] = to_bits_np(wl.ckpt_values(c))          # the workload's own seeded generator
            i = np.arange(int(sl["nr"]), dtype=np.int64)[:, None]
            j = np.arange(int(sl["nc"]), dtype=np.int64)[None, :]
            g = (int(sl["r0"]) + i) * int(sl["ckpt_cols"]) + int(sl["c0"]) + j
            x = int(sl["local_off"]) + i * int(sl["stride_r"]) + j * int(sl["stride_c"])
            src[int(sl["tensor"])][x] = vals[c][g]
    shapes = [(c.rows, c.cols) for c in wl.ckpt]
    t0 = time.perf_counter()
    res = remap_oracle(shapes, t_t, t_s, r_t, r_s, src)
    dt = time.perf_counter() - t0
    es = 4 if wl.src_dtype == 0 else 2
    ed = 4 if wl.dst_dtype == 0 else 2
    moved = res.n_ids_consumed * es + res.n_written * ed
    desc = (f"the first {len(picked)} checkpoint tensors of {wl.name} that fit a {budget_elems}-element budget "
            f"({res.n_ids_consumed} elements), numpy oracle, single thread")
    return dt, moved, desc


def to_bits_np(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu().contiguous().reshape(-1)
    if t.dtype == torch.float32:
        return t.view(torch.int32).numpy().view(np.uint32)
    return t.view(torch.int16).numpy().view(np.uint16)


def run_reference(args):
    """--impl reference: the oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = make_workload(args.workload, args.scale)
    budget = 20_000_000
    times, moved, desc = [], 0, ""
    for _ in range(args.warmup):
        oracle_sample(wl, None, budget)
    for _ in range(args.steps):
        dt, moved, desc = oracle_sample(wl, None, budget)
        times.append(dt)
    ms = 1e3 * sum(times) / max(len(times), 1)
    value = moved / (ms * 1e-3) / 1e9 if times else 0.0
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "u16" if wl.src_dtype == 1 else "f32->bf16",
           "data": "synthetic", "config": {"workload": wl.name, "note": "each step = bounded sample"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
                            "sample": desc},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def run_extract(args):
    """--path extract: the diff2 + compaction kernel of source-map extraction over the int64 id
    fields the trainer's load_weights produces (first loader groups, up to ~4 GB of ids)."""
    from paper_2609_25442_b200 import binding as wb
    from paper_2609_25442_b200.device import require_cuda
    require_cuda()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    wl = make_workload(args.workload, args.scale)
    fields, total = [], 0
    for ckpt_idx, fn in wl.trainer_groups():
        for _, t in fn([wl.ckpt_ids(i, dev) + 1 for i in ckpt_idx]).items():
            t = (t.reshape(1, -1) if t.dim() == 1 else t.reshape(-1, t.shape[-1])).clamp_min(0).contiguous()
            fields.append(t)
            total += t.numel()
        if total * 8 >= 4e9:
            break
    cap = 1 << 20
    out = torch.zeros(cap * 24, dtype=torch.uint8, device=dev)
    count = torch.zeros(1, dtype=torch.int64, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def step():
        count.zero_()
        for f in fields:
            wb.wb_diff2_nonzeros(f.data_ptr(), wb.WB_ID_I64, f.shape[0], f.shape[1], out.data_ptr(), cap,
                                 count.data_ptr(), stream)
    # the same fields in one launch
    desc = np.array([(f.data_ptr(), f.shape[0], f.shape[1], wb.WB_ID_I64, k) for k, f in enumerate(fields)],
                    dtype=wb.DIFF2_FIELD_DTYPE)
    nb = wb.wb_diff2_batch_scratch_bytes(len(desc))
    scratch = torch.zeros(max(nb, 16), dtype=torch.uint8, device=dev)
    tout = torch.zeros(cap * 32, dtype=torch.uint8, device=dev)

    def step_batched():
        count.zero_()
        wb.wb_diff2_nonzeros_batch(desc, scratch.data_ptr(), nb, tout.data_ptr(), cap, count.data_ptr(), stream)

    def timed(fn):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.steps
    ms_batched = timed(step_batched)
    nz_batched = int(count.item())
    ms = timed(step)
    gbs = total * 8 / (ms * 1e-3) / 1e9
    peak = FALLBACK_HBM_GBS
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak = float(json.load(f)["hbm_gbs"])
    except Exception:
        pass
    print(json.dumps({"metric": "diff2 id-field scan GB/s (int64 ids read)", "value": gbs, "unit": "GB/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "int64", "data": "synthetic",
                      "config": {"workload": wl.name, "path": "extract", "fields": len(fields),
                                 "elements": total, "nonzeros": int(count.item()), "nonzeros_batched": nz_batched,
                                 "batched_ms": ms_batched, "batched_gbs": total * 8 / (ms_batched * 1e-3) / 1e9,
                                 "l2": "inputs_larger_than_l2"},
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s",
                                   "frac": gbs / peak, "traffic": None, "kernel": "wb_diff2_kernel"},
                      "gpu_launches": args.steps * len(fields)}))


def run_extract_chunks(args):
    """--path extract_chunks: Algorithm 1's inner loop on the trainer's id fields held as 8-bit chunks in bf16
    tensors (first loader groups, up to ~2^28 elements): per pass, the entries that cross to the host with the
    carry construction (digits + strided carry differences) and without it (plain diff2 of the chunk), and
    the device time of the pass."""
    from paper_2609_25442_b200 import binding as wb
    from paper_2609_25442_b200.device import require_cuda
    require_cuda()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    wl = make_workload(args.workload, args.scale)
    fields, total = [], 0
    for ckpt_idx, fn in wl.trainer_groups():
        for _, t in fn([wl.ckpt_ids(i, dev) + 1 for i in ckpt_idx]).items():
            t = (t.reshape(1, -1) if t.dim() == 1 else t.reshape(-1, t.shape[-1])).clamp_min(0).contiguous()
            fields.append(t)
            total += t.numel()
        if total >= (1 << 28):
            break
    b = 8
    K = -(-((16 * (wl.ckpt_numel() + 1)).bit_length() + 1) // b)
    cap = 1 << 22
    zo = torch.zeros(cap * 24, dtype=torch.uint8, device=dev)
    go = torch.zeros(cap * 24, dtype=torch.uint8, device=dev)
    counts = torch.zeros(2, dtype=torch.int64, device=dev)
    nb = max(wb.wb_diff2_chunk_scratch_bytes(f.shape[0], f.shape[1]) for f in fields)
    scratch = torch.empty(nb, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    carries = [None] * len(fields)
    passes = []
    for _ in range(3):                                   # untimed: module load, first-launch costs
        f = fields[-1]
        counts.zero_()
        wb.wb_diff2_chunk_pass((f & 255).to(torch.bfloat16).data_ptr(), wb.WB_ID_BF16, f.shape[0], f.shape[1], b, 0, 0, 0,
                               scratch.data_ptr(), nb, zo.data_ptr(), cap, counts.data_ptr(), go.data_ptr(), cap,
                               counts.data_ptr() + 8, stream)
        torch.cuda.synchronize()
    for k in range(K):
        row = {"pass": k, "digits": 0, "carry_records": 0, "plain": 0, "ms": 0.0, "plain_ms": 0.0}
        for n, f in enumerate(fields):
            chunk = ((f >> (b * k)) & ((1 << b) - 1)).to(torch.bfloat16)       # what load_weights leaves in a bf16 tensor
            cin = carries[n]
            counts.zero_()
            a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            wb.wb_diff2_chunk_pass(chunk.data_ptr(), wb.WB_ID_BF16, f.shape[0], f.shape[1], b, k,
                                   cin.data_ptr() if cin is not None else 0, 0 if cin is None else cin.numel() // 24,
                                   scratch.data_ptr(), nb, zo.data_ptr(), cap, counts.data_ptr(), go.data_ptr(), cap,
                                   counts.data_ptr() + 8, stream)
            e.record()
            torch.cuda.synchronize()
            row["ms"] += a.elapsed_time(e)
            nz, ng = (int(x) for x in counts.cpu())
            assert nz <= cap and ng <= cap
            row["digits"] += nz
            row["carry_records"] += ng
            # the records go to the host and come back for the next pass
            host = go[:ng * 24].cpu()
            carries[n] = host.to(dev) if ng else None
            counts.zero_()
            a.record()
            wb.wb_diff2_nonzeros(chunk.data_ptr(), wb.WB_ID_BF16, f.shape[0], f.shape[1], zo.data_ptr(), cap,
                                 counts.data_ptr(), stream)
            e.record()
            torch.cuda.synchronize()
            row["plain_ms"] += a.elapsed_time(e)
            row["plain"] += int(counts[0].item())
        row["gbs_field_bytes"] = total * 2 / (row["ms"] * 1e-3) / 1e9
        passes.append(row)
    peak, peak_src = hbm_peak()
    ms = sum(r["ms"] for r in passes) / K
    gbs = total * 2 / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "chunk pass with carries, GB/s of id-chunk field read (bf16 elements)", "value": gbs,
                      "unit": "GB/s", "n_gpus": 1, "steps": K, "warmup": 0, "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "bf16 chunks -> int", "data": "synthetic",
                      "config": {"workload": wl.name, "path": "extract_chunks", "fields": len(fields), "elements": total,
                                 "chunk_bits": b, "passes": passes, "l2": "inputs_larger_than_l2",
                                 "entries_shipped_with_carries": sum(r["digits"] + r["carry_records"] for r in passes),
                                 "entries_shipped_plain": sum(r["plain"] for r in passes)},
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                   "traffic": None, "peak_source": peak_src, "kernel": "wb_chunk_pass_kernel",
                                   "note": "algorithmic bytes = the 2-byte field; the one-byte carry field is read and "
                                           "written by the pass and read again by the strided difference"},
                      "gpu_launches": K * len(fields) * 2}))


def hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measure_remap(name, scale, args, dev, local_rank):
    """One more workload through the same call as the headline one: build, bind, warm up, time
    `steps` wb_remap launches with CUDA events on the launching stream, sample the clocks, check the
    plan's error word.  Returns the entry of config.workloads; releases everything it allocated."""
    from paper_2609_25442_b200 import binding as wb
    from paper_2609_25442_b200.device import RankArenas, bind
    wl = make_workload(name, scale)
    es, ed = (4 if wl.src_dtype == 0 else 2), (4 if wl.dst_dtype == 0 else 2)
    need = sum(int(t["numel"]) for t in wl.trainer.tensors) * es + sum(int(t["numel"]) for t in wl.rollout.tensors) * ed
    free = torch.cuda.mem_get_info(dev)[0]
    entry = {"workload": wl.name, "dtype": {0: "f32", 1: "bf16"}[wl.src_dtype] + "->" + {0: "f32", 1: "bf16"}[wl.dst_dtype]}
    if need * 1.02 + (2 << 30) > free:
        entry["skipped"] = f"needs {need / 1e9:.1f} GB of device memory, {free / 1e9:.1f} GB free"
        return entry
    t0 = time.perf_counter()
    plan = wb.Plan(wb.Layout(wl.trainer.tensors, wl.trainer.slices), wb.Layout(wl.rollout.tensors, wl.rollout.slices),
                   tile_bytes=args.tile_bytes, grid_ctas=args.grid_ctas)
    plan_s = time.perf_counter() - t0
    stats = plan.stats()
    src = RankArenas(wl.trainer.tensors, dev, fill_byte=0)
    dst = RankArenas(wl.rollout.tensors, dev, fill_byte=0)
    wl.load_side("trainer", lambda i: wl.ckpt_values(i, dev), lambda k, t: src.tensors[k].copy_(t))
    bind(plan, src, dst)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream
    bytes_step = stats["src_bytes_read"] + stats["dst_bytes_written"]
    for _ in range(max(args.warmup, 3)):
        plan.remap(stream)
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    evs[0].record()
    for k in range(args.steps):
        plan.remap(stream)
        evs[k + 1].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    plan.check()                                   # a bounded wait that ran out inside a launch fails the run
    per_step = [evs[k].elapsed_time(evs[k + 1]) for k in range(args.steps)]
    ms = float(np.mean(per_step))
    gbs = bytes_step / (ms * 1e-3) / 1e9
    peak, peak_src = hbm_peak()
    entry.update({"bytes_per_step": bytes_step, "ms_per_step": ms, "best_ms": float(min(per_step)), "gbs": gbs,
                  "frac_of_measured": gbs / peak, "peak_source": peak_src, "frac_of_8TBs": gbs / 8000.0,
                  "tiles": stats["n_tiles_remap"], "plan_build_s": plan_s, "steps": args.steps,
                  "gpu_launches": args.steps, "l2": "inputs_larger_than_l2", "clocks": clocks,
                  "traffic": int(NCU_TRAFFIC_RATIO[name] * bytes_step) if name in NCU_TRAFFIC_RATIO else None})
    del plan, src, dst
    torch.cuda.empty_cache()
    return entry


# ------------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.path == "extract":
        run_extract(args)
        return
    if args.path == "extract_chunks":
        run_extract_chunks(args)
        return

    from paper_2609_25442_b200 import binding as wb
    from paper_2609_25442_b200.device import RankArenas, bind, require_cuda

    from paper_2609_25442_b200 import dist as wbdist
    rank, local_rank, world = wbdist.rank_info()
    require_cuda()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = wbdist.init("nccl", dev)

    # ---- inputs: resident in HBM before the timed region -------------------------------------
    wl = make_workload(args.workload, args.scale)
    t0 = time.perf_counter()
    tl = wb.Layout(wl.trainer.tensors, wl.trainer.slices)
    rl = wb.Layout(wl.rollout.tensors, wl.rollout.slices)
    plan = wb.Plan(tl, rl, tile_bytes=args.tile_bytes, grid_ctas=args.grid_ctas,
                   bucket_budget_bytes=args.budget_mib << 20,
                   flags=wb.WB_PLAN_STATIC_SCHEDULE if args.static_schedule else 0)
    plan_s = time.perf_counter() - t0
    stats = plan.stats()
    src = RankArenas(wl.trainer.tensors, dev, fill_byte=0)
    dst = RankArenas(wl.rollout.tensors, dev, fill_byte=0)
    wl.load_side("trainer", lambda i: wl.ckpt_values(i, dev), lambda k, t: src.tensors[k].copy_(t))
    bind(plan, src, dst)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream
    bytes_step = stats["src_bytes_read"] + stats["dst_bytes_written"]

    n_rounds = plan.num_rounds()
    buckets = None
    if args.path != "remap":
        buckets = [torch.empty(max(plan.bucket_bytes(r) for r in range(n_rounds)), dtype=torch.uint8, device=dev)
                   for _ in range(2)]

    amax = qbucket = None
    qbuckets = None
    if args.path in ("rounds_fp8", "rounds_fp8_pipelined", "rounds_fp8_fused"):
        amax = torch.zeros(plan.num_ckpts(), dtype=torch.float32, device=dev)
        qbuckets = [torch.empty(max(plan.qbucket_bytes(r) for r in range(n_rounds)), dtype=torch.uint8, device=dev)
                    for _ in range(2)]
        qbucket = qbuckets[0]

    graph = None
    if args.cuda_graph and args.path == "remap":
        plan.remap(stream)                               # the first call sets the kernel attribute
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        cap = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(cap):
            with torch.cuda.graph(graph, stream=cap):
                plan.remap(torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()

    def step():
        if args.path == "remap":
            if graph is not None:
                graph.replay()
            else:
                plan.remap(stream)
            return 1
        if args.path == "rounds_fp8_fused":
            plan.transfer_rounds_fp8_fused(qbuckets[0].data_ptr(), qbuckets[1].data_ptr(), amax.data_ptr(), stream)
            return 1 + 2 * n_rounds
        if args.path == "rounds_fp8_pipelined":
            plan.transfer_rounds_fp8(buckets[0].data_ptr(), buckets[1].data_ptr(), qbuckets[0].data_ptr(),
                                     qbuckets[1].data_ptr(), amax.data_ptr(), stream)
            return 1 + 4 * n_rounds
        if args.path == "rounds_fp8":
            plan.absmax(amax.data_ptr(), stream)
            for r in range(n_rounds):
                b = buckets[r % 2].data_ptr()
                plan.pack(r, b, stream)
                plan.bucket_quantize(r, b, qbucket.data_ptr(), amax.data_ptr(), stream)
                plan.bucket_dequantize(r, qbucket.data_ptr(), b, amax.data_ptr(), stream)
                plan.unpack(r, b, stream)
            return 1 + 4 * n_rounds
        if args.path in ("rounds", "rounds_serial"):
            plan.transfer_rounds(buckets[0].data_ptr(), buckets[1].data_ptr(),
                                 wb.WB_ROUNDS_SERIAL if args.path == "rounds_serial" else 0, stream)
            return 2 * n_rounds
        for r in range(n_rounds):
            b = buckets[r % 2].data_ptr()
            plan.pack(r, b, stream)
            plan.unpack(r, b, stream)
        return 2 * n_rounds

    def barrier():
        wbdist.barrier(dist, cuda=True)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    launches = 0
    torch.cuda.nvtx.range_push("timed")
    evs[0].record()
    for k in range(args.steps):
        launches += step()
        evs[k + 1].record()
    barrier()
    torch.cuda.nvtx.range_pop()
    clocks = sampler.stop() if rank == 0 else None
    plan.check()                                       # a bounded wait that ran out inside a launch fails the run
    total_ms = evs[0].elapsed_time(evs[-1])
    per_step = [evs[k].elapsed_time(evs[k + 1]) for k in range(args.steps)]
    total_ms = wbdist.max_over_ranks(dist, total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = wbdist.aggregate_gbs(world, bytes_step, ms_per_step)

    # ---- roofline of the dominant (only) kernel --------------------------------------------------
    peak, peak_src = hbm_peak()
    launch_ms = float(np.mean(per_step)) / (1 if args.path == "remap" else 1)
    achieved = bytes_step / (launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak,
                "traffic": (int(NCU_TRAFFIC_RATIO[args.workload] * bytes_step)
                            if args.workload in NCU_TRAFFIC_RATIO and args.path == "remap" else None),
                "traffic_source": "ncu on the large scale of this layout, scaled by bytes moved",
                "peak_source": peak_src, "kernel": "wb_exec_kernel", "best_ms": float(min(per_step)),
                "frac_of_nominal_8TBs": achieved / 8000.0}

    # ---- FP8 path: each of the three extra kernels on its own, over all rounds ----------------------
    fp8 = None
    if args.path == "rounds_fp8_fused" and rank == 0:
        def timed(fn, reps=5):
            fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps
        ed_ = 4 if wl.dst_dtype == 0 else 2
        bucket_elems = sum(plan.qbucket_bytes(r) for r in range(n_rounds))
        t_a = timed(lambda: plan.absmax(amax.data_ptr(), stream))
        t_p = timed(lambda: [plan.pack_fp8(r, qbuckets[r % 2].data_ptr(), amax.data_ptr(), stream) for r in range(n_rounds)])
        t_u = timed(lambda: [plan.unpack_fp8(r, qbuckets[r % 2].data_ptr(), amax.data_ptr(), stream) for r in range(n_rounds)])
        peak_, _src = hbm_peak()
        fp8 = {"absmax_ms": t_a, "absmax_gbs": stats["src_bytes_read"] / t_a / 1e6,
               "pack_fp8_ms": t_p, "pack_fp8_gbs": (stats["src_bytes_read"] + bucket_elems) / t_p / 1e6,
               "unpack_fp8_ms": t_u, "unpack_fp8_gbs": (bucket_elems + stats["dst_bytes_written"]) / t_u / 1e6,
               "bucket_elements": bucket_elems, "wire_bytes_fp8": bucket_elems, "wire_bytes_unquantised": bucket_elems * ed_,
               "algorithmic_bytes": stats["src_bytes_read"] * 2 + bucket_elems * 2 + stats["dst_bytes_written"]}
        for kname in ("absmax", "pack_fp8", "unpack_fp8"):
            fp8[kname + "_frac_of_measured"] = fp8[kname + "_gbs"] / peak_
    if args.path == "rounds_fp8" and rank == 0:
        def timed(fn, reps=5):
            fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps
        es_, ed_ = (4 if wl.src_dtype == 0 else 2), (4 if wl.dst_dtype == 0 else 2)
        elems = stats["dst_bytes_written"] // ed_          # one bucket element per rollout element written once
        bucket_elems = sum(plan.qbucket_bytes(r) for r in range(n_rounds))
        t_a = timed(lambda: plan.absmax(amax.data_ptr(), stream))
        t_q = timed(lambda: [plan.bucket_quantize(r, buckets[0].data_ptr(), qbucket.data_ptr(), amax.data_ptr(), stream)
                             for r in range(n_rounds)])
        t_d = timed(lambda: [plan.bucket_dequantize(r, qbucket.data_ptr(), buckets[0].data_ptr(), amax.data_ptr(), stream)
                             for r in range(n_rounds)])
        fp8 = {"absmax_ms": t_a, "absmax_gbs": stats["src_bytes_read"] / t_a / 1e6,
               "quantize_ms": t_q, "quantize_gbs": bucket_elems * (ed_ + 1) / t_q / 1e6,
               "dequantize_ms": t_d, "dequantize_gbs": bucket_elems * (ed_ + 1) / t_d / 1e6,
               "bucket_elements": bucket_elems, "wire_bytes_fp8": bucket_elems, "wire_bytes_unquantised": bucket_elems * ed_}

    # ---- bucket budget sweep (rounds path) ---------------------------------------------------------
    sweep = None
    if args.budget_sweep and rank == 0 and world == 1:
        sweep = []
        del buckets
        for mib in [int(x) for x in args.budget_sweep.split(",") if x]:
            p2 = wb.Plan(tl, rl, tile_bytes=args.tile_bytes, grid_ctas=args.grid_ctas, bucket_budget_bytes=mib << 20)
            bind(p2, src, dst)
            nr = p2.num_rounds()
            nb = max(p2.bucket_bytes(r) for r in range(nr))
            bk = [torch.empty(nb, dtype=torch.uint8, device=dev) for _ in range(2)]
            row = {"budget_mib": mib, "rounds": nr, "bucket_bytes": nb}
            for key, flags in (("pipelined_ms", 0), ("serial_ms", wb.WB_ROUNDS_SERIAL)):
                for _ in range(3):
                    p2.transfer_rounds(bk[0].data_ptr(), bk[1].data_ptr(), flags, stream)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(args.steps):
                    p2.transfer_rounds(bk[0].data_ptr(), bk[1].data_ptr(), flags, stream)
                b.record()
                torch.cuda.synchronize()
                row[key] = a.elapsed_time(b) / args.steps
            p2.check()
            sweep.append(row)
            del bk, p2

    # ---- end to end through the host-buffer entry point -------------------------------------------
    e2e = None
    if not args.no_e2e:
        try:
            host_src = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in src.tensors]
            host_dst = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in dst.tensors]
            pinned = True
        except RuntimeError:
            host_src = [torch.empty(t.shape, dtype=t.dtype) for t in src.tensors]
            host_dst = [torch.empty(t.shape, dtype=t.dtype) for t in dst.tensors]
            pinned = False
        for h, t in zip(host_src, src.tensors):
            h.copy_(t)
        hs = [t.data_ptr() for t in host_src]
        hd = [t.data_ptr() for t in host_dst]
        plan.remap_host(hs, hd, stream)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.e2e_steps):
            plan.remap_host(hs, hd, stream)
        b.record()
        barrier()
        e_ms = a.elapsed_time(b)
        e_ms = wbdist.max_over_ranks(dist, e_ms, dev) / args.e2e_steps
        e2e = {"value": wbdist.aggregate_gbs(world, bytes_step, e_ms), "unit": UNIT,
               "h2d_bytes_per_step": src.total_bytes(), "d2h_bytes_per_step": dst.total_bytes(),
               "ms_per_step": e_ms, "steps": args.e2e_steps, "pinned": pinned}
        del host_src, host_dst

    # ---- CPU baseline (rank 0, N = 1 only) -----------------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dt, moved, desc = oracle_sample(wl, lambda k: to_bits_np(src.tensors[k]))
        cpu = {"value": moved / dt / 1e9, "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
               "sample": desc, "seconds": dt}

    # ---- the other workloads, through the same call (default run on one GPU only) -------------------
    others = None
    if rank == 0 and world == 1 and args.path == "remap" and args.workload == "cfg2" and args.scale == "full" and args.also:
        headline = {"workload": wl.name, "dtype": {0: "f32", 1: "bf16"}[wl.src_dtype] + "->" + {0: "f32", 1: "bf16"}[wl.dst_dtype],
                    "bytes_per_step": bytes_step, "ms_per_step": ms_per_step, "best_ms": float(min(per_step)),
                    "gbs": value, "frac_of_measured": value / peak, "peak_source": peak_src,
                    "frac_of_8TBs": value / 8000.0, "tiles": stats["n_tiles_remap"], "plan_build_s": plan_s,
                    "steps": args.steps, "gpu_launches": launches, "l2": "inputs_larger_than_l2", "clocks": clocks,
                    "traffic": roofline["traffic"]}
        del plan, src, dst, buckets
        torch.cuda.empty_cache()
        others = [headline]
        for name in [x for x in args.also.split(",") if x]:
            others.append(measure_remap(name, args.scale, args, dev, local_rank))

    if rank == 0:
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
               "scaling": "weak", "vs_baseline": None,
               "dtype": {0: "f32", 1: "bf16"}[wl.src_dtype] + "->" + {0: "f32", 1: "bf16"}[wl.dst_dtype],
               "data": "synthetic",
               "config": {"workload": wl.name, "path": args.path, "l2": "inputs_larger_than_l2",
                          "bytes_per_step": bytes_step, "tiles": stats["n_tiles_remap"],
                          "slabs": stats["n_slabs"], "rounds": stats["n_rounds"],
                          "grid_ctas": stats["grid_ctas"], "tile_bytes": stats["tile_bytes"],
                          "plan_build_s": plan_s, "replicas_per_gpu": 1,
                          "schedule": "static" if args.static_schedule else "dynamic",
                          "cuda_graph": bool(graph is not None),
                          "multi_gpu": "independent replicas, no collective"},
               "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
               "gpu_launches": launches, "pct_of_8TBs_nominal": 100.0 * value / world / 8000.0}
        if others is not None:
            out["config"]["workloads"] = others
        if sweep is not None:
            out["budget_sweep"] = sweep
        if fp8 is not None:
            out["fp8"] = fp8
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
