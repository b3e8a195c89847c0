"""wb_remap_static: the remap for callers that cannot allocate device memory (an inference
engine whose KV-cache pool already owns all free HBM, a fixed start-up memory budget).  Its
tile table lives in the library's fixed 4 MiB device array instead of a cudaMalloc'd arena.
The output must equal the CPU oracle's rollout tensors, and what the ordinary bind + wb_remap
path writes, bit for bit, on two calls in a row that use different plans (so stale contents of
the shared array would show).

This file is named to be collected last."""
import gc

import numpy as np
import pytest
import torch

from gpu_util import DeviceCase, oracle_for
from paper_2609_25442_b200 import binding as wb
from paper_2609_25442_b200.device import RankArenas
from wb_workloads import WB_BF16, Layout, make_workload

pytestmark = pytest.mark.gpu


def _reference_and_static(device, name, scale, **opts):
    case = DeviceCase(make_workload(name, scale), device, **opts)
    want = oracle_for(case).dst                           # the CPU oracle
    case.plan.remap()                                     # existing entry point
    torch.cuda.synchronize()
    for got, w in zip(case.dst_bits(), want):
        assert np.array_equal(got, w)
    case.reset_dst()
    # a second, never-bound plan of the same layouts goes through the no-allocation entry point
    plan = wb.Plan(wb.Layout(case.trainer.tensors, case.trainer.slices),
                   wb.Layout(case.rollout.tensors, case.rollout.slices), **opts)
    return case, plan, want


def test_static_scratch_matches_bound_remap_twice_in_a_row():
    device = torch.device("cuda:0")
    stream = torch.cuda.current_stream().cuda_stream
    a_case, a_plan, a_want = _reference_and_static(device, "cfg3", "small")      # fp32 -> bf16, fan-out
    b_case, b_plan, b_want = _reference_and_static(device, "cfg1b", "full")      # padding, replicas
    gc.collect()                                  # plans of earlier tests free their arenas now, not later
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    wb.wb_remap_static(a_plan, a_case.src.pointers(), a_case.dst.pointers(), 0, stream)
    wb.wb_remap_static(b_plan, b_case.src.pointers(), b_case.dst.pointers(), wb.WB_STATIC_SYNC_CHECK, stream)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before            # no device memory was taken
    for got, want in zip(a_case.dst_bits(), a_want):
        assert np.array_equal(got, want)
    for got, want in zip(b_case.dst_bits(), b_want):
        assert np.array_equal(got, want)
    assert a_case.gaps_intact() and b_case.gaps_intact()
    # and once more with the first plan: the array now holds the second plan's table
    a_case.reset_dst()
    wb.wb_remap_static(a_plan, a_case.src.pointers(), a_case.dst.pointers(), wb.WB_STATIC_SYNC_CHECK, stream)
    for got, want in zip(a_case.dst_bits(), a_want):
        assert np.array_equal(got, want)


def test_static_scratch_refuses_plans_beyond_its_limit():
    device = torch.device("cuda:0")
    n = 100_000_000                                  # one 200 MB tensor cut into ~98,000 small tiles
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T", 0, WB_BF16, n)
    rl.add_tensor("R", 0, WB_BF16, n)
    tl.add_slice(0, 0, n, 1, 0, 1, n, 0, 0, 1, n)
    rl.add_slice(0, 0, n, 1, 0, 1, n, 0, 0, 1, n)
    tl.freeze(); rl.freeze()
    big = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices), tile_bytes=4096)
    assert big.stats()["n_tiles_remap"] * 48 > wb.WB_STATIC_SCRATCH_BYTES
    src = RankArenas(tl.tensors, device, fill_byte=1)
    dst = RankArenas(rl.tensors, device, fill_byte=0xCD)
    with pytest.raises(wb.WbError) as e:
        wb.wb_remap_static(big, src.pointers(), dst.pointers())
    assert e.value.name == "WB_ERR_STATIC_LIMIT"
    torch.cuda.synchronize()
    assert bool((dst.arenas[0] == 0xCD).all())        # nothing was launched
    # the same layouts with the default tile size fit and run
    ok = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices))
    wb.wb_remap_static(ok, src.pointers(), dst.pointers(), wb.WB_STATIC_SYNC_CHECK)
    assert torch.equal(dst.tensors[0].view(torch.int16), src.tensors[0].view(torch.int16))
