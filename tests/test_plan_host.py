"""Host logic of the library: C-ABI surface, layout validation, the planner's invariants,
and the tile tables executed on the host against the oracle.  No GPU needed."""
import ctypes
import os
import re

import numpy as np
import pytest

from helpers import ckpt_shapes, fuzz_case, random_bits, scatter_checkpoint, to_bits
from oracle import checkpoint_view, remap_oracle
from oracle.cast import cast_bits
from paper_2609_25442_b200 import binding as wb
from plan_interp import run_table
from wb_workloads import SLICE_DTYPE, TENSOR_DTYPE, WB_BF16, WB_F32, Layout, make_workload
from wb_workloads.rng import SplitMix64

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SMALL = [("cfg1", "full"), ("cfg1b", "full"), ("cfg1c", "full"), ("cfg2", "small"),
         ("cfg3", "small"), ("cfg4", "small"), ("cfg5", "small")]
BITS = {WB_F32: np.uint32, WB_BF16: np.uint16}


def build(tl: Layout, rl: Layout, **opts):
    a = wb.Layout(tl.tensors, tl.slices)
    b = wb.Layout(rl.tensors, rl.slices)
    return wb.Plan(a, b, **opts)


# ---- ABI surface -----------------------------------------------------------------------------
def test_library_exports_every_declared_symbol():
    lib = wb.load()
    header = open(os.path.join(ROOT, "include", "wb.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(wb_[a-z0-9_]+)\s*\(", header))
    assert {"wb_layout_describe", "wb_plan_build", "wb_pack", "wb_unpack", "wb_remap"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(wb.EXPORTS)


def test_struct_sizes_match_the_generators():
    assert ctypes.sizeof(wb.wb_slice) == SLICE_DTYPE.itemsize == 88
    assert ctypes.sizeof(wb.wb_tensor_desc) == TENSOR_DTYPE.itemsize == 16
    for (name, _), f in zip(wb.wb_slice._fields_, SLICE_DTYPE.names):
        assert getattr(wb.wb_slice, name).offset == SLICE_DTYPE.fields[f][1]
    assert wb.wb_launches_per_call() == 1
    assert "sm_100a" in wb.wb_version()


# ---- plans reproduce the oracle when executed on the host -----------------------------------------
def _check_plan_against_oracle(shapes, tl, rl, src, plan, src_dt, dst_dt):
    plan.verify()
    want = remap_oracle(shapes, tl.tensors, tl.slices, rl.tensors, rl.slices, src,
                        [np.full(int(t["numel"]), 0xBEEF, BITS[dst_dt]) for t in rl.tensors])
    # fused remap
    dst = [np.full(int(t["numel"]), 0xBEEF, BITS[dst_dt]) for t in rl.tensors]
    reads = [np.zeros(int(t["numel"]), np.int32) for t in tl.tensors]
    writes = [np.zeros(int(t["numel"]), np.int32) for t in rl.tensors]
    run_table(plan.tiles(wb.WB_TABLE_REMAP), src, dst, None, src_dt, dst_dt, reads, writes)
    for k in range(len(dst)):
        assert np.array_equal(dst[k], want.dst[k]), k
        assert np.array_equal(writes[k] == 1, want.written[k]) and writes[k].max(initial=0) <= 1
    assert max(int(r.max(initial=0)) for r in reads) <= 1           # no source element read twice
    assert sum(int(r.sum()) for r in reads) == want.n_ids_consumed   # every consumed id read once
    # pack -> bucket -> unpack, round by round
    dst2 = [np.full(int(t["numel"]), 0xBEEF, BITS[dst_dt]) for t in rl.tensors]
    reads2 = [np.zeros(int(t["numel"]), np.int32) for t in tl.tensors]
    for r in range(plan.num_rounds()):
        nb = plan.bucket_bytes(r)
        assert nb % 16 == 0
        bucket = np.full(nb // BITS[dst_dt]().itemsize, 0x7A7A, BITS[dst_dt])
        bw = np.zeros(bucket.size, np.int32)
        run_table(plan.tiles(wb.WB_TABLE_PACK, r), src, None, bucket, src_dt, dst_dt, reads2,
                  bucket_writes=bw)
        assert bw.max(initial=0) <= 1
        # directory: each payload is its checkpoint rectangle, row-major, destination dtype
        for e in plan.bucket_entries(r):
            t = int(e["ckpt_tensor"])
            view, held = checkpoint_view(t, shapes[t], tl.slices, src)
            r0, c0, nr, nc = (int(e[k]) for k in ("r0", "c0", "nr", "nc"))
            rect = cast_bits(view[r0:r0 + nr, c0:c0 + nc].reshape(-1), src_dt, dst_dt)
            off = int(e["bucket_off"]) // bucket.itemsize
            assert int(e["bucket_off"]) % 16 == 0
            assert np.array_equal(bucket[off:off + nr * nc], rect)
            assert (bw[off:off + nr * nc] == 1).all()
        run_table(plan.tiles(wb.WB_TABLE_UNPACK, r), None, dst2, bucket, dst_dt, dst_dt)
    for k in range(len(dst2)):
        assert np.array_equal(dst2[k], want.dst[k]), k
    assert max(int(r.max(initial=0)) for r in reads2) <= 1
    return want


@pytest.mark.parametrize("name,scale", SMALL)
def test_plan_tables_reproduce_oracle(name, scale):
    wl = make_workload(name, scale)
    src = [to_bits(t) for t in wl.trainer_weights()]
    budget = 0 if name != "cfg3" else 1 << 20          # cfg3: force several rounds
    plan = build(wl.trainer, wl.rollout, bucket_budget_bytes=budget, tile_bytes=16384)
    want = _check_plan_against_oracle(ckpt_shapes(wl), wl.trainer, wl.rollout, src, plan,
                                      wl.src_dtype, wl.dst_dtype)
    st = plan.stats()
    assert st["src_elems_read"] == wl.ckpt_numel() == want.n_ids_consumed
    assert st["dst_elems_written"] == want.n_written
    if name == "cfg3":
        assert st["n_rounds"] > 4 and st["n_fanout_slabs"] > 0
        assert st["bucket_bytes_max"] <= 1 << 20


@pytest.mark.parametrize("seed", range(240))
def test_fuzz_plans(seed):
    src_dt, dst_dt = [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)][seed % 4]
    shapes, tl, rl = fuzz_case(5000 + seed, src_dt, dst_dt, max_dim=70)
    rng = np.random.default_rng(seed)
    ck = [random_bits(rng, r * c, src_dt) for (r, c) in shapes]
    src = scatter_checkpoint(tl, ck)
    plan = build(tl, rl, tile_bytes=4096, bucket_budget_bytes=[0, 4096, 16384][seed % 3], grid_ctas=7)
    _check_plan_against_oracle(shapes, tl, rl, src, plan, src_dt, dst_dt)


def test_inverse_plan_is_identity():
    wl = make_workload("cfg1b")
    tl, rl = wl.trainer.swapped_dtype(WB_BF16), wl.rollout.swapped_dtype(WB_BF16)
    rng = np.random.default_rng(0)
    ck = [rng.integers(0, 1 << 16, c.numel, dtype=np.uint64).astype(np.uint16) for c in wl.ckpt]
    src = scatter_checkpoint(tl, ck, fill_bits=0x1111)
    fwd, inv = build(tl, rl), build(rl, tl)
    mid = [np.zeros(int(t["numel"]), np.uint16) for t in rl.tensors]
    run_table(fwd.tiles(wb.WB_TABLE_REMAP), src, mid, None, WB_BF16, WB_BF16)
    back = [np.full(int(t["numel"]), 0x1111, np.uint16) for t in tl.tensors]
    run_table(inv.tiles(wb.WB_TABLE_REMAP), mid, back, None, WB_BF16, WB_BF16)
    for a, b in zip(src, back):
        assert np.array_equal(a, b)
    # the inverse writes the norms to every trainer replica from one read (fan-out)
    assert inv.stats()["n_fanout_slabs"] > 0 and inv.stats()["src_elems_read"] == wl.ckpt_numel()


# ---- de-duplication -------------------------------------------------------------------------------
def test_trainer_replicas_each_supply_a_distinct_slice():
    wl = make_workload("cfg1")          # norms are replicated on both TP ranks
    plan = build(wl.trainer, wl.rollout)
    st = plan.stats()
    assert st["replica_elems_skipped"] == 5 * 256          # 2 layers x 2 norms + final norm
    egress = [plan.rank_bytes(0, r) for r in range(4)]
    assert sum(egress) == wl.ckpt_numel() * 4 == st["src_bytes_read"]   # exactly one model copy
    norm_tensor = wl.rollout.index("r0.final_norm")
    srcs = {int(t["src_tensor"]) for t in plan.tiles(wb.WB_TABLE_REMAP) if int(t["dst_tensor"]) == norm_tensor}
    ranks = {int(wl.trainer.tensors[s]["rank"]) // 2 for s in srcs}      # tp = rank // W
    assert ranks == {0, 1}
    lazy = build(wl.trainer, wl.rollout, flags=wb.WB_PLAN_NO_REPLICA_SPLIT)
    srcs = {int(t["src_tensor"]) for t in lazy.tiles(wb.WB_TABLE_REMAP) if int(t["dst_tensor"]) == norm_tensor}
    assert {int(wl.trainer.tensors[s]["rank"]) // 2 for s in srcs} == {0}


def test_rollout_replicas_share_one_read():
    wl = make_workload("cfg3", "small")
    plan = build(wl.trainer, wl.rollout)
    st = plan.stats()
    H = wl.meta["spec"].H
    n_norms = 2 * wl.meta["spec"].L + 1
    assert st["src_elems_read"] == wl.ckpt_numel()
    assert st["dst_elems_written"] == wl.ckpt_numel() + n_norms * H
    ingress = [plan.rank_bytes(1, r) for r in range(2)]
    assert sum(ingress) == wl.ckpt_numel() * 2                # each id enters the rollout side once
    assert abs(ingress[0] - ingress[1]) <= 2 * H


# ---- full-size plans: byte totals, balance, table overhead ------------------------------------------
@pytest.mark.parametrize("name,src_bytes,dst_bytes", [
    ("cfg2", 16_060_522_496, 16_060_522_496),
    ("cfg3", 32_121_044_992, 16_061_054_976),
    ("cfg4", 61_064_220_672, 61_064_220_672),
    ("cfg5", None, None)])
def test_full_size_plans(name, src_bytes, dst_bytes):
    wl = make_workload(name, "full")
    plan = build(wl.trainer, wl.rollout)
    plan.verify()
    st = plan.stats()
    r, w = wl.algorithmic_bytes()
    assert (st["src_bytes_read"], st["dst_bytes_written"]) == (r, w)
    if src_bytes:
        assert (r, w) == (src_bytes, dst_bytes)
    assert st["table_bytes"] < 0.01 * (r + w)                      # descriptors << payload
    assert st["bucket_bytes_max"] <= 4 << 30
    assert st["n_rounds"] == plan.num_rounds() >= -(-w // (4 << 30))
    sizes = [plan.bucket_bytes(k) for k in range(plan.num_rounds())]
    assert max(sizes) - min(sizes) <= 0.1 * max(sizes)              # roughly equal rounds
    assert st["remap_cta_bytes_max"] <= 1.06 * st["remap_cta_bytes_mean"]
    assert sum(plan.rank_bytes(0, k) for k in range(8)) == r
    assert st["build_seconds"] < 5.0


# ---- error paths: nothing is built, a status comes back -----------------------------------------------
def _tiny():
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T", 0, WB_F32, 16)
    rl.add_tensor("R", 0, WB_BF16, 16)
    return tl, rl


def _expect(status_name, fn):
    with pytest.raises(wb.WbError) as e:
        fn()
    assert e.value.name == status_name, e.value


def test_error_slice_leaves_checkpoint_tensor():
    tl, _ = _tiny()
    tl.add_slice(0, 0, 4, 1, 0, 4, 4, 2, 0, 3, 4)
    tl.freeze()
    _expect("WB_ERR_OUT_OF_RANGE", lambda: wb.Layout(tl.tensors, tl.slices))


def test_error_slice_leaves_local_tensor():
    tl, _ = _tiny()
    tl.add_slice(0, 4, 4, 1, 0, 4, 4, 0, 0, 4, 4)
    tl.freeze()
    _expect("WB_ERR_OUT_OF_RANGE", lambda: wb.Layout(tl.tensors, tl.slices))


def test_error_bad_strides_and_indices():
    tl, _ = _tiny()
    tl.add_slice(0, 0, 2, 3, 0, 4, 4, 0, 0, 2, 2)
    tl.freeze()
    _expect("WB_ERR_INVALID_ARG", lambda: wb.Layout(tl.tensors, tl.slices))
    tl2, _ = _tiny()
    tl2.add_slice(5, 0, 4, 1, 0, 4, 4, 0, 0, 4, 4)
    tl2.freeze()
    _expect("WB_ERR_INVALID_ARG", lambda: wb.Layout(tl2.tensors, tl2.slices))
    tl3, _ = _tiny()
    tl3.add_slice(0, 0, 2, 1, 0, 4, 4, 0, 0, 4, 4)      # rows overlap: pitch 2 < 4 columns
    tl3.freeze()
    _expect("WB_ERR_INVALID_ARG", lambda: wb.Layout(tl3.tensors, tl3.slices))


def test_error_dtype_and_shape_mismatch():
    t = np.array([(0, 7, 16)], dtype=TENSOR_DTYPE)
    _expect("WB_ERR_DTYPE", lambda: wb.Layout(t, np.zeros(0, SLICE_DTYPE)))
    t = np.array([(0, 0, 16), (0, 1, 16)], dtype=TENSOR_DTYPE)
    _expect("WB_ERR_DTYPE", lambda: wb.Layout(t, np.zeros(0, SLICE_DTYPE)))
    tl, _ = _tiny()
    tl.add_slice(0, 0, 4, 1, 0, 4, 4, 0, 0, 2, 4)
    tl.add_slice(0, 8, 4, 1, 0, 2, 8, 0, 0, 1, 8)
    tl.freeze()
    _expect("WB_ERR_SHAPE_MISMATCH", lambda: wb.Layout(tl.tensors, tl.slices))
    tl, rl = _tiny()
    tl.add_slice(0, 0, 4, 1, 0, 4, 4, 0, 0, 4, 4)
    rl.add_slice(0, 0, 8, 1, 0, 2, 8, 0, 0, 2, 8)
    tl.freeze(); rl.freeze()
    _expect("WB_ERR_SHAPE_MISMATCH", lambda: build(tl, rl))


def test_error_uncovered_and_overlap():
    tl, rl = _tiny()
    tl.add_slice(0, 0, 4, 1, 0, 4, 4, 0, 0, 3, 4)           # row 3 held by nobody
    rl.add_slice(0, 0, 4, 1, 0, 4, 4, 0, 0, 4, 4)
    tl.freeze(); rl.freeze()
    _expect("WB_ERR_UNCOVERED", lambda: build(tl, rl))
    tl, rl = _tiny()
    tl.add_slice(0, 0, 4, 1, 0, 4, 4, 0, 0, 4, 4)
    rl.add_slice(0, 0, 4, 1, 1, 4, 4, 0, 0, 4, 4)           # checkpoint tensor 1 unknown to the trainer
    tl.freeze(); rl.freeze()
    _expect("WB_ERR_UNCOVERED", lambda: build(tl, rl))
    tl, rl = _tiny()
    tl.add_slice(0, 0, 4, 1, 0, 4, 4, 0, 0, 4, 4)
    rl.add_slice(0, 0, 4, 1, 0, 4, 4, 0, 0, 2, 4)
    rl.add_slice(0, 6, 4, 1, 0, 4, 4, 2, 0, 2, 4)           # lands on elements 6.. already described
    tl.freeze(); rl.freeze()
    _expect("WB_ERR_DST_OVERLAP", lambda: build(tl, rl))


def test_error_bucket_too_small_and_unbound_execution():
    wl = make_workload("cfg1")
    _expect("WB_ERR_BUCKET_TOO_SMALL", lambda: build(wl.trainer, wl.rollout, bucket_budget_bytes=64))
    plan = build(wl.trainer, wl.rollout)
    _expect("WB_ERR_NOT_BOUND", lambda: plan.remap())
    _expect("WB_ERR_INVALID_ARG", lambda: plan.pack(99, 16))
    _expect("WB_ERR_NOT_BOUND", lambda: plan.transfer_rounds(256, 512))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.transfer_rounds(256, 256))       # one bucket given twice
    _expect("WB_ERR_INVALID_ARG", lambda: plan.transfer_rounds(256, 0))         # second bucket missing
    _expect("WB_ERR_INVALID_ARG", lambda: plan.transfer_rounds(258, 512))       # not 16-byte aligned
    _expect("WB_ERR_INVALID_ARG", lambda: plan.transfer_rounds(256, 512, flags=8))
    _expect("WB_ERR_NOT_BOUND", lambda: plan.transfer_rounds(256, 0, flags=wb.WB_ROUNDS_SERIAL))
    # FP8 bucket quantisation: host-side queries work on any plan, device calls need a binding
    assert plan.num_ckpts() == len(wl.ckpt) and plan.ckpt_ids().tolist() == list(range(len(wl.ckpt)))
    assert plan.qbucket_bytes(0) * 2 == plan.bucket_bytes(0) and plan.qbucket_bytes(99) == 0
    _expect("WB_ERR_NOT_BOUND", lambda: plan.absmax(256))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.absmax(0))
    _expect("WB_ERR_NOT_BOUND", lambda: plan.bucket_quantize(0, 256, 512, 1024))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.bucket_quantize(0, 258, 512, 1024))     # not 16-byte aligned
    _expect("WB_ERR_INVALID_ARG", lambda: plan.bucket_dequantize(99, 256, 512, 1024))  # no such round
    _expect("WB_ERR_NOT_BOUND", lambda: plan.transfer_rounds_fp8(256, 512, 1024, 2048, 4096))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.transfer_rounds_fp8(256, 256, 1024, 2048, 4096))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.transfer_rounds_fp8(256, 512, 1024, 2050, 4096))
    # the fused forms and the rank subsets likewise
    _expect("WB_ERR_NOT_BOUND", lambda: plan.pack_fp8(0, 256, 1024))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.pack_fp8(0, 258, 1024))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.unpack_fp8(99, 256, 1024))
    _expect("WB_ERR_NOT_BOUND", lambda: plan.transfer_rounds_fp8_fused(256, 512, 1024))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.transfer_rounds_fp8_fused(256, 256, 1024))
    _expect("WB_ERR_NOT_BOUND", lambda: plan.pack_ranks(0, [0], 256))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.pack_ranks(0, [0], 258))
    _expect("WB_ERR_INVALID_ARG", lambda: plan.unpack_ranks(99, [0], 256))
    nt, nr = plan.num_ranks()
    assert (nt, nr) == (4, 1)                                  # TP2 x FSDP2 trainer ranks, one rollout rank
    regions = plan.bucket_regions(0)
    assert sorted((int(g["receiver"]), int(g["sender"])) for g in regions) == [(0, s) for s in range(4)]
    assert all(int(g["off"]) % 256 == 0 for g in regions) and int(regions["bytes"].sum()) <= plan.bucket_bytes(0)
    entries = plan.bucket_entries(0)
    for e in entries:                                          # every payload lies in the region of its pair
        g = regions[(regions["receiver"] == e["receiver"]) & (regions["sender"] == e["sender"])][0]
        size = int(e["nr"]) * int(e["nc"]) * 2
        assert int(g["off"]) <= int(e["bucket_off"]) and int(e["bucket_off"]) + size <= int(g["off"]) + int(g["bytes"])
    _expect("WB_ERR_INVALID_ARG", lambda: plan.bind([0] * plan.n_src, [0] * plan.n_dst))
    lib = wb.load()
    assert lib.wb_remap(None, None) == 1
    assert lib.wb_plan_build(None, None, None, None) == 1
    assert lib.wb_plan_num_rounds(None) == 0


def test_interleaved_column_blocks_are_not_an_overlap():
    # two column blocks of one matrix stored interleaved in one local tensor: bounding
    # intervals overlap, elements do not
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T", 0, WB_F32, 32)
    rl.add_tensor("R", 0, WB_F32, 32)
    tl.add_slice(0, 0, 8, 1, 0, 4, 8, 0, 0, 4, 8)
    rl.add_slice(0, 0, 8, 1, 0, 4, 8, 0, 0, 4, 3)
    rl.add_slice(0, 3, 8, 1, 0, 4, 8, 0, 3, 4, 5)
    tl.freeze(); rl.freeze()
    plan = build(tl, rl)
    plan.verify()
    src = [np.arange(32, dtype=np.uint32)]
    dst = [np.zeros(32, np.uint32)]
    run_table(plan.tiles(wb.WB_TABLE_REMAP), src, dst, None, WB_F32, WB_F32)
    assert np.array_equal(dst[0], src[0])


@pytest.mark.parametrize("dts", [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_BF16, WB_F32)])
def test_seam_flags_pair_up_between_staged_transposing_tiles(dts):
    """A transposing slab is cut into tiles along its rows.  WB_TILE_ROWS_AFTER on a tile and
    WB_TILE_ROWS_BEFORE on the tile that holds the next rows of the same columns come in pairs, only
    between tiles the executor stages in chunks (rows of at least 128 source bytes, at least 16 of them,
    at least 8 KiB moved), and never on other kinds of tile - in the fused table and in the unpack
    tables alike."""
    es = 4 if dts[0] == WB_F32 else 2
    ed = 4 if dts[1] == WB_F32 else 2
    found = 0
    for (R, C, tile_bytes) in [(1000, 300, 65536), (130, 500, 4096), (2000, 40, 32768), (70, 4000, 0), (4096, 130, 0)]:
        tl, rl = Layout("t"), Layout("r")
        tl.add_tensor("T", 0, dts[0], R * C)
        tl.add_slice(0, 0, C, 1, 0, R, C, 0, 0, R, C)
        rl.add_tensor("R", 0, dts[1], R * C)
        rl.add_slice(0, 0, 1, R, 0, R, C, 0, 0, R, C)            # checkpoint (i, j) -> local j*R + i
        tl.freeze(); rl.freeze()
        plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices), tile_bytes=tile_bytes,
                       bucket_budget_bytes=1 << 20)
        plan.verify()
        tables = [plan.tiles(wb.WB_TABLE_REMAP)]
        for r in range(plan.num_rounds()):
            tables.append(plan.tiles(wb.WB_TABLE_PACK, r))
            tables.append(plan.tiles(wb.WB_TABLE_UNPACK, r))
        for k, t in enumerate(tables):
            src_es = ed if (k and k % 2 == 0) else es           # an unpack table reads the bucket (rollout dtype)
            before = (t["flags"] & wb.WB_TILE_ROWS_BEFORE) != 0
            after = (t["flags"] & wb.WB_TILE_ROWS_AFTER) != 0
            staged = ((t["kind"] == 1) & (t["nc"].astype(np.int64) * src_es >= 128) & (t["nr"] >= 16) &
                      (t["nr"].astype(np.int64) * t["nc"] * (src_es + ed) >= 8192))
            assert not (before & ~staged).any() and not (after & ~staged).any()
            # the tile below continues the destination runs: its first element follows this tile's last row
            below = {(int(x["dst_tensor"]), int(x["dst_off"])): i for i, x in enumerate(t)}
            for i in np.nonzero(after)[0]:
                x = t[i]
                assert int(x["dst_sr"]) == 1
                j = below.get((int(x["dst_tensor"]), int(x["dst_off"]) + int(x["nr"])))
                assert j is not None and before[j] and int(t[j]["nc"]) == int(x["nc"])
                assert int(t[j]["src_off"]) == int(x["src_off"]) + int(x["nr"]) * int(x["src_sr"])
                found += 1
            assert before.sum() == after.sum()
    assert found > 20


def test_flat_range_helper_gives_the_rectangles_of_a_flat_shard():
    """wb_layout_add_flat_range against brute force on ids (every element of the flat range is described
    exactly once, at the local offset it has in the shard) and against the generator's own statement."""
    from wb_workloads.configs import flat_range_rects
    rng = SplitMix64(77)
    cases = [(1, 1, 0, 1), (4, 6, 0, 24), (4, 6, 0, 0), (4, 6, 5, 7), (4, 6, 6, 12), (4, 6, 7, 11), (4, 6, 3, 23)]
    for _ in range(300):
        rows, cols = rng.randint(1, 12), rng.randint(1, 12)
        b = rng.randint(0, rows * cols)
        cases.append((rows, cols, b, rng.randint(b, rows * cols)))
    for rows, cols, b, e in cases:
        local_off = 5
        got = wb.wb_layout_add_flat_range(3, local_off, 9, rows, cols, b, e)
        assert len(got) <= 3
        ids = np.arange(rows * cols)
        local = np.full(local_off + (e - b), -1)
        local[local_off:] = ids[b:e]
        seen = np.zeros(local.size, bool)
        for s in got:
            assert (int(s["tensor"]), int(s["ckpt"]), int(s["ckpt_rows"]), int(s["ckpt_cols"])) == (3, 9, rows, cols)
            for i in range(int(s["nr"])):
                for j in range(int(s["nc"])):
                    x = int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])
                    assert local[x] == (int(s["r0"]) + i) * cols + int(s["c0"]) + j and not seen[x]
                    seen[x] = True
        assert seen[local_off:].all() and not seen[:local_off].any()
        want = flat_range_rects(cols, b, e)
        assert [(int(s["r0"]), int(s["c0"]), int(s["nr"]), int(s["nc"]), int(s["local_off"]) - local_off + b)
                for s in got] == want
    with pytest.raises(wb.WbError) as err:
        wb.wb_layout_add_flat_range(0, 0, 0, 4, 6, 5, 25)
    assert err.value.name == "WB_ERR_OUT_OF_RANGE"
    with pytest.raises(wb.WbError) as err:
        wb.wb_layout_add_flat_range(0, 0, 0, 4, 6, 7, 5)
    assert err.value.name == "WB_ERR_OUT_OF_RANGE"
    with pytest.raises(wb.WbError) as err:
        wb.wb_layout_add_flat_range(0, 0, 0, 4, 0, 0, 0)
    assert err.value.name == "WB_ERR_INVALID_ARG"
    # the records are accepted by wb_layout_describe as they are
    sl = wb.wb_layout_add_flat_range(0, 0, 0, 4, 6, 3, 23)
    wb.Layout(np.array([(0, WB_F32, 20)], TENSOR_DTYPE), sl)
