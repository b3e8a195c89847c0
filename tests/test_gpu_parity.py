"""Parity of the CUDA path against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from gpu_util import CANARY, DeviceCase, oracle_for, prefill_bits
from helpers import ckpt_shapes, from_bits, fuzz_case, random_bits, scatter_checkpoint, to_bits
from oracle import checkpoint_view, remap_oracle
from oracle.cast import cast_bits, f32_to_bf16_bits
from paper_2609_25442_b200 import binding as wb
from paper_2609_25442_b200.device import RankArenas, bind
from wb_workloads import WB_BF16, WB_F32, Layout, make_workload

pytestmark = pytest.mark.gpu
BITS = {WB_F32: np.uint32, WB_BF16: np.uint16}

CASES = [("cfg1", "full"), ("cfg1b", "full"), ("cfg1c", "full"), ("cfg2", "small"), ("cfg3", "small"),
         ("cfg4", "small"), ("cfg5", "small"), ("cfg2", "medium"), ("cfg3", "medium"),
         ("cfg4", "medium"), ("cfg5", "medium")]


@pytest.fixture(scope="module")
def device():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def assert_dst_equals(case, want):
    got = case.dst_bits()
    for k in range(len(got)):
        if not np.array_equal(got[k], want.dst[k]):
            bad = np.nonzero(got[k] != want.dst[k])[0]
            raise AssertionError(f"{case.rollout.names[k]}: {bad.size} of {got[k].size} elements differ, "
                                 f"first at {bad[:5]}")
    assert case.gaps_intact()


@pytest.mark.parametrize("name,scale", CASES)
def test_remap_matches_oracle(device, name, scale):
    case = DeviceCase(make_workload(name, scale), device)
    want = oracle_for(case)
    case.plan.remap()
    torch.cuda.synchronize()
    assert_dst_equals(case, want)
    # a second call on the same plan gives the same result (the plan is reused every update)
    case.reset_dst()
    case.plan.remap()
    torch.cuda.synchronize()
    assert_dst_equals(case, want)


@pytest.mark.parametrize("name,scale,budget", [
    ("cfg1", "full", 0), ("cfg1b", "full", 1 << 20), ("cfg3", "small", 1 << 20), ("cfg4", "small", 1 << 19),
    ("cfg5", "small", 1 << 18), ("cfg2", "medium", 16 << 20), ("cfg3", "medium", 32 << 20),
    ("cfg5", "medium", 16 << 20)])
def test_pack_unpack_matches_oracle(device, name, scale, budget):
    wl = make_workload(name, scale)
    case = DeviceCase(wl, device, bucket_budget_bytes=budget)
    want = oracle_for(case)
    src_bits = case.src_bits()
    shapes = ckpt_shapes(wl)
    n_rounds = case.plan.num_rounds()
    if budget:
        assert n_rounds > 1
    views = {}
    for r in range(n_rounds):
        nb = case.plan.bucket_bytes(r)
        bucket = torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=device)
        case.plan.pack(r, bucket.data_ptr())
        torch.cuda.synchronize()
        assert bool((bucket[nb:] == 0x5A).all())
        raw = bucket[:nb].cpu().numpy().view(BITS[wl.dst_dtype])
        covered = np.zeros(raw.size, bool)
        for e in case.plan.bucket_entries(r):
            t = int(e["ckpt_tensor"])
            if t not in views:
                views[t] = checkpoint_view(t, shapes[t], case.trainer.slices, src_bits)[0]
            r0, c0, nr, nc = (int(e[k]) for k in ("r0", "c0", "nr", "nc"))
            rect = cast_bits(views[t][r0:r0 + nr, c0:c0 + nc].reshape(-1), wl.src_dtype, wl.dst_dtype)
            off = int(e["bucket_off"]) // raw.itemsize
            assert np.array_equal(raw[off:off + nr * nc], rect), (r, t)
            covered[off:off + nr * nc] = True
        pad = 0x5A5A if raw.itemsize == 2 else 0x5A5A5A5A
        assert (raw[~covered] == pad).all()          # alignment padding is never written
        case.plan.unpack(r, bucket.data_ptr())
        torch.cuda.synchronize()
    assert_dst_equals(case, want)


@pytest.mark.parametrize("name,scale,budget", [
    ("cfg1", "full", 0), ("cfg1b", "full", 1 << 20), ("cfg3", "small", 1 << 20), ("cfg4", "small", 1 << 19),
    ("cfg5", "small", 1 << 18), ("cfg2", "medium", 16 << 20), ("cfg3", "medium", 32 << 20),
    ("cfg5", "medium", 16 << 20)])
def test_pipelined_rounds_match_oracle(device, name, scale, budget):
    """Depth-2 bucket pipeline (Section 3.2 / Section 4): all rounds through two buckets on two
    internal streams give the same rollout tensors as the fused remap, on the caller's stream."""
    wl = make_workload(name, scale)
    case = DeviceCase(wl, device, bucket_budget_bytes=budget)
    want = oracle_for(case)
    n_rounds = case.plan.num_rounds()
    if budget:
        assert n_rounds > 2                     # the second use of a bucket is exercised
    nb = max(case.plan.bucket_bytes(r) for r in range(n_rounds))
    buckets = [torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=device) for _ in range(2)]
    side = torch.cuda.Stream(device=device)
    for flags, stream in [(0, None), (wb.WB_ROUNDS_SERIAL, None), (0, side), (0, side)]:
        case.reset_dst()
        torch.cuda.synchronize()
        sp = 0 if stream is None else stream.cuda_stream
        case.plan.transfer_rounds(buckets[0].data_ptr(), buckets[1].data_ptr(), flags, sp)
        if stream is not None:
            # back to back on the same stream: the second transfer is ordered after the first
            case.plan.transfer_rounds(buckets[0].data_ptr(), buckets[1].data_ptr(), flags, sp)
            stream.synchronize()                # the caller's stream alone covers all internal work
        else:
            torch.cuda.synchronize()
        assert_dst_equals(case, want)
        case.plan.check()
        for b in buckets:
            assert bool((b[nb:] == 0x5A).all())
    with pytest.raises(wb.WbError):
        case.plan.transfer_rounds(buckets[0].data_ptr(), buckets[0].data_ptr())     # one bucket twice
    with pytest.raises(wb.WbError):
        case.plan.transfer_rounds(buckets[0].data_ptr() + 2, buckets[1].data_ptr())  # misaligned


@pytest.mark.parametrize("seed", range(160))
def test_fuzz_layouts(device, seed):
    src_dt, dst_dt = [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)][seed % 4]
    shapes, tl, rl = fuzz_case(9000 + seed, src_dt, dst_dt, max_dim=[40, 150, 300][seed % 3])
    rng = np.random.default_rng(seed)
    ck = [random_bits(rng, r * c, src_dt) for (r, c) in shapes]
    src_host = scatter_checkpoint(tl, ck)
    src = RankArenas(tl.tensors, device, fill_byte=0)
    dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
    for t, h in zip(src.tensors, src_host):
        t.copy_(from_bits(h))
    plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices),
                   tile_bytes=[4096, 65536][seed % 2], bucket_budget_bytes=[0, 8192][seed % 2])
    bind(plan, src, dst)
    want = remap_oracle(shapes, tl.tensors, tl.slices, rl.tensors, rl.slices, src_host,
                        prefill_bits(rl, BITS[dst_dt]))
    plan.remap()
    torch.cuda.synchronize()
    for k, t in enumerate(dst.tensors):
        assert np.array_equal(to_bits(t), want.dst[k]), k
    for a in dst.arenas.values():
        a.fill_(CANARY)
    for r in range(plan.num_rounds()):
        bucket = torch.empty(plan.bucket_bytes(r) + 16, dtype=torch.uint8, device=device)
        plan.pack(r, bucket.data_ptr())
        plan.unpack(r, bucket.data_ptr())
    torch.cuda.synchronize()
    for k, t in enumerate(dst.tensors):
        assert np.array_equal(to_bits(t), want.dst[k]), k


@pytest.mark.parametrize("seed", range(40))
def test_fuzz_layouts_with_larger_tensors(device, seed):
    """The same fuzz with dimensions up to 2500, so that staged rows, staged transposition chunks and
    multi-tile slabs are reached; automatic, 64 KiB and 4 KiB tiles."""
    src_dt, dst_dt = [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)][seed % 4]
    shapes, tl, rl = fuzz_case(50000 + seed, src_dt, dst_dt, max_dim=[300, 900, 2500][seed % 3])
    rng = np.random.default_rng(seed)
    ck = [random_bits(rng, r * c, src_dt) for (r, c) in shapes]
    src_host = scatter_checkpoint(tl, ck)
    src = RankArenas(tl.tensors, device, fill_byte=0)
    dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
    for t, h in zip(src.tensors, src_host):
        t.copy_(from_bits(h))
    plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices),
                   tile_bytes=[0, 65536, 4096][seed % 3], bucket_budget_bytes=[0, 1 << 16][seed % 2])
    bind(plan, src, dst)
    want = remap_oracle(shapes, tl.tensors, tl.slices, rl.tensors, rl.slices, src_host,
                        prefill_bits(rl, BITS[dst_dt]))
    plan.remap()
    torch.cuda.synchronize()
    for k, t in enumerate(dst.tensors):
        assert np.array_equal(to_bits(t), want.dst[k]), k
    for a in dst.arenas.values():
        a.fill_(CANARY)
    for r in range(plan.num_rounds()):
        bucket = torch.empty(plan.bucket_bytes(r) + 16, dtype=torch.uint8, device=device)
        plan.pack(r, bucket.data_ptr())
        plan.unpack(r, bucket.data_ptr())
    torch.cuda.synchronize()
    for k, t in enumerate(dst.tensors):
        assert np.array_equal(to_bits(t), want.dst[k]), k
    plan.check()


def _one_tensor_plan(n, src_dt, dst_dt, device, src_off=0, dst_off=0):
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T", 0, src_dt, n + src_off)
    rl.add_tensor("R", 0, dst_dt, n + dst_off)
    tl.add_slice(0, src_off, n, 1, 0, 1, n, 0, 0, 1, n)
    rl.add_slice(0, dst_off, n, 1, 0, 1, n, 0, 0, 1, n)
    tl.freeze(); rl.freeze()
    src = RankArenas(tl.tensors, device)
    dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
    plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices))
    bind(plan, src, dst)
    return plan, src, dst


def test_cast_all_fp32_patterns(device):
    """Every one of the 2^32 fp32 bit patterns through the kernel's fp32 -> bf16 path, NaNs
    included, against the oracle's integer rounding."""
    n = 1 << 26
    plan, src, dst = _one_tensor_plan(n, WB_F32, WB_BF16, device)
    ar = torch.arange(n, dtype=torch.int64, device=device)
    for chunk in range(64):
        src.tensors[0].view(torch.int32).copy_((ar + chunk * n).to(torch.int32))   # wraps to the pattern
        plan.remap()
        torch.cuda.synchronize()
        got = to_bits(dst.tensors[0])
        pats = (np.arange(n, dtype=np.uint64) + chunk * n).astype(np.uint32)
        want = f32_to_bf16_bits(pats)
        assert np.array_equal(got, want), chunk


def test_same_dtype_is_a_bit_copy(device):
    n = 1 << 16
    plan, src, dst = _one_tensor_plan(n, WB_BF16, WB_BF16, device, src_off=3, dst_off=5)
    src.tensors[0].view(torch.int16)[3:].copy_(torch.arange(n, device=device).to(torch.int16))
    plan.remap()
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(dst.tensors[0])[5:], np.arange(n, dtype=np.uint16))
    assert (to_bits(dst.tensors[0])[:5] == 0xCDCD).all()
    # fp32: NaN payloads, signalling NaNs and subnormals survive
    n = 1 << 24
    plan, src, dst = _one_tensor_plan(n, WB_F32, WB_F32, device, src_off=1, dst_off=2)
    g = torch.Generator(device=device); g.manual_seed(1)
    pats = torch.randint(-(1 << 31), (1 << 31) - 1, (n,), dtype=torch.int64, device=device, generator=g).to(torch.int32)
    src.tensors[0].view(torch.int32)[1:].copy_(pats)
    plan.remap()
    torch.cuda.synchronize()
    assert torch.equal(dst.tensors[0].view(torch.int32)[2:], pats)


def test_widening_bf16_to_fp32(device):
    n = 1 << 16
    plan, src, dst = _one_tensor_plan(n, WB_BF16, WB_F32, device, src_off=1)
    src.tensors[0].view(torch.int16)[1:].copy_(torch.arange(n, device=device).to(torch.int16))
    plan.remap()
    torch.cuda.synchronize()
    want = cast_bits(np.arange(n, dtype=np.uint16), WB_BF16, WB_F32)
    assert np.array_equal(to_bits(dst.tensors[0]), want)


@pytest.mark.parametrize("src_off,dst_off", [(0, 0), (1, 0), (0, 1), (3, 7), (5, 2), (4, 4)])
@pytest.mark.parametrize("dts", [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32)])
def test_unaligned_runs(device, src_off, dst_off, dts):
    """Runs that start off a 16-byte boundary on either side, of every length around the
    vector width, must not touch a neighbouring element."""
    for n in list(range(1, 40)) + [255, 256, 257, 4099, 70001]:
        plan, src, dst = _one_tensor_plan(n, dts[0], dts[1], device, src_off, dst_off)
        rng = np.random.default_rng(n)
        bits = random_bits(rng, n + src_off, dts[0])
        src.tensors[0].copy_(from_bits(bits))
        plan.remap()
        torch.cuda.synchronize()
        got = to_bits(dst.tensors[0])
        want = cast_bits(bits[src_off:], dts[0], dts[1])
        assert np.array_equal(got[dst_off:], want), n
        assert (got[:dst_off] == (0xCDCD if dts[1] == WB_BF16 else 0xCDCDCDCD)).all()


TRANS_SHAPES = [(16, 64), (17, 65), (15, 300), (40, 124), (41, 125), (63, 123), (64, 124), (65, 125), (71, 247),
                (72, 248), (73, 249), (64, 496), (129, 497), (200, 1000), (333, 130), (1, 700), (700, 1), (8, 2048),
                (55, 121), (56, 120), (57, 241), (87, 119), (88, 120), (89, 121), (96, 240), (176, 122), (177, 481)]


@pytest.mark.parametrize("dts", [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)])
@pytest.mark.parametrize("skew", [(0, 0, 0), (1, 3, 0), (2, 5, 7), (4, 8, 4)])
@pytest.mark.parametrize("flags", [0, wb.WB_PLAN_NO_TENSOR_MAPS])
def test_transposition_shapes(device, dts, skew, flags):
    """dst[j, i] = cast(src[i, j]) for shapes on both sides of every block and chunk size of the
    transposing paths (chunks staged by tensor-map loads, and - WB_PLAN_NO_TENSOR_MAPS - by per-lane
    copies), with the source starting `so` elements into its tensor, the destination `do`,
    and the source rows `extra` elements longer than the part that is moved (so row starts fall on
    every alignment).  The oracle is numpy's transpose of the seeded bits; the element before and
    after every destination must keep the canary."""
    so, do, extra = skew
    for (R, C) in TRANS_SHAPES:
        pitch = C + extra
        tl, rl = Layout("t"), Layout("r")
        tl.add_tensor("T", 0, dts[0], so + R * pitch)
        # the source matrix is the left C columns of a wider [R, pitch] matrix, which is checkpoint tensor 0
        tl.add_slice(0, so, pitch, 1, 0, R, pitch, 0, 0, R, pitch)
        rl.add_tensor("R", 0, dts[1], do + R * C + 3)
        rl.add_slice(0, do, 1, R, 0, R, pitch, 0, 0, R, C)        # checkpoint (i, j) -> local do + j*R + i
        tl.freeze(); rl.freeze()
        plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices), flags=flags)
        src = RankArenas(tl.tensors, device, fill_byte=0)
        dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
        bind(plan, src, dst)
        rng = np.random.default_rng(R * 1000 + C)
        bits = random_bits(rng, so + R * pitch, dts[0])
        src.tensors[0].copy_(from_bits(bits).to(device))
        plan.remap()
        torch.cuda.synchronize()
        plan.check()
        got = to_bits(dst.tensors[0])
        m = bits[so:].reshape(R, pitch)[:, :C]
        want = cast_bits(np.ascontiguousarray(m.T).reshape(-1), dts[0], dts[1])
        assert np.array_equal(got[do:do + R * C], want), (R, C)
        canary = 0xCDCD if dts[1] == WB_BF16 else 0xCDCDCDCD
        assert (got[:do] == canary).all() and (got[do + R * C:] == canary).all(), (R, C)


@pytest.mark.parametrize("seed", range(6))
def test_fuzz_transposing_slabs(device, seed):
    """Random transposed slabs - rows 8..3000, columns 8..1200, every offset and pitch remainder on
    both sides, one to three destination tensors, tile sizes from 4 KiB up, all four dtype pairs, with
    and without tensor maps - through the fused call, the two-pass rounds and the staged host call.
    The oracle is numpy's transpose of the seeded bits; gaps and padding must keep the canary."""
    rng = np.random.default_rng(4000 + seed)
    for case in range(40):
        dts = [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)][case % 4]
        R, C = int(rng.integers(8, 3000)), int(rng.integers(8, 1200))
        so, do, sx, dx = (int(rng.integers(0, 9)) for _ in range(4))
        sp, dp = C + sx, R + dx
        k = int(rng.integers(1, 4))
        tl, rl = Layout("t"), Layout("r")
        tl.add_tensor("T", 0, dts[0], so + R * sp)
        tl.add_slice(0, so, sp, 1, 0, R, sp, 0, 0, R, sp)
        bounds = [int(b) for b in np.linspace(0, C, k + 1)]
        parts = [(bounds[g], bounds[g + 1]) for g in range(k) if bounds[g + 1] > bounds[g]]
        for g, (c0, c1) in enumerate(parts):
            t = rl.add_tensor(f"R{g}", g % 2, dts[1], do + (c1 - c0) * dp + 3)
            rl.add_slice(t, do, 1, dp, 0, R, sp, 0, c0, R, c1 - c0)      # checkpoint (i, j) -> do + (j - c0) * dp + i
        tl.freeze(); rl.freeze()
        plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices),
                       tile_bytes=int(rng.choice([0, 4096, 16384, 65536])),
                       flags=int(rng.choice([0, 0, wb.WB_PLAN_NO_TENSOR_MAPS])),
                       bucket_budget_bytes=int(rng.choice([0, 1 << 18])), host_group_kib=int(rng.choice([64, 512])))
        src = RankArenas(tl.tensors, device, fill_byte=0)
        dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
        bind(plan, src, dst)
        bits = random_bits(rng, so + R * sp, dts[0])
        src.tensors[0].copy_(from_bits(bits).to(device))
        if case % 3 == 0:
            plan.remap()
        elif case % 3 == 1:
            for r in range(plan.num_rounds()):
                bucket = torch.empty(plan.bucket_bytes(r) + 16, dtype=torch.uint8, device=device)
                plan.pack(r, bucket.data_ptr())
                plan.unpack(r, bucket.data_ptr())
        else:
            hs = [t.cpu().pin_memory() for t in src.tensors]
            hd = [t.cpu().pin_memory() for t in dst.tensors]
            for a in src.arenas.values():
                a.zero_()
            plan.remap_host([t.data_ptr() for t in hs], [t.data_ptr() for t in hd])
            torch.cuda.synchronize()
            for t, h in zip(dst.tensors, hd):
                t.copy_(h)
        torch.cuda.synchronize()
        plan.check()
        m = bits[so:].reshape(R, sp)
        canary = 0xCDCD if dts[1] == WB_BF16 else 0xCDCDCDCD
        for g, (c0, c1) in enumerate(parts):
            got = to_bits(dst.tensors[g])
            want = cast_bits(np.ascontiguousarray(m[:, c0:c1].T).reshape(-1), dts[0], dts[1]).reshape(c1 - c0, R)
            body = got[do:do + (c1 - c0) * dp].reshape(c1 - c0, dp)
            assert np.array_equal(body[:, :R], want), (seed, case, R, C, g)
            assert (body[:, R:] == canary).all() and (got[:do] == canary).all() and (got[do + (c1 - c0) * dp:] == canary).all(), (seed, case)


ROW_SHAPES = [(16, 64), (17, 65), (40, 100), (64, 127), (100, 128), (176, 129), (177, 200), (300, 249), (301, 250),
              (90, 252), (91, 253), (92, 254), (700, 131), (15, 200), (2000, 67)]


@pytest.mark.parametrize("dts", [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)])
@pytest.mark.parametrize("skew", [(0, 0, 3, 0), (1, 3, 0, 5), (2, 5, 7, 0), (4, 8, 4, 8)])
def test_short_row_shapes(device, dts, skew):
    """dst[i, j] = cast(src[i, j]) for rows below 1 KiB (the warp-level short-row path and the runs of
    small tiles): the source starts `so` elements into its tensor and its rows are `sx` elements longer
    than the part that is moved, the destination likewise with `do` and `dx`, so that row starts fall
    on every alignment and the destination is packed or strided.  The element before and after every
    destination row must keep the canary."""
    so, do, sx, dx = skew
    for (R, C) in ROW_SHAPES:
        sp, dp = C + sx, C + dx
        tl, rl = Layout("t"), Layout("r")
        tl.add_tensor("T", 0, dts[0], so + R * sp)
        rl.add_tensor("R", 0, dts[1], do + R * dp + 3)
        # checkpoint tensor 0 is the wider [R, sp] source matrix; the rollout keeps its left C columns
        tl.add_slice(0, so, sp, 1, 0, R, sp, 0, 0, R, sp)
        rl.add_slice(0, do, dp, 1, 0, R, sp, 0, 0, R, C)
        tl.freeze(); rl.freeze()
        plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices))
        src = RankArenas(tl.tensors, device, fill_byte=0)
        dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
        bind(plan, src, dst)
        rng = np.random.default_rng(R * 1000 + C)
        bits = random_bits(rng, so + R * sp, dts[0])
        src.tensors[0].copy_(from_bits(bits).to(device))
        plan.remap()
        torch.cuda.synchronize()
        plan.check()
        got = to_bits(dst.tensors[0])
        want = cast_bits(np.ascontiguousarray(bits[so:].reshape(R, sp)[:, :C]).reshape(-1), dts[0], dts[1]).reshape(R, C)
        canary = 0xCDCD if dts[1] == WB_BF16 else 0xCDCDCDCD
        body = got[do:do + R * dp].reshape(R, dp)
        assert np.array_equal(body[:, :C], want), (R, C)
        assert (body[:, C:] == canary).all() and (got[:do] == canary).all() and (got[do + R * dp:] == canary).all(), (R, C)


def test_rebinding_rebuilds_the_tensor_maps(device):
    """The tensor maps of transposing tiles hold device addresses: binding the plan to other trainer
    tensors (here at another alignment) must re-encode them, and the old tensors may then be freed."""
    wl = make_workload("cfg5", "medium")
    case = DeviceCase(wl, device)
    want = oracle_for(case)
    case.plan.remap()
    torch.cuda.synchronize()
    assert_dst_equals(case, want)
    # a second set of trainer tensors, every one 4 bytes further from a 16-byte boundary, same contents
    flat = [torch.zeros(t.numel() + 8, dtype=t.dtype, device=device) for t in case.src.tensors]
    shifted = [f[4 // f.element_size():4 // f.element_size() + t.numel()] for f, t in zip(flat, case.src.tensors)]
    for a, b in zip(shifted, case.src.tensors):
        a.copy_(b)
    case.plan.bind([t.data_ptr() for t in shifted], [t.data_ptr() for t in case.dst.tensors])
    for t in case.src.tensors:
        t.zero_()                        # reading the old tensors would now give zeros
    case.reset_dst()
    case.plan.remap()
    torch.cuda.synchronize()
    case.plan.check()
    assert_dst_equals(case, want)


def test_inverse_remap_restores_the_trainer(device):
    wl = make_workload("cfg1b")
    tl, rl = wl.trainer.swapped_dtype(WB_BF16), wl.rollout.swapped_dtype(WB_BF16)
    fwd = DeviceCase(wl, device, trainer=tl, rollout=rl)
    fwd.plan.remap()
    inv_plan = wb.Plan(wb.Layout(rl.tensors, rl.slices), wb.Layout(tl.tensors, tl.slices))
    back = RankArenas(tl.tensors, device, fill_byte=0)      # trainer padding was loaded as zeros
    bind(inv_plan, fwd.dst, back)
    inv_plan.remap()
    torch.cuda.synchronize()
    for a, b in zip(fwd.src.tensors, back.tensors):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_remap_from_host_buffers(device):
    wl = make_workload("cfg3", "small")
    case = DeviceCase(wl, device)
    want = oracle_for(case)
    host_src = [t.cpu().pin_memory() for t in case.src.tensors]
    host_dst = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in case.dst.tensors]
    for t in case.src.tensors:
        t.zero_()
    case.plan.remap_host([t.data_ptr() for t in host_src], [t.data_ptr() for t in host_dst])
    torch.cuda.synchronize()
    for k, t in enumerate(host_dst):
        assert np.array_equal(to_bits(t), want.dst[k])


@pytest.mark.parametrize("name,scale,kib", [("cfg5", "medium", 512), ("cfg3", "medium", 2048), ("cfg2", "medium", 4096)])
def test_remap_from_host_buffers_in_many_stages(device, name, scale, kib):
    """wb_remap_host with small pipeline stages: a stage's kernel may only read what its own uploads
    brought (the trainer tensors on the device hold zeros beforehand), including the source rows a
    transposing tile reads across the seam to the tile below, which may belong to the next stage."""
    wl = make_workload(name, scale)
    case = DeviceCase(wl, device, host_group_kib=kib)
    want = oracle_for(case)
    host_src = [t.cpu().pin_memory() for t in case.src.tensors]
    host_dst = [torch.full(t.shape, -1, dtype=torch.int16 if t.element_size() == 2 else torch.int32).view(t.dtype).pin_memory()
                for t in case.dst.tensors]
    for a in case.src.arenas.values():
        a.zero_()
    case.plan.remap_host([t.data_ptr() for t in host_src], [t.data_ptr() for t in host_dst])
    torch.cuda.synchronize()
    case.plan.check()
    for k, t in enumerate(host_dst):
        assert np.array_equal(to_bits(t), want.dst[k]), k


def test_empty_layouts_launch_nothing(device):
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T", 0, WB_F32, 16)
    rl.add_tensor("R", 0, WB_BF16, 16)
    tl.freeze(); rl.freeze()
    plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices))
    plan.verify()
    st = plan.stats()
    assert st["n_tiles_remap"] == 0 and st["src_elems_read"] == 0 and plan.num_rounds() == 1
    src = RankArenas(tl.tensors, device, fill_byte=1)
    dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
    bind(plan, src, dst)
    plan.remap()
    bucket = torch.zeros(64, dtype=torch.uint8, device=device)
    plan.pack(0, bucket.data_ptr())
    plan.unpack(0, bucket.data_ptr())
    torch.cuda.synchronize()
    plan.check()
    assert (to_bits(dst.tensors[0]) == 0xCDCD).all()


def test_offsets_beyond_32_bits(device):
    """One tensor of 4.4 G elements (8.8 GB a side): element offsets, tile counts and bucket offsets
    need 64 bits.  Trainer: two flat shards; rollout: one tensor, so slabs start deep inside."""
    n = (1 << 32) + 123_456_789
    if torch.cuda.mem_get_info()[0] < 2 * 2 * n + (8 << 30):
        pytest.skip("needs ~26 GB of free device memory")
    half = n // 2 + 7
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T0", 0, WB_BF16, half)
    tl.add_tensor("T1", 1, WB_BF16, n - half)
    rl.add_tensor("R", 0, WB_BF16, n)
    tl.add_slice(0, 0, n, 1, 0, 1, n, 0, 0, 1, half)
    tl.add_slice(1, 0, n, 1, 0, 1, n, 0, half, 1, n - half)
    rl.add_slice(0, 0, n, 1, 0, 1, n, 0, 0, 1, n)
    tl.freeze(); rl.freeze()
    plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices))
    plan.verify()
    assert plan.stats()["src_elems_read"] == n and plan.num_rounds() >= 3
    src = RankArenas(tl.tensors, device)
    dst = RankArenas(rl.tensors, device, fill_byte=CANARY)
    g = torch.Generator(device=device); g.manual_seed(3)
    for t in src.tensors:                       # random 16-bit patterns, generated in pieces
        v = t.view(torch.int16)
        for a in range(0, v.numel(), 1 << 28):
            b = min(a + (1 << 28), v.numel())
            v[a:b] = torch.randint(-32768, 32767, (b - a,), dtype=torch.int16, device=device, generator=g)
    bind(plan, src, dst)
    plan.remap()
    torch.cuda.synchronize()
    out = dst.tensors[0].view(torch.int16)
    assert torch.equal(out[:half], src.tensors[0].view(torch.int16))
    assert torch.equal(out[half:], src.tensors[1].view(torch.int16))
    # the two-pass path over the same range
    dst.arenas[0].fill_(CANARY)
    bucket = torch.empty(max(plan.bucket_bytes(r) for r in range(plan.num_rounds())), dtype=torch.uint8, device=device)
    for r in range(plan.num_rounds()):
        plan.pack(r, bucket.data_ptr())
        plan.unpack(r, bucket.data_ptr())
    torch.cuda.synchronize()
    plan.check()
    assert torch.equal(out[:half], src.tensors[0].view(torch.int16))
    assert torch.equal(out[half:], src.tensors[1].view(torch.int16))


@pytest.mark.parametrize("name,scale", [("cfg1b", "full"), ("cfg3", "small"), ("cfg5", "small"), ("cfg2", "medium")])
def test_static_schedule_gives_the_same_result(device, name, scale):
    """WB_PLAN_STATIC_SCHEDULE: every thread block walks the planner's fixed tile range instead of
    drawing batches at run time; the output must not depend on the schedule."""
    case = DeviceCase(make_workload(name, scale), device, flags=wb.WB_PLAN_STATIC_SCHEDULE,
                      bucket_budget_bytes=1 << 20)
    want = oracle_for(case)
    case.plan.remap()
    torch.cuda.synchronize()
    case.plan.check()
    assert_dst_equals(case, want)
    case.reset_dst()
    for r in range(case.plan.num_rounds()):
        bucket = torch.empty(case.plan.bucket_bytes(r), dtype=torch.uint8, device=device)
        case.plan.pack(r, bucket.data_ptr())
        case.plan.unpack(r, bucket.data_ptr())
    torch.cuda.synchronize()
    case.plan.check()
    assert_dst_equals(case, want)


def test_bounded_wait_gives_up_and_the_context_survives(device):
    """Every wait inside the kernels has a time limit.  A wait on a barrier that nothing signals runs
    out, reports through the error word, and the kernel ends normally: later work still runs."""
    import time
    t0 = time.perf_counter()
    status = wb.wb_wait_probe(50, torch.cuda.current_stream().cuda_stream)
    dt = time.perf_counter() - t0
    assert status == 11                      # WB_ERR_INTERNAL: the wait gave up as designed
    assert 0.04 < dt < 1.5
    case = DeviceCase(make_workload("cfg1"), device)     # the context is still usable
    want = oracle_for(case)
    case.plan.remap()
    torch.cuda.synchronize()
    case.plan.check()
    assert_dst_equals(case, want)


def test_replica_consistency_check(device):
    """The plan reads a replicated region from one replica; wb_plan_check_replicas verifies the
    assumption behind that on the bound tensors."""
    wl = make_workload("cfg1")                    # norms live on both TP ranks
    case = DeviceCase(wl, device)
    assert case.plan.check_replicas() == 0
    k = wl.trainer.index("t2.final.flat")          # TP rank 1's copy of final_norm starts this shard
    case.src.tensors[k][3] += 1.0
    case.src.tensors[k][200] += 1.0
    assert case.plan.check_replicas() == 2
    wl4 = make_workload("cfg4", "small")           # no replicas at all
    assert DeviceCase(wl4, device).plan.check_replicas() == 0


def test_remap_in_a_cuda_graph(device):
    """wb_remap is one kernel launch on the caller's stream, so it can be captured into a CUDA graph and
    replayed (after one ordinary call, which sets the kernel's shared-memory attribute)."""
    case = DeviceCase(make_workload("cfg1b"), device)
    want = oracle_for(case)
    case.plan.remap()                                   # outside capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream(device=device)
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            case.plan.remap(torch.cuda.current_stream().cuda_stream)
    for _ in range(3):
        case.reset_dst()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert_dst_equals(case, want)
    case.plan.check()


@pytest.mark.parametrize("name,scale,budget", [
    ("cfg1b", "full", 1 << 20), ("cfg3", "small", 1 << 20), ("cfg4", "small", 1 << 19), ("cfg5", "small", 1 << 18),
    ("cfg3", "medium", 32 << 20), ("cfg5", "medium", 16 << 20)])
def test_rank_subsets_compose_to_the_whole_round(device, name, scale, budget):
    """wb_pack_ranks / wb_unpack_ranks (Section 3.2: every worker packs its own shards and assembles its
    own parameters): a trainer rank's call writes exactly its (receiver, sender) regions of the bucket,
    the calls of all ranks together fill the bucket wb_pack fills, and assembling the rollout ranks one
    group at a time gives the oracle's tensors."""
    wl = make_workload(name, scale)
    case = DeviceCase(wl, device, bucket_budget_bytes=budget)
    want = oracle_for(case)
    plan = case.plan
    nt, nr = plan.num_ranks()
    rng = np.random.default_rng(5)
    for r in range(plan.num_rounds()):
        nb = plan.bucket_bytes(r)
        whole = torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=device)
        plan.pack(r, whole.data_ptr())
        regions = plan.bucket_regions(r)
        parts = torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=device)
        # one rank alone: only its regions change
        for v in range(nt):
            alone = torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=device)
            plan.pack_ranks(r, [v], alone.data_ptr())
            torch.cuda.synchronize()
            mine = torch.zeros(nb + 64, dtype=torch.bool, device=device)
            for g in regions:
                if int(g["sender"]) == v:
                    mine[int(g["off"]):int(g["off"]) + int(g["bytes"])] = True
            assert torch.equal(alone[mine], whole[mine]) and bool((alone[~mine] == 0x5A).all()), (r, v)
        # a random grouping of the ranks (lists with gaps and duplicates) fills the whole bucket
        order = rng.permutation(nt)
        cut = int(rng.integers(0, nt + 1))
        for group in (order[:cut], order[cut:]):
            plan.pack_ranks(r, [int(x) for x in group] + [int(x) for x in group[:1]], parts.data_ptr())
        torch.cuda.synchronize()
        assert torch.equal(parts, whole), r
        order = rng.permutation(nr)
        cut = int(rng.integers(0, nr + 1))
        for group in (order[:cut], order[cut:]):
            plan.unpack_ranks(r, [int(x) for x in group], parts.data_ptr())
    torch.cuda.synchronize()
    assert_dst_equals(case, want)
    plan.check()
    with pytest.raises(wb.WbError):
        plan.pack_ranks(0, [nt], whole.data_ptr())
    with pytest.raises(wb.WbError):
        plan.unpack_ranks(0, [nr], whole.data_ptr())
    plan.pack_ranks(0, [], whole.data_ptr())          # an empty set launches nothing
