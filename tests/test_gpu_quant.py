"""FP8 quantisation of transfer buckets on the GPU against the oracle: the per-tensor maxima, the
quantised bucket of every round, the dequantised bucket, and the rollout tensors after assembly."""
import numpy as np
import pytest
import torch

from gpu_util import DeviceCase
from helpers import ckpt_shapes, from_bits, to_bits
from oracle import checkpoint_view, quant
from oracle.cast import cast_bits
from paper_2609_25442_b200 import binding as wb
from paper_2609_25442_b200.device import RankArenas, bind
from wb_workloads import WB_BF16, WB_F32, Layout, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BITS = {WB_F32: np.uint32, WB_BF16: np.uint16}


def same_bits(a, b, dtype):
    """Bitwise equality; for fp32, NaN payloads of a product are not fixed by IEEE 754, so NaN-ness is compared."""
    if dtype != WB_F32:
        return np.array_equal(a, b)
    fa, fb = np.asarray(a).view(np.float32), np.asarray(b).view(np.float32)
    return np.array_equal(np.isnan(fa), np.isnan(fb)) and np.array_equal(a[~np.isnan(fa)], b[~np.isnan(fb)])


def run_quantised_transfer(case, wl_src_dtype, wl_dst_dtype, shapes, ckpt_of_id, keep=None):
    """pack -> quantise -> dequantise -> unpack for every round, checking each stage against the oracle.
    Returns the oracle's dequantised checkpoint tensors (destination dtype bits)."""
    plan = case.plan
    dev = case.device
    ids = plan.ckpt_ids()
    src_bits = case.src_bits()
    views = {int(t): cast_bits(checkpoint_view(int(t), shapes[ckpt_of_id(int(t))], case.trainer.slices, src_bits)[0],
                               wl_src_dtype, wl_dst_dtype) for t in ids}
    # the gather: one maximum per checkpoint tensor
    amax = torch.full((len(ids),), 7.0, dtype=torch.float32, device=dev)          # must be overwritten
    plan.absmax(amax.data_ptr())
    torch.cuda.synchronize()
    got_amax = amax.cpu().numpy().view(np.uint32)
    want_amax = np.array([quant.amax_bits(views[int(t)].reshape(-1), wl_dst_dtype) for t in ids], np.uint32)
    assert np.array_equal(got_amax, want_amax)
    scales = {int(t): quant.scale_of(want_amax[k]) for k, t in enumerate(ids)}
    rscales = {int(t): quant.rscale_of(want_amax[k]) for k, t in enumerate(ids)}
    ed = 2 if wl_dst_dtype == WB_BF16 else 4
    for r in range(plan.num_rounds()):
        nb = plan.bucket_bytes(r)
        assert plan.qbucket_bytes(r) == nb // ed
        bucket = torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=dev)
        qb = torch.full((nb // ed + 64,), 0xA5, dtype=torch.uint8, device=dev)
        plan.pack(r, bucket.data_ptr())
        plan.bucket_quantize(r, bucket.data_ptr(), qb.data_ptr(), amax.data_ptr())
        bucket2 = torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=dev)
        plan.bucket_dequantize(r, qb.data_ptr(), bucket2.data_ptr(), amax.data_ptr())
        torch.cuda.synchronize()
        q = qb.cpu().numpy()
        if keep is not None:
            keep.append(q.copy())
        b2 = bucket2[:nb].cpu().numpy().view(BITS[wl_dst_dtype])
        covered = np.zeros(nb // ed, bool)
        for e in plan.bucket_entries(r):
            t = int(e["ckpt_tensor"])
            r0, c0, nr, nc = (int(e[k]) for k in ("r0", "c0", "nr", "nc"))
            rect = views[t][r0:r0 + nr, c0:c0 + nc].reshape(-1)
            off = int(e["bucket_off"]) // ed
            codes = quant.quantize(rect, wl_dst_dtype, scales[t], rscales[t])
            assert np.array_equal(q[off:off + nr * nc], codes), (r, t)
            back = quant.dequantize(codes, wl_dst_dtype, scales[t])
            assert same_bits(b2[off:off + nr * nc], back, wl_dst_dtype), (r, t)
            covered[off:off + nr * nc] = True
        assert (q[:nb // ed][~covered] == 0xA5).all() and (q[nb // ed:] == 0xA5).all()   # padding never written
        pad = 0x5A5A if ed == 2 else 0x5A5A5A5A
        assert (b2[~covered] == pad).all() and bool((bucket2[nb:] == 0x5A).all())
        plan.unpack(r, bucket2.data_ptr())
    torch.cuda.synchronize()
    plan.check()
    return {t: quant.dequantize(quant.quantize(v.reshape(-1), wl_dst_dtype, scales[t], rscales[t]), wl_dst_dtype,
                                scales[t]).reshape(v.shape) for t, v in views.items()}


@pytest.mark.parametrize("name,scale,budget", [
    ("cfg1", "full", 0), ("cfg1b", "full", 1 << 20), ("cfg3", "small", 1 << 20), ("cfg4", "small", 1 << 19),
    ("cfg5", "small", 1 << 18), ("cfg2", "medium", 16 << 20), ("cfg5", "medium", 16 << 20)])
def test_quantised_rounds_match_the_oracle(name, scale, budget):
    wl = make_workload(name, scale)
    case = DeviceCase(wl, torch.device(DEV), bucket_budget_bytes=budget)
    shapes = ckpt_shapes(wl)
    want = run_quantised_transfer(case, wl.src_dtype, wl.dst_dtype, shapes, lambda t: t)
    # the rollout tensors hold the dequantised checkpoint tensors, in the rollout layout
    dst_bits = case.dst_bits()
    for t, v in want.items():
        got = checkpoint_view(t, shapes[t], case.rollout.slices, dst_bits)[0]
        assert np.array_equal(got, v), wl.ckpt[t].name
    assert case.gaps_intact()


def run_fused_transfer(case, qbuckets, dst_reset):
    """wb_pack_fp8 must write exactly the FP8 bucket that wb_pack + wb_bucket_quantize wrote (checked against the
    oracle by the caller, padding and guard bytes included); wb_unpack_fp8 then assembles from it."""
    plan, dev = case.plan, case.device
    amax = torch.zeros(plan.num_ckpts(), dtype=torch.float32, device=dev)
    plan.absmax(amax.data_ptr())
    dst_reset()
    for r in range(plan.num_rounds()):
        qb = torch.full((len(qbuckets[r]),), 0xA5, dtype=torch.uint8, device=dev)
        plan.pack_fp8(r, qb.data_ptr(), amax.data_ptr())
        torch.cuda.synchronize()
        assert np.array_equal(qb.cpu().numpy(), qbuckets[r]), r
        plan.unpack_fp8(r, qb.data_ptr(), amax.data_ptr())
    torch.cuda.synchronize()
    plan.check()


@pytest.mark.parametrize("name,scale,budget", [
    ("cfg1", "full", 0), ("cfg1b", "full", 1 << 20), ("cfg3", "small", 1 << 20), ("cfg4", "small", 1 << 19),
    ("cfg5", "small", 1 << 18), ("cfg2", "medium", 16 << 20), ("cfg5", "medium", 16 << 20)])
def test_fused_quantised_rounds_match_the_oracle(name, scale, budget):
    """The fused kernels (quantise while packing, dequantise while assembling) against the oracle: the FP8
    bucket of every round and the rollout tensors, bit for bit."""
    wl = make_workload(name, scale)
    case = DeviceCase(wl, torch.device(DEV), bucket_budget_bytes=budget)
    shapes = ckpt_shapes(wl)
    kept = []
    want = run_quantised_transfer(case, wl.src_dtype, wl.dst_dtype, shapes, lambda t: t, keep=kept)
    run_fused_transfer(case, kept, case.reset_dst)
    dst_bits = case.dst_bits()
    for t, v in want.items():
        got = checkpoint_view(t, shapes[t], case.rollout.slices, dst_bits)[0]
        assert np.array_equal(got, v), wl.ckpt[t].name
    assert case.gaps_intact()
    # and pipelined over two FP8 buckets
    plan, dev = case.plan, case.device
    nq = max(plan.qbucket_bytes(r) for r in range(plan.num_rounds()))
    q = [torch.full((nq + 64,), 0xA5, dtype=torch.uint8, device=dev) for _ in range(2)]
    amax = torch.zeros(plan.num_ckpts(), dtype=torch.float32, device=dev)
    side = torch.cuda.Stream(device=dev)
    for stream in (None, side):
        case.reset_dst()
        torch.cuda.synchronize()
        plan.transfer_rounds_fp8_fused(q[0].data_ptr(), q[1].data_ptr(), amax.data_ptr(), 0 if stream is None else stream.cuda_stream)
        (torch.cuda if stream is None else stream).synchronize()
        dst_bits = case.dst_bits()
        for t, v in want.items():
            assert np.array_equal(checkpoint_view(t, shapes[t], case.rollout.slices, dst_bits)[0], v), wl.ckpt[t].name
        plan.check()
        assert all(bool((x[nq:] == 0xA5).all()) for x in q)


@pytest.mark.parametrize("dts", [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)])
def test_special_tensors(dts):
    """All-zero tensors (scale 1), a tensor with an infinity (scale infinite), one with a NaN (no scale), odd
    lengths (scalar tails), values that land exactly between two codes, tensors of tiny magnitudes (the
    reciprocal scale overflows: encoded by division; zeros must stay zeros), a subnormal maximum so small
    that amax / 448 rounds to zero (scale = smallest subnormal), and a maximum of FLT_MAX."""
    sdt, ddt = dts
    n = 1003
    rng = np.random.default_rng(3)
    vals = [np.zeros(n, np.float32),
            rng.normal(0, 1, n).astype(np.float32),
            np.concatenate([[np.inf, -3.0, 0.5], rng.normal(0, 1, n - 3)]).astype(np.float32),
            np.concatenate([[np.nan, 2.0], rng.normal(0, 1, n - 2)]).astype(np.float32),
            # amax = 448, so the scale is 1 and the midpoints between codes are hit exactly
            np.concatenate([[448.0, -448.0, 1.0625, 1.1875, 0.0009765625, 17.0, 27.0, 464.0 / 2], rng.uniform(-448, 448, n - 8)]
                           ).astype(np.float32),
            np.concatenate([[0.0, 1e-37, -5e-38, 2e-38, -0.0], rng.normal(0, 3e-38, n - 5)]).astype(np.float32),
            np.concatenate([[0.0, 1.2e-39, -0.0], rng.normal(0, 4e-40, n - 3)]).astype(np.float32),       # subnormals
            (np.concatenate([[0, 150, -3, 1, -0.0], rng.integers(-150, 151, n - 5)]) * 2.0 ** -149).astype(np.float32),
            np.concatenate([[3.4028234663852886e38, 0.0, -1e38], np.clip(rng.normal(0, 1e38, n - 3), -3e38, 3e38)]).astype(np.float32)]
    if WB_BF16 in (sdt, ddt):
        # bf16 on either side: the fp32 subnormal-count tensor would round to zero or to coarse steps; use bf16's own
        # smallest subnormals (2^-133) instead, and the largest finite bf16 value
        vals[7] = (np.concatenate([[0, 2, -1, 1, -0.0], rng.integers(-2, 3, n - 5)]) * 2.0 ** -133).astype(np.float32)
        vals[8] = np.concatenate([[3.3895313892515355e38, 0.0, -1e38], np.clip(rng.normal(0, 1e38, n - 3), -3e38, 3e38)]).astype(np.float32)
    tl, rl = Layout("t"), Layout("r")
    for k in range(len(vals)):
        tl.add_tensor(f"T{k}", k % 2, sdt, n)
        tl.add_slice(k, 0, n, 1, k, 1, n, 0, 0, 1, n)
        rl.add_tensor(f"R{k}", 0, ddt, n)
        rl.add_slice(k, 0, n, 1, k, 1, n, 0, 0, 1, n)
    tl.freeze(); rl.freeze()

    class Case:
        pass
    case = Case()
    case.device = torch.device(DEV)
    case.trainer, case.rollout = tl, rl
    case.plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices), bucket_budget_bytes=4096)
    src = RankArenas(tl.tensors, case.device, fill_byte=0)
    dst = RankArenas(rl.tensors, case.device, fill_byte=0xCD)
    for k, v in enumerate(vals):
        t = torch.from_numpy(v)
        src.tensors[k].copy_((t if sdt == WB_F32 else t.to(torch.bfloat16)).to(case.device))
    bind(case.plan, src, dst)
    case.src_bits = lambda: [to_bits(t) for t in src.tensors]
    assert case.plan.num_rounds() > 1
    kept = []
    want = run_quantised_transfer(case, sdt, ddt, [(1, n)] * len(vals), lambda t: t, keep=kept)
    for k in range(len(vals)):
        got = to_bits(dst.tensors[k])
        assert same_bits(got, want[k].reshape(-1), ddt), k
    # the fused kernels on the same tensors (tiny magnitudes take the division rule there too)
    def reset():
        for a in dst.arenas.values():
            a.fill_(0xCD)
    run_fused_transfer(case, kept, reset)
    for k in range(len(vals)):
        assert same_bits(to_bits(dst.tensors[k]), want[k].reshape(-1), ddt), k


def test_rebinding_rebuilds_the_work_lists():
    """The amax work list holds device addresses: binding the plan to other tensors must rebuild it."""
    wl = make_workload("cfg1b")
    dev = torch.device(DEV)
    case = DeviceCase(wl, dev)
    plan = case.plan
    amax = torch.zeros(plan.num_ckpts(), dtype=torch.float32, device=dev)
    plan.absmax(amax.data_ptr())
    torch.cuda.synchronize()
    first = amax.clone()
    # a second set of trainer tensors with every value doubled (exact in fp32)
    src2 = RankArenas(wl.trainer.tensors, dev, fill_byte=0)
    for a, b in zip(src2.tensors, case.src.tensors):
        a.copy_(b * 2)
    bind(plan, src2, case.dst)
    plan.absmax(amax.data_ptr())
    torch.cuda.synchronize()
    assert torch.equal(amax, first * 2) and bool((first > 0).all())
    # and the old tensors may be gone by now
    case.src = None
    plan.absmax(amax.data_ptr())
    torch.cuda.synchronize()
    assert torch.equal(amax, first * 2)


@pytest.mark.parametrize("name,scale,budget", [("cfg1b", "full", 1 << 20), ("cfg3", "small", 1 << 20),
                                               ("cfg5", "medium", 16 << 20)])
def test_pipelined_quantised_rounds(name, scale, budget):
    """wb_transfer_rounds_fp8 (two bucket pairs in flight on two internal streams) leaves the rollout tensors
    the step-by-step quantised transfer leaves, which is the oracle's."""
    wl = make_workload(name, scale)
    dev = torch.device(DEV)
    case = DeviceCase(wl, dev, bucket_budget_bytes=budget)
    shapes = ckpt_shapes(wl)
    want = run_quantised_transfer(case, wl.src_dtype, wl.dst_dtype, shapes, lambda t: t)
    plan = case.plan
    assert plan.num_rounds() > 2
    nb = max(plan.bucket_bytes(r) for r in range(plan.num_rounds()))
    nq = max(plan.qbucket_bytes(r) for r in range(plan.num_rounds()))
    b = [torch.full((nb + 64,), 0x5A, dtype=torch.uint8, device=dev) for _ in range(2)]
    q = [torch.full((nq + 64,), 0xA5, dtype=torch.uint8, device=dev) for _ in range(2)]
    amax = torch.zeros(plan.num_ckpts(), dtype=torch.float32, device=dev)
    side = torch.cuda.Stream(device=dev)
    for stream in (None, side):
        case.reset_dst()
        torch.cuda.synchronize()
        sp = 0 if stream is None else stream.cuda_stream
        plan.transfer_rounds_fp8(b[0].data_ptr(), b[1].data_ptr(), q[0].data_ptr(), q[1].data_ptr(), amax.data_ptr(), sp)
        (torch.cuda if stream is None else stream).synchronize()
        dst_bits = case.dst_bits()
        for t, v in want.items():
            assert np.array_equal(checkpoint_view(t, shapes[t], case.rollout.slices, dst_bits)[0], v), wl.ckpt[t].name
        plan.check()
        assert all(bool((x[nb:] == 0x5A).all()) for x in b) and all(bool((x[nq:] == 0xA5).all()) for x in q)
    with pytest.raises(wb.WbError):
        plan.transfer_rounds_fp8(b[0].data_ptr(), b[0].data_ptr(), q[0].data_ptr(), q[1].data_ptr(), amax.data_ptr())
