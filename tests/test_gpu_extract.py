"""Source-map extraction on the GPU: the diff2 kernel against the oracle's definition, and the whole
chain -- chunked id probe through the parameters' own dtype, diff2 + compaction on the device,
recombination and scan on the host -- producing source maps that drive the same transfer."""
import numpy as np
import pytest
import torch

from gpu_util import DeviceCase
from helpers import ckpt_shapes, predict_ids, to_bits
from oracle import remap_oracle
from oracle.extract import diff2, id_chunk, nonzeros
from paper_2609_25442_b200 import binding as wb
from paper_2609_25442_b200.device import RankArenas, bind
from wb_workloads import WB_BF16, WB_F32, Layout, make_workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def gpu_entries(field: torch.Tensor, kind: int, cap: int = 1 << 16):
    """Run wb_diff2_nonzeros on a 2-D device tensor; returns (sorted entries, count reported)."""
    field = field.contiguous()
    out = torch.zeros(cap * 24, dtype=torch.uint8, device=field.device)
    count = torch.zeros(1, dtype=torch.int64, device=field.device)
    wb.wb_diff2_nonzeros(field.data_ptr(), kind, field.shape[0], field.shape[1], out.data_ptr(), cap,
                         count.data_ptr(), torch.cuda.current_stream().cuda_stream)
    n = int(count.item())
    e = out.cpu().numpy().view(wb.DIFF2_ENTRY_DTYPE)[:min(n, cap)].copy()
    return np.sort(e, order=["row", "col"]), n


def oracle_entries(a: np.ndarray):
    nz = nonzeros(diff2(a))
    return np.array(nz, dtype=wb.DIFF2_ENTRY_DTYPE) if nz else np.zeros(0, wb.DIFF2_ENTRY_DTYPE)


@pytest.mark.parametrize("shape", [(1, 1), (1, 100003), (7, 33), (257, 1023), (1000, 2), (3, 70001)])
def test_diff2_kernel_matches_the_definition(shape):
    rng = np.random.default_rng(shape[0] * 131 + shape[1])
    # piecewise-affine field with a few random rectangles, plus some isolated noise
    a = np.zeros(shape, np.int64)
    for _ in range(6):
        i0, j0 = rng.integers(0, shape[0]), rng.integers(0, shape[1])
        ni, nj = rng.integers(1, shape[0] - i0 + 1), rng.integers(1, shape[1] - j0 + 1)
        ii, jj = np.meshgrid(np.arange(ni), np.arange(nj), indexing="ij")
        a[i0:i0 + ni, j0:j0 + nj] = int(rng.integers(1, 1 << 40)) + ii * int(rng.integers(1, 1 << 20)) + jj
    for _ in range(5):
        a[rng.integers(0, shape[0]), rng.integers(0, shape[1])] = int(rng.integers(1, 1 << 45))
    want = oracle_entries(a)
    got, n = gpu_entries(torch.from_numpy(a).to(DEV), wb.WB_ID_I64)
    assert n == len(want) and np.array_equal(got, want)


def _piecewise_affine(shape, rng, n_rect=8):
    a = np.zeros(shape, np.int64)
    for _ in range(n_rect):
        i0, j0 = rng.integers(0, shape[0]), rng.integers(0, shape[1])
        ni, nj = rng.integers(1, shape[0] - i0 + 1), rng.integers(1, shape[1] - j0 + 1)
        a[i0:i0 + ni, j0:j0 + nj] = (int(rng.integers(1, 1 << 40)) + np.arange(ni)[:, None] * int(rng.integers(1, 1 << 20))
                                     + np.arange(nj)[None, :])
    return a


def test_diff2_kernel_on_a_field_of_many_row_blocks():
    """More (strip, row block) tasks than resident warps: the rows per task are rebalanced, warps walk
    several tasks each, and rectangle edges fall on every position relative to the task seams."""
    rng = np.random.default_rng(77)
    a = _piecewise_affine((40000, 1100), rng, n_rect=24)
    for i in (0, 1, 2, 63, 64, 65, 84, 85, 86, 169, 170, 39999):        # isolated entries around likely seams
        a[i, rng.integers(0, 1100)] += int(rng.integers(1, 1 << 30))
    want = oracle_entries(a)
    got, n = gpu_entries(torch.from_numpy(a).to(DEV), wb.WB_ID_I64, cap=1 << 18)
    assert n == len(want) and np.array_equal(got, want)


@pytest.mark.parametrize("shape", [(1, 4099), (1, 4096), (9, 514), (9, 515), (130, 260)])
@pytest.mark.parametrize("skew", [1, 2, 3])
def test_diff2_kernel_at_any_alignment_of_the_field(shape, skew):
    """Fields that start `skew` elements into an allocation: rows whose first element is not on the
    boundary the vector loads want take the element-wise loads, with the same result."""
    rng = np.random.default_rng(shape[0] * 7 + shape[1] + skew)
    a = _piecewise_affine(shape, rng)
    n = a.size
    want = oracle_entries(a)
    buf = torch.zeros(n + 8, dtype=torch.int64, device=DEV)
    buf[skew:skew + n] = torch.from_numpy(a.reshape(-1)).to(DEV)
    got, cnt = gpu_entries(buf[skew:skew + n].view(*shape), wb.WB_ID_I64)
    assert cnt == len(want) and np.array_equal(got, want)
    # 16-bit chunks of the same field, as raw bits
    c16 = id_chunk(a, 0, 16)
    b16 = torch.zeros(n + 8, dtype=torch.int16, device=DEV)
    b16[skew:skew + n] = torch.from_numpy(c16.astype(np.uint16).view(np.int16).reshape(-1)).to(DEV)
    got16, _ = gpu_entries(b16[skew:skew + n].view(*shape), wb.WB_ID_U16, 1 << 17)
    assert np.array_equal(got16, oracle_entries(c16))
    # 24-bit chunks held in fp32
    c24 = id_chunk(a, 0, 24)
    b32 = torch.zeros(n + 8, dtype=torch.float32, device=DEV)
    b32[skew:skew + n] = torch.from_numpy(c24.astype(np.float32).reshape(-1)).to(DEV)
    got32, _ = gpu_entries(b32[skew:skew + n].view(*shape), wb.WB_ID_F32, 1 << 17)
    assert np.array_equal(got32, oracle_entries(c24))


def test_diff2_kernel_reads_chunks_in_the_parameter_dtypes():
    rng = np.random.default_rng(5)
    ids = rng.integers(1, 1 << 34, size=(61, 517)).astype(np.int64)
    c16 = id_chunk(ids, 1, 16)
    t16 = torch.from_numpy(c16.astype(np.uint16).view(np.int16)).to(DEV)          # raw bits of a bf16 tensor
    assert np.array_equal(gpu_entries(t16, wb.WB_ID_U16, 1 << 17)[0], oracle_entries(c16))
    c8 = id_chunk(ids, 2, 8)
    tb = torch.from_numpy(c8.astype(np.float32)).to(torch.bfloat16).to(DEV)        # 0..255 are exact in bf16
    assert np.array_equal(gpu_entries(tb, wb.WB_ID_BF16, 1 << 17)[0], oracle_entries(c8))
    c24 = id_chunk(ids, 0, 24)
    tf = torch.from_numpy(c24.astype(np.float32)).to(DEV)                          # < 2^24: exact in fp32
    assert np.array_equal(gpu_entries(tf, wb.WB_ID_F32, 1 << 17)[0], oracle_entries(c24))


def test_diff2_kernel_reports_overflow_of_the_list():
    a = torch.arange(1, 4097, dtype=torch.int64, device=DEV).view(64, 64) ** 2     # nothing cancels
    got, n = gpu_entries(a, wb.WB_ID_I64, cap=100)
    assert n > 100 and len(got) == 100
    full, n2 = gpu_entries(a, wb.WB_ID_I64, cap=8192)
    assert n2 == n == len(full)


def batch_entries(tensors, kind, cap=1 << 20):
    """wb_diff2_nonzeros_batch over {tag: 2-D device tensor}; returns {tag: sorted plain entries}."""
    tags = sorted(tensors)
    fields = np.array([(tensors[t].data_ptr(), tensors[t].shape[0], tensors[t].shape[1], kind, t) for t in tags],
                      dtype=wb.DIFF2_FIELD_DTYPE)
    nb = wb.wb_diff2_batch_scratch_bytes(len(fields))
    scratch = torch.zeros(max(nb, 16), dtype=torch.uint8, device=DEV)
    out = torch.zeros(cap * 32, dtype=torch.uint8, device=DEV)
    count = torch.zeros(1, dtype=torch.int64, device=DEV)
    wb.wb_diff2_nonzeros_batch(fields, scratch.data_ptr(), nb, out.data_ptr(), cap, count.data_ptr(),
                               torch.cuda.current_stream().cuda_stream)
    n = int(count.item())
    assert n <= cap
    e = out.cpu().numpy().view(wb.DIFF2_TAGGED_ENTRY_DTYPE)[:n]
    res = {}
    for t in tags:
        m = e[e["tag"] == t]
        plain = np.zeros(len(m), wb.DIFF2_ENTRY_DTYPE)
        for f in ("row", "col", "value"):
            plain[f] = m[f]
        res[t] = np.sort(plain, order=["row", "col"])
    return res


def extract_on_gpu(wl, side, chunk_bits, batched=False):
    """Algorithm 1 on one side: K passes of load_weights with b-bit id chunks in the parameters' own
    dtype, diff2 per local tensor on the device, recombination and scan in the library."""
    declared = wl.trainer if side == "trainer" else wl.rollout
    dt = wl.src_dtype if side == "trainer" else wl.dst_dtype
    tdt = torch.float32 if dt == WB_F32 else torch.bfloat16
    if dt == WB_F32:
        kind = wb.WB_ID_F32
    else:
        kind = wb.WB_ID_U16 if chunk_bits == 16 else wb.WB_ID_BF16
    K = -(-int(wl.ckpt_numel() + 1).bit_length() // chunk_bits)
    passes = [dict() for _ in range(declared.n_tensors)]
    shapes = {}
    for k in range(K):
        def values(i, k=k):
            part = ((wl.ckpt_ids(i, DEV) + 1) >> (chunk_bits * k)) & ((1 << chunk_bits) - 1)
            if kind == wb.WB_ID_U16:
                return part.to(torch.int16).view(torch.bfloat16)     # raw 16-bit payload
            return part.to(tdt)                                       # an exactly representable integer

        def sink(t, x, k=k):
            x = x.reshape(1, -1) if x.dim() == 1 else x.reshape(-1, x.shape[-1])
            if x.dtype not in (torch.float32, torch.bfloat16):        # integer padding of the loaders
                x = x.clamp_min(0)
            shapes[t] = tuple(x.shape)
            if batched:
                held[t] = x.contiguous()
                return
            passes[t][k], n = gpu_entries(x, kind, cap=1 << 18)
            assert n == len(passes[t][k])
        held = {}
        wl.load_side_shaped(side, values, sink)
        if batched:                                   # every local tensor of the pass in one launch
            for t, ent in batch_entries(held, kind).items():
                passes[t][k] = ent
    base = wl.ckpt_base().astype(np.uint64)
    rows = np.array([c.rows for c in wl.ckpt], np.uint64)
    cols = np.array([c.cols for c in wl.ckpt], np.uint64)
    lay = Layout(side)
    for t in range(declared.n_tensors):
        d = declared.tensors[t]
        lay.add_tensor(declared.names[t], int(d["rank"]), int(d["dtype"]), int(d["numel"]))
        z = wb.wb_diff2_recombine([passes[t][k] for k in range(K)], chunk_bits)
        for s in wb.wb_scan_slices(z, shapes[t][0], shapes[t][1], base, rows, cols, t):
            lay.add_slice(int(s["tensor"]), int(s["local_off"]), int(s["stride_r"]), int(s["stride_c"]),
                          int(s["ckpt"]), int(s["ckpt_rows"]), int(s["ckpt_cols"]),
                          int(s["r0"]), int(s["c0"]), int(s["nr"]), int(s["nc"]))
    return lay.freeze()


@pytest.mark.parametrize("name,scale,bits", [("cfg3", "small", 16), ("cfg4", "small", 16), ("cfg4", "small", 8),
                                              ("cfg5", "small", 16), ("cfg1b", "full", 16)])
def test_extracted_source_maps_give_the_same_remap(name, scale, bits):
    wl = make_workload(name, scale)
    batched = name in ("cfg5", "cfg4")                # the many-tensor configurations go through the batched scan
    tl = extract_on_gpu(wl, "trainer", bits, batched)
    rl = extract_on_gpu(wl, "rollout", bits, batched)
    for lay, declared in ((tl, wl.trainer), (rl, wl.rollout)):
        for a, b in zip(predict_ids(lay, wl), predict_ids(declared, wl)):
            assert np.array_equal(a, b)                # same source map, element for element
    case = DeviceCase(wl, torch.device(DEV), trainer=tl, rollout=rl)
    want = remap_oracle(ckpt_shapes(wl), wl.trainer.tensors, wl.trainer.slices, wl.rollout.tensors,
                        wl.rollout.slices, case.src_bits())
    case.plan.remap()
    torch.cuda.synchronize()
    case.plan.check()
    for k, got in enumerate(case.dst_bits()):
        assert np.array_equal(got[want.written[k]], want.dst[k][want.written[k]]), wl.rollout.names[k]


def test_batched_diff2_over_many_fields():
    """One launch over fields of every kind and shape (one-row, thin, wide, tall, empty) returns, per tag,
    exactly the entries of the definition."""
    rng = np.random.default_rng(21)
    shapes = [(1, 1), (1, 5000), (7, 33), (300, 700), (2, 9000), (0, 10), (1000, 3), (65, 257), (129, 1)] * 3
    shapes += [(4100, 4100), (1, 16800000)]       # large fields: launched on their own by the entry point
    tensors, want, desc = [], {}, []
    for k, shp in enumerate(shapes):
        kind = [wb.WB_ID_I64, wb.WB_ID_U16, wb.WB_ID_F32, wb.WB_ID_BF16][k % 4]
        if shp[0] * shp[1] == 0:
            desc.append((0, shp[0], shp[1], kind, k))
            continue
        a = _piecewise_affine(shp, rng, n_rect=4)
        if kind == wb.WB_ID_I64:
            t, ref = torch.from_numpy(a).to(DEV), a
        elif kind == wb.WB_ID_U16:
            ref = id_chunk(a, 0, 16)
            t = torch.from_numpy(ref.astype(np.uint16).view(np.int16)).to(DEV)
        elif kind == wb.WB_ID_F32:
            ref = id_chunk(a, 0, 24)
            t = torch.from_numpy(ref.astype(np.float32)).to(DEV)
        else:
            ref = id_chunk(a, 1, 8)
            t = torch.from_numpy(ref.astype(np.float32)).to(torch.bfloat16).to(DEV)
        tensors.append(t)
        want[k] = oracle_entries(ref)
        desc.append((t.data_ptr(), shp[0], shp[1], kind, k))
    fields = np.array(desc, dtype=wb.DIFF2_FIELD_DTYPE)
    nb = wb.wb_diff2_batch_scratch_bytes(len(fields))
    scratch = torch.zeros(nb, dtype=torch.uint8, device=DEV)
    cap = 1 << 18
    out = torch.zeros(cap * 32, dtype=torch.uint8, device=DEV)
    count = torch.zeros(1, dtype=torch.int64, device=DEV)
    wb.wb_diff2_nonzeros_batch(fields, scratch.data_ptr(), nb, out.data_ptr(), cap, count.data_ptr(),
                               torch.cuda.current_stream().cuda_stream)
    n = int(count.item())
    assert n == sum(len(v) for v in want.values()) and n <= cap
    e = out.cpu().numpy().view(wb.DIFF2_TAGGED_ENTRY_DTYPE)[:n]
    for k, w in want.items():
        mine = np.sort(e[e["tag"] == k], order=["row", "col"])
        assert len(mine) == len(w), k
        assert np.array_equal(mine["row"], w["row"]) and np.array_equal(mine["col"], w["col"]) \
            and np.array_equal(mine["value"], w["value"]), k
    assert set(np.unique(e["tag"]).tolist()) <= set(want)


# ---- chunk passes with carries (Algorithm 1, inner loop) --------------------------------------------------
from oracle.extract import chunk_passes, recombine


def _as_entries(dense: np.ndarray):
    nz = nonzeros(dense)
    return np.array(nz, dtype=wb.DIFF2_ENTRY_DTYPE) if nz else np.zeros(0, wb.DIFF2_ENTRY_DTYPE)


def _chunk_tensor(ids: np.ndarray, k: int, b: int):
    """Chunk k of the ids the way a parameter tensor holds it: an 8-bit chunk as a bf16 value (exact), a
    16-bit chunk as the raw pattern of a 16-bit element."""
    c = id_chunk(ids, k, b)
    if b == 8:
        return torch.from_numpy(c.astype(np.float32)).to(torch.bfloat16).to(DEV), wb.WB_ID_BF16
    return torch.from_numpy(c.astype(np.uint16).view(np.int16)).to(DEV), wb.WB_ID_U16


def gpu_chunk_passes(ids: np.ndarray, b: int, n_passes: int, cap: int = 1 << 18):
    rows, cols = ids.shape
    nb = wb.wb_diff2_chunk_scratch_bytes(rows, cols)
    scratch = torch.full((nb,), 0x77, dtype=torch.uint8, device=DEV)           # contents must not matter
    stream = torch.cuda.current_stream().cuda_stream
    z_lists, g_lists = [], []
    carry = np.zeros(0, wb.DIFF2_ENTRY_DTYPE)
    for k in range(n_passes):
        field, kind = _chunk_tensor(ids, k, b)
        zo = torch.zeros(cap * 24, dtype=torch.uint8, device=DEV)
        go = torch.zeros(cap * 24, dtype=torch.uint8, device=DEV)
        counts = torch.zeros(2, dtype=torch.int64, device=DEV)
        cin = torch.from_numpy(carry.view(np.uint8).copy()).to(DEV) if len(carry) else None   # host -> device
        wb.wb_diff2_chunk_pass(field.data_ptr(), kind, rows, cols, b, k, cin.data_ptr() if cin is not None else 0,
                               len(carry), scratch.data_ptr(), nb, zo.data_ptr(), cap, counts.data_ptr(),
                               go.data_ptr(), cap, counts.data_ptr() + 8, stream)
        nz, ng = (int(x) for x in counts.cpu())
        assert nz <= cap and ng <= cap
        z = np.sort(zo.cpu().numpy().view(wb.DIFF2_ENTRY_DTYPE)[:nz].copy(), order=["row", "col"])
        carry = np.sort(go.cpu().numpy().view(wb.DIFF2_ENTRY_DTYPE)[:ng].copy(), order=["row", "col"])   # device -> host
        z_lists.append(z)
        g_lists.append(carry)
    return z_lists, g_lists


def _check_chunk_passes(ids: np.ndarray, b: int):
    K = -(-((16 * int(ids.max())).bit_length() + 1) // b)
    h_z, h_g, last = chunk_passes(ids, b, K)
    assert not last.any()
    z_lists, g_lists = gpu_chunk_passes(ids, b, K)
    for k in range(K):
        assert np.array_equal(z_lists[k], _as_entries(h_z[k])), (k, "digits")
        assert np.array_equal(g_lists[k], _as_entries(h_g[k])), (k, "carries")
    assert len(g_lists[-1]) == 0
    # the library's Recombine on the device's lists is diff2 of the full ids
    assert np.array_equal(wb.wb_diff2_recombine(z_lists, b), oracle_entries(ids))
    return sum(len(z) + len(g) for z, g in zip(z_lists, g_lists))


@pytest.mark.parametrize("b", [8, 16])
@pytest.mark.parametrize("shape,pitch,transposed", [
    ((1, 100003), 0, False), ((1, 1 << 20), 0, False), ((300, 1024), 1024, False), ((300, 1000), 4096, False),
    ((700, 1000), 4099, False), ((700, 1000), 4099, True), ((2, 70001), 70001, False), ((1000, 3), 3, False),
    ((513, 260), 260, False), ((2048, 2048), 2048, False),
    # 4 MiB and more with rows on 16-byte boundaries: the bulk-copy ring kernels
    ((1, 1 << 22), 0, False), ((1100, 4096), 4096, False), ((1100, 4096), 3 * 8192, False), ((1500, 2048), 4104, False),
    ((1500, 2048), 4099, True)])
def test_chunk_pass_matches_the_oracle_on_affine_fields(shape, pitch, transposed, b):
    """One slice-copy rectangle over the whole tensor, ids far enough up that several chunks are in play."""
    i = np.arange(shape[0], dtype=np.int64)[:, None]
    j = np.arange(shape[1], dtype=np.int64)[None, :]
    base = (1 << 33) + 98765
    ids = base + (j * pitch + i if transposed else i * max(pitch, 1) + j)
    shipped = _check_chunk_passes(ids, b)
    if shape == (1, 1 << 20):
        # a flat shard: a handful of entries per pass, where the bare 8-bit chunk carries a cluster per 256 ids
        assert shipped <= 8 * 6
        assert b != 8 or np.count_nonzero(diff2(id_chunk(ids, 0, 8))) >= (1 << 20) // 256


@pytest.mark.parametrize("b", [8, 16])
def test_chunk_pass_on_piecewise_affine_fields_with_padding(b):
    rng = np.random.default_rng(21 + b)
    for shape in [(7, 33), (257, 1023), (64, 5000)]:
        a = np.zeros(shape, np.int64)
        for _ in range(6):
            i0, j0 = rng.integers(0, shape[0]), rng.integers(0, shape[1])
            ni, nj = rng.integers(1, shape[0] - i0 + 1), rng.integers(1, shape[1] - j0 + 1)
            a[i0:i0 + ni, j0:j0 + nj] = (int(rng.integers(1, 1 << 40)) + np.arange(ni)[:, None] * int(rng.integers(1, 1 << 20))
                                         + np.arange(nj)[None, :])
        _check_chunk_passes(a, b)


@pytest.mark.parametrize("name,side", [("cfg3", "trainer"), ("cfg5", "rollout"), ("cfg2", "trainer")])
def test_chunk_passes_on_workload_tensors(name, side):
    """The largest local tensors of a configuration through 8-bit chunk passes."""
    wl = make_workload(name, "small")
    out = []

    def sink(k, t):
        t = t.reshape(1, -1) if t.dim() == 1 else t.reshape(-1, t.shape[-1])
        out.append(t.clamp_min(0).numpy())
    wl.load_side_shaped(side, lambda i: wl.ckpt_ids(i) + 1 + (1 << 30), sink)     # ids pushed up: more chunks matter
    for f in sorted(out, key=lambda f: -f.size)[:4]:
        f = np.where(f > (1 << 30), f, 0)                                          # padding stays "no source"
        _check_chunk_passes(f, 8)


# ---- the bulk-copy ring kernels (fields of 4 MiB or more whose rows start on 16-byte boundaries) ------------
def _noisy(a, rng, rows, cols, maxval):
    """Isolated entries around the seams of the ring kernels: strip edges (3968-byte pieces), the 16-byte windows
    where one warp's part of a row ends and the next begins (every 496 bytes), unit and band edges."""
    es = a.dtype.itemsize
    for byte in (0, 16, 480, 496, 512, 3952, 3968, 3984, 4096, 7936, 32768, 32784):
        for d in (-2, -1, 0, 1, 2):
            c = byte // es + d
            if 0 <= c < a.shape[1]:
                a[rng.integers(0, a.shape[0]), c] = rng.integers(1, maxval)
    for r in rows:
        if 0 <= r < a.shape[0]:
            a[r, rng.integers(0, a.shape[1])] = rng.integers(1, maxval)
    for c in cols:
        if 0 <= c < a.shape[1]:
            a[rng.integers(0, a.shape[0]), c] = rng.integers(1, maxval)
    return a


@pytest.mark.parametrize("kind,shape", [
    ("i64", (1, 3_000_000)), ("i64", (1, 600_002)), ("u16", (1, 4_000_000)), ("f32", (1, 2_000_004)),
    ("i64", (700, 1100)), ("i64", (5000, 498)), ("u16", (600, 4000)), ("u16", (2100, 1984 + 8)), ("bf16", (1200, 2048)),
    ("f32", (900, 1500)), ("f32", (4100, 512))])
def test_ring_kernels_match_the_definition(kind, shape):
    rng = np.random.default_rng(sum(map(ord, kind)) * 1000003 + shape[0] * 7919 + shape[1])
    maxval = {"i64": 1 << 40, "u16": 1 << 16, "bf16": 256, "f32": 1 << 24}[kind]
    a = np.zeros(shape, np.int64)
    for _ in range(6):                                   # a few affine rectangles
        i0, j0 = rng.integers(0, shape[0]), rng.integers(0, shape[1])
        ni, nj = rng.integers(1, shape[0] - i0 + 1), rng.integers(1, shape[1] - j0 + 1)
        base = int(rng.integers(1, maxval // 4))
        pitch = int(rng.integers(1, max(2, maxval // (4 * max(ni, 1) * 2)))) if shape[0] > 1 else 0
        a[i0:i0 + ni, j0:j0 + nj] = (base + np.arange(ni)[:, None] * pitch + np.arange(nj)[None, :]) % maxval
    _noisy(a, rng, rows=(0, 1, 2, 7, 8, 9, 63, 64, 65, 66, shape[0] - 1), cols=(0, 1, shape[1] - 2, shape[1] - 1), maxval=maxval)
    want = oracle_entries(a)
    if kind == "i64":
        t, k = torch.from_numpy(a), wb.WB_ID_I64
    elif kind == "u16":
        t, k = torch.from_numpy(a.astype(np.uint16).view(np.int16)), wb.WB_ID_U16
    elif kind == "bf16":
        t, k = torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16), wb.WB_ID_BF16
    else:
        t, k = torch.from_numpy(a.astype(np.float32)), wb.WB_ID_F32
    assert t.numel() * t.element_size() >= 4 << 20 and (shape[1] * t.element_size()) % 16 == 0
    got, n = gpu_entries(t.to(DEV), k, cap=1 << 18)
    assert n == len(want) and np.array_equal(got, want)
