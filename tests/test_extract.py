"""Source-map extraction (Section 3.1, Appendix B): pins for the diff2 oracle, and the host
scanner / recombiner of the library checked against the id probe on every small workload."""
import numpy as np
import pytest
import torch

from helpers import ckpt_shapes, predict_ids, scatter_checkpoint, to_bits
from oracle import remap_oracle
from oracle.extract import diff1, diff2, id_chunk, nonzeros, recombine, undo_diff2
from paper_2609_25442_b200 import binding as wb
from plan_interp import run_table
from wb_workloads import WB_BF16, Layout, make_workload

SMALL = [("cfg1b", "full"), ("cfg1c", "full"), ("cfg2", "small"), ("cfg3", "small"), ("cfg4", "small"),
         ("cfg5", "small")]


def entries(d):
    nz = nonzeros(d)
    return np.array(nz, dtype=wb.DIFF2_ENTRY_DTYPE) if nz else np.zeros(0, wb.DIFF2_ENTRY_DTYPE)


def id_fields(wl, side):
    """2-D id field of every local tensor: ids are 1-based, 0 where nothing was loaded."""
    layout = wl.trainer if side == "trainer" else wl.rollout
    out = [None] * layout.n_tensors

    def sink(k, t):
        t = t.reshape(1, -1) if t.dim() == 1 else t.reshape(-1, t.shape[-1])
        out[k] = t.clamp_min(0).numpy()          # the loaders pad integer tensors with -1
    wl.load_side_shaped(side, lambda i: wl.ckpt_ids(i) + 1, sink)
    return out


# ---- the oracle's diff2 against what the paper and mathematics fix ------------------------------------
def test_diff2_is_the_3x3_kernel_of_the_paper():
    from scipy.signal import convolve2d
    rng = np.random.default_rng(0)
    a = rng.integers(0, 1 << 30, size=(37, 53)).astype(np.int64)
    k = np.outer([1, -2, 1], [1, -2, 1])                 # Appendix B: outer product of [1,-2,1] with itself
    want = convolve2d(a, k, mode="full")[:37, :53]        # causal, zeros outside
    assert np.array_equal(diff2(a), want)


def test_diff2_is_lossless():
    rng = np.random.default_rng(1)
    a = rng.integers(0, 1 << 40, size=(29, 31)).astype(np.int64)
    assert np.array_equal(undo_diff2(diff2(a)), a)
    assert np.array_equal(np.cumsum(np.cumsum(diff1(a), 0), 1), a)


@pytest.mark.parametrize("transposed", [False, True])
def test_affine_rectangle_leaves_at_most_16_entries_at_its_corners(transposed):
    rng = np.random.default_rng(2)
    for _ in range(50):
        R, C = 40, 50
        i0, j0 = rng.integers(0, 20, 2)
        ni, nj = rng.integers(1, 18, 2)
        base, pitch = int(rng.integers(1, 1 << 33)), int(rng.integers(20, 5000))
        a = np.zeros((R, C), np.int64)
        ii, jj = np.meshgrid(np.arange(ni), np.arange(nj), indexing="ij")
        a[i0:i0 + ni, j0:j0 + nj] = base + (jj * pitch + ii if transposed else ii * pitch + jj)
        nz = nonzeros(diff2(a))
        assert len(nz) <= 16
        for (i, j, _) in nz:                                # 2x2 neighbourhoods of the four corners
            assert i in (i0, i0 + 1, i0 + ni, i0 + ni + 1) and j in (j0, j0 + 1, j0 + nj, j0 + nj + 1)
        assert nz[0] == (i0, j0, base)                      # the first entry is the first id


@pytest.mark.parametrize("b", [8, 16])
def test_chunk_diffs_recombine_to_the_full_diff(b):
    wl = make_workload("cfg3", "small")
    field = id_fields(wl, "trainer")[5]
    K = -(-int(wl.ckpt_numel() + 1).bit_length() // b)
    parts = [diff2(id_chunk(field, k, b)) for k in range(K)]
    assert np.array_equal(recombine(parts, b), diff2(field))
    got = wb.wb_diff2_recombine([entries(p) for p in parts], b)     # the library's Recombine
    assert np.array_equal(got, entries(diff2(field)))
    assert sum(len(entries(p)) for p in parts) > len(got)           # the chunks alone carry wrap artifacts


# ---- the library's ScanSliceMappings ---------------------------------------------------------------------
def extract_layout(wl, side, fields):
    declared = wl.trainer if side == "trainer" else wl.rollout
    base = wl.ckpt_base().astype(np.uint64)
    rows = np.array([c.rows for c in wl.ckpt], np.uint64)
    cols = np.array([c.cols for c in wl.ckpt], np.uint64)
    lay = Layout(side)
    n_entries = 0
    for k, f in enumerate(fields):
        d = declared.tensors[k]
        lay.add_tensor(declared.names[k], int(d["rank"]), int(d["dtype"]), int(d["numel"]))
        e = entries(diff2(f))
        n_entries += len(e)
        for s in wb.wb_scan_slices(e, f.shape[0], f.shape[1], base, rows, cols, k):
            lay.add_slice(int(s["tensor"]), int(s["local_off"]), int(s["stride_r"]), int(s["stride_c"]),
                          int(s["ckpt"]), int(s["ckpt_rows"]), int(s["ckpt_cols"]),
                          int(s["r0"]), int(s["c0"]), int(s["nr"]), int(s["nc"]))
    return lay.freeze(), n_entries


@pytest.mark.parametrize("name,scale", SMALL)
@pytest.mark.parametrize("side", ["trainer", "rollout"])
def test_scanned_source_map_reproduces_the_id_field(name, scale, side):
    wl = make_workload(name, scale)
    fields = id_fields(wl, side)
    lay, n_entries = extract_layout(wl, side, fields)
    for k, (p, f) in enumerate(zip(predict_ids(lay, wl), fields)):
        assert np.array_equal(p + 1, f.reshape(-1)), lay.names[k]      # 0 stays "no source"
    declared = wl.trainer if side == "trainer" else wl.rollout
    assert n_entries <= 16 * max(len(lay.slices), len(declared.slices))   # O(number of operations)


def test_extracted_source_maps_drive_the_same_transfer():
    wl = make_workload("cfg1b")
    tl, _ = extract_layout(wl, "trainer", id_fields(wl, "trainer"))
    rl, _ = extract_layout(wl, "rollout", id_fields(wl, "rollout"))
    src = [to_bits(t) for t in wl.trainer_weights()]
    want = remap_oracle(ckpt_shapes(wl), wl.trainer.tensors, wl.trainer.slices, wl.rollout.tensors,
                        wl.rollout.slices, src)
    plan = wb.Plan(wb.Layout(tl.tensors, tl.slices), wb.Layout(rl.tensors, rl.slices))
    plan.verify()
    dst = [np.zeros(int(t["numel"]), np.uint16) for t in rl.tensors]
    run_table(plan.tiles(wb.WB_TABLE_REMAP), src, dst, None, wl.src_dtype, wl.dst_dtype)
    for a, b in zip(dst, want.dst):
        assert np.array_equal(a, b)
    assert plan.stats()["src_elems_read"] == wl.ckpt_numel()


def test_scan_rejects_fields_no_slice_copy_produces():
    base = np.array([0, 64], np.uint64)
    one = np.array([8], np.uint64)
    a = np.outer(np.arange(1, 9), np.arange(1, 9)).astype(np.int64)      # bilinear, not affine
    with pytest.raises(wb.WbError):
        wb.wb_scan_slices(entries(diff2(a)), 8, 8, base, one, one, 0)
    far = np.array([(9, 0, 5)], wb.DIFF2_ENTRY_DTYPE)
    with pytest.raises(wb.WbError) as e:
        wb.wb_scan_slices(far, 8, 8, base, one, one, 0)
    assert e.value.name == "WB_ERR_OUT_OF_RANGE"


def test_diff2_kernel_entry_point_checks_its_arguments_on_the_host():
    """Size limits are refused before anything is launched (no GPU needed to see them)."""
    lib = wb.load()
    import ctypes as C
    lib.wb_diff2_nonzeros.argtypes = [C.c_void_p, C.c_uint32, C.c_uint64, C.c_uint64, C.c_void_p, C.c_uint64,
                                      C.c_void_p, C.c_void_p]
    dummy = C.c_uint64(0)
    p = C.addressof(dummy)
    INVALID = 1
    assert lib.wb_diff2_nonzeros(None, 0, 4, 4, p, 1, p, None) == INVALID
    assert lib.wb_diff2_nonzeros(p, 9, 4, 4, p, 1, p, None) == INVALID              # unknown field kind
    assert lib.wb_diff2_nonzeros(p, 0, 1 << 31, 2, p, 1, p, None) == INVALID        # several rows: < 2^31 rows
    assert lib.wb_diff2_nonzeros(p, 0, 2, 1 << 31, p, 1, p, None) == INVALID
    assert lib.wb_diff2_nonzeros(p, 0, 1, (1 << 48) + 1, p, 1, p, None) == INVALID
    assert lib.wb_diff2_nonzeros(p, 0, 0, 4, p, 1, p, None) == 0                    # empty field: nothing to do


def test_batched_diff2_entry_point_checks_its_arguments_on_the_host():
    fields = np.zeros(2, wb.DIFF2_FIELD_DTYPE)
    fields["field"] = 4096
    fields["rows"], fields["cols"] = 4, 4
    assert wb.wb_diff2_batch_scratch_bytes(2) >= 2 * 32
    with pytest.raises(wb.WbError):                              # scratch too small
        wb.wb_diff2_nonzeros_batch(fields, 4096, 8, 4096, 1, 4096)
    with pytest.raises(wb.WbError):                              # scratch not 16-byte aligned
        wb.wb_diff2_nonzeros_batch(fields, 4100, 1024, 4096, 1, 4096)
    bad = fields.copy()
    bad["id_kind"][1] = 7
    with pytest.raises(wb.WbError):                              # unknown field kind
        wb.wb_diff2_nonzeros_batch(bad, 4096, 1024, 4096, 1, 4096)
    empty = fields.copy()
    empty["rows"] = 0
    wb.wb_diff2_nonzeros_batch(empty, 4096, 1024, 4096, 1, 4096)   # only empty fields: nothing is launched
    wb.wb_diff2_nonzeros_batch(fields[:0], 0, 0, 4096, 1, 4096)    # no fields at all


# ---- Algorithm 1's chunk passes with carries (the oracle's reading, pinned to diff2 of the full ids) -------
from oracle.extract import carry_stride, chunk_passes, emit_carry, expand_carry, strided_diff1


def _balanced_digits(v: int, b: int, n: int):
    """Digits d_k in [-2^(b-1), 2^(b-1)) with v = sum d_k 2^(bk), in Python integers."""
    out = []
    for _ in range(n):
        d = ((v + (1 << (b - 1))) % (1 << b)) - (1 << (b - 1))
        out.append(d)
        v = (v - d) >> b
    assert v == 0
    return out


def test_strided_diff1_is_lossless_and_is_diff1_at_stride_one():
    rng = np.random.default_rng(4)
    for shape in [(1, 1000), (37, 53), (300, 7), (5, 700)]:
        c = rng.integers(-17, 18, size=shape)
        assert np.array_equal(strided_diff1(c, 1)[:, 1:], diff1(c)[:, 1:])      # away from the left edge, where the
        for s in (1, 2, 3, 16, 256, 65536):                                     # flat order wraps into the row above
            g = strided_diff1(c, s)
            assert np.array_equal(expand_carry(g, s), c)
        # written out for one element: left neighbour s back in flat order, upper neighbour s rows up
        if shape == (37, 53):
            g, s, f = strided_diff1(c, 3), 3, c.reshape(-1)
            x = 20 * 53 + 1
            assert g.reshape(-1)[x] == f[x] - f[x - s] - f[x - s * 53] + f[x - s - s * 53]
            assert g.reshape(-1)[2] == f[2] and g.reshape(-1)[5] == f[5] - f[2]


def test_emit_carry_splits_into_a_balanced_digit_and_a_carry():
    d = np.array([[0, 1, -1, 127, 128, -128, -129, 255, 256, -256, 4096 * 3 + 5, -(1 << 40) - 3]], np.int64)
    z, c = emit_carry(d, 8)
    assert np.array_equal(z + (c << 8), d) and z.min() >= -128 and z.max() <= 127
    assert z.tolist()[0][:10] == [0, 1, -1, 127, -128, -128, 127, -1, 0, 0]
    assert c.tolist()[0][:10] == [0, 0, 0, 0, 1, 0, -1, 1, 1, -1]


@pytest.mark.parametrize("b", [8, 16])
@pytest.mark.parametrize("name,side,pick", [("cfg3", "trainer", 5), ("cfg5", "rollout", None), ("cfg1b", "trainer", None)])
def test_chunk_passes_give_the_balanced_digits_of_the_full_diff(name, side, pick, b):
    """Algorithm 1 with carries: Recombine(H_Z) = diff2(full ids), the field comes back by two prefix sums,
    every Z_k holds exactly the k-th balanced digit of diff2(ids) - so it is as sparse as diff2(ids) - and
    the carry out of the last pass is zero."""
    wl = make_workload(name, "small" if name != "cfg1b" else "full")
    fields = id_fields(wl, side)
    fields = [fields[pick]] if pick is not None else sorted(fields, key=lambda f: -f.size)[:6]
    bits = (16 * (wl.ckpt_numel() + 1)).bit_length() + 1
    K = -(-bits // b)
    for f in fields:
        h_z, h_g, last = chunk_passes(f, b, K)
        full = diff2(f)
        assert np.array_equal(recombine(h_z, b), full)
        assert np.array_equal(undo_diff2(recombine(h_z, b)), f)
        assert not last.any()
        for (i, j) in zip(*np.nonzero(full)):
            assert [int(z[i, j]) for z in h_z] == _balanced_digits(int(full[i, j]), b, K)
        assert all(not z[full == 0].any() for z in h_z)
        # the library's Recombine takes the same lists
        got = wb.wb_diff2_recombine([entries(z) for z in h_z], b)
        assert np.array_equal(got, entries(full))


def test_entries_shipped_per_pass_stay_bounded_where_plain_chunk_diffs_do_not():
    """A field of 2^24 ids as one flat shard and as a 4096 x 4096 tensor filled by two slice copies: every
    pass ships a handful of entries (digits + strided carry differences), while diff2 of a bare 8-bit
    chunk carries one cluster of wrap artifacts per 256 consecutive ids."""
    n = 1 << 24
    flat = (np.arange(n, dtype=np.int64) + 1 + 12345).reshape(1, n)
    two = flat.reshape(4096, 4096).copy()
    two[2048:, :] += 7 * 4096 * 4096 + 999 * 4096                  # a second checkpoint tensor further on
    for field, n_ops in ((flat, 1), (two, 2)):
        K = -(-((16 * int(field.max())).bit_length() + 1) // 8)
        h_z, h_g, last = chunk_passes(field, 8, K)
        assert np.array_equal(recombine(h_z, 8), diff2(field)) and not last.any()
        for k in range(K):
            shipped = np.count_nonzero(h_z[k]) + np.count_nonzero(h_g[k])
            assert shipped <= 32 * n_ops, (k, shipped)
        if field.shape[0] == 1:                   # (rows 4096 ids apart repeat their wrap pattern: those cancel vertically)
            assert np.count_nonzero(diff2(id_chunk(field, 0, 8))) >= n // 256


def test_chunk_pass_entry_point_checks_its_arguments_on_the_host():
    """Bad arguments are refused before anything is launched (no GPU needed to see them)."""
    nb = wb.wb_diff2_chunk_scratch_bytes(4, 4)
    assert nb >= 16 + (1 << 18)
    ok = dict(field_ptr=4096, id_kind=wb.WB_ID_U16, rows=4, cols=4, chunk_bits=8, pass_index=0, carry_in_ptr=0, n_carry_in=0,
              scratch_ptr=8192, scratch_bytes=nb, z_out_ptr=4096, z_cap=1, z_count_ptr=4096, carry_out_ptr=4096, carry_cap=1,
              carry_count_ptr=4096)
    for bad in (dict(field_ptr=0), dict(id_kind=9), dict(chunk_bits=12), dict(pass_index=8), dict(scratch_ptr=8200),
                dict(scratch_bytes=nb - 1), dict(n_carry_in=3), dict(pass_index=1, n_carry_in=3), dict(z_count_ptr=0),
                dict(rows=1 << 31, cols=2)):
        with pytest.raises(wb.WbError) as e:
            wb.wb_diff2_chunk_pass(**{**ok, **bad})
        assert e.value.name == "WB_ERR_INVALID_ARG", bad
    wb.wb_diff2_chunk_pass(**{**ok, "rows": 0})          # an empty field: nothing to do
