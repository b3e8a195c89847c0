"""Thin ctypes binding of the C ABI in include/wb.h.

Argument marshalling only: every step of the remap runs inside libwb.so.  Function and
type names mirror the header.  There is no fallback: if the library cannot be built or
loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

WB_OK = 0
WB_F32, WB_BF16 = 0, 1
WB_TABLE_REMAP, WB_TABLE_PACK, WB_TABLE_UNPACK = 0, 1, 2
WB_TILE_FANOUT_CONT = 1
WB_PLAN_NO_REPLICA_SPLIT = 1
WB_PLAN_STATIC_SCHEDULE = 2
WB_PLAN_NO_TENSOR_MAPS = 4
WB_TILE_ROWS_BEFORE, WB_TILE_ROWS_AFTER = 2, 4

STATUS_NAMES = {
    0: "WB_OK", 1: "WB_ERR_INVALID_ARG", 2: "WB_ERR_DTYPE", 3: "WB_ERR_SHAPE_MISMATCH",
    4: "WB_ERR_OUT_OF_RANGE", 5: "WB_ERR_DST_OVERLAP", 6: "WB_ERR_UNCOVERED",
    7: "WB_ERR_BUCKET_TOO_SMALL", 8: "WB_ERR_OOM", 9: "WB_ERR_CUDA", 10: "WB_ERR_NOT_BOUND",
    11: "WB_ERR_INTERNAL", 12: "WB_ERR_STATIC_LIMIT", 13: "WB_ERR_REPLICA_MISMATCH",
}


class WbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        self.name = STATUS_NAMES.get(status, str(status))
        msg = _lib.wb_status_str(status).decode() if _lib is not None else ""
        super().__init__(f"{where}: {self.name} ({msg})")


class wb_tensor_desc(C.Structure):
    _fields_ = [("rank", C.c_uint32), ("dtype", C.c_uint32), ("numel", C.c_uint64)]


class wb_slice(C.Structure):
    _fields_ = [("tensor", C.c_uint32), ("reserved", C.c_uint32), ("local_off", C.c_uint64),
                ("stride_r", C.c_int64), ("stride_c", C.c_int64),
                ("ckpt_tensor", C.c_uint64), ("ckpt_rows", C.c_uint64), ("ckpt_cols", C.c_uint64),
                ("r0", C.c_uint64), ("c0", C.c_uint64), ("nr", C.c_uint64), ("nc", C.c_uint64)]


class wb_plan_opts(C.Structure):
    _fields_ = [("bucket_budget_bytes", C.c_uint64), ("tile_bytes", C.c_uint32),
                ("grid_ctas", C.c_uint32), ("flags", C.c_uint32), ("host_group_kib", C.c_uint32)]


class wb_plan_stats_t(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "n_ckpt_tensors", "n_slabs", "n_fanout_slabs", "n_rounds", "n_tiles_remap", "n_tiles_pack",
        "n_tiles_unpack", "src_elems_read", "dst_elems_written", "src_bytes_read",
        "dst_bytes_written", "replica_elems_skipped", "bucket_bytes_total", "bucket_bytes_max",
        "table_bytes", "remap_cta_bytes_max", "remap_cta_bytes_mean")] + \
        [("grid_ctas", C.c_uint32), ("tile_bytes", C.c_uint32), ("build_seconds", C.c_double)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


BUCKET_ENTRY_DTYPE = np.dtype([
    ("sender", "<u4"), ("receiver", "<u4"), ("ckpt_tensor", "<u8"), ("r0", "<u8"), ("c0", "<u8"),
    ("nr", "<u8"), ("nc", "<u8"), ("bucket_off", "<u8"), ("dtype", "<u4"), ("n_dst", "<u4")])
TILE_VIEW_DTYPE = np.dtype([
    ("src_tensor", "<i4"), ("dst_tensor", "<i4"), ("src_off", "<u8"), ("dst_off", "<u8"),
    ("nr", "<u4"), ("nc", "<u4"), ("src_sr", "<u4"), ("src_sc", "<u4"), ("dst_sr", "<u4"),
    ("dst_sc", "<u4"), ("kind", "<u4"), ("flags", "<u4"), ("cta", "<u4"), ("reserved", "<u4")])
BUCKET_REGION_DTYPE = np.dtype([("receiver", "<u4"), ("sender", "<u4"), ("off", "<u8"), ("bytes", "<u8")])
assert BUCKET_ENTRY_DTYPE.itemsize == 64 and TILE_VIEW_DTYPE.itemsize == 64 and BUCKET_REGION_DTYPE.itemsize == 24

EXPORTS = [
    "wb_layout_describe", "wb_layout_free", "wb_layout_add_flat_range", "wb_plan_build", "wb_plan_free", "wb_plan_verify",
    "wb_plan_stats", "wb_plan_rank_bytes", "wb_plan_num_rounds", "wb_plan_bucket_bytes",
    "wb_plan_bucket_entries", "wb_plan_bucket_regions", "wb_plan_num_ranks", "wb_pack_ranks", "wb_unpack_ranks", "wb_plan_rank_tiles",
    "wb_plan_tiles", "wb_plan_bind", "wb_remap", "wb_pack", "wb_unpack",
    "wb_remap_host", "wb_remap_static", "wb_plan_check", "wb_transfer_rounds",
    "wb_plan_num_ckpts", "wb_plan_ckpt_ids", "wb_plan_qbucket_bytes", "wb_absmax", "wb_bucket_quantize",
    "wb_bucket_dequantize", "wb_transfer_rounds_fp8", "wb_pack_fp8", "wb_unpack_fp8", "wb_transfer_rounds_fp8_fused",
    "wb_diff2_nonzeros", "wb_diff2_nonzeros_batch", "wb_diff2_batch_scratch_bytes", "wb_diff2_recombine", "wb_diff2_chunk_pass", "wb_diff2_chunk_scratch_bytes", "wb_scan_slices", "wb_route_account", "wb_wait_probe", "wb_plan_check_replicas", "wb_launches_per_call", "wb_status_str", "wb_version",
]

_lib: Optional[C.CDLL] = None


def lib_path() -> str:
    return _build.LIB


def load() -> C.CDLL:
    """Build (if stale) and load libwb.so; raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    lib = C.CDLL(path)
    vp, sz = C.c_void_p, C.c_size_t
    lib.wb_layout_describe.argtypes = [vp, sz, vp, sz, C.POINTER(vp)]
    lib.wb_layout_free.argtypes = [vp]
    lib.wb_layout_free.restype = None
    lib.wb_layout_add_flat_range.argtypes = [C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint64,
                                             C.c_uint64, vp, sz, C.POINTER(sz)]
    lib.wb_plan_build.argtypes = [vp, vp, C.POINTER(wb_plan_opts), C.POINTER(vp)]
    lib.wb_plan_free.argtypes = [vp]
    lib.wb_plan_free.restype = None
    lib.wb_plan_verify.argtypes = [vp]
    lib.wb_plan_stats.argtypes = [vp, C.POINTER(wb_plan_stats_t)]
    lib.wb_plan_rank_bytes.argtypes = [vp, C.c_int, C.c_uint32, C.POINTER(C.c_uint64)]
    lib.wb_plan_num_rounds.argtypes = [vp]
    lib.wb_plan_num_rounds.restype = sz
    lib.wb_plan_bucket_bytes.argtypes = [vp, sz]
    lib.wb_plan_bucket_bytes.restype = sz
    lib.wb_plan_bucket_entries.argtypes = [vp, sz, vp, sz, C.POINTER(sz)]
    lib.wb_plan_tiles.argtypes = [vp, C.c_int, sz, vp, sz, C.POINTER(sz)]
    lib.wb_plan_bucket_regions.argtypes = [vp, sz, vp, sz, C.POINTER(sz)]
    lib.wb_plan_num_ranks.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
    lib.wb_plan_rank_tiles.argtypes = [vp, C.c_int, sz, C.c_uint32, C.POINTER(sz), C.POINTER(sz)]
    lib.wb_pack_ranks.argtypes = [vp, sz, vp, sz, vp, vp]
    lib.wb_unpack_ranks.argtypes = [vp, sz, vp, sz, vp, vp]
    lib.wb_plan_bind.argtypes = [vp, vp, sz, vp, sz]
    lib.wb_remap.argtypes = [vp, vp]
    lib.wb_pack.argtypes = [vp, sz, vp, vp]
    lib.wb_unpack.argtypes = [vp, sz, vp, vp]
    lib.wb_remap_host.argtypes = [vp, vp, sz, vp, sz, vp]
    lib.wb_transfer_rounds.argtypes = [vp, vp, vp, C.c_uint32, vp]
    lib.wb_plan_num_ckpts.argtypes = [vp]
    lib.wb_plan_num_ckpts.restype = sz
    lib.wb_plan_ckpt_ids.argtypes = [vp, vp, sz]
    lib.wb_plan_qbucket_bytes.argtypes = [vp, sz]
    lib.wb_plan_qbucket_bytes.restype = sz
    lib.wb_absmax.argtypes = [vp, vp, vp]
    lib.wb_bucket_quantize.argtypes = [vp, sz, vp, vp, vp, vp]
    lib.wb_bucket_dequantize.argtypes = [vp, sz, vp, vp, vp, vp]
    lib.wb_transfer_rounds_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.wb_pack_fp8.argtypes = [vp, sz, vp, vp, vp]
    lib.wb_unpack_fp8.argtypes = [vp, sz, vp, vp, vp]
    lib.wb_transfer_rounds_fp8_fused.argtypes = [vp, vp, vp, vp, vp]
    lib.wb_remap_static.argtypes = [vp, vp, sz, vp, sz, C.c_uint32, vp]
    lib.wb_plan_check.argtypes = [vp]
    lib.wb_wait_probe.argtypes = [C.c_uint32, vp]
    lib.wb_plan_check_replicas.argtypes = [vp, C.POINTER(C.c_uint64), vp]
    lib.wb_route_account.argtypes = [vp, vp, sz, vp, sz, C.c_double, C.c_double, vp, vp, vp, sz]
    lib.wb_diff2_nonzeros.argtypes = [vp, C.c_uint32, C.c_uint64, C.c_uint64, vp, C.c_uint64, vp, vp]
    lib.wb_diff2_recombine.argtypes = [vp, vp, sz, C.c_uint32, vp, sz, C.POINTER(sz)]
    lib.wb_scan_slices.argtypes = [vp, sz, C.c_uint64, C.c_uint64, vp, vp, vp, sz, C.c_uint32, C.c_uint64,
                                   vp, sz, C.POINTER(sz)]
    lib.wb_launches_per_call.restype = C.c_int
    lib.wb_status_str.argtypes = [C.c_int]
    lib.wb_status_str.restype = C.c_char_p
    lib.wb_version.restype = C.c_char_p
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != WB_OK:
        raise WbError(status, where)


def _ptr_array(ptrs: Sequence[int]):
    arr = (C.c_void_p * max(len(ptrs), 1))()
    for i, p in enumerate(ptrs):
        arr[i] = p
    return arr


class Layout:
    """Owns a wb_layout*."""

    def __init__(self, tensors: np.ndarray, slices: np.ndarray):
        lib = load()
        tensors = np.ascontiguousarray(tensors)
        slices = np.ascontiguousarray(slices)
        assert tensors.dtype.itemsize == C.sizeof(wb_tensor_desc)
        assert slices.dtype.itemsize == C.sizeof(wb_slice)
        self.n_tensors = len(tensors)
        self.handle = C.c_void_p()
        _check(lib.wb_layout_describe(tensors.ctypes.data, len(tensors), slices.ctypes.data,
                                      len(slices), C.byref(self.handle)), "wb_layout_describe")

    def __del__(self):
        if _lib is not None and getattr(self, "handle", None):
            _lib.wb_layout_free(self.handle)
            self.handle = None


def wb_layout_describe(tensors: np.ndarray, slices: np.ndarray) -> Layout:
    return Layout(tensors, slices)


def wb_layout_add_flat_range(tensor: int, local_off: int, ckpt_tensor: int, ckpt_rows: int, ckpt_cols: int,
                             begin: int, end: int) -> np.ndarray:
    """The <= 3 slice records of flat checkpoint range [begin, end) held contiguously from local_off on."""
    lib = load()
    out = np.zeros(3, SLICE_DTYPE)
    n = C.c_size_t()
    _check(lib.wb_layout_add_flat_range(tensor, local_off, ckpt_tensor, ckpt_rows, ckpt_cols, begin, end,
                                        out.ctypes.data, 3, C.byref(n)), "wb_layout_add_flat_range")
    return out[:n.value]


class Plan:
    """Owns a wb_plan*."""

    def __init__(self, trainer: Layout, rollout: Layout, bucket_budget_bytes: int = 0,
                 tile_bytes: int = 0, grid_ctas: int = 0, flags: int = 0, host_group_kib: int = 0):
        lib = load()
        opts = wb_plan_opts(bucket_budget_bytes, tile_bytes, grid_ctas, flags, host_group_kib)
        self.handle = C.c_void_p()
        self.n_src, self.n_dst = trainer.n_tensors, rollout.n_tensors
        _check(lib.wb_plan_build(trainer.handle, rollout.handle, C.byref(opts), C.byref(self.handle)),
               "wb_plan_build")

    def __del__(self):
        if _lib is not None and getattr(self, "handle", None):
            _lib.wb_plan_free(self.handle)
            self.handle = None

    # ---- host queries ---------------------------------------------------------------------
    def verify(self) -> None:
        _check(_lib.wb_plan_verify(self.handle), "wb_plan_verify")

    def stats(self) -> dict:
        st = wb_plan_stats_t()
        _check(_lib.wb_plan_stats(self.handle, C.byref(st)), "wb_plan_stats")
        return st.as_dict()

    def rank_bytes(self, side: int, rank: int) -> int:
        out = C.c_uint64()
        _check(_lib.wb_plan_rank_bytes(self.handle, side, rank, C.byref(out)), "wb_plan_rank_bytes")
        return out.value

    def num_rounds(self) -> int:
        return _lib.wb_plan_num_rounds(self.handle)

    def bucket_bytes(self, rnd: int) -> int:
        return _lib.wb_plan_bucket_bytes(self.handle, rnd)

    def bucket_entries(self, rnd: int) -> np.ndarray:
        n = C.c_size_t()
        _check(_lib.wb_plan_bucket_entries(self.handle, rnd, None, 0, C.byref(n)), "wb_plan_bucket_entries")
        out = np.zeros(n.value, BUCKET_ENTRY_DTYPE)
        _check(_lib.wb_plan_bucket_entries(self.handle, rnd, out.ctypes.data, n.value, C.byref(n)),
               "wb_plan_bucket_entries")
        return out

    def bucket_regions(self, rnd: int) -> np.ndarray:
        n = C.c_size_t()
        _check(_lib.wb_plan_bucket_regions(self.handle, rnd, None, 0, C.byref(n)), "wb_plan_bucket_regions")
        out = np.zeros(n.value, BUCKET_REGION_DTYPE)
        _check(_lib.wb_plan_bucket_regions(self.handle, rnd, out.ctypes.data, n.value, C.byref(n)),
               "wb_plan_bucket_regions")
        return out

    def num_ranks(self):
        a, b = C.c_uint32(), C.c_uint32()
        _check(_lib.wb_plan_num_ranks(self.handle, C.byref(a), C.byref(b)), "wb_plan_num_ranks")
        return a.value, b.value

    def rank_tiles(self, which: int, rnd: int, rank: int) -> np.ndarray:
        """The tile views of one virtual rank in a round's pack / unpack table."""
        a, n = C.c_size_t(), C.c_size_t()
        _check(_lib.wb_plan_rank_tiles(self.handle, which, rnd, rank, C.byref(a), C.byref(n)), "wb_plan_rank_tiles")
        return self.tiles(which, rnd)[a.value:a.value + n.value]

    def tiles(self, which: int, rnd: int = 0) -> np.ndarray:
        n = C.c_size_t()
        _check(_lib.wb_plan_tiles(self.handle, which, rnd, None, 0, C.byref(n)), "wb_plan_tiles")
        out = np.zeros(n.value, TILE_VIEW_DTYPE)
        _check(_lib.wb_plan_tiles(self.handle, which, rnd, out.ctypes.data, n.value, C.byref(n)),
               "wb_plan_tiles")
        return out

    # ---- device ------------------------------------------------------------------------------
    def bind(self, src_ptrs: Sequence[int], dst_ptrs: Sequence[int]) -> None:
        a, b = _ptr_array(src_ptrs), _ptr_array(dst_ptrs)
        _check(_lib.wb_plan_bind(self.handle, a, len(src_ptrs), b, len(dst_ptrs)), "wb_plan_bind")

    def check(self) -> None:
        _check(_lib.wb_plan_check(self.handle), "wb_plan_check")

    def check_replicas(self, stream: int = 0) -> int:
        """Number of elements in which trainer replicas differ (0 = consistent)."""
        n = C.c_uint64()
        st = _lib.wb_plan_check_replicas(self.handle, C.byref(n), stream)
        if st not in (WB_OK, 13):
            raise WbError(st, "wb_plan_check_replicas")
        return n.value

    def remap(self, stream: int = 0) -> None:
        _check(_lib.wb_remap(self.handle, stream), "wb_remap")

    def pack(self, rnd: int, bucket_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_pack(self.handle, rnd, bucket_ptr, stream), "wb_pack")

    def unpack(self, rnd: int, bucket_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_unpack(self.handle, rnd, bucket_ptr, stream), "wb_unpack")

    def pack_ranks(self, rnd: int, ranks: Sequence[int], bucket_ptr: int, stream: int = 0) -> None:
        r = np.ascontiguousarray(ranks, dtype=np.uint32)
        _check(_lib.wb_pack_ranks(self.handle, rnd, r.ctypes.data, len(r), bucket_ptr, stream), "wb_pack_ranks")

    def unpack_ranks(self, rnd: int, ranks: Sequence[int], bucket_ptr: int, stream: int = 0) -> None:
        r = np.ascontiguousarray(ranks, dtype=np.uint32)
        _check(_lib.wb_unpack_ranks(self.handle, rnd, r.ctypes.data, len(r), bucket_ptr, stream), "wb_unpack_ranks")

    def transfer_rounds(self, bucket0_ptr: int, bucket1_ptr: int, flags: int = 0, stream: int = 0) -> None:
        _check(_lib.wb_transfer_rounds(self.handle, bucket0_ptr, bucket1_ptr, flags, stream), "wb_transfer_rounds")

    # ---- FP8 quantisation of buckets ----------------------------------------------------------
    def num_ckpts(self) -> int:
        return int(_lib.wb_plan_num_ckpts(self.handle))

    def ckpt_ids(self) -> np.ndarray:
        out = np.zeros(self.num_ckpts(), np.uint64)
        _check(_lib.wb_plan_ckpt_ids(self.handle, out.ctypes.data, out.size), "wb_plan_ckpt_ids")
        return out

    def qbucket_bytes(self, rnd: int) -> int:
        return int(_lib.wb_plan_qbucket_bytes(self.handle, rnd))

    def absmax(self, amax_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_absmax(self.handle, amax_ptr, stream), "wb_absmax")

    def bucket_quantize(self, rnd: int, bucket_ptr: int, qbucket_ptr: int, amax_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_bucket_quantize(self.handle, rnd, bucket_ptr, qbucket_ptr, amax_ptr, stream),
               "wb_bucket_quantize")

    def bucket_dequantize(self, rnd: int, qbucket_ptr: int, bucket_ptr: int, amax_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_bucket_dequantize(self.handle, rnd, qbucket_ptr, bucket_ptr, amax_ptr, stream),
               "wb_bucket_dequantize")

    def transfer_rounds_fp8(self, bucket0: int, bucket1: int, qbucket0: int, qbucket1: int, amax_ptr: int,
                            stream: int = 0) -> None:
        _check(_lib.wb_transfer_rounds_fp8(self.handle, bucket0, bucket1, qbucket0, qbucket1, amax_ptr, stream),
               "wb_transfer_rounds_fp8")

    def pack_fp8(self, rnd: int, qbucket_ptr: int, amax_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_pack_fp8(self.handle, rnd, qbucket_ptr, amax_ptr, stream), "wb_pack_fp8")

    def unpack_fp8(self, rnd: int, qbucket_ptr: int, amax_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_unpack_fp8(self.handle, rnd, qbucket_ptr, amax_ptr, stream), "wb_unpack_fp8")

    def transfer_rounds_fp8_fused(self, qbucket0: int, qbucket1: int, amax_ptr: int, stream: int = 0) -> None:
        _check(_lib.wb_transfer_rounds_fp8_fused(self.handle, qbucket0, qbucket1, amax_ptr, stream),
               "wb_transfer_rounds_fp8_fused")

    def remap_host(self, host_src_ptrs: Sequence[int], host_dst_ptrs: Sequence[int], stream: int = 0) -> None:
        a, b = _ptr_array(host_src_ptrs), _ptr_array(host_dst_ptrs)
        _check(_lib.wb_remap_host(self.handle, a, len(host_src_ptrs), b, len(host_dst_ptrs), stream),
               "wb_remap_host")


WB_ROUNDS_SERIAL = 1
WB_STATIC_SCRATCH_BYTES = 4 << 20
WB_STATIC_SYNC_CHECK = 1


def wb_remap_static(plan: Plan, src_ptrs: Sequence[int], dst_ptrs: Sequence[int], flags: int = 0,
                    stream: int = 0) -> None:
    """wb_remap without any device allocation: the plan is not bound; its tile table goes into
    the library's fixed 4 MiB device array (see include/wb.h for who needs this and the rules:
    first call per device outside stream capture, overlapping calls race, larger plans are
    refused with WB_ERR_STATIC_LIMIT)."""
    load()
    a, b = _ptr_array(src_ptrs), _ptr_array(dst_ptrs)
    _check(_lib.wb_remap_static(plan.handle, a, len(src_ptrs), b, len(dst_ptrs), flags, stream),
           "wb_remap_static")


def wb_plan_build(trainer: Layout, rollout: Layout, **opts) -> Plan:
    return Plan(trainer, rollout, **opts)


def wb_launches_per_call() -> int:
    return load().wb_launches_per_call()


def wb_version() -> str:
    return load().wb_version().decode()


# ---- source-map extraction ------------------------------------------------------------------------
WB_ID_I64, WB_ID_U16, WB_ID_F32, WB_ID_BF16 = 0, 1, 2, 3
DIFF2_ENTRY_DTYPE = np.dtype([("row", "<u8"), ("col", "<u8"), ("value", "<i8")])
SLICE_DTYPE = np.dtype([
    ("tensor", "<u4"), ("_pad", "<u4"), ("local_off", "<u8"), ("stride_r", "<i8"), ("stride_c", "<i8"),
    ("ckpt", "<u8"), ("ckpt_rows", "<u8"), ("ckpt_cols", "<u8"),
    ("r0", "<u8"), ("c0", "<u8"), ("nr", "<u8"), ("nc", "<u8")])
assert SLICE_DTYPE.itemsize == C.sizeof(wb_slice)


def wb_diff2_nonzeros(field_ptr: int, id_kind: int, rows: int, cols: int, out_ptr: int, cap: int,
                      count_ptr: int, stream: int = 0) -> None:
    """diff2 of a device id field, non-zeros appended to a device list (all pointers are device)."""
    load()
    _check(_lib.wb_diff2_nonzeros(field_ptr, id_kind, rows, cols, out_ptr, cap, count_ptr, stream),
           "wb_diff2_nonzeros")


DIFF2_FIELD_DTYPE = np.dtype([("field", "<u8"), ("rows", "<u8"), ("cols", "<u8"), ("id_kind", "<u4"), ("tag", "<u4")])
DIFF2_TAGGED_ENTRY_DTYPE = np.dtype([("row", "<u8"), ("col", "<u8"), ("value", "<i8"), ("tag", "<u4"), ("reserved", "<u4")])
assert DIFF2_FIELD_DTYPE.itemsize == 32 and DIFF2_TAGGED_ENTRY_DTYPE.itemsize == 32


def wb_diff2_batch_scratch_bytes(n_fields: int) -> int:
    load()
    _lib.wb_diff2_batch_scratch_bytes.restype = C.c_size_t
    _lib.wb_diff2_batch_scratch_bytes.argtypes = [C.c_size_t]
    return int(_lib.wb_diff2_batch_scratch_bytes(n_fields))


def wb_diff2_nonzeros_batch(fields: np.ndarray, scratch_ptr: int, scratch_bytes: int, out_ptr: int, cap: int,
                            count_ptr: int, stream: int = 0) -> None:
    """diff2 of many device id fields in one launch; `fields` is a host array of DIFF2_FIELD_DTYPE."""
    load()
    fields = np.ascontiguousarray(fields, dtype=DIFF2_FIELD_DTYPE)
    _lib.wb_diff2_nonzeros_batch.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p, C.c_uint64,
                                             C.c_void_p, C.c_void_p]
    _check(_lib.wb_diff2_nonzeros_batch(fields.ctypes.data, len(fields), scratch_ptr, scratch_bytes, out_ptr, cap,
                                        count_ptr, stream), "wb_diff2_nonzeros_batch")


def wb_diff2_chunk_scratch_bytes(rows: int, cols: int) -> int:
    lib = load()
    lib.wb_diff2_chunk_scratch_bytes.restype = C.c_size_t
    lib.wb_diff2_chunk_scratch_bytes.argtypes = [C.c_uint64, C.c_uint64]
    return int(lib.wb_diff2_chunk_scratch_bytes(rows, cols))


def wb_diff2_chunk_pass(field_ptr: int, id_kind: int, rows: int, cols: int, chunk_bits: int, pass_index: int,
                        carry_in_ptr: int, n_carry_in: int, scratch_ptr: int, scratch_bytes: int, z_out_ptr: int,
                        z_cap: int, z_count_ptr: int, carry_out_ptr: int, carry_cap: int, carry_count_ptr: int,
                        stream: int = 0) -> None:
    """One chunk pass of Algorithm 1 with carries for one device tensor (all pointers are device)."""
    lib = load()
    lib.wb_diff2_chunk_pass.argtypes = [C.c_void_p, C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32,
                                        C.c_void_p, C.c_uint64, C.c_void_p, C.c_size_t, C.c_void_p, C.c_uint64,
                                        C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p]
    _check(lib.wb_diff2_chunk_pass(field_ptr, id_kind, rows, cols, chunk_bits, pass_index, carry_in_ptr, n_carry_in,
                                   scratch_ptr, scratch_bytes, z_out_ptr, z_cap, z_count_ptr, carry_out_ptr, carry_cap,
                                   carry_count_ptr, stream), "wb_diff2_chunk_pass")


def wb_diff2_recombine(passes: Sequence[np.ndarray], chunk_bits: int) -> np.ndarray:
    load()
    passes = [np.ascontiguousarray(p, dtype=DIFF2_ENTRY_DTYPE) for p in passes]
    ptrs = _ptr_array([p.ctypes.data for p in passes])
    counts = (C.c_size_t * max(len(passes), 1))(*[len(p) for p in passes])
    n = C.c_size_t()
    _check(_lib.wb_diff2_recombine(ptrs, counts, len(passes), chunk_bits, None, 0, C.byref(n)), "wb_diff2_recombine")
    out = np.zeros(n.value, DIFF2_ENTRY_DTYPE)
    _check(_lib.wb_diff2_recombine(ptrs, counts, len(passes), chunk_bits, out.ctypes.data, n.value, C.byref(n)),
           "wb_diff2_recombine")
    return out


def wb_scan_slices(entries: np.ndarray, rows: int, cols: int, ckpt_base: np.ndarray, ckpt_rows: np.ndarray,
                   ckpt_cols: np.ndarray, tensor: int, elem_off: int = 0) -> np.ndarray:
    load()
    entries = np.ascontiguousarray(entries, dtype=DIFF2_ENTRY_DTYPE)
    base = np.ascontiguousarray(ckpt_base, dtype=np.uint64)
    cr = np.ascontiguousarray(ckpt_rows, dtype=np.uint64)
    cc = np.ascontiguousarray(ckpt_cols, dtype=np.uint64)
    assert len(base) == len(cr) + 1 == len(cc) + 1
    n = C.c_size_t()
    args = (entries.ctypes.data, len(entries), rows, cols, base.ctypes.data, cr.ctypes.data, cc.ctypes.data,
            len(cr), tensor, elem_off)
    _check(_lib.wb_scan_slices(*args, None, 0, C.byref(n)), "wb_scan_slices")
    out = np.zeros(n.value, SLICE_DTYPE)
    _check(_lib.wb_scan_slices(*args, out.ctypes.data, n.value, C.byref(n)), "wb_scan_slices")
    return out


# ---- three-stage routing, traffic accounting ---------------------------------------------------------
class wb_route_stats_t(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "model_bytes", "receive_bytes", "external_bytes", "internal_bytes", "direct_rdma_bytes",
        "max_trainer_rank_egress", "max_rollout_rank_rdma_ingress", "max_node_rdma_ingress")] + \
        [("t_min_seconds", C.c_double)]


def wb_route_account(plan: Plan, trainer_node: Sequence[int], rollout_node: Sequence[int], n_nodes: int,
                     trainer_gbs: float = 0.0, node_gbs: float = 0.0):
    """Returns (stats dict, per-node RDMA ingress, per-node required bytes M_v)."""
    load()
    tn = np.ascontiguousarray(trainer_node, dtype=np.uint32)
    rn = np.ascontiguousarray(rollout_node, dtype=np.uint32)
    st = wb_route_stats_t()
    ing = np.zeros(n_nodes, np.uint64)
    req = np.zeros(n_nodes, np.uint64)
    _check(_lib.wb_route_account(plan.handle, tn.ctypes.data, len(tn), rn.ctypes.data, len(rn), trainer_gbs,
                                 node_gbs, C.byref(st), ing.ctypes.data, req.ctypes.data, n_nodes),
           "wb_route_account")
    return {n: getattr(st, n) for n, _ in st._fields_}, ing, req


def wb_wait_probe(limit_ms: int, stream: int = 0) -> int:
    """Returns the raw status: WB_ERR_INTERNAL (11) means the bounded wait gave up as designed."""
    return load().wb_wait_probe(limit_ms, stream)
