"""Plain data containers for workloads: tensor tables, slice lists, value recipes."""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, Iterator, List, Optional, Sequence, Tuple

import numpy as np
import torch

WB_F32 = 0
WB_BF16 = 1

# One slice-copy operation of a source map (Section 3.1): the rectangle
# [r0, r0+nr) x [c0, c0+nc) of checkpoint tensor `ckpt` (viewed as a row-major
# ckpt_rows x ckpt_cols matrix) lives in local tensor `tensor`; checkpoint
# element (r0+i, c0+j) is local element local_off + i*stride_r + j*stride_c.
SLICE_DTYPE = np.dtype([
    ("tensor", "<u4"), ("_pad", "<u4"), ("local_off", "<u8"),
    ("stride_r", "<i8"), ("stride_c", "<i8"),
    ("ckpt", "<u8"), ("ckpt_rows", "<u8"), ("ckpt_cols", "<u8"),
    ("r0", "<u8"), ("c0", "<u8"), ("nr", "<u8"), ("nc", "<u8"),
])
assert SLICE_DTYPE.itemsize == 88

# One local tensor of a virtual rank.
TENSOR_DTYPE = np.dtype([("rank", "<u4"), ("dtype", "<u4"), ("numel", "<u8")])
assert TENSOR_DTYPE.itemsize == 16


def dtype_size(dt: int) -> int:
    return 4 if dt == WB_F32 else 2


def torch_dtype(dt: int) -> torch.dtype:
    return torch.float32 if dt == WB_F32 else torch.bfloat16


def bits_dtype(dt: int):
    return np.uint32 if dt == WB_F32 else np.uint16


def torch_bits_dtype(dt: int) -> torch.dtype:
    # same-width signed integer view (torch has full support for these)
    return torch.int32 if dt == WB_F32 else torch.int16


@dataclass
class CkptTensor:
    name: str
    rows: int
    cols: int

    @property
    def numel(self) -> int:
        return self.rows * self.cols


class Layout:
    """One side's source map: local tensor table + slice list."""

    def __init__(self, side: str):
        self.side = side
        self.names: List[str] = []
        self._index: Dict[str, int] = {}
        self._tensors: List[Tuple[int, int, int]] = []
        self._slices: List[tuple] = []
        self._frozen = False
        self.tensors: np.ndarray = np.zeros(0, TENSOR_DTYPE)
        self.slices: np.ndarray = np.zeros(0, SLICE_DTYPE)

    def add_tensor(self, name: str, rank: int, dtype: int, numel: int) -> int:
        assert name not in self._index, name
        idx = len(self.names)
        self.names.append(name)
        self._index[name] = idx
        self._tensors.append((rank, dtype, numel))
        return idx

    def index(self, name: str) -> int:
        return self._index[name]

    def add_slice(self, tensor: int, local_off: int, stride_r: int, stride_c: int,
                  ckpt: int, ckpt_rows: int, ckpt_cols: int,
                  r0: int, c0: int, nr: int, nc: int) -> None:
        if nr == 0 or nc == 0:
            return
        self._slices.append((tensor, 0, local_off, stride_r, stride_c, ckpt,
                             ckpt_rows, ckpt_cols, r0, c0, nr, nc))

    def freeze(self) -> "Layout":
        self.tensors = np.array(self._tensors, dtype=TENSOR_DTYPE) if self._tensors \
            else np.zeros(0, TENSOR_DTYPE)
        self.slices = np.array(self._slices, dtype=SLICE_DTYPE) if self._slices \
            else np.zeros(0, SLICE_DTYPE)
        self._frozen = True
        return self

    @property
    def n_tensors(self) -> int:
        return len(self.names)

    def total_bytes(self) -> int:
        return int(sum(int(t["numel"]) * dtype_size(int(t["dtype"])) for t in self.tensors))

    def swapped_dtype(self, dtype: int) -> "Layout":
        """Same layout with every local tensor's dtype replaced."""
        out = Layout(self.side)
        out.names = list(self.names)
        out._index = dict(self._index)
        out._tensors = [(r, dtype, n) for (r, _, n) in self._tensors]
        out._slices = list(self._slices)
        return out.freeze()


# A procedural loader group: the checkpoint tensors it needs (indices into the
# checkpoint table) and a function that turns them (2-D torch tensors, in that
# order) into {local tensor name: flat torch tensor}.  Written with tensor ops
# (cat / chunk / stack / transpose / pad), never through the slice lists.
LoaderGroup = Tuple[List[int], Callable[[List[torch.Tensor]], Dict[str, torch.Tensor]]]


@dataclass
class Workload:
    name: str
    seed: int
    dist: str                      # "normal0.02" | "uniform"
    src_dtype: int
    dst_dtype: int
    ckpt: List[CkptTensor]
    trainer: Layout
    rollout: Layout
    trainer_groups: Callable[[], Iterator[LoaderGroup]]
    rollout_groups: Callable[[], Iterator[LoaderGroup]]
    pad_value: float = 0.0
    meta: dict = field(default_factory=dict)

    # ---- checkpoint coordinates -------------------------------------------------
    def ckpt_base(self) -> np.ndarray:
        """Global id of element (0,0) of every checkpoint tensor (exclusive prefix sum)."""
        n = np.array([t.numel for t in self.ckpt], dtype=np.int64)
        base = np.zeros(len(n) + 1, dtype=np.int64)
        np.cumsum(n, out=base[1:])
        return base

    def ckpt_numel(self) -> int:
        return int(sum(t.numel for t in self.ckpt))

    # ---- values --------------------------------------------------------------------
    def ckpt_values(self, idx: int, device="cpu") -> torch.Tensor:
        """Seeded values of checkpoint tensor `idx`, in the source dtype, shape [rows, cols]."""
        t = self.ckpt[idx]
        g = torch.Generator(device=device)
        g.manual_seed((self.seed * 1_000_003 + idx * 7919 + 12345) & 0x7FFFFFFFFFFF)
        if self.dist == "normal0.02":
            v = torch.empty(t.rows, t.cols, dtype=torch.float32, device=device)
            v.normal_(0.0, 0.02, generator=g)
        elif self.dist == "uniform":
            v = torch.empty(t.rows, t.cols, dtype=torch.float32, device=device)
            v.uniform_(-1.0, 1.0, generator=g)
        else:
            raise ValueError(self.dist)
        return v.to(torch_dtype(self.src_dtype))

    def ckpt_ids(self, idx: int, device="cpu") -> torch.Tensor:
        """Global ids (int64) of checkpoint tensor `idx`, shape [rows, cols] (the id probe)."""
        t = self.ckpt[idx]
        base = int(self.ckpt_base()[idx])
        return torch.arange(base, base + t.numel, dtype=torch.int64, device=device).view(t.rows, t.cols)

    # ---- procedural load_weights ------------------------------------------------------
    def load_side(self, side: str, values: Callable[[int], torch.Tensor],
                  sink: Callable[[int, torch.Tensor], None]) -> None:
        """Run the procedural load_weights of `side`: for every loader group fetch the
        checkpoint tensors with `values(idx)` and hand each produced local tensor to
        `sink(local_index, flat_tensor)`."""
        layout = self.trainer if side == "trainer" else self.rollout
        groups = self.trainer_groups if side == "trainer" else self.rollout_groups
        for ckpt_idx, fn in groups():
            out = fn([values(i) for i in ckpt_idx])
            for name, t in out.items():
                sink(layout.index(name), t.reshape(-1))

    def load_side_shaped(self, side: str, values: Callable[[int], torch.Tensor],
                         sink: Callable[[int, torch.Tensor], None]) -> None:
        """Like load_side, but hands over each local tensor with the shape load_weights gives it
        (the 2-D view used by source-map extraction is [prod(shape[:-1]), shape[-1]])."""
        layout = self.trainer if side == "trainer" else self.rollout
        groups = self.trainer_groups if side == "trainer" else self.rollout_groups
        for ckpt_idx, fn in groups():
            for name, t in fn([values(i) for i in ckpt_idx]).items():
                sink(layout.index(name), t)

    def load_side_to_list(self, side: str, values: Callable[[int], torch.Tensor]) -> List[torch.Tensor]:
        layout = self.trainer if side == "trainer" else self.rollout
        out: List[Optional[torch.Tensor]] = [None] * layout.n_tensors

        def sink(i, t):
            assert out[i] is None, layout.names[i]
            assert t.numel() == int(layout.tensors[i]["numel"]), \
                (layout.names[i], t.numel(), int(layout.tensors[i]["numel"]))
            out[i] = t.contiguous()
        self.load_side(side, values, sink)
        for i, t in enumerate(out):
            assert t is not None, layout.names[i]
        return out  # type: ignore

    def trainer_weights(self, device="cpu") -> List[torch.Tensor]:
        """Trainer local tensors filled with the seeded weights (padding = pad_value)."""
        return self.load_side_to_list("trainer", lambda i: self.ckpt_values(i, device))

    # ---- accounting ----------------------------------------------------------------------
    def algorithmic_bytes(self) -> Tuple[int, int]:
        """(bytes read, bytes written) by one full remap: every rollout element described by
        the rollout source map is written once; every distinct checkpoint element any
        rollout slice consumes is read once.  Computed here only from slice extents
        (rollout replicas counted once on the read side via `meta['distinct_read_elems']`
        when the builder knows it, else assumed replica-free)."""
        written = int(np.sum(self.rollout.slices["nr"].astype(np.int64) *
                             self.rollout.slices["nc"].astype(np.int64)))
        read = int(self.meta.get("distinct_read_elems", written))
        return read * dtype_size(self.src_dtype), written * dtype_size(self.dst_dtype)
