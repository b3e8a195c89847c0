"""The remap, stated element by element (test infrastructure).

Definition (Section 3.1 of the paper): the checkpoint is the common coordinate system.
Give checkpoint element (r, c) of checkpoint tensor t the id (t, r*cols_t + c).  A
trainer source map S sends a trainer element y to the id that supplies it; a rollout
source map D does the same for a rollout element x.  The transfer must leave

        dst[x] = cast(src[y])   for every described x, for any y with S(y) = D(x).

Replication, de-duplication, rounds and buckets (Section 3.2) only decide *how* the
bytes travel; they do not change this result.  The functions below apply the definition
one checkpoint tensor at a time with a `holder` table (which trainer element supplies
each id), and count reads and writes so the exactly-once properties can be asserted.

Inputs are plain numpy: tensor tables and slice tables with the field names of a
slice-copy operation (tensor, local_off, stride_r, stride_c, ckpt, ckpt_rows, ckpt_cols,
r0, c0, nr, nc), and one raw-bits array per local tensor (uint32 for fp32, uint16 for
bf16).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from .cast import cast_bits


class UncoveredError(Exception):
    """A rollout element needs a checkpoint id that no trainer element holds."""


class ReplicaMismatchError(Exception):
    """Two trainer elements with the same checkpoint id hold different bits."""


class DoubleWriteError(Exception):
    """A rollout element is described by more than one slice-copy operation."""


@dataclass
class OracleResult:
    dst: List[np.ndarray]                 # expected rollout buffers (raw bits)
    written: List[np.ndarray]             # per rollout tensor: bool mask of described elements
    n_written: int = 0                    # rollout elements written (each exactly once)
    n_ids_consumed: int = 0               # distinct checkpoint ids read by >= 1 rollout element
    n_ids_held: int = 0                   # distinct checkpoint ids some trainer element holds
    n_replica_elems: int = 0              # trainer elements that duplicate an already-held id
    max_fanout: int = 0                   # most rollout elements fed by one id
    per_ckpt_consumed: Dict[int, int] = field(default_factory=dict)


def _slice_grid(s) -> Tuple[np.ndarray, np.ndarray]:
    """For one slice-copy op: (flat checkpoint index g, local element index x), both
    arrays of shape [nr, nc]."""
    i = np.arange(int(s["nr"]), dtype=np.int64)[:, None]
    j = np.arange(int(s["nc"]), dtype=np.int64)[None, :]
    g = (int(s["r0"]) + i) * int(s["ckpt_cols"]) + (int(s["c0"]) + j)
    x = int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])
    return g, x


def _group_by_ckpt(slices: np.ndarray) -> Dict[int, np.ndarray]:
    order = np.argsort(slices["ckpt"], kind="stable")
    out: Dict[int, List[int]] = {}
    for k in order:
        out.setdefault(int(slices["ckpt"][k]), []).append(int(k))
    return {t: np.array(v, dtype=np.int64) for t, v in out.items()}


def _build_holder(t_slices: np.ndarray, idx: np.ndarray, numel: int,
                  src: Sequence[np.ndarray]):
    """holder[g] = (trainer tensor, element) of the first trainer element (in slice
    order) that holds checkpoint element g; later holders must carry identical bits."""
    hold_t = np.full(numel, -1, dtype=np.int64)
    hold_y = np.zeros(numel, dtype=np.int64)
    hold_bits = None
    n_replica = 0
    for k in idx:
        s = t_slices[k]
        g, y = _slice_grid(s)
        g = g.ravel()
        y = y.ravel()
        tensor = int(s["tensor"])
        buf = src[tensor]
        if y.size and (y.min() < 0 or y.max() >= buf.size):
            raise IndexError(f"trainer slice {int(k)} leaves local tensor {tensor}")
        if g.size and (g.max() >= numel):
            raise IndexError(f"trainer slice {int(k)} leaves its checkpoint tensor")
        bits = buf[y]
        if hold_bits is None:
            hold_bits = np.zeros(numel, dtype=buf.dtype)
        empty = hold_t[g] < 0
        dup = ~empty
        if dup.any():
            if not np.array_equal(hold_bits[g[dup]], bits[dup]):
                raise ReplicaMismatchError(f"trainer slice {int(k)} disagrees with an earlier replica")
            n_replica += int(dup.sum())
        ge = g[empty]
        hold_t[ge] = tensor
        hold_y[ge] = y[empty]
        hold_bits[ge] = bits[empty]
    return hold_t, hold_y, hold_bits, n_replica


def remap_oracle(ckpt_shapes: Sequence[Tuple[int, int]],
                 trainer_tensors: np.ndarray, trainer_slices: np.ndarray,
                 rollout_tensors: np.ndarray, rollout_slices: np.ndarray,
                 src: Sequence[np.ndarray],
                 dst_prefill: Optional[Sequence[np.ndarray]] = None,
                 only_ckpt: Optional[Sequence[int]] = None) -> OracleResult:
    """Expected rollout buffers for the given trainer buffers.

    `dst_prefill` gives the initial contents of the rollout buffers; elements no rollout
    slice describes (padding) keep them.  `only_ckpt` restricts the pass to some
    checkpoint tensors (used to bound the CPU-baseline timing sample).
    """
    bits_of = {0: np.uint32, 1: np.uint16}
    dst = []
    for k, t in enumerate(rollout_tensors):
        if dst_prefill is not None:
            dst.append(np.array(dst_prefill[k], copy=True))
        else:
            dst.append(np.zeros(int(t["numel"]), dtype=bits_of[int(t["dtype"])]))
    writes = [np.zeros(int(t["numel"]), dtype=np.uint8) for t in rollout_tensors]
    res = OracleResult(dst=dst, written=[])

    t_by = _group_by_ckpt(trainer_slices)
    r_by = _group_by_ckpt(rollout_slices)
    todo = sorted(r_by.keys()) if only_ckpt is None else [t for t in only_ckpt if t in r_by]
    for t in todo:
        rows, cols = ckpt_shapes[t]
        numel = rows * cols
        if t in t_by:
            hold_t, hold_y, hold_bits, n_rep = _build_holder(trainer_slices, t_by[t], numel, src)
            res.n_replica_elems += n_rep
            res.n_ids_held += int((hold_t >= 0).sum())
        else:
            hold_t = np.full(numel, -1, dtype=np.int64)
            hold_bits = None
        reads = np.zeros(numel, dtype=np.int32)
        for k in r_by[t]:
            s = rollout_slices[k]
            if int(s["ckpt_rows"]) != rows or int(s["ckpt_cols"]) != cols:
                raise ValueError(f"rollout slice {int(k)}: checkpoint shape mismatch")
            g, x = _slice_grid(s)
            g = g.ravel()
            x = x.ravel()
            tensor = int(s["tensor"])
            if x.size and (x.min() < 0 or x.max() >= dst[tensor].size):
                raise IndexError(f"rollout slice {int(k)} leaves local tensor {tensor}")
            if (hold_t[g] < 0).any():
                raise UncoveredError(f"rollout slice {int(k)} needs ids of checkpoint tensor {t} "
                                     f"that no trainer holds")
            src_dtype = int(trainer_tensors[int(hold_t[g[0]])]["dtype"]) if g.size else 0
            dst_dtype = int(rollout_tensors[tensor]["dtype"])
            dst[tensor][x] = cast_bits(hold_bits[g], src_dtype, dst_dtype)
            np.add.at(writes[tensor], x, 1)
            np.add.at(reads, g, 1)
        consumed = int((reads > 0).sum())
        res.n_ids_consumed += consumed
        res.per_ckpt_consumed[t] = consumed
        if reads.size:
            res.max_fanout = max(res.max_fanout, int(reads.max()))
    for k, w in enumerate(writes):
        if (w > 1).any():
            raise DoubleWriteError(f"rollout tensor {k}: element written {int(w.max())} times")
        res.n_written += int(w.sum())
        res.written.append(w.astype(bool))
    return res


def checkpoint_view(t: int, ckpt_shape: Tuple[int, int], trainer_slices: np.ndarray,
                    src: Sequence[np.ndarray]) -> Tuple[np.ndarray, np.ndarray]:
    """The checkpoint tensor t as the trainer buffers hold it: (bits [rows, cols] in the
    source dtype, held mask).  This is "checkpoint format" (Section 3.2), used to check
    packed transfer buckets element by element."""
    rows, cols = ckpt_shape
    idx = np.nonzero(trainer_slices["ckpt"] == t)[0]
    hold_t, _, hold_bits, _ = _build_holder(trainer_slices, idx, rows * cols, src)
    if hold_bits is None:
        hold_bits = np.zeros(rows * cols, dtype=np.uint16)
    return hold_bits.reshape(rows, cols), (hold_t >= 0).reshape(rows, cols)


# ----------------------------------------------------------------------------------------
# one element at a time (for sampling outputs of runs too large to materialise on the host)
# ----------------------------------------------------------------------------------------
class SampleIndex:
    """Per-tensor / per-checkpoint-tensor lists of slices, so that single elements can be
    resolved without touching whole tensors."""

    def __init__(self, trainer_slices: np.ndarray, rollout_slices: np.ndarray):
        self.t_slices = trainer_slices
        self.r_slices = rollout_slices
        self.r_by_tensor: Dict[int, List[int]] = {}
        for k in range(len(rollout_slices)):
            self.r_by_tensor.setdefault(int(rollout_slices["tensor"][k]), []).append(k)
        self.t_by_ckpt: Dict[int, List[int]] = {}
        for k in range(len(trainer_slices)):
            self.t_by_ckpt.setdefault(int(trainer_slices["ckpt"][k]), []).append(k)


def _locate(s, x: int) -> Optional[Tuple[int, int]]:
    """(i, j) with local_off + i*stride_r + j*stride_c == x inside the slice, or None."""
    nr, nc = int(s["nr"]), int(s["nc"])
    sr, sc = int(s["stride_r"]), int(s["stride_c"])
    d = x - int(s["local_off"])
    if d < 0:
        return None
    if nr == 1 and nc == 1:
        return (0, 0) if d == 0 else None
    if nc == 1:                               # one column: only stride_r matters
        return (d // sr, 0) if (d % sr == 0 and d // sr < nr) else None
    if nr == 1:                               # one row: only stride_c matters
        return (0, d // sc) if (d % sc == 0 and d // sc < nc) else None
    # the two shapes a slice-copy op takes: rows contiguous (stride_c == 1) or, when
    # transposed, columns contiguous (stride_r == 1)
    if sc == 1:
        i, j = divmod(d, sr)
        return (i, j) if (i < nr and j < nc) else None
    if sr == 1:
        j, i = divmod(d, sc)
        return (i, j) if (i < nr and j < nc) else None
    for i in range(nr):                       # general strides: exhaustive (tiny cases only)
        rem = d - i * sr
        if rem >= 0 and rem % sc == 0 and rem // sc < nc:
            return i, rem // sc
    return None


def source_of_rollout_element(index: SampleIndex, tensor: int, x: int):
    """Resolve one rollout element: returns (ckpt tensor, r, c, trainer tensor, y) or None
    if no rollout slice describes x.  Raises UncoveredError if no trainer holds the id."""
    for k in index.r_by_tensor.get(tensor, ()):
        s = index.r_slices[k]
        ij = _locate(s, x)
        if ij is None:
            continue
        t = int(s["ckpt"])
        r = int(s["r0"]) + ij[0]
        c = int(s["c0"]) + ij[1]
        for m in index.t_by_ckpt.get(t, ()):
            u = index.t_slices[m]
            if int(u["r0"]) <= r < int(u["r0"]) + int(u["nr"]) and \
               int(u["c0"]) <= c < int(u["c0"]) + int(u["nc"]):
                y = int(u["local_off"]) + (r - int(u["r0"])) * int(u["stride_r"]) + \
                    (c - int(u["c0"])) * int(u["stride_c"])
                return t, r, c, int(u["tensor"]), y
        raise UncoveredError(f"checkpoint element ({t},{r},{c}) held by no trainer")
    return None
