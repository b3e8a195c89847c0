"""Shared test utilities: bit views, the id probe, fuzz layouts.  No method arithmetic
from either the oracle or the library lives here."""
import numpy as np
import torch

from wb_workloads import SLICE_DTYPE, TENSOR_DTYPE, WB_BF16, WB_F32, Layout
from wb_workloads.rng import SplitMix64


def to_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns of a float32 / bfloat16 tensor as uint32 / uint16."""
    t = t.detach().cpu().contiguous().reshape(-1)
    if t.dtype == torch.float32:
        return t.view(torch.int32).numpy().view(np.uint32).copy()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    raise TypeError(t.dtype)


def from_bits(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32).copy()).view(torch.float32)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    raise TypeError(a.dtype)


def ckpt_shapes(wl):
    return [(c.rows, c.cols) for c in wl.ckpt]


def predict_ids(layout: Layout, wl):
    """What the slice list says each local element's checkpoint id is (-1 = undescribed)."""
    base = wl.ckpt_base()
    out = [np.full(int(t["numel"]), -1, np.int64) for t in layout.tensors]
    for s in layout.slices:
        i = np.arange(int(s["nr"]), dtype=np.int64)[:, None]
        j = np.arange(int(s["nc"]), dtype=np.int64)[None, :]
        g = base[int(s["ckpt"])] + (int(s["r0"]) + i) * int(s["ckpt_cols"]) + int(s["c0"]) + j
        x = int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])
        buf = out[int(s["tensor"])]
        assert (buf[x] == -1).all(), "slice list describes a local element twice"
        buf[x] = g
    return out


def probe_ids(wl, side):
    """The id probe: load an id-valued checkpoint through the procedural load_weights."""
    return [t.numpy() for t in wl.load_side_to_list(side, lambda i: wl.ckpt_ids(i))]


def random_partition(rng: SplitMix64, rows: int, cols: int, max_parts: int):
    """Random guillotine partition of a rows x cols matrix into rectangles."""
    rects = [(0, 0, rows, cols)]
    target = rng.randint(1, max_parts)
    guard = 0
    while len(rects) < target and guard < 50:
        guard += 1
        k = rng.randint(0, len(rects) - 1)
        r0, c0, nr, nc = rects[k]
        if rng.uniform() < 0.5 and nr > 1:
            cut = rng.randint(1, nr - 1)
            rects[k] = (r0, c0, cut, nc)
            rects.append((r0 + cut, c0, nr - cut, nc))
        elif nc > 1:
            cut = rng.randint(1, nc - 1)
            rects[k] = (r0, c0, nr, cut)
            rects.append((r0, c0 + cut, nr, nc - cut))
    return rects


def fuzz_case(seed: int, src_dtype=WB_F32, dst_dtype=WB_BF16, n_ckpt=None, max_dim=40,
              replicas=True):
    """Random affine source maps: every checkpoint tensor gets an independent random
    rectangle partition on each side; every rectangle lands in a random local tensor at a
    random offset with random pitch padding, optionally transposed; some trainer
    rectangles are replicated on a second rank, some rollout rectangles too (fan-out).
    Returns (ckpt shapes, trainer Layout, rollout Layout)."""
    rng = SplitMix64(seed)
    n_ckpt = n_ckpt or rng.randint(1, 6)
    shapes = [(rng.randint(1, max_dim), rng.randint(1, max_dim)) for _ in range(n_ckpt)]

    def side(name, dtype, n_local):
        lay = Layout(name)
        # local tensors are filled by appending regions; sizes fixed at the end
        cursor = [rng.randint(0, 5) for _ in range(n_local)]
        pending = []
        for t, (rows, cols) in enumerate(shapes):
            rects = random_partition(rng, rows, cols, 6)
            extra = []
            if replicas:
                for r in rects:
                    if rng.uniform() < 0.25:
                        extra.append(r)
                if rng.uniform() < 0.5:      # a replica that straddles partition boundaries
                    a0, b0 = rng.randint(0, rows - 1), rng.randint(0, cols - 1)
                    extra.append((a0, b0, rng.randint(1, rows - a0), rng.randint(1, cols - b0)))
            for (r0, c0, nr, nc) in rects + extra:
                loc = rng.randint(0, n_local - 1)
                transposed = rng.uniform() < 0.3
                if transposed:
                    pitch = nr + rng.randint(0, 3)
                    sr, sc = 1, pitch
                    span = (nc - 1) * pitch + nr
                else:
                    pitch = nc + rng.randint(0, 3)
                    sr, sc = pitch, 1
                    span = (nr - 1) * pitch + nc
                off = cursor[loc]
                cursor[loc] = off + span + rng.randint(0, 4)
                pending.append((loc, off, sr, sc, t, rows, cols, r0, c0, nr, nc))
        for k in range(n_local):
            lay.add_tensor(f"{name}{k}", k % 4, dtype, cursor[k] + 1)
        for p in pending:
            lay.add_slice(*p)
        return lay.freeze()

    return shapes, side("t", src_dtype, rng.randint(1, 4)), side("r", dst_dtype, rng.randint(1, 4))


def random_bits(rng: np.random.Generator, n: int, dtype: int) -> np.ndarray:
    """Random finite, non-NaN bit patterns (values are irrelevant to the data path)."""
    if dtype == WB_F32:
        v = rng.standard_normal(n).astype(np.float32)
        return v.view(np.uint32).copy()
    v = torch.from_numpy(rng.standard_normal(n).astype(np.float32)).to(torch.bfloat16)
    return to_bits(v)


def scatter_checkpoint(layout: Layout, ckpt_bits, fill_bits=None):
    """load_weights by slice list: copy checkpoint bits into local buffers (used by the
    fuzz cases, whose layouts have no procedural loader)."""
    out = []
    for t in layout.tensors:
        dt = np.uint32 if int(t["dtype"]) == WB_F32 else np.uint16
        a = np.zeros(int(t["numel"]), dtype=dt)
        if fill_bits is not None:
            a[:] = fill_bits
        out.append(a)
    for s in layout.slices:
        i = np.arange(int(s["nr"]), dtype=np.int64)[:, None]
        j = np.arange(int(s["nc"]), dtype=np.int64)[None, :]
        g = (int(s["r0"]) + i) * int(s["ckpt_cols"]) + int(s["c0"]) + j
        x = int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])
        out[int(s["tensor"])][x] = ckpt_bits[int(s["ckpt"])].reshape(-1)[g]
    return out
