"""The benchmark's own configurations at full size, in the launch configuration bench.py times
(default plan options), checked three ways that need no host copy of the model:

  * every rollout tensor equals the procedural rollout load_weights (torch cat / stack / chunk /
    transpose) of the seeded checkpoint -- all elements;
  * the id probe of Section 3.1 / Algorithm 1 run THROUGH the GPU path: the checkpoint is filled
    with b-bit chunks of each element's global id (b = 16 raw bits for a bit copy, b = 8 exact
    small integers for fp32 -> bf16), remapped, and compared with the ids the rollout layout
    expects -- all elements, every chunk;
  * sampled outputs resolved one by one by the CPU oracle (which rollout slice, which checkpoint
    element, which trainer element, oracle cast).
"""
import numpy as np
import pytest
import torch

from gpu_util import CANARY, DeviceCase
from oracle import SampleIndex, source_of_rollout_element
from oracle.cast import cast_bits
from wb_workloads import WB_BF16, WB_F32, make_workload
from wb_workloads.types import torch_dtype

pytestmark = pytest.mark.gpu
INT_VIEW = {torch.float32: torch.int32, torch.bfloat16: torch.int16}


def check_against_procedural(case, values):
    """Reload the trainer arenas from `values`, remap, and compare every rollout tensor with the
    procedural rollout loader applied to the same checkpoint values (cast by torch)."""
    wl = case.wl
    dst_dt = torch_dtype(wl.dst_dtype)
    case.load_trainer(values)
    case.reset_dst()
    case.plan.remap()
    torch.cuda.synchronize()
    case.plan.check()
    bad = []

    def sink(k, want):
        got = case.dst.tensors[k]
        if not torch.equal(got.view(INT_VIEW[got.dtype]), want.contiguous().view(INT_VIEW[want.dtype])):
            bad.append(case.rollout.names[k])
    wl.load_side("rollout", lambda i: values(i).to(dst_dt), sink)
    assert not bad, f"{len(bad)} rollout tensors differ, e.g. {bad[:5]}"


def gaps_intact(case):
    """The bytes between consecutive local tensors of each rollout arena still hold the canary."""
    by_rank = {}
    for t, d in zip(case.dst.tensors, case.rollout.tensors):
        by_rank.setdefault(int(d["rank"]), []).append(t)
    for r, arena in case.dst.arenas.items():
        base = arena.data_ptr()
        spans = sorted((t.data_ptr() - base, t.numel() * t.element_size()) for t in by_rank.get(r, []))
        pos = 0
        for off, n in spans:
            if off > pos and not bool((arena[pos:off] == CANARY).all()):
                return False
            pos = off + n
        if pos < arena.numel() and not bool((arena[pos:] == CANARY).all()):
            return False
    return True


def sample_against_oracle(case, n_samples, seed):
    wl = case.wl
    rng = np.random.default_rng(seed)
    index = SampleIndex(case.trainer.slices, case.rollout.slices)
    numel = case.rollout.tensors["numel"].astype(np.float64)
    picks = []
    for k in rng.choice(len(numel), size=n_samples, p=numel / numel.sum()):
        picks.append((int(k), int(rng.integers(0, int(numel[k])))))
    # the corners of randomly chosen rollout slices (slab boundaries are where indexing goes wrong)
    for s in case.rollout.slices[rng.integers(0, len(case.rollout.slices), size=n_samples // 4)]:
        for (i, j) in ((0, 0), (int(s["nr"]) - 1, int(s["nc"]) - 1), (0, int(s["nc"]) - 1), (int(s["nr"]) - 1, 0)):
            picks.append((int(s["tensor"]), int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])))
    src_t, src_y, dst_t, dst_x = [], [], [], []
    for (k, x) in picks:
        hit = source_of_rollout_element(index, k, x)
        if hit is None:
            continue                      # padding on the rollout side (none in these layouts)
        src_t.append(hit[3]); src_y.append(hit[4]); dst_t.append(k); dst_x.append(x)
    assert len(src_t) >= n_samples

    def gather(tensors, which, where):
        out = np.zeros(len(which), dtype=np.uint32)
        which, where = np.array(which), np.array(where)
        for t in np.unique(which):
            m = which == t
            view = tensors[t].view(INT_VIEW[tensors[t].dtype])
            vals = view[torch.from_numpy(where[m]).to(view.device)].cpu().numpy()
            out[m] = vals.astype(np.int64) & (0xFFFFFFFF if vals.dtype == np.int32 else 0xFFFF)
        return out
    src_bits = gather(case.src.tensors, src_t, src_y)
    dst_bits = gather(case.dst.tensors, dst_t, dst_x)
    src_bits = src_bits.astype(np.uint32 if wl.src_dtype == WB_F32 else np.uint16)
    want = cast_bits(src_bits, wl.src_dtype, wl.dst_dtype)
    assert np.array_equal(dst_bits.astype(want.dtype), want)


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg5", "cfg4"])
def test_full_size_configuration(name):
    device = torch.device("cuda:0")
    wl = make_workload(name, "full")
    need = wl.trainer.total_bytes() + wl.rollout.total_bytes() + (12 << 30)
    torch.cuda.empty_cache()
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    case = DeviceCase(wl, device)                       # default options = bench.py's launch configuration
    st = case.plan.stats()
    r, w = wl.algorithmic_bytes()
    assert (st["src_bytes_read"], st["dst_bytes_written"]) == (r, w)

    # 1. seeded weights, all elements, against the procedural rollout loader
    check_against_procedural(case, lambda i: wl.ckpt_values(i, device))
    assert gaps_intact(case)
    # 2. sampled outputs against the CPU oracle (same buffers)
    sample_against_oracle(case, 4000, seed=wl.seed)

    # 3. chunked id probe through the GPU path
    bits_needed = int(wl.ckpt_numel()).bit_length()
    same = wl.src_dtype == wl.dst_dtype
    b = 16 if same else 8
    src_dt = torch_dtype(wl.src_dtype)
    for chunk in range(-(-bits_needed // b)):
        def values(i, chunk=chunk):
            part = (wl.ckpt_ids(i, device) >> (b * chunk)) & ((1 << b) - 1)
            if same and src_dt == torch.bfloat16:
                return part.to(torch.int16).view(torch.bfloat16)      # raw 16-bit payload
            return part.to(src_dt)                                       # 0..255, exact in bf16
        check_against_procedural(case, values)
    del case
    torch.cuda.empty_cache()
