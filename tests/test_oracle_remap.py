"""Pins for the remap oracle: things fixed by the definition of correspondence
(Section 3.1) and by plain mathematics, none of which re-type the oracle's own code."""
import os

import numpy as np
import pytest
import torch

from helpers import (ckpt_shapes, from_bits, fuzz_case, probe_ids, random_bits,
                     scatter_checkpoint, to_bits)
from oracle import (DoubleWriteError, ReplicaMismatchError, SampleIndex, UncoveredError,
                    checkpoint_view, remap_oracle, source_of_rollout_element)
from wb_workloads import SLICE_DTYPE, WB_BF16, WB_F32, Layout, make_workload

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "micro_4x6.txt")
SMALL = [("cfg1", "full"), ("cfg1b", "full"), ("cfg1c", "full"), ("cfg2", "small"),
         ("cfg3", "small"), ("cfg4", "small"), ("cfg5", "small")]


def run_oracle(wl, src_bits, prefill=None, **kw):
    return remap_oracle(ckpt_shapes(wl), wl.trainer.tensors, wl.trainer.slices,
                        wl.rollout.tensors, wl.rollout.slices, src_bits, prefill, **kw)


def torch_cast_bits(t: torch.Tensor, dst_dtype: int) -> np.ndarray:
    return to_bits(t.to(torch.bfloat16 if dst_dtype == WB_BF16 else torch.float32))


# ---- the hand-worked micro case ----------------------------------------------------------
def _load_micro():
    vals, slices = {}, []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, rest = line.split(":")
            if key == "slice":
                p = rest.split()
                slices.append((p[0], [int(v) for v in p[1:]]))
            else:
                vals[key] = np.array([float(v) for v in rest.split()], dtype=np.float32)
    return vals, slices


def test_micro_case_by_hand():
    vals, slices = _load_micro()
    tl, rl = Layout("trainer"), Layout("rollout")
    for k in range(2):
        tl.add_tensor(f"T{k}", k, WB_F32, 12)
        rl.add_tensor(f"R{k}", k, WB_BF16, 12)
    for side, (t, off, sr, sc, r0, c0, nr, nc) in slices:
        (tl if side == "T" else rl).add_slice(t, off, sr, sc, 0, 4, 6, r0, c0, nr, nc)
    tl.freeze(); rl.freeze()
    src = [vals["T0"].view(np.uint32), vals["T1"].view(np.uint32)]
    res = remap_oracle([(4, 6)], tl.tensors, tl.slices, rl.tensors, rl.slices, src)
    for k in range(2):
        got = from_bits(res.dst[k]).to(torch.float32).numpy()
        assert np.array_equal(got, vals[f"R{k}"])
    assert res.n_written == 24 and res.n_ids_consumed == 24 and res.max_fanout == 1


# ---- brute force: join on materialised ids, no rectangle arithmetic ------------------------
@pytest.mark.parametrize("name", ["cfg1", "cfg1b", "cfg1c"])
def test_brute_force_id_join(name):
    wl = make_workload(name)
    src = wl.trainer_weights()
    t_ids = probe_ids(wl, "trainer")          # id of every trainer element (-1 = padding)
    r_ids = probe_ids(wl, "rollout")          # id of every rollout element
    all_ids = np.concatenate(t_ids)
    all_vals = torch.cat(src)
    keep = all_ids >= 0
    ids_k, pos_k = all_ids[keep], np.nonzero(keep)[0]
    order = np.argsort(ids_k, kind="stable")
    sorted_ids, sorted_pos = ids_k[order], pos_k[order]
    res = run_oracle(wl, [to_bits(t) for t in src])
    for k, rid in enumerate(r_ids):
        assert (rid >= 0).all()
        at = np.searchsorted(sorted_ids, rid, side="left")
        assert np.array_equal(sorted_ids[at], rid)           # some trainer holds every id
        want = torch_cast_bits(all_vals[torch.from_numpy(sorted_pos[at])], wl.dst_dtype)
        assert np.array_equal(res.dst[k], want), wl.rollout.names[k]
    # replicas (norms on both TP ranks) carry the same bits, so "any y" is well defined
    uniq, counts = np.unique(ids_k, return_counts=True)
    assert res.n_replica_elems == int((counts - 1).sum()) > 0
    assert res.n_ids_held == uniq.size == wl.ckpt_numel()


# ---- library-routine statement: rollout tensors are cat / stack / chunk of the checkpoint ----
@pytest.mark.parametrize("name,scale", SMALL)
def test_equals_procedural_rollout_load(name, scale):
    wl = make_workload(name, scale)
    src = wl.trainer_weights()
    res = run_oracle(wl, [to_bits(t) for t in src])
    want = wl.load_side_to_list(
        "rollout", lambda i: wl.ckpt_values(i).to(torch.bfloat16 if wl.dst_dtype == WB_BF16 else torch.float32))
    for k, w in enumerate(want):
        assert np.array_equal(res.dst[k], to_bits(w)), wl.rollout.names[k]


def test_fused_qkv_is_a_concatenation():
    wl = make_workload("cfg1")
    res = run_oracle(wl, [to_bits(t) for t in wl.trainer_weights()])
    ix = {c.name: i for i, c in enumerate(wl.ckpt)}
    bf = lambda n: wl.ckpt_values(ix[n]).to(torch.bfloat16)
    qkv = torch.cat([bf("layers.1.q_proj"), bf("layers.1.k_proj"), bf("layers.1.v_proj")], 0)
    assert qkv.shape == (512, 256)
    assert np.array_equal(res.dst[wl.rollout.index("r0.layers.1.qkv_proj")], to_bits(qkv))
    gu = torch.cat([bf("layers.0.gate_proj"), bf("layers.0.up_proj")], 0)
    assert gu.shape == (1376, 256)
    assert np.array_equal(res.dst[wl.rollout.index("r0.layers.0.gate_up_proj")], to_bits(gu))


# ---- exactly-once invariants ---------------------------------------------------------------
@pytest.mark.parametrize("name,scale", SMALL)
def test_exactly_once_counters(name, scale):
    wl = make_workload(name, scale)
    src = [to_bits(t) for t in wl.trainer_weights()]
    prefill = [np.full(int(t["numel"]), 0xDEAD, dtype=np.uint16) for t in wl.rollout.tensors]
    res = run_oracle(wl, src, prefill)
    described = int(np.sum(wl.rollout.slices["nr"].astype(np.int64) * wl.rollout.slices["nc"].astype(np.int64)))
    assert res.n_written == described
    assert res.n_ids_consumed == wl.ckpt_numel()            # every id is needed, read once
    assert sum(int(w.sum()) for w in res.written) == described
    assert res.max_fanout == (2 if name == "cfg3" else 1)   # cfg3: norms on both rollout ranks
    for k, w in enumerate(res.written):                     # undescribed elements keep the prefill
        assert (res.dst[k][~w] == 0xDEAD).all()


def test_padding_never_read():
    wl = make_workload("cfg1b")
    src = wl.trainer_weights()
    a = run_oracle(wl, [to_bits(t) for t in src])
    ids = probe_ids(wl, "trainer")
    poisoned = []
    for t, i in zip(src, ids):
        t = t.clone()
        t[torch.from_numpy(i < 0)] = float("nan")
        poisoned.append(to_bits(t))
    b = run_oracle(wl, poisoned)
    for x, y in zip(a.dst, b.dst):
        assert np.array_equal(x, y)


# ---- inverse ---------------------------------------------------------------------------------
@pytest.mark.parametrize("name,scale", [("cfg1b", "full"), ("cfg3", "small"), ("cfg5", "small")])
def test_inverse_remap_is_identity(name, scale):
    wl = make_workload(name, scale)
    tl = wl.trainer.swapped_dtype(WB_BF16)
    rl = wl.rollout.swapped_dtype(WB_BF16)
    rng = np.random.default_rng(1)
    ck_bits = [rng.integers(0, 1 << 16, size=c.numel, dtype=np.uint64).astype(np.uint16) for c in wl.ckpt]
    src = scatter_checkpoint(tl, ck_bits, fill_bits=0xAAAA)
    fwd = remap_oracle(ckpt_shapes(wl), tl.tensors, tl.slices, rl.tensors, rl.slices, src)
    prefill = [np.full(int(t["numel"]), 0xAAAA, dtype=np.uint16) for t in tl.tensors]
    back = remap_oracle(ckpt_shapes(wl), rl.tensors, rl.slices, tl.tensors, tl.slices, fwd.dst, prefill)
    for a, b in zip(src, back.dst):
        assert np.array_equal(a, b)


# ---- error detection ---------------------------------------------------------------------------
def _two_by_two():
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T", 0, WB_F32, 4)
    rl.add_tensor("R", 0, WB_F32, 4)
    return tl, rl


def test_uncovered_is_reported():
    tl, rl = _two_by_two()
    tl.add_slice(0, 0, 2, 1, 0, 2, 2, 0, 0, 1, 2)            # only row 0 held
    rl.add_slice(0, 0, 2, 1, 0, 2, 2, 0, 0, 2, 2)
    tl.freeze(); rl.freeze()
    with pytest.raises(UncoveredError):
        remap_oracle([(2, 2)], tl.tensors, tl.slices, rl.tensors, rl.slices, [np.zeros(4, np.uint32)])


def test_double_write_is_reported():
    tl, rl = _two_by_two()
    tl.add_slice(0, 0, 2, 1, 0, 2, 2, 0, 0, 2, 2)
    rl.add_slice(0, 0, 2, 1, 0, 2, 2, 0, 0, 2, 2)
    rl.add_slice(0, 3, 2, 1, 0, 2, 2, 0, 0, 1, 1)
    tl.freeze(); rl.freeze()
    with pytest.raises(DoubleWriteError):
        remap_oracle([(2, 2)], tl.tensors, tl.slices, rl.tensors, rl.slices, [np.zeros(4, np.uint32)])


def test_replica_mismatch_is_reported():
    tl, rl = Layout("t"), Layout("r")
    tl.add_tensor("T0", 0, WB_F32, 4); tl.add_tensor("T1", 1, WB_F32, 4)
    rl.add_tensor("R", 0, WB_F32, 4)
    tl.add_slice(0, 0, 2, 1, 0, 2, 2, 0, 0, 2, 2)
    tl.add_slice(1, 0, 2, 1, 0, 2, 2, 0, 0, 2, 2)
    rl.add_slice(0, 0, 2, 1, 0, 2, 2, 0, 0, 2, 2)
    tl.freeze(); rl.freeze()
    good = [np.arange(4, dtype=np.uint32), np.arange(4, dtype=np.uint32)]
    remap_oracle([(2, 2)], tl.tensors, tl.slices, rl.tensors, rl.slices, good)
    bad = [np.arange(4, dtype=np.uint32), np.array([0, 1, 2, 9], dtype=np.uint32)]
    with pytest.raises(ReplicaMismatchError):
        remap_oracle([(2, 2)], tl.tensors, tl.slices, rl.tensors, rl.slices, bad)


# ---- the per-element resolver agrees with the whole-tensor pass ----------------------------------
@pytest.mark.parametrize("name,scale", [("cfg1b", "full"), ("cfg3", "small"), ("cfg4", "small"), ("cfg5", "small")])
def test_single_element_resolver(name, scale):
    wl = make_workload(name, scale)
    src = [to_bits(t) for t in wl.trainer_weights()]
    res = run_oracle(wl, src)
    t_ids, r_ids = probe_ids(wl, "trainer"), probe_ids(wl, "rollout")
    base = wl.ckpt_base()
    index = SampleIndex(wl.trainer.slices, wl.rollout.slices)
    rng = np.random.default_rng(2)
    for _ in range(3000):
        k = int(rng.integers(0, wl.rollout.n_tensors))
        x = int(rng.integers(0, int(wl.rollout.tensors[k]["numel"])))
        got = source_of_rollout_element(index, k, x)
        if r_ids[k][x] < 0:
            assert got is None
            continue
        t, r, c, st, y = got
        assert base[t] + r * wl.ckpt[t].cols + c == r_ids[k][x]      # right id
        assert t_ids[st][y] == r_ids[k][x]                            # a trainer element with that id
    # padding of a flat shard resolves to "undescribed" on the trainer side of the inverse
    inv = SampleIndex(wl.rollout.slices, wl.trainer.slices)
    for k in range(wl.trainer.n_tensors):
        pads = np.nonzero(t_ids[k] < 0)[0]
        for x in pads[:3]:
            assert source_of_rollout_element(inv, k, int(x)) is None


# ---- checkpoint format -----------------------------------------------------------------------------
@pytest.mark.parametrize("name,scale", [("cfg1b", "full"), ("cfg4", "small"), ("cfg5", "small")])
def test_checkpoint_view_recovers_the_seeded_checkpoint(name, scale):
    wl = make_workload(name, scale)
    src = [to_bits(t) for t in wl.trainer_weights()]
    for t in range(0, len(wl.ckpt), max(1, len(wl.ckpt) // 25)):
        bits, held = checkpoint_view(t, (wl.ckpt[t].rows, wl.ckpt[t].cols), wl.trainer.slices, src)
        assert held.all()
        assert np.array_equal(bits.reshape(-1), to_bits(wl.ckpt_values(t)))


# ---- fuzz: random affine source maps against a dictionary join --------------------------------------
@pytest.mark.parametrize("seed", range(200))
def test_fuzz_against_dictionary_join(seed):
    src_dt, dst_dt = [(WB_F32, WB_BF16), (WB_BF16, WB_BF16), (WB_F32, WB_F32), (WB_BF16, WB_F32)][seed % 4]
    shapes, tl, rl = fuzz_case(1000 + seed, src_dt, dst_dt)
    rng = np.random.default_rng(seed)
    ck_bits = [random_bits(rng, r * c, src_dt) for (r, c) in shapes]
    src = scatter_checkpoint(tl, ck_bits)
    res = remap_oracle(shapes, tl.tensors, tl.slices, rl.tensors, rl.slices, src)
    # dictionary join, one element at a time
    holder = {}
    for s in tl.slices:
        for i in range(int(s["nr"])):
            for j in range(int(s["nc"])):
                key = (int(s["ckpt"]), int(s["r0"]) + i, int(s["c0"]) + j)
                y = int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])
                holder.setdefault(key, src[int(s["tensor"])][y])
    want = [np.zeros(int(t["numel"]), dtype=np.uint16 if dst_dt == WB_BF16 else np.uint32) for t in rl.tensors]
    for s in rl.slices:
        for i in range(int(s["nr"])):
            for j in range(int(s["nc"])):
                key = (int(s["ckpt"]), int(s["r0"]) + i, int(s["c0"]) + j)
                x = int(s["local_off"]) + i * int(s["stride_r"]) + j * int(s["stride_c"])
                v = from_bits(np.array([holder[key]]))
                want[int(s["tensor"])][x] = torch_cast_bits(v, dst_dt)[0]
    for a, b in zip(res.dst, want):
        assert np.array_equal(a, b)
