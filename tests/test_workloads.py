"""The workload generators: slice lists against the procedural load_weights (id probe,
Section 3.1), byte totals, and the stress recipe."""
import numpy as np
import pytest
import torch

from helpers import predict_ids, probe_ids
from wb_workloads import make_workload
from wb_workloads.configs import _chunk_bounds, flat_range_rects

SMALL = [("cfg1", "full"), ("cfg1b", "full"), ("cfg1c", "full"), ("cfg2", "small"),
         ("cfg3", "small"), ("cfg4", "small"), ("cfg5", "small")]


@pytest.mark.parametrize("name,scale", SMALL)
@pytest.mark.parametrize("side", ["trainer", "rollout"])
def test_id_probe_matches_slice_list(name, scale, side):
    wl = make_workload(name, scale)
    lay = wl.trainer if side == "trainer" else wl.rollout
    pred = predict_ids(lay, wl)
    got = probe_ids(wl, side)
    for k, (p, g) in enumerate(zip(pred, got)):
        assert np.array_equal(p, g), (name, side, lay.names[k])


def test_padding_is_exercised_by_cfg1b():
    wl = make_workload("cfg1b")
    pad = sum(int((p < 0).sum()) for p in predict_ids(wl.trainer, wl))
    assert pad > 0
    wl1 = make_workload("cfg1")
    assert sum(int((p < 0).sum()) for p in predict_ids(wl1.trainer, wl1)) == 0


def test_full_size_byte_totals():
    # model sizes: 8B shape = 8,030,261,248 parameters; the 30B-A3B shape = 30,532,110,336
    # parameters = 61.06 GB in bf16 (Table 2 of the paper lists 30.5 B / 61.1 GB)
    wl2 = make_workload("cfg2", "full")
    assert wl2.ckpt_numel() == 8_030_261_248
    assert wl2.algorithmic_bytes() == (16_060_522_496, 16_060_522_496)
    wl3 = make_workload("cfg3", "full")
    r, w = wl3.algorithmic_bytes()
    assert r == 32_121_044_992
    assert w == 16_060_522_496 + 65 * 4096 * 2      # norms written on both rollout ranks
    wl4 = make_workload("cfg4", "full")
    assert len(wl4.ckpt) == 18_771
    assert wl4.ckpt_numel() == 30_532_110_336
    assert wl4.algorithmic_bytes() == (61_064_220_672, 61_064_220_672)


def test_cfg1_shapes():
    wl = make_workload("cfg1")
    assert wl.ckpt_numel() == 1_975_552
    names = wl.rollout.names
    qkv = wl.rollout.tensors[names.index("r0.layers.0.qkv_proj")]
    assert int(qkv["numel"]) == (4 + 2 + 2) * 64 * 256
    gu = wl.rollout.tensors[names.index("r0.layers.0.gate_up_proj")]
    assert int(gu["numel"]) == 2 * 688 * 256
    assert set(int(t["rank"]) for t in wl.trainer.tensors) == {0, 1, 2, 3}


def test_chunk_bounds_follow_torch_chunk():
    for n in (1, 2, 7, 16, 17, 100):
        for k in range(2, 9):
            ours = [e - b for b, e in _chunk_bounds(n, k)]
            ref = [c.numel() for c in torch.arange(n).chunk(k)]
            assert ours == ref, (n, k)
    assert [e - b for b, e in _chunk_bounds(17, 8)] == [3, 3, 3, 3, 3, 2]


def test_flat_range_rects_cover_the_range():
    for cols in (1, 3, 7):
        for b in range(0, 25):
            for e in range(b, 30):
                cells = []
                for (r0, c0, nr, nc, f) in flat_range_rects(cols, b, e):
                    assert f == r0 * cols + c0
                    for i in range(nr):
                        for j in range(nc):
                            cells.append((r0 + i) * cols + c0 + j)
                assert cells == list(range(b, e))


def test_stress_recipe_is_deterministic_and_in_range():
    a = make_workload("cfg5", "small")
    b = make_workload("cfg5", "small")
    assert a.meta["recipe"] == b.meta["recipe"]
    assert np.array_equal(a.trainer.slices, b.trainer.slices)
    for (tk, tp, rk, rp, tr) in a.meta["recipe"]:
        assert tk != rk and tp != rp and 2 <= tp <= 8 and 2 <= rp <= 8
    frac = np.mean([r[4] for r in a.meta["recipe"]])
    assert 0.2 < frac < 0.4


def test_stress_full_shapes():
    wl = make_workload("cfg5", "full")
    assert len(wl.ckpt) == 4000
    for c in wl.ckpt:
        assert 16 <= c.rows < 8192 and 16 <= c.cols < 8192 and c.rows * c.cols * 4 <= 1 << 26
