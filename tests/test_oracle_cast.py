"""Pins for the oracle's casts: exact rational arithmetic, the torch CPU cast as a
library routine (non-NaN inputs), and a hand-worked special-value table."""
import os
from fractions import Fraction

import numpy as np
import torch

from oracle.cast import BF16, F32, bf16_to_f32_bits, cast_bits, f32_to_bf16_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "cast_special_values.txt")


def _bf16_value(p: int) -> Fraction:
    """Exact value of a finite bf16 pattern; the Inf pattern counts as 2^128, the value
    IEEE rounding compares against when deciding overflow."""
    sign = -1 if p & 0x8000 else 1
    e = (p >> 7) & 0xFF
    m = p & 0x7F
    if e == 0xFF:
        assert m == 0
        return sign * Fraction(2) ** 128
    if e == 0:
        return sign * Fraction(m, 128) * Fraction(2) ** -126
    return sign * (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)


def _nearest_even(u: int) -> int:
    """RNE by exact comparison of the two neighbouring bf16 values."""
    x = Fraction(float(np.array([u], dtype=np.uint32).view(np.float32)[0]))
    lo = u >> 16                       # truncation toward zero (same sign)
    hi = lo + 1                        # next pattern away from zero
    dlo = abs(x - _bf16_value(lo))
    dhi = abs(_bf16_value(hi) - x)
    if dlo < dhi:
        return lo
    if dhi < dlo:
        return hi
    return lo if lo % 2 == 0 else hi


def test_rne_against_exact_rationals():
    rng = np.random.default_rng(7)
    pats = rng.integers(0, 1 << 32, size=4000, dtype=np.uint64).astype(np.uint32)
    # dense coverage around ties and binade edges
    hi = rng.integers(0, 1 << 16, size=600, dtype=np.uint64).astype(np.uint32) << 16
    edge = np.concatenate([hi | 0x7FFF, hi | 0x8000, hi | 0x8001, hi | 0xFFFF, hi])
    pats = np.concatenate([pats, edge])
    finite = (pats & 0x7F800000) != 0x7F800000
    pats = pats[finite]
    got = f32_to_bf16_bits(pats)
    for u, g in zip(pats.tolist(), got.tolist()):
        assert g == _nearest_even(u), hex(u)


def test_matches_torch_cpu_on_non_nan():
    rng = np.random.default_rng(11)
    lows = np.array([0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x4000, 0xC000] +
                    rng.integers(0, 1 << 16, size=24).tolist(), dtype=np.uint32)
    highs = np.arange(1 << 16, dtype=np.uint32) << 16
    pats = (highs[:, None] | lows[None, :]).reshape(-1)
    pats = np.concatenate([pats, rng.integers(0, 1 << 32, size=1 << 21, dtype=np.uint64).astype(np.uint32)])
    not_nan = (pats & 0x7FFFFFFF) <= 0x7F800000
    pats = pats[not_nan]
    ref = torch.from_numpy(pats.view(np.int32)).view(torch.float32).to(torch.bfloat16)
    ref = ref.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(f32_to_bf16_bits(pats), ref)


def test_special_value_table():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b = line.split()[:2]
            rows.append((int(a, 16), int(b, 16)))
    assert len(rows) >= 25
    got = f32_to_bf16_bits(np.array([r[0] for r in rows], dtype=np.uint32))
    for (u, want), g in zip(rows, got.tolist()):
        assert g == want, hex(u)


def test_every_nan_is_canonical():
    rng = np.random.default_rng(3)
    mant = rng.integers(1, 1 << 23, size=10000, dtype=np.uint64).astype(np.uint32)
    for sign in (0, 0x80000000):
        pats = (np.uint32(sign) | np.uint32(0x7F800000) | mant).astype(np.uint32)
        assert (f32_to_bf16_bits(pats) == 0x7FFF).all()


def test_widening_is_exact_and_inverts_narrowing():
    all16 = np.arange(1 << 16, dtype=np.uint16)
    wide = bf16_to_f32_bits(all16)
    ref = torch.from_numpy(all16.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32)
    ref = ref.view(torch.int32).numpy().view(np.uint32)
    nan = (all16 & 0x7FFF) > 0x7F80
    assert np.array_equal(wide[~nan], ref[~nan])
    assert np.array_equal(f32_to_bf16_bits(wide)[~nan], all16[~nan])


def test_same_dtype_is_a_bit_copy():
    all16 = np.arange(1 << 16, dtype=np.uint16)
    assert np.array_equal(cast_bits(all16, BF16, BF16), all16)
    rng = np.random.default_rng(5)
    p = rng.integers(0, 1 << 32, size=1 << 16, dtype=np.uint64).astype(np.uint32)
    assert np.array_equal(cast_bits(p, F32, F32), p)
