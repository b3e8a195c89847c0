"""Pins for the oracle's FP8 (E4M3) quantisation of a bucket: the format against its definition and
against torch's CPU float8 type, rounding against exact rational arithmetic, the scale rule."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle.cast import BF16, F32, f32_to_bf16_bits
from oracle import quant


def test_decode_is_the_format_definition_and_torchs_table():
    codes = np.arange(256, dtype=np.uint8)
    got = quant.e4m3_decode(codes)
    # definition: sign, 4-bit exponent with bias 7, 3-bit mantissa, subnormals at exponent 0
    for c in range(256):
        s, e, m = c >> 7, (c >> 3) & 15, c & 7
        if e == 15 and m == 7:
            assert np.isnan(got[c])
            continue
        v = Fraction(m, 8) * Fraction(1, 64) if e == 0 else (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7)
        assert Fraction(float(got[c])) == (-v if s else v), c
    assert float(np.nanmax(got)) == 448.0
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    assert np.array_equal(ref[~np.isnan(ref)], got[~np.isnan(got)])


def _nearest_even_code(x: Fraction, table):
    """Brute force over the non-negative finite codes: nearest value, ties to the even code."""
    best = None
    for c, v in table:
        d = abs(x - v)
        if best is None or d < best[0] or (d == best[0] and c % 2 == 0 and best[1] % 2 == 1):
            best = (d, c)
    return best[1]


def test_encode_rounds_to_nearest_even_exactly():
    table = [(c, Fraction(float(v))) for c, v in enumerate(quant.e4m3_decode(np.arange(127, dtype=np.uint8)))]
    rng = np.random.default_rng(11)
    xs = np.concatenate([
        rng.uniform(0, 448, 3000), rng.uniform(0, 2.0 ** -5, 2000), rng.uniform(0, 2.0 ** -8, 1000),
        # every midpoint between neighbouring codes and its two fp32 neighbours
        np.array([float((table[c][1] + table[c + 1][1]) / 2) for c in range(126)]),
    ]).astype(np.float32)
    mids = xs[-126:]
    xs = np.concatenate([xs, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(1000))])
    got = quant.e4m3_encode(xs)
    for x, g in zip(xs, got):
        assert g == _nearest_even_code(Fraction(float(x)), table), (float(x), int(g))
    # the sign is carried, zero keeps its sign
    assert np.array_equal(quant.e4m3_encode(-xs), got | 0x80)
    assert quant.e4m3_encode(np.float32([0.0, -0.0])).tolist() == [0x00, 0x80]


def test_encode_saturates_and_maps_nan():
    x = np.float32([448.0, 464.0, 464.1, 480.0, 1e9, np.inf, -np.inf, -500.0, np.nan])
    assert quant.e4m3_encode(x).tolist() == [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0xFE, 0x7F]


def test_encode_equals_torch_inside_the_finite_range():
    """torch's CPU cast to float8_e4m3fn rounds to nearest even too; it differs only beyond 464, where it
    gives NaN instead of saturating."""
    rng = np.random.default_rng(12)
    x = np.concatenate([rng.normal(0, 100, 200000), rng.normal(0, 0.01, 100000), rng.uniform(-464, 464, 100000)])
    x = x.astype(np.float32)
    x = x[np.abs(x) <= 464]
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(quant.e4m3_encode(x), ref)


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_scale_and_round_trip(dtype):
    rng = np.random.default_rng(13)
    v = rng.normal(0, 0.02, 50000).astype(np.float32)
    bits = v.view(np.uint32) if dtype == F32 else f32_to_bf16_bits(v.view(np.uint32))
    amax = quant.amax_bits(bits, dtype)
    vals = quant.to_f32(bits, dtype)
    assert np.array([amax], np.uint32).view(np.float32)[0] == np.abs(vals).max()
    s = quant.scale_of(amax)
    assert s == np.float32(np.abs(vals).max() / np.float32(448))
    r = quant.rscale_of(amax)
    assert r == np.float32(np.float32(448) / np.abs(vals).max())
    q = quant.quantize(bits, dtype, r)
    assert (q & 0x7F).max() <= 0x7E                          # nothing overflows: |x * r| <= 448 (1 + 2^-23)
    assert (q[np.argmax(np.abs(vals))] & 0x7F) == 0x7E       # the largest element lands on the largest code
    back = quant.to_f32(quant.dequantize(q, dtype, s), dtype)
    # E4M3 keeps 4 significant bits: relative error <= 2^-4 for normal codes, absolute <= s * 2^-10 below
    err = np.abs(back.astype(np.float64) - vals)
    bound = np.maximum(np.abs(vals) * 2.0 ** -4, float(s) * 2.0 ** -10) * 1.01 + 1e-12
    assert (err <= bound).all()


def test_degenerate_scales():
    assert quant.scale_of(np.uint32(0)) == np.float32(1.0)                       # all-zero tensor
    zeros = np.zeros(8, np.uint16)
    assert quant.rscale_of(np.uint32(0)) == np.float32(1.0)
    assert quant.quantize(zeros, BF16, quant.rscale_of(quant.amax_bits(zeros, BF16))).tolist() == [0] * 8
    nan_bits = np.array([0x3F80, 0x7FC0, 0xBF80], np.uint16)                      # 1, NaN, -1 in bf16
    amax = quant.amax_bits(nan_bits, BF16)
    assert amax > 0x7F800000                                                      # the NaN wins the maximum
    q = quant.quantize(nan_bits, BF16, quant.rscale_of(amax))
    assert q.tolist() == [0x7F, 0x7F, 0x7F]                                       # no scale: everything is NaN
    assert quant.amax_bits(np.zeros(0, np.uint16), BF16) == 0
