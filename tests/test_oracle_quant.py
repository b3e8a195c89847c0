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


def _round_to_f32(q: Fraction) -> float:
    """A non-negative rational rounded to the nearest fp32 value, ties to the even mantissa, in integer
    arithmetic (subnormals included; beyond the largest finite value -> inf)."""
    if q == 0:
        return 0.0
    e = q.numerator.bit_length() - q.denominator.bit_length()       # 2^(e-1) < q < 2^(e+1)
    if Fraction(2) ** e > q:
        e -= 1                                                      # now 2^e <= q < 2^(e+1)
    quantum = Fraction(2) ** (max(e, -126) - 23)                    # spacing of fp32 values in q's binade
    n, rem = divmod(q, quantum)
    n = int(n)
    if rem * 2 > quantum or (rem * 2 == quantum and n % 2 == 1):
        n += 1
    v = n * quantum
    if v >= Fraction(2) ** 128:
        return float("inf")
    return float(v)                                                 # exact: v is an fp32 value


def _f32(bits: int) -> np.float32:
    return np.array([bits], np.uint32).view(np.float32)[0]


# magnitudes across the whole fp32 range: smallest subnormal, subnormals around the point where amax / 448
# rounds to zero, largest subnormal, smallest normal, around 448 / FLT_MAX (where 448 / amax overflows),
# ordinary values, powers of two, the largest finite value
AMAX_BITS = [1, 2, 100, 223, 224, 225, 226, 447, 448, 449, 1000, 0x0007FFFF, 0x007FFFFF, 0x00800000, 0x00800001,
             int(np.float32(1e-37).view(np.uint32)), 0x03000000, 0x03DFFFFF, 0x03E00000, 0x03E00001, 0x03E00002, 0x04000000,
             0x3CA3D70A, 0x3F800000, 0x3F800001, 0x43E00000, 0x43E00001, 0x7F000000, 0x7F7FFFFF]


def test_scale_and_reciprocal_are_the_correctly_rounded_quotients():
    rng = np.random.default_rng(14)
    cases = AMAX_BITS + [int(b) for b in rng.integers(1, 0x7F800000, 400)]
    for b in cases:
        a = Fraction(float(_f32(b)))
        s, r = quant.scale_of(np.uint32(b)), quant.rscale_of(np.uint32(b))
        assert s.dtype == np.float32 and r.dtype == np.float32
        want_s = _round_to_f32(a / 448)
        if want_s == 0.0:
            want_s = 2.0 ** -149                 # never zero for a tensor that is not
        assert float(s) == want_s, hex(b)
        assert float(r) == _round_to_f32(Fraction(448) / a), hex(b)
        assert s > 0
    # the threshold of the division rule: 448 / amax is finite above 1.75 * 2^-120 = 448 / 2^128
    assert np.isinf(quant.rscale_of(np.uint32(0x03E00000))) and np.isfinite(quant.rscale_of(np.uint32(0x03E00001)))


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_zero_stays_zero_and_amax_stays_amax_for_every_scale(dtype):
    """The rule is total: whatever the tensor's magnitude, zeros come back as zeros (sign kept), nothing
    becomes NaN or infinite, and the largest element comes back within E4M3's resolution."""
    for b in AMAX_BITS:
        if dtype == BF16:
            b &= 0xFFFF0000                      # a bf16 value
            if b == 0:
                continue
        a = float(_f32(b))
        vals = np.array([0.0, -0.0, a, -a, a / 2, -a / 3, a / 448, a / 1000], np.float32)
        bits = vals.view(np.uint32) if dtype == F32 else f32_to_bf16_bits(vals.view(np.uint32))
        vals = quant.to_f32(bits, dtype)
        amax = quant.amax_bits(bits, dtype)
        assert amax == b
        s, r = quant.scale_of(amax), quant.rscale_of(amax)
        q = quant.quantize(bits, dtype, s, r)
        assert q[0] == 0x00 and q[1] == 0x80, hex(b)
        assert ((q & 0x7F) != 0x7F).all(), hex(b)
        if float(s) >= 2.0 ** -140:              # (a subnormal s is itself rounded: by at most 2^-10 here)
            assert (q[2] & 0x7F) >= 0x7C, hex(b) # amax lands on one of the top codes (384 .. 448)
        back_bits = quant.dequantize(q, dtype, s)
        back = quant.to_f32(back_bits, dtype).astype(np.float64)
        assert back_bits[0] == 0 and back_bits[1] == (0x80000000 if dtype == F32 else 0x8000), hex(b)
        assert np.isfinite(back).all(), hex(b)
        assert abs(back[2] - a) <= a / 8 + 2.0 ** -149, (hex(b), back[2], a)
        assert np.array_equal(np.signbit(back), np.signbit(vals))


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_round_trip_error_over_the_whole_range(dtype):
    """Tensors whose magnitude is drawn log-uniformly from the whole fp32 range, elements N(0, 1) times it:
    E4M3 keeps 4 significant bits, so the relative error is at most 2^-4 for normal codes and the absolute
    error at most s * 2^-10 below; a subnormal s carries a relative error of its own of at most 2^-150 / s,
    which shows when the largest elements saturate, and the destination dtype rounds once more
    (relatively, or by half a subnormal step)."""
    rng = np.random.default_rng(13)
    eps_dst = 2.0 ** -24 if dtype == F32 else 2.0 ** -9
    tiny_dst = 2.0 ** -149 if dtype == F32 else 2.0 ** -134      # half a subnormal step of the destination dtype, at least
    for trial in range(120):
        mag = 2.0 ** rng.uniform(-149, 125) if trial else 0.02
        v = (rng.normal(0, 1, 4000) * mag).astype(np.float32)
        bits = v.view(np.uint32) if dtype == F32 else f32_to_bf16_bits(v.view(np.uint32))
        vals = quant.to_f32(bits, dtype)
        if not np.isfinite(vals).all() or not vals.any():
            continue
        amax = quant.amax_bits(bits, dtype)
        assert _f32(int(amax)) == np.abs(vals).max()
        s, r = quant.scale_of(amax), quant.rscale_of(amax)
        q = quant.quantize(bits, dtype, s, r)
        assert (q & 0x7F).max() <= 0x7E                          # nothing overflows or turns NaN
        if float(s) >= 2.0 ** -126:
            assert (q[np.argmax(np.abs(vals))] & 0x7F) == 0x7E   # the largest element lands on the largest code
        back = quant.to_f32(quant.dequantize(q, dtype, s), dtype).astype(np.float64)
        err = np.abs(back - vals.astype(np.float64))
        rel = 2.0 ** -4 + 2.0 ** -149 / float(s) + eps_dst
        bound = np.maximum(np.abs(vals) * rel, float(s) * 2.0 ** -10) * 1.001 + tiny_dst + np.abs(back) * eps_dst
        assert (err <= bound).all(), (trial, mag, float(np.max(err / bound)))


def test_degenerate_scales():
    assert quant.scale_of(np.uint32(0)) == np.float32(1.0)                       # all-zero tensor
    zeros = np.zeros(8, np.uint16)
    assert quant.rscale_of(np.uint32(0)) == np.float32(1.0)
    a0 = quant.amax_bits(zeros, BF16)
    assert quant.quantize(zeros, BF16, quant.scale_of(a0), quant.rscale_of(a0)).tolist() == [0] * 8
    nan_bits = np.array([0x3F80, 0x7FC0, 0xBF80], np.uint16)                      # 1, NaN, -1 in bf16
    amax = quant.amax_bits(nan_bits, BF16)
    assert amax > 0x7F800000                                                      # the NaN wins the maximum
    q = quant.quantize(nan_bits, BF16, quant.scale_of(amax), quant.rscale_of(amax))
    assert q.tolist() == [0x7F, 0x7F, 0x7F]                                       # no scale: everything is NaN
    assert quant.amax_bits(np.zeros(0, np.uint16), BF16) == 0
    # the example that a reciprocal-only rule gets wrong: zeros must not become NaN, small elements must
    # not all saturate to +-amax
    tiny = np.float32([0.0, 1e-37, -5e-38, 2e-38]).view(np.uint32)
    a = quant.amax_bits(tiny, F32)
    s, r = quant.scale_of(a), quant.rscale_of(a)
    q = quant.quantize(tiny, F32, s, r)
    assert q.tolist() == [0x00, 0x7E, 0xF6, 0x6B]            # 0, 448, -224, 89.6 -> 88 (x / s, s = 1e-37 / 448)
    back = quant.dequantize(q, F32, s).view(np.float32)
    assert back[0] == 0 and np.allclose(back[1:], [1e-37, -5e-38, 2e-38], rtol=2.0 ** -4, atol=0)
