"""Element casts of the remap, on raw bit patterns (test infrastructure).

The paper moves weights between equal precisions (Section 3.1 requires load_weights to
preserve same-dtype values; Section 5 "Parameter precision mismatch" leaves anything
else to future work).  The benchmark adds an elementwise fp32 -> bf16 narrowing with
round-to-nearest, ties-to-even; it needs no gather, so it does not conflict with the
paper's traffic argument.
"""
import numpy as np

F32 = 0
BF16 = 1

BF16_CANONICAL_NAN = 0x7FFF


def f32_to_bf16_bits(u32: np.ndarray) -> np.ndarray:
    """fp32 bit patterns -> bf16 bit patterns, round to nearest, ties to even.

    Integer form: add 0x7FFF plus the lowest kept bit, then drop 16 bits.  The carry
    out of the mantissa bumps the exponent, so rounding up to the next binade and
    overflow to +-Inf fall out of the addition; subnormals round like everything else;
    the sign bit is never touched.  Every NaN maps to the canonical 0x7FFF (our reading,
    chosen to equal what the sm_100 `cvt.rn.bf16x2.f32` instruction returns).
    """
    u = np.asarray(u32).astype(np.uint64)
    is_nan = (u & 0x7FFFFFFF) > 0x7F800000
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    out = np.where(is_nan, np.uint64(BF16_CANONICAL_NAN), rounded)
    return out.astype(np.uint16)


def bf16_to_f32_bits(u16: np.ndarray) -> np.ndarray:
    """bf16 -> fp32 widening is exact: the bf16 pattern becomes the high half."""
    return (np.asarray(u16).astype(np.uint32) << 16).astype(np.uint32)


def cast_bits(bits: np.ndarray, src_dtype: int, dst_dtype: int) -> np.ndarray:
    if src_dtype == dst_dtype:
        return np.asarray(bits).copy()           # same dtype: pure bit copy
    if src_dtype == F32 and dst_dtype == BF16:
        return f32_to_bf16_bits(bits)
    if src_dtype == BF16 and dst_dtype == F32:
        return bf16_to_f32_bits(bits)
    raise ValueError((src_dtype, dst_dtype))
