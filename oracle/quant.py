"""FP8 quantisation of a transfer bucket (test infrastructure).

Section 5 of the paper ("Parameter precision mismatch") only sketches this step: trainer tensors
are quantised before the transfer, which needs the full tensor gathered first, so in every round
the trainers first gather the shards of the tensors that are to be quantised.  It fixes no
quantisation rule.  The reading taken here (parity unpinned by the paper, pinned to the arithmetic
below):

  format   FP8 E4M3 (4 exponent bits, bias 7, 3 mantissa bits, no infinities, largest finite
           value 448, NaN = S.1111.111).
  scale    one per checkpoint tensor: s = amax / 448 and its counterpart r = 448 / amax, both one
           fp32 division, amax the largest magnitude of the tensor's elements in the destination
           dtype (the "gather"); s = r = 1 if amax = 0.  A quotient amax / 448 that rounds to zero
           (amax at most 224 units of the smallest subnormal) is replaced by the smallest subnormal,
           2^-149, so that s is never zero for a tensor that is not.
  encode   q = e4m3(x * r): fp32 multiplication with the reciprocal scale (the convention of FP8
           training libraries: one division per tensor, none per element), round to nearest with
           ties to even, magnitudes beyond the largest finite value saturate to it, NaN -> 0x7F.
           The rule must be total: for amax below 448 / FLT_MAX (about 1.3e-36, still a normal
           number) r overflows to infinity, which would turn every zero into NaN and every other
           element into +-amax.  A tensor whose r is not finite is therefore encoded by division,
           q = e4m3(x / s), which is finite for every element because s is not zero.  (A NaN amax
           keeps r and s NaN: the whole tensor is NaN either way.)
  decode   x' = cast_dst(value(q) * s): fp32 multiplication, then the destination dtype's rounding.

The quantised object is the bucket payload (checkpoint format, destination dtype), so for an
fp32 -> bf16 transfer the value quantised is the bf16 one.
"""
import numpy as np

from .cast import f32_to_bf16_bits, bf16_to_f32_bits, F32, BF16

E4M3_MAX = 448.0
E4M3_NAN = 0x7F


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """Value of every E4M3 code as float32 (exact); S.1111.111 is NaN."""
    c = np.asarray(codes).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 7
    normal = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    sub = (m / 8.0) * 2.0 ** -6
    v = np.where(e == 0, sub, normal)
    v = np.where((e == 15) & (m == 7), np.nan, v)
    return (sign * v).astype(np.float32)


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """float32 values -> E4M3 codes: nearest representable value, ties to the even code, saturating
    at +-448, NaN -> 0x7F.  Works in float64, where fp32 values, the spacing of the target grid
    (a power of two) and their quotient are all exact."""
    x = np.asarray(x, dtype=np.float32)
    a = np.abs(x.astype(np.float64))
    nan = np.isnan(a)
    a = np.where(nan, 0.0, a)
    a = np.minimum(a, 1e30)                                   # infinities saturate below
    _, ex = np.frexp(np.maximum(a, 2.0 ** -20))               # a = f * 2^ex, f in [0.5, 1)
    e = np.maximum(ex - 1, -6)                                # binade of a, not below the smallest normal one
    quantum = np.exp2((e - 3).astype(np.float64))             # spacing of representable values there
    v = np.rint(a / quantum) * quantum                        # rint: half to even; a carry lands on the next binade
    v = np.minimum(v, E4M3_MAX)
    # value -> code
    _, vx = np.frexp(np.maximum(v, 2.0 ** -20))
    ve = vx - 1
    is_sub = v < 2.0 ** -6
    code_sub = np.rint(v / 2.0 ** -9).astype(np.int64)        # 0..7
    mant = np.rint((v / np.exp2(ve.astype(np.float64)) - 1.0) * 8.0).astype(np.int64)
    code_norm = ((ve + 7) << 3) | mant
    code = np.where(is_sub, code_sub, code_norm)
    code = np.where(np.signbit(x), code | 0x80, code)
    code = np.where(nan, E4M3_NAN, code)
    return code.astype(np.uint8)


def to_f32(bits: np.ndarray, dtype: int) -> np.ndarray:
    """Destination-dtype bit patterns as float32 values (bf16 widens exactly)."""
    if dtype == F32:
        return np.asarray(bits, dtype=np.uint32).view(np.float32)
    return bf16_to_f32_bits(bits).view(np.float32)


def from_f32(v: np.ndarray, dtype: int) -> np.ndarray:
    u = np.asarray(v, dtype=np.float32).view(np.uint32)
    return u.copy() if dtype == F32 else f32_to_bf16_bits(u)


def amax_bits(bits: np.ndarray, dtype: int) -> np.uint32:
    """Largest magnitude as an fp32 bit pattern, compared as unsigned integers of the sign-cleared
    patterns (so a NaN, whose pattern exceeds infinity's, wins: the tensor then has no scale)."""
    if np.asarray(bits).size == 0:
        return np.uint32(0)
    u = to_f32(bits, dtype).view(np.uint32) & np.uint32(0x7FFFFFFF)
    return np.uint32(u.max())


def scale_of(amax: np.uint32) -> np.float32:
    """The scale amax / 448 (fp32 division; 1 for an all-zero tensor; never zero otherwise: a
    quotient that rounds to zero becomes the smallest subnormal)."""
    a = np.array([amax], np.uint32).view(np.float32)[0]
    if a == 0:
        return np.float32(1.0)
    with np.errstate(invalid="ignore", under="ignore"):
        s = np.float32(a / np.float32(E4M3_MAX))
    if s == 0:
        s = np.array([1], np.uint32).view(np.float32)[0]          # 2^-149
    return s


def rscale_of(amax: np.uint32) -> np.float32:
    """The reciprocal scale 448 / amax (fp32 division; 1 for an all-zero tensor)."""
    a = np.array([amax], np.uint32).view(np.float32)[0]
    if a == 0:
        return np.float32(1.0)
    with np.errstate(invalid="ignore", divide="ignore", over="ignore"):
        return np.float32(np.float32(E4M3_MAX) / a)


def quantize(bits: np.ndarray, dtype: int, scale: np.float32, rscale: np.float32) -> np.ndarray:
    """Codes of a tensor's elements: x * rscale, or x / scale when rscale is not finite (a tensor
    of tiny magnitudes, or one that holds a NaN)."""
    x = to_f32(bits, dtype)
    with np.errstate(invalid="ignore", over="ignore", under="ignore", divide="ignore"):
        y = x * np.float32(rscale) if np.isfinite(rscale) else x / np.float32(scale)
    return e4m3_encode(y)


def dequantize(codes: np.ndarray, dtype: int, scale: np.float32) -> np.ndarray:
    with np.errstate(invalid="ignore", over="ignore", under="ignore"):
        v = e4m3_decode(codes) * np.float32(scale)
    return from_f32(v, dtype)
