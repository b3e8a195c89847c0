"""Difference encoding of an id field (test infrastructure).

Appendix B of the paper ("Difference encoding"): let A be the identifier field of an in-GPU
tensor, A[i, j] = the checkpoint position that supplies element (i, j), viewed as 2-D, with
A = 0 outside the tensor.  Eq. (diff1):

    diff1(A)[i, j] = A[i, j] - A[i-1, j] - A[i, j-1] + A[i-1, j-1]

and Eq. (diff2): diff2 = diff1(diff1(A)).  diff1 is inverted by a 2-D prefix sum, so diff2 is
lossless.  Over a rectangle filled by one slice-copy operation the field is affine (with or
without transposition), so diff2 vanishes except in a constant-size neighbourhood of the
rectangle's corners.  Chunked ids (Algorithm 1, MakeIdChunk): chunk k of width b of position p
is floor(p / 2^(b k)) mod 2^b, and by linearity sum_k 2^(b k) diff2(chunk_k) = diff2(ids)
(Algorithm 1, Recombine).

Ids here start at 1 so that 0 means "no source" (padding).
"""
import numpy as np


def diff1(a: np.ndarray) -> np.ndarray:
    """Eq. (diff1), written out with the zero convention for negative indices."""
    a = np.asarray(a, dtype=np.int64)
    out = a.copy()
    out[1:, :] -= a[:-1, :]
    out[:, 1:] -= a[:, :-1]
    out[1:, 1:] += a[:-1, :-1]
    return out


def diff2(a: np.ndarray) -> np.ndarray:
    """Eq. (diff2): diff1 applied twice."""
    return diff1(diff1(a))


def undo_diff2(d: np.ndarray) -> np.ndarray:
    """Inverse of diff2: two 2-D prefix sums."""
    x = np.asarray(d, dtype=np.int64)
    for _ in range(2):
        x = np.cumsum(np.cumsum(x, axis=0), axis=1)
    return x


def nonzeros(d: np.ndarray):
    """(row, col, value) of the non-zero entries, sorted by (row, col)."""
    r, c = np.nonzero(d)
    return [(int(i), int(j), int(d[i, j])) for i, j in zip(r, c)]


def id_chunk(ids: np.ndarray, k: int, b: int) -> np.ndarray:
    """Algorithm 1, MakeIdChunk: floor(p / 2^(b k)) mod 2^b."""
    return (np.asarray(ids, dtype=np.int64) >> (b * k)) & ((1 << b) - 1)


def recombine(chunk_diffs, b: int) -> np.ndarray:
    """Algorithm 1, Recombine: sum_k 2^(b k) * diff2(chunk_k)."""
    out = np.zeros_like(np.asarray(chunk_diffs[0], dtype=np.int64))
    for k, d in enumerate(chunk_diffs):
        out += np.asarray(d, dtype=np.int64) << (b * k)
    return out


# ---- Algorithm 1, inner loop: chunk passes with carries -------------------------------------------
# The paper only sketches this part (Appendix B, last two paragraphs of "Difference encoding"): diff2 of
# a truncated id chunk overflows at regularly spaced positions, the overflow has to be carried into
# the next chunk, and a strided difference over the diff2 tensors cancels the periodic artifacts so
# that O(N_c) entries remain.  The reading written out here (parity unpinned by the paper, pinned to
# Recombine(H_Z) = diff2(full ids)):
#
#   A_k = chunk k of the ids, so ids = sum_k 2^(bk) A_k and diff2(ids) = sum_k 2^(bk) diff2(A_k).
#   That sum is evaluated like a multi-digit addition, least significant chunk first:
#     D_k = diff2(A_k) + Gamma_k              Gamma_0 = 0, Gamma_k = the carry out of pass k-1
#     EmitCarry(D_k) splits D_k = Z_k + 2^b C_k, Z_k the balanced b-bit digit in [-2^(b-1), 2^(b-1))
#     H_Z[k] = NonZeros(Z_k),  H_Gamma[k] = NonZeros(StridedDiff1(C_k)),  Gamma_(k+1) = C_k
#   Wherever diff2(ids) = 0 every digit Z_k is 0 (induction: D_k is a multiple of 2^b there), so the
#   Z_k are the balanced digits of the O(N_c) entries of diff2(ids).  The carries C_k are not sparse:
#   they are non-zero wherever chunk k wraps, every s_k = 2^(b(k+1)) consecutive ids of a run.  Along a
#   run of consecutive ids - which continues from one row into the next when a rectangle spans the full
#   width of its tensor - those positions have period s_k in the row-major flat index x = i * cols + j,
#   and when the id pitch between rows is a multiple of s_k every row repeats the one above.  So
#   StridedDiff1 is Eq. (diff1) with the left neighbour s_k elements back in flat order and the upper
#   neighbour s_k rows up:
#       G[x] = C[x] - C[x - s_k] - C[x - s_k cols] + C[x - s_k - s_k cols]      (C = 0 before the tensor)
#   It vanishes inside a slice-copy rectangle except, for a rectangle narrower than its tensor whose id
#   pitch is not a multiple of s_k, in its first s_k rows and columns.  ExpandCarry is the inverse: a
#   prefix sum over every s_k-th element of the flat order, then over every s_k-th row.


def emit_carry(d: np.ndarray, b: int):
    """Algorithm 1, EmitCarry: D = Z + 2^b C with Z the balanced b-bit digit.  Returns (Z, C)."""
    d = np.asarray(d, dtype=np.int64)
    half = 1 << (b - 1)
    z = ((d + half) & ((1 << b) - 1)) - half
    return z, (d - z) >> b


def carry_stride(b: int, k: int) -> int:
    """Spacing of the wraps of chunk k along a run of consecutive ids."""
    return 1 << (b * (k + 1))


def _shifted(flat: np.ndarray, t: int) -> np.ndarray:
    """flat[x - t], zero where x < t."""
    out = np.zeros_like(flat)
    if t < flat.size:
        out[t:] = flat[:flat.size - t]
    return out


def strided_diff1(c: np.ndarray, s: int) -> np.ndarray:
    """Algorithm 1, StridedDiff1: Eq. (diff1) with the left neighbour s elements back in row-major flat
    order and the upper neighbour s rows up (zero before the start of the tensor)."""
    c = np.asarray(c, dtype=np.int64)
    flat = c.reshape(-1)
    up = s * c.shape[1]
    return (flat - _shifted(flat, s) - _shifted(flat, up) + _shifted(flat, s + up)).reshape(c.shape)


def _strided_prefix(flat: np.ndarray, t: int) -> np.ndarray:
    """y[x] = flat[x] + y[x - t]: a running sum over every t-th element."""
    if t >= flat.size:
        return flat.copy()
    pad = (-flat.size) % t
    blocks = np.concatenate([flat, np.zeros(pad, flat.dtype)]).reshape(-1, t)
    return np.cumsum(blocks, axis=0).reshape(-1)[:flat.size]


def expand_carry(g: np.ndarray, s: int) -> np.ndarray:
    """Algorithm 1, ExpandCarry: the inverse of strided_diff1."""
    g = np.asarray(g, dtype=np.int64)
    flat = _strided_prefix(g.reshape(-1), s)
    return _strided_prefix(flat, s * g.shape[1]).reshape(g.shape)


def chunk_passes(ids: np.ndarray, b: int, n_passes: int):
    """Algorithm 1, the loop over k for one tensor.  Returns (H_Z, H_Gamma, last carry): the digit
    fields Z_k and the strided differences of the carries, one per pass, as dense arrays (the caller
    takes their non-zeros), and the carry out of the last pass (zero when n_passes * b bits hold
    diff2(ids))."""
    h_z, h_gamma = [], []
    gamma = None
    for k in range(n_passes):
        a = id_chunk(ids, k, b)                       # load_weights(MakeIdChunk(k, b))
        d = diff2(a)
        if k > 0:                                     # D <- D + ExpandCarry(H_Gamma[k-1])
            d = d + expand_carry(h_gamma[k - 1], carry_stride(b, k - 1))
        z, gamma = emit_carry(d, b)
        h_z.append(z)
        h_gamma.append(strided_diff1(gamma, carry_stride(b, k)))
    return h_z, h_gamma, gamma
