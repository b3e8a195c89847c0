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
