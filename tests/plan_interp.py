"""Host-side execution of a plan's tile tables with numpy, for checking the planner without
a GPU.  It follows only the documented meaning of a tile view (include/wb.h):
dst[dst_off + i*dst_sr + j*dst_sc] = cast(src[src_off + i*src_sr + j*src_sc])."""
import numpy as np

from oracle.cast import cast_bits
from paper_2609_25442_b200 import binding as wb


def _idx(off, nr, nc, sr, sc):
    i = np.arange(nr, dtype=np.int64)[:, None]
    j = np.arange(nc, dtype=np.int64)[None, :]
    return (int(off) + i * int(sr) + j * int(sc)).ravel()


def run_table(tiles, src_bufs, dst_bufs, bucket, src_dtype, dst_dtype, read_counts=None,
              write_counts=None, bucket_writes=None):
    """Execute tile views.  Tensor index -1 addresses `bucket` (elements of the bucket dtype)."""
    last = None
    for t in tiles:
        nr, nc = int(t["nr"]), int(t["nc"])
        cont = bool(int(t["flags"]) & wb.WB_TILE_FANOUT_CONT)
        if not cont:
            si = _idx(t["src_off"], nr, nc, t["src_sr"], t["src_sc"])
            sbuf = bucket if int(t["src_tensor"]) < 0 else src_bufs[int(t["src_tensor"])]
            assert si.min() >= 0 and si.max() < sbuf.size
            if read_counts is not None and int(t["src_tensor"]) >= 0:
                np.add.at(read_counts[int(t["src_tensor"])], si, 1)
            last = cast_bits(sbuf[si], src_dtype, dst_dtype)
        di = _idx(t["dst_off"], nr, nc, t["dst_sr"], t["dst_sc"])
        if int(t["dst_tensor"]) < 0:
            assert di.max() < bucket.size
            bucket[di] = last
            if bucket_writes is not None:
                np.add.at(bucket_writes, di, 1)
        else:
            dbuf = dst_bufs[int(t["dst_tensor"])]
            assert di.min() >= 0 and di.max() < dbuf.size
            dbuf[di] = last
            if write_counts is not None:
                np.add.at(write_counts[int(t["dst_tensor"])], di, 1)
