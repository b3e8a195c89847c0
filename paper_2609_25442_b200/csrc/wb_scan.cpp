// Source-map extraction, host part (Algorithm 1 of the paper: Recombine and ScanSliceMappings).
//
// The id field A of a local tensor is never materialised here.  Its diff2 entries D(p, q) determine
// it through two 2-D prefix sums:  A(i, j) = sum_{p<=i, q<=j} (i-p+1)(j-q+1) D(p, q).  The weight
// also vanishes for p = i+1 and q = j+1, so an entry may be counted one row / column early.  Grid
// lines are put at every row r such that r or r+1 carries an entry (same for columns); on the cell
// that starts at (r, c) the entries with p <= r+1, q <= c+1 are exactly the contributing ones, and
//     A(i, j) = (i+1)(j+1) S0 - (i+1) Sq - (j+1) Sp + Spq
// with S0 = sum D, Sp = sum p D, Sq = sum q D, Spq = sum p q D over them.  A field written by
// slice-copy operations is affine on every cell (S0 = 0 unless the cell is one row or one column
// thin); equal neighbouring cells are merged back into the rectangles the operations filled, and
// every rectangle is translated into checkpoint coordinates.
#include <algorithm>
#include <new>
#include <vector>

#include "wb_internal.h"

namespace {

typedef __int128 i128;

struct Affine {        // id(i, j) = a + b*i + c*j in absolute local coordinates
  i128 a, b, c;
  bool operator==(const Affine& o) const { return a == o.a && b == o.b && c == o.c; }
  bool zero() const { return a == 0 && b == 0 && c == 0; }
};

struct Seg { uint64_t j0, j1, i0; Affine f; };

struct Ckpts {
  const uint64_t* base; const uint64_t* rows; const uint64_t* cols; size_t n;
  // checkpoint tensor holding global position g (0-based)
  bool find(uint64_t g, size_t* t) const {
    if (n == 0 || g >= base[n]) return false;
    size_t lo = 0, hi = n;            // base[lo] <= g < base[hi]
    while (hi - lo > 1) {
      const size_t mid = (lo + hi) / 2;
      if (base[mid] <= g) lo = mid; else hi = mid;
    }
    *t = lo;
    return true;
  }
};

struct Emitter {
  wb_slice* out; size_t cap; size_t n = 0;
  uint32_t tensor; uint64_t elem_off, view_cols;
  void push(uint64_t local, int64_t sr, int64_t sc, const Ckpts& ck, size_t t, uint64_t r0, uint64_t c0,
            uint64_t nr, uint64_t nc) {
    if (out && n < cap) {
      wb_slice s{};
      s.tensor = tensor; s.local_off = elem_off + local; s.stride_r = sr; s.stride_c = sc;
      s.ckpt_tensor = t; s.ckpt_rows = ck.rows[t]; s.ckpt_cols = ck.cols[t];
      s.r0 = r0; s.c0 = c0; s.nr = nr; s.nc = nc;
      out[n] = s;
    }
    ++n;
  }
};

// A run of `len` consecutive positions starting at g, stored contiguously from local element
// `local`: split at checkpoint row and tensor boundaries into <= 3 rectangles per tensor.
bool emit_run(Emitter& em, const Ckpts& ck, uint64_t g, uint64_t len, uint64_t local) {
  while (len) {
    size_t t;
    if (!ck.find(g, &t)) return false;
    const uint64_t C = ck.cols[t], R = ck.rows[t];
    const uint64_t r = (g - ck.base[t]) / C, c = (g - ck.base[t]) % C;
    uint64_t take;
    if (c != 0 || len < C) {
      take = std::min(len, C - c);
      em.push(local, (int64_t)C, 1, ck, t, r, c, 1, take);
    } else {
      const uint64_t m = std::min(len / C, R - r);
      take = m * C;
      em.push(local, (int64_t)C, 1, ck, t, r, 0, m, C);
    }
    g += take; local += take; len -= take;
  }
  return true;
}

// One maximal rectangle [i0,i1) x [j0,j1) of the local view with id = a + b i + c j.
bool emit_rect(Emitter& em, const Ckpts& ck, uint64_t i0, uint64_t i1, uint64_t j0, uint64_t j1, const Affine& f);
bool emit_rect(Emitter& em, const Ckpts& ck, uint64_t i0, uint64_t i1, uint64_t j0, uint64_t j1, const Affine& f) {
  const uint64_t ni = i1 - i0, nj = j1 - j0, W = em.view_cols;
  const i128 id00 = f.a + f.b * (i128)i0 + f.c * (i128)j0;
  if (id00 < 1) return false;
  const uint64_t g00 = (uint64_t)(id00 - 1);
  size_t t;
  if (!ck.find(g00, &t)) return false;
  const uint64_t C = ck.cols[t], R = ck.rows[t];
  const uint64_t r0 = (g00 - ck.base[t]) / C, c0 = (g00 - ck.base[t]) % C;
  const uint64_t local = i0 * W + j0;
  const bool along_j = nj == 1 ? !(ni > 1 && f.b == 1) : f.c == 1;
  if (along_j) {
    // ids advance by one along local columns (same orientation as the checkpoint)
    if (nj <= C - c0 && (ni == 1 || (f.b == (i128)C && r0 + ni <= R))) {
      em.push(local, (int64_t)W, 1, ck, t, r0, c0, ni, nj);
      return true;
    }
    for (uint64_t i = i0; i < i1; ++i) {       // rows that wrap over checkpoint rows: run by run
      const i128 id = f.a + f.b * (i128)i + f.c * (i128)j0;
      if (id < 1 || !emit_run(em, ck, (uint64_t)(id - 1), nj, i * W + j0)) return false;
    }
    return true;
  }
  // transposed: ids advance by one along local rows, by a checkpoint row along local columns
  if ((ni == 1 || f.b == 1) && (nj == 1 || f.c == (i128)C) && ni <= C - c0 && r0 + nj <= R) {
    em.push(local, 1, (int64_t)W, ck, t, r0, c0, nj, ni);
    return true;
  }
  // neither shape as a whole (e.g. two unrelated one-element pieces that happen to be "affine"):
  // row by row, and a thin piece element by element
  if (ni > 1 && nj > 1) {
    for (uint64_t i = i0; i < i1; ++i)
      if (!emit_rect(em, ck, i, i + 1, j0, j1, f)) return false;
    return true;
  }
  if (ni * nj == 1) return false;
  for (uint64_t i = i0; i < i1; ++i)
    for (uint64_t j = j0; j < j1; ++j)
      if (!emit_rect(em, ck, i, i + 1, j, j + 1, f)) return false;
  return true;
}

}  // namespace

extern "C" wb_status wb_diff2_recombine(const wb_diff2_entry* const* passes, const size_t* counts, size_t n_passes,
                                        uint32_t chunk_bits, wb_diff2_entry* out, size_t cap, size_t* n_out) {
  if (!n_out || (n_passes && (!passes || !counts)) || chunk_bits == 0 || chunk_bits > 32 ||
      (uint64_t)chunk_bits * n_passes > 64) return WB_ERR_INVALID_ARG;
  try {
    std::vector<wb_diff2_entry> all;
    for (size_t k = 0; k < n_passes; ++k)
      for (size_t e = 0; e < counts[k]; ++e) {
        wb_diff2_entry x = passes[k][e];
        x.value = (int64_t)((uint64_t)x.value << (chunk_bits * k));   // times 2^(b k), exact mod 2^64
        all.push_back(x);
      }
    std::sort(all.begin(), all.end(), [](const wb_diff2_entry& a, const wb_diff2_entry& b) {
      return a.row != b.row ? a.row < b.row : a.col < b.col;
    });
    size_t n = 0;
    for (size_t e = 0; e < all.size();) {
      size_t f = e;
      int64_t v = 0;
      while (f < all.size() && all[f].row == all[e].row && all[f].col == all[e].col) v += all[f++].value;
      if (v != 0) {
        if (out && n < cap) out[n] = wb_diff2_entry{all[e].row, all[e].col, v};
        ++n;
      }
      e = f;
    }
    *n_out = n;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  return WB_OK;
}

extern "C" wb_status wb_scan_slices(const wb_diff2_entry* nz, size_t n, uint64_t rows, uint64_t cols,
                                    const uint64_t* ckpt_base, const uint64_t* ckpt_rows, const uint64_t* ckpt_cols,
                                    size_t n_ckpt, uint32_t tensor, uint64_t elem_off, wb_slice* out, size_t cap,
                                    size_t* n_out) {
  if (!n_out || (n && !nz) || !ckpt_base || !ckpt_rows || !ckpt_cols || rows == 0 || cols == 0)
    return WB_ERR_INVALID_ARG;
  const Ckpts ck{ckpt_base, ckpt_rows, ckpt_cols, n_ckpt};
  Emitter em{out, cap, 0, tensor, elem_off, cols};
  try {
    std::vector<wb_diff2_entry> e(nz, nz + n);
    std::sort(e.begin(), e.end(), [](const wb_diff2_entry& a, const wb_diff2_entry& b) {
      return a.row != b.row ? a.row < b.row : a.col < b.col;
    });
    std::vector<uint64_t> R{0}, C{0};
    for (const auto& x : e) {
      if (x.row >= rows || x.col >= cols) return WB_ERR_OUT_OF_RANGE;
      R.push_back(x.row); C.push_back(x.col);
      if (x.row) R.push_back(x.row - 1);
      if (x.col) C.push_back(x.col - 1);
    }
    std::sort(R.begin(), R.end()); R.erase(std::unique(R.begin(), R.end()), R.end());
    std::sort(C.begin(), C.end()); C.erase(std::unique(C.begin(), C.end()), C.end());
    const size_t nc = C.size();
    // column-wise running sums, carried from grid row to grid row
    struct Sums { i128 s0, sp, sq, spq; };
    std::vector<Sums> col(nc, Sums{0, 0, 0, 0});
    std::vector<Seg> open, now;
    size_t cur = 0;
    for (size_t k = 0; k < R.size(); ++k) {
      for (; cur < e.size() && e[cur].row <= R[k] + 1; ++cur) {
        // the first grid column c with c + 1 >= q
        const uint64_t q = e[cur].col;
        const size_t l = q ? std::lower_bound(C.begin(), C.end(), q - 1) - C.begin() : 0;
        const i128 v = e[cur].value, p = e[cur].row;
        col[l].s0 += v; col[l].sp += p * v; col[l].sq += (i128)q * v; col[l].spq += p * (i128)q * v;
      }
      const uint64_t i0 = R[k], i1 = k + 1 < R.size() ? R[k + 1] : rows;
      // cells of this grid row, merged along columns
      now.clear();
      Sums s{0, 0, 0, 0};
      for (size_t l = 0; l < nc; ++l) {
        s.s0 += col[l].s0; s.sp += col[l].sp; s.sq += col[l].sq; s.spq += col[l].spq;
        const uint64_t j0 = C[l], j1 = l + 1 < nc ? C[l + 1] : cols;
        Affine f;
        if (s.s0 == 0) {
          f = Affine{s.spq - s.sq - s.sp, -s.sq, -s.sp};
        } else if (i1 - i0 == 1) {           // one row: only the slope along j is defined
          const i128 r1 = (i128)i0 + 1;
          f = Affine{r1 * s.s0 - r1 * s.sq - s.sp + s.spq, 0, r1 * s.s0 - s.sp};
        } else if (j1 - j0 == 1) {           // one column: only the slope along i is defined
          const i128 c1 = (i128)j0 + 1;
          f = Affine{c1 * s.s0 - s.sq - c1 * s.sp + s.spq, c1 * s.s0 - s.sq, 0};
        } else {
          return WB_ERR_INVALID_ARG;         // bilinear over a 2-D cell: not a field of slice copies
        }
        if (f.zero()) continue;
        if (!now.empty() && now.back().j1 == j0 && now.back().f == f) now.back().j1 = j1;
        else now.push_back(Seg{j0, j1, i0, f});
      }
      // rectangles that continue keep their first row; the others are complete
      for (const Seg& o : open) {
        bool cont = false;
        for (Seg& s2 : now)
          if (s2.j0 == o.j0 && s2.j1 == o.j1 && s2.f == o.f) { s2.i0 = o.i0; cont = true; break; }
        if (!cont && !emit_rect(em, ck, o.i0, R[k], o.j0, o.j1, o.f)) return WB_ERR_INVALID_ARG;
      }
      open.swap(now);
    }
    for (const Seg& o : open)
      if (!emit_rect(em, ck, o.i0, rows, o.j0, o.j1, o.f)) return WB_ERR_INVALID_ARG;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  *n_out = em.n;
  return WB_OK;
}
