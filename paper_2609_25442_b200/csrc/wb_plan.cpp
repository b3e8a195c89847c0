// The transfer planner (Section 3.2), single-GPU form.  Host only; no CUDA call.
//
//   correspondence   per checkpoint tensor, intersect source rectangles with destination
//                    rectangles (Section 3.1: overlap of source maps)
//   de-duplication   source replicas each supply a distinct slice; destination replicas
//                    are fed from one read (fan-out), each being the designated receiver
//                    of a distinct slice                     (Section 3.2, three-stage plan)
//   tiles            slabs cut into near-equal-byte tiles, contiguous tile ranges per
//                    thread block balanced by bytes
//   rounds           payload chunks assigned to roughly equal rounds whose buckets fit the
//                    budget (Section 3.2: the transfer runs in rounds, each a batch;
//                    Appendix D: the round count follows from the buffer budget)
#include <algorithm>
#include <chrono>
#include <cstring>
#include <map>
#include <new>
#include <numeric>

#include "wb_internal.h"

using namespace wbi;

namespace {

constexpr uint64_t kDefaultBudget = 4ull << 30;
constexpr uint32_t kDefaultTileBytes = 512u << 10;
constexpr uint32_t kDefaultGrid = wbi::kNumSMs * wbi::kCtasPerSM;
constexpr uint64_t kPayloadAlign = 16;
constexpr uint64_t kRegionAlign = 256;

inline uint32_t esize(uint32_t dt) { return dt == WB_F32 ? 4u : 2u; }
inline uint64_t roundup(uint64_t x, uint64_t m) { return (x + m - 1) / m * m; }

// a - b as up to four disjoint rectangles
void subtract(const Rect& a, const Rect& b, std::vector<Rect>* out) {
  Rect x;
  if (!intersect(a, b, &x)) { out->push_back(a); return; }
  if (x.r0 > a.r0) out->push_back(Rect{a.r0, a.c0, x.r0 - a.r0, a.nc});
  if (x.r1() < a.r1()) out->push_back(Rect{x.r1(), a.c0, a.r1() - x.r1(), a.nc});
  if (x.c0 > a.c0) out->push_back(Rect{x.r0, a.c0, x.nr, x.c0 - a.c0});
  if (x.c1() < a.c1()) out->push_back(Rect{x.r0, x.c1(), x.nr, a.c1() - x.c1()});
}

// Split a rectangle into at most m contiguous, near-equal pieces: by rows when there are
// enough rows, else by columns on 128-element boundaries when the row is long enough.
void split_rect(const Rect& r, uint32_t m, std::vector<Rect>* out) {
  if (m <= 1 || r.area() < 2) { out->push_back(r); return; }
  if (r.nr >= m) {
    for (uint32_t k = 0; k < m; ++k) {
      uint64_t a = r.nr * k / m, b = r.nr * (k + 1) / m;
      if (b > a) out->push_back(Rect{r.r0 + a, r.c0, b - a, r.nc});
    }
    return;
  }
  const bool aligned = r.nc >= 128ull * m;
  uint64_t prev = 0;
  for (uint32_t k = 0; k < m; ++k) {
    uint64_t b = r.nc * (k + 1) / m;
    if (aligned && k + 1 < m) b = b / 128 * 128;
    if (k + 1 == m) b = r.nc;
    if (b > prev) out->push_back(Rect{r.r0, r.c0 + prev, r.nr, b - prev});
    prev = b > prev ? b : prev;
  }
}

// ---- footprints: exact overlap test of strided element sets inside one tensor ------------
struct Footprint {
  int64_t tensor;
  uint64_t off, runs, len, pitch;   // `runs` runs of `len` elements, `pitch` apart
  uint64_t lo() const { return off; }
  uint64_t hi() const { return off + (runs - 1) * pitch + len; }   // exclusive
};

Footprint footprint(int64_t tensor, uint64_t off, uint64_t nr, uint64_t nc, uint64_t sr, uint64_t sc) {
  // every tile / slice has unit stride along one axis, or a degenerate axis
  if (nr == 1 && nc == 1) return Footprint{tensor, off, 1, 1, 1};
  if (nc == 1) return sr == 1 ? Footprint{tensor, off, 1, nr, 1} : Footprint{tensor, off, nr, 1, sr};
  if (nr == 1) return sc == 1 ? Footprint{tensor, off, 1, nc, 1} : Footprint{tensor, off, nc, 1, sc};
  if (sc == 1) return (sr == nc) ? Footprint{tensor, off, 1, nr * nc, 1} : Footprint{tensor, off, nr, nc, sr};
  return (sc == nr) ? Footprint{tensor, off, 1, nr * nc, 1} : Footprint{tensor, off, nc, nr, sc};
}

bool run_hits(const Footprint& b, uint64_t a, uint64_t len) {   // [a, a+len) vs b
  if (a + len <= b.lo() || a >= b.hi()) return false;
  if (b.runs == 1) return true;
  // run k of b is [off + k*pitch, off + k*pitch + b.len); it touches [a, a+len) iff
  // k_lo <= k <= k_hi with the bounds below
  uint64_t k_hi = (a + len - 1 - b.off) / b.pitch;
  if (k_hi > b.runs - 1) k_hi = b.runs - 1;
  uint64_t k_lo = 0;
  if (a >= b.off + b.len) k_lo = (a - b.off - b.len) / b.pitch + 1;
  return k_lo <= k_hi;
}

bool overlaps(const Footprint& a, const Footprint& b) {
  const Footprint& x = a.runs <= b.runs ? a : b;
  const Footprint& y = a.runs <= b.runs ? b : a;
  for (uint64_t k = 0; k < x.runs; ++k)
    if (run_hits(y, x.off + k * x.pitch, x.len)) return true;
  return false;
}

// true if any two footprints share an element
bool any_overlap(std::vector<Footprint>& f) {
  std::sort(f.begin(), f.end(), [](const Footprint& a, const Footprint& b) {
    return a.tensor != b.tensor ? a.tensor < b.tensor : a.off < b.off;
  });
  for (size_t i = 0; i < f.size(); ++i)
    for (size_t j = i + 1; j < f.size() && f[j].tensor == f[i].tensor && f[j].lo() < f[i].hi(); ++j)
      if (overlaps(f[i], f[j])) return true;
  return false;
}

// ---- copy operations and tiling --------------------------------------------------------------
struct Ref {            // where a checkpoint rectangle's element (i, j) lives: off + i*sr + j*sc
  int32_t tensor;
  uint64_t off, sr, sc;
};

Ref ref_of(const NSlice& s, const Rect& sub) {
  return Ref{(int32_t)s.tensor, s.elem(sub.r0, sub.c0), s.sr(), s.sc()};
}

struct TileBuilder {
  TileTable* tab;
  uint32_t es, ed, tile_bytes;
  bool ok = true;

  void emit(const Ref& src, const Ref* dsts, uint32_t n_dst, uint64_t i0, uint64_t j0,
            uint64_t ni, uint64_t nj, uint32_t kind, uint32_t seam = 0) {
    HTile t{};
    t.seam = seam;
    auto fits = [&](uint64_t v) { if (v >= (1ull << 32)) ok = false; return (uint32_t)v; };
    t.src_tensor = src.tensor;
    t.src_off = src.off + i0 * src.sr + j0 * src.sc;
    t.dst_tensor = dsts[0].tensor;
    t.dst_off = dsts[0].off + i0 * dsts[0].sr + j0 * dsts[0].sc;
    t.nr = fits(ni); t.nc = fits(nj);
    t.ssr = fits(src.sr); t.ssc = fits(src.sc);
    t.dsr = fits(dsts[0].sr); t.dsc = fits(dsts[0].sc);
    t.kind = kind;
    t.n_extra = n_dst - 1;
    t.extra = (uint32_t)tab->extras.size();
    if (n_dst - 1 > 255) ok = false;
    for (uint32_t d = 1; d < n_dst; ++d)
      tab->extras.push_back(HDst{dsts[d].tensor, dsts[d].off + i0 * dsts[d].sr + j0 * dsts[d].sc,
                                 fits(dsts[d].sr), fits(dsts[d].sc)});
    t.bytes = ni * nj * ((uint64_t)es + (uint64_t)ed * n_dst);
    tab->tiles.push_back(t);
  }

  // Copy the nr x nc checkpoint rectangle from src to every dst.
  void add(Ref src, std::vector<Ref> dsts, uint64_t nr, uint64_t nc) {
    const uint32_t n_dst = (uint32_t)dsts.size();
    // degenerate extents: their strides are never used; give them a canonical value
    if (nr == 1) { src.sr = 0; for (auto& d : dsts) d.sr = 0; }
    if (nc == 1) { src.sc = 0; for (auto& d : dsts) d.sc = 0; }
    // make j the axis along which the source is contiguous
    bool swap = (nc == 1 && nr > 1) || (nr > 1 && nc > 1 && src.sc != 1 && src.sr == 1);
    if (swap) {
      std::swap(nr, nc);
      std::swap(src.sr, src.sc);
      for (auto& d : dsts) std::swap(d.sr, d.sc);
    }
    const uint64_t be = (uint64_t)es + (uint64_t)ed * n_dst;
    const uint64_t T = std::max<uint64_t>(1024, tile_bytes / be);   // target elements per tile
    if (nr == 1) {
      bool unit = (nc == 1) || src.sc == 1;
      for (auto& d : dsts) unit = unit && (nc == 1 || d.sc == 1);
      const uint32_t kind = unit ? KIND_ROWS : KIND_ELEM;
      if (nc == 1) { src.sc = 1; for (auto& d : dsts) d.sc = 1; }
      uint64_t n_tiles = (nc + T - 1) / T;
      uint64_t chunk = roundup((nc + n_tiles - 1) / n_tiles, 512);
      for (uint64_t j = 0; j < nc; j += chunk)
        emit(src, dsts.data(), n_dst, 0, j, 1, std::min(chunk, nc - j), kind);
      return;
    }
    // two real axes; the source has unit stride along j
    bool rows = src.sc == 1, trans = src.sc == 1;
    for (auto& d : dsts) { rows = rows && d.sc == 1; trans = trans && d.sr == 1; }
    if (rows) {
      bool contiguous = src.sr == nc;
      for (auto& d : dsts) contiguous = contiguous && d.sr == nc;
      if (contiguous) {       // collapses to one run
        Ref s1 = src; s1.sr = 0;
        std::vector<Ref> d1 = dsts;
        for (auto& d : d1) d.sr = 0;
        const uint64_t n = nr * nc;
        uint64_t n_tiles = (n + T - 1) / T;
        uint64_t chunk = roundup((n + n_tiles - 1) / n_tiles, 512);
        for (uint64_t j = 0; j < n; j += chunk)
          emit(s1, d1.data(), n_dst, 0, j, 1, std::min(chunk, n - j), KIND_ROWS);
        return;
      }
      if (nc >= 2 * T) {      // very long rows: cut columns as well
        uint64_t n_tiles = (nc + T - 1) / T;
        uint64_t chunk = roundup((nc + n_tiles - 1) / n_tiles, 512);
        for (uint64_t i = 0; i < nr; ++i)
          for (uint64_t j = 0; j < nc; j += chunk)
            emit(src, dsts.data(), n_dst, i, j, 1, std::min(chunk, nc - j), KIND_ROWS);
        return;
      }
      uint64_t per = std::max<uint64_t>(1, T / nc);
      uint64_t n_tiles = (nr + per - 1) / per;
      per = (nr + n_tiles - 1) / n_tiles;
      for (uint64_t i = 0; i < nr; i += per)
        emit(src, dsts.data(), n_dst, i, 0, std::min(per, nr - i), nc, KIND_ROWS);
      return;
    }
    const uint32_t kind = trans ? KIND_TRANS : KIND_ELEM;
    // 2-D blocks, multiples of 64 on both axes where the extent allows
    // transposed: one staged transposition chunk of the executor wide (480 source bytes) and as tall
    // as the tile size allows, so that a tile writes long pieces of few destination runs and the
    // element stores at the two ends of a run piece are rare
#ifndef WB_TRANS_NARROW_MIN_BYTES
#define WB_TRANS_NARROW_MIN_BYTES (1u << 20)
#endif
    // (small slabs keep four chunks per tile: there the number of tiles matters more)
    const bool narrow = nr * nc * (uint64_t)(es + ed) >= WB_TRANS_NARROW_MIN_BYTES;
    uint64_t tc = std::min<uint64_t>(nc, trans ? (narrow ? 480 / es : 480) : 512);
    if (trans && nc > tc) {
      // equal column shares instead of full tiles plus a thin remainder (which would be too narrow
      // for the staged path)
      const uint64_t n_col = (nc + tc - 1) / tc;
      tc = std::min<uint64_t>(tc, roundup((nc + n_col - 1) / n_col, 8));
    }
    uint64_t tr = std::min<uint64_t>(nr, std::max<uint64_t>(64, roundup(T / tc, 64)));
    if (trans && nr > tr) {
      // equal row shares too (multiples of a chunk's 64 rows): no tile of a few left-over rows
      const uint64_t n_row = (nr + tr - 1) / tr;
      tr = std::min<uint64_t>(tr, roundup((nr + n_row - 1) / n_row, 64));
    }
    if (trans) {
      // rows fastest: consecutive tiles continue the same destination runs; where two neighbours in
      // a column are both staged by the executor, destination windows may cross their seam
      for (uint64_t j = 0; j < nc; j += tc) {
        const uint64_t w = std::min(tc, nc - j);
        auto staged = [&](uint64_t i) {
          return i < nr && staged_transposition(kind, n_dst - 1, std::min(tr, nr - i), w, es, ed);
        };
        for (uint64_t i = 0; i < nr; i += tr) {
          uint32_t seam = 0;
          if (staged(i)) {
            if (i > 0 && staged(i - tr)) seam |= kTileRowsBefore;
            if (staged(i + tr)) seam |= kTileRowsAfter;
          }
          emit(src, dsts.data(), n_dst, i, j, std::min(tr, nr - i), w, kind, seam);
        }
      }
      return;
    }
    for (uint64_t i = 0; i < nr; i += tr)
      for (uint64_t j = 0; j < nc; j += tc)
        emit(src, dsts.data(), n_dst, i, j, std::min(tr, nr - i), std::min(tc, nc - j), kind);
  }
};

// Contiguous tile ranges per thread block, balanced by bytes plus a per-tile overhead.
void assign_ctas(TileTable* tab, uint32_t grid) {
  const uint64_t kOverhead = 8192;   // a tile's fixed cost, expressed in bytes
  uint64_t total = 0;
  for (auto& t : tab->tiles) total += t.bytes + kOverhead;
  tab->cta_begin.assign(grid + 1, 0);
  std::vector<uint64_t> load(grid, 0);
  uint64_t acc = 0;
  uint32_t c = 0;
  for (size_t k = 0; k < tab->tiles.size(); ++k) {
    const uint64_t w = tab->tiles[k].bytes + kOverhead;
    // the block whose share [c*total/grid, (c+1)*total/grid) of the weight holds the
    // tile's midpoint; midpoints increase, so ranges are contiguous
    uint64_t want = (uint64_t)(((unsigned __int128)(2 * acc + w) * grid) / (2 * (unsigned __int128)total));
    if (want > grid - 1) want = grid - 1;
    while (c < want) {
      ++c;
      tab->cta_begin[c] = (uint32_t)k;
    }
    tab->tiles[k].cta = c;
    load[c] += tab->tiles[k].bytes;
    acc += w;
  }
  for (uint32_t k = c + 1; k <= grid; ++k) tab->cta_begin[k] = (uint32_t)tab->tiles.size();
  tab->bytes_total = 0;
  tab->bytes_max_cta = 0;
  for (uint32_t k = 0; k < grid; ++k) {
    tab->bytes_total += load[k];
    tab->bytes_max_cta = std::max(tab->bytes_max_cta, load[k]);
  }
}

}  // namespace

// =================================================================================================
extern "C" wb_status wb_plan_build(const wb_layout* trainer, const wb_layout* rollout,
                                   const wb_plan_opts* opts_in, wb_plan** out) {
  if (!trainer || !rollout || !out) return WB_ERR_INVALID_ARG;
  const auto t_start = std::chrono::steady_clock::now();
  wb_plan* P = new (std::nothrow) wb_plan();
  if (!P) return WB_ERR_OOM;
  auto fail = [&](wb_status s) { delete P; return s; };
  try {
    P->src = *trainer;
    P->dst = *rollout;
    if (opts_in) P->opts = *opts_in;
    if (P->opts.bucket_budget_bytes == 0) P->opts.bucket_budget_bytes = kDefaultBudget;
    const bool auto_tile = P->opts.tile_bytes == 0;
    if (!auto_tile && P->opts.tile_bytes < 4096) P->opts.tile_bytes = 4096;
    if (P->opts.grid_ctas == 0) P->opts.grid_ctas = kDefaultGrid;
    if (P->opts.grid_ctas > (1u << 20)) return fail(WB_ERR_INVALID_ARG);
    P->grid = P->opts.grid_ctas;
    const wb_layout& S = P->src;
    const wb_layout& D = P->dst;
    const uint32_t es = esize(S.dtype), ed = esize(D.dtype);
    P->egress.assign(std::max<uint32_t>(S.n_ranks, 1), 0);
    P->ingress.assign(std::max<uint32_t>(D.n_ranks, 1), 0);

    // ---- a destination element may be described only once ---------------------------------
    {
      std::vector<Footprint> f;
      f.reserve(D.slices.size());
      for (const NSlice& s : D.slices)
        f.push_back(footprint(s.tensor, s.off, s.rect.nr, s.rect.nc, s.sr(), s.sc()));
      if (any_overlap(f)) return fail(WB_ERR_DST_OVERLAP);
    }

    // ---- correspondence + de-duplication, one checkpoint tensor at a time -------------------
    struct Piece { Rect rect; uint32_t slice; };
    struct Hit { uint32_t dslice; Rect rect; };
    std::vector<Piece> pieces;
    std::vector<Rect> owned, frags, tmp;
    std::vector<uint32_t> owned_by;
    std::vector<uint32_t> order;
    std::vector<Hit> hits;
    std::vector<uint64_t> covered;
    uint64_t replica_skipped = 0;
    size_t si = 0;   // cursor into S.ckpts (both sorted by id)
    for (size_t di = 0; di < D.ckpts.size(); ++di) {
      const CkptInfo& dc = D.ckpts[di];
      while (si < S.ckpts.size() && S.ckpts[si].id < dc.id) ++si;
      if (si == S.ckpts.size() || S.ckpts[si].id != dc.id) return fail(WB_ERR_UNCOVERED);
      const CkptInfo& sc = S.ckpts[si];
      if (sc.rows != dc.rows || sc.cols != dc.cols) return fail(WB_ERR_SHAPE_MISMATCH);

      // group source slices with identical rectangles (replicas), ascending rank inside
      order.resize(sc.count);
      std::iota(order.begin(), order.end(), sc.first);
      std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
        const NSlice& x = S.slices[a]; const NSlice& y = S.slices[b];
        if (x.rect.r0 != y.rect.r0) return x.rect.r0 < y.rect.r0;
        if (x.rect.c0 != y.rect.c0) return x.rect.c0 < y.rect.c0;
        if (x.rect.nr != y.rect.nr) return x.rect.nr < y.rect.nr;
        if (x.rect.nc != y.rect.nc) return x.rect.nc < y.rect.nc;
        const uint32_t rx = S.tensors[x.tensor].rank, ry = S.tensors[y.tensor].rank;
        if (rx != ry) return rx < ry;
        return a < b;
      });
      pieces.clear();
      owned.clear();
      owned_by.clear();
      uint64_t held_area = 0, slice_area = 0;
      for (size_t g0 = 0; g0 < order.size();) {
        size_t g1 = g0 + 1;
        const Rect& gr = S.slices[order[g0]].rect;
        while (g1 < order.size()) {
          const Rect& o = S.slices[order[g1]].rect;
          if (o.r0 != gr.r0 || o.c0 != gr.c0 || o.nr != gr.nr || o.nc != gr.nc) break;
          ++g1;
        }
        const uint32_t m = (uint32_t)(g1 - g0);
        slice_area += gr.area() * m;
        // replicas are assumed identical; remember which pairs a consistency check must compare
        for (uint32_t k = 1; k < m; ++k) P->replica_pairs.push_back(ReplicaPair{order[g0], order[g0 + k], gr});
        // keep only what no earlier group already owns
        frags.assign(1, gr);
        for (size_t oi = 0; oi < owned.size(); ++oi) {
          const Rect& o = owned[oi];
          Rect both;
          if (!intersect(gr, o, &both)) continue;
          P->replica_pairs.push_back(ReplicaPair{owned_by[oi], order[g0], both});
          tmp.clear();
          for (const Rect& f : frags) subtract(f, o, &tmp);
          frags.swap(tmp);
          if (frags.empty()) break;
        }
        for (const Rect& f : frags) {
          owned.push_back(f);
          owned_by.push_back(order[g0]);
          held_area += f.area();
          if (m == 1 || (P->opts.flags & WB_PLAN_NO_REPLICA_SPLIT)) {
            pieces.push_back(Piece{f, order[g0]});
          } else {
            tmp.clear();
            split_rect(f, m, &tmp);
            for (size_t k = 0; k < tmp.size(); ++k) pieces.push_back(Piece{tmp[k], order[g0 + k]});
          }
        }
        g0 = g1;
      }
      replica_skipped += slice_area - held_area;

      // destination rectangles against the (disjoint) source pieces
      covered.assign(dc.count, 0);
      uint64_t consumed_here = 0;
      for (const Piece& pc : pieces) {
        hits.clear();
        for (uint32_t k = 0; k < dc.count; ++k) {
          Rect x;
          if (intersect(pc.rect, D.slices[dc.first + k].rect, &x)) {
            hits.push_back(Hit{dc.first + k, x});
            covered[k] += x.area();
          }
        }
        if (hits.empty()) continue;
        bool disjoint = true;
        for (size_t a = 0; a < hits.size() && disjoint; ++a)
          for (size_t b = a + 1; b < hits.size(); ++b)
            if (intersect(hits[a].rect, hits[b].rect, nullptr)) { disjoint = false; break; }
        auto add_slab = [&](const Rect& r, const uint32_t* ds, uint32_t nd) {
          // destination replicas: each is the designated receiver of a distinct slice
          tmp.clear();
          split_rect(r, nd, &tmp);
          for (size_t k = 0; k < tmp.size(); ++k) {
            Slab sl{};
            sl.ckpt_index = (uint32_t)di;
            sl.rect = tmp[k];
            sl.src_slice = pc.slice;
            sl.dst_begin = (uint32_t)P->slab_dsts.size();
            sl.dst_count = nd;
            for (uint32_t d = 0; d < nd; ++d) P->slab_dsts.push_back(ds[d]);
            sl.sender = S.tensors[S.slices[pc.slice].tensor].rank;
            sl.receiver = D.tensors[D.slices[ds[k % nd]].tensor].rank;
            P->slabs.push_back(sl);
            consumed_here += tmp[k].area();
          }
        };
        if (disjoint) {
          for (const Hit& h : hits) add_slab(h.rect, &h.dslice, 1);
        } else {
          // overlapping destination rectangles (replicas): decompose on the grid of their
          // boundaries and merge cells with the same set of destinations
          std::vector<uint64_t> ys, xs;
          for (const Hit& h : hits) {
            ys.push_back(h.rect.r0); ys.push_back(h.rect.r1());
            xs.push_back(h.rect.c0); xs.push_back(h.rect.c1());
          }
          std::sort(ys.begin(), ys.end()); ys.erase(std::unique(ys.begin(), ys.end()), ys.end());
          std::sort(xs.begin(), xs.end()); xs.erase(std::unique(xs.begin(), xs.end()), xs.end());
          struct Open { uint64_t c0, c1, r0, r1; std::vector<uint32_t> set; };
          std::vector<Open> open, next;
          auto flush = [&](const Open& o) {
            add_slab(Rect{o.r0, o.c0, o.r1 - o.r0, o.c1 - o.c0}, o.set.data(), (uint32_t)o.set.size());
          };
          for (size_t a = 0; a + 1 < ys.size(); ++a) {
            next.clear();
            for (size_t b = 0; b + 1 < xs.size(); ++b) {
              std::vector<uint32_t> set;
              Rect cell{ys[a], xs[b], ys[a + 1] - ys[a], xs[b + 1] - xs[b]};
              for (const Hit& h : hits)
                if (intersect(cell, h.rect, nullptr)) set.push_back(h.dslice);
              if (set.empty()) continue;
              if (!next.empty() && next.back().c1 == xs[b] && next.back().set == set)
                next.back().c1 = xs[b + 1];
              else
                next.push_back(Open{xs[b], xs[b + 1], ys[a], ys[a + 1], set});
            }
            // extend open rectangles downwards where the band repeats them
            for (Open& o : open) {
              bool extended = false;
              for (Open& n : next)
                if (n.r0 == ys[a] && n.c0 == o.c0 && n.c1 == o.c1 && n.set == o.set && o.r1 == ys[a]) {
                  n.r0 = o.r0; extended = true; break;
                }
              if (!extended) flush(o);
            }
            open.swap(next);
          }
          for (const Open& o : open) flush(o);
        }
      }
      for (uint32_t k = 0; k < dc.count; ++k)
        if (covered[k] != D.slices[dc.first + k].rect.area()) return fail(WB_ERR_UNCOVERED);
      P->stats.src_elems_read += consumed_here;
    }
    P->stats.n_ckpt_tensors = D.ckpts.size();
    P->stats.replica_elems_skipped = replica_skipped;

    // ---- accounting ---------------------------------------------------------------------------
    for (const Slab& sl : P->slabs) {
      P->egress[sl.sender] += sl.rect.area() * es;
      P->ingress[sl.receiver] += sl.rect.area() * ed;
      P->stats.dst_elems_written += sl.rect.area() * sl.dst_count;
      if (sl.dst_count > 1) P->stats.n_fanout_slabs++;
    }
    P->stats.n_slabs = P->slabs.size();
    P->stats.src_bytes_read = P->stats.src_elems_read * es;
    P->stats.dst_bytes_written = P->stats.dst_elems_written * ed;

    if (auto_tile) {
      // about 16 tiles per thread block, within [32 KiB, 512 KiB]
      uint64_t tb = (P->stats.src_bytes_read + P->stats.dst_bytes_written) / ((uint64_t)P->opts.grid_ctas * 16);
      tb = std::min<uint64_t>(std::max<uint64_t>(tb, 32u << 10), kDefaultTileBytes);
      P->opts.tile_bytes = (uint32_t)(tb / 4096 * 4096);
    }

    // ---- fused remap table ------------------------------------------------------------------------
    auto slab_refs = [&](const Slab& sl, const Rect& sub, Ref* src, std::vector<Ref>* dsts) {
      *src = ref_of(S.slices[sl.src_slice], sub);
      dsts->clear();
      for (uint32_t d = 0; d < sl.dst_count; ++d)
        dsts->push_back(ref_of(D.slices[P->slab_dsts[sl.dst_begin + d]], sub));
    };
    {
      TileBuilder tb{&P->remap, es, ed, P->opts.tile_bytes};
      Ref src; std::vector<Ref> dsts;
      // Tiles of one checkpoint tensor are emitted slab by slab; they are then ordered by the address
      // of their strided side (rows a pitch apart: several slabs cut the same rows into column
      // pieces), so that tiles which touch the same rows, lines and DRAM pages run close in time.
      std::vector<std::pair<size_t, size_t>> ranges;     // [first, last) tile of each checkpoint tensor
      uint32_t cur_ckpt = UINT32_MAX;
      for (const Slab& sl : P->slabs) {
        if (sl.ckpt_index != cur_ckpt) {
          if (!ranges.empty()) ranges.back().second = P->remap.tiles.size();
          ranges.push_back({P->remap.tiles.size(), 0});
          cur_ckpt = sl.ckpt_index;
        }
        slab_refs(sl, sl.rect, &src, &dsts);
        tb.add(src, dsts, sl.rect.nr, sl.rect.nc);
      }
      if (!ranges.empty()) ranges.back().second = P->remap.tiles.size();
      if (!tb.ok) return fail(WB_ERR_INVALID_ARG);
      for (auto& rg : ranges) {
        auto key = [](const HTile& t) {
          // 0: source rows strided, by source address; 1: destination strided, by destination address; 2: as emitted
          if (t.kind == KIND_ROWS && t.nr > 1 && t.ssr > t.nc) return std::make_tuple(0, (int64_t)t.src_tensor, t.src_off);
          if (t.kind == KIND_ROWS && t.nr > 1 && t.dsr > t.nc) return std::make_tuple(1, (int64_t)t.dst_tensor, t.dst_off);
          return std::make_tuple(2, (int64_t)0, (uint64_t)0);
        };
        std::stable_sort(P->remap.tiles.begin() + rg.first, P->remap.tiles.begin() + rg.second,
                         [&](const HTile& a, const HTile& b) { return key(a) < key(b); });
      }
      assign_ctas(&P->remap, P->grid);
    }

    // ---- rounds and buckets -------------------------------------------------------------------------
    {
      const uint64_t budget = P->opts.bucket_budget_bytes;
      uint64_t chunk_max = std::min<uint64_t>(64ull << 20, budget / 16);
      chunk_max = std::max<uint64_t>(chunk_max, 4096);
      if (budget < 2 * kRegionAlign) return fail(WB_ERR_BUCKET_TOO_SMALL);
      // cut slabs into payload chunks of at most chunk_max bytes (row blocks, else column runs)
      struct Chunk { uint32_t slab; Rect rect; uint64_t bytes; };
      std::vector<Chunk> chunks;
      uint64_t total = 0;
      const uint64_t max_elems = std::max<uint64_t>(1, chunk_max / ed);
      for (uint32_t k = 0; k < P->slabs.size(); ++k) {
        const Rect& r = P->slabs[k].rect;
        auto push = [&](const Rect& c) {
          uint64_t b = roundup(c.area() * ed, kPayloadAlign);
          chunks.push_back(Chunk{k, c, b});
          total += b;
        };
        if (r.area() <= max_elems) { push(r); continue; }
        if (r.nc <= max_elems) {
          uint64_t per = max_elems / r.nc;
          uint64_t n = (r.nr + per - 1) / per;
          per = (r.nr + n - 1) / n;
          for (uint64_t i = 0; i < r.nr; i += per)
            push(Rect{r.r0 + i, r.c0, std::min(per, r.nr - i), r.nc});
        } else {
          for (uint64_t i = 0; i < r.nr; ++i)
            for (uint64_t j = 0; j < r.nc; j += max_elems)
              push(Rect{r.r0 + i, r.c0 + j, 1, std::min(max_elems, r.nc - j)});
        }
      }
      uint64_t n_rounds = std::max<uint64_t>(1, (total + budget - 1) / budget);
      for (int attempt = 0; attempt < 64; ++attempt, ++n_rounds) {
        P->rounds.assign(n_rounds, Round{});
        // chunk c goes to the round whose share of the running total holds its start
        uint64_t acc = 0;
        std::vector<std::vector<uint32_t>> members(n_rounds);
        for (uint32_t c = 0; c < chunks.size(); ++c) {
          uint64_t r = total ? (uint64_t)((unsigned __int128)acc * n_rounds / total) : 0;
          if (r >= n_rounds) r = n_rounds - 1;
          members[r].push_back(c);
          acc += chunks[c].bytes;
        }
        bool fits = true;
        for (uint64_t r = 0; r < n_rounds && fits; ++r) {
          // bucket layout: one region per (receiver, sender), payloads in checkpoint order
          auto& m = members[r];
          std::stable_sort(m.begin(), m.end(), [&](uint32_t a, uint32_t b) {
            const Slab& x = P->slabs[chunks[a].slab]; const Slab& y = P->slabs[chunks[b].slab];
            if (x.receiver != y.receiver) return x.receiver < y.receiver;
            return x.sender < y.sender;
          });
          uint64_t off = 0;
          int64_t last_pair = -1;
          Round& R = P->rounds[r];
          R.payloads.reserve(m.size());
          for (uint32_t c : m) {
            const Slab& sl = P->slabs[chunks[c].slab];
            int64_t pair = (int64_t)sl.receiver * (1ll << 32) + sl.sender;
            if (pair != last_pair) {
              off = roundup(off, kRegionAlign);
              last_pair = pair;
              R.regions.push_back(Region{sl.receiver, sl.sender, off, 0});
            }
            R.payloads.push_back(Payload{chunks[c].slab, chunks[c].rect, off});
            off += chunks[c].bytes;
            R.regions.back().bytes = off - R.regions.back().off;
          }
          R.bucket_bytes = roundup(off, kPayloadAlign);
          if (R.bucket_bytes > budget) fits = false;
        }
        if (fits) break;
        if (attempt == 63 || n_rounds > chunks.size() + 1) return fail(WB_ERR_BUCKET_TOO_SMALL);
        n_rounds += n_rounds / 50;   // (the loop adds one more)
      }
      // per-round tile tables
      Ref src; std::vector<Ref> dsts;
      // Pack tiles are grouped by sender rank and unpack tiles by receiver rank, so that the work of a
      // set of virtual ranks - what one GPU of a multi-GPU deployment would execute, Section 3.2's
      // per-worker packing and assembly - is a contiguous tile range of the round's table.
      std::vector<uint32_t> by_sender;
      for (Round& R : P->rounds) {
        TileBuilder pk{&R.pack, es, ed, P->opts.tile_bytes};
        TileBuilder up{&R.unpack, ed, ed, P->opts.tile_bytes};
        by_sender.resize(R.payloads.size());
        std::iota(by_sender.begin(), by_sender.end(), 0u);
        std::stable_sort(by_sender.begin(), by_sender.end(), [&](uint32_t a, uint32_t b) {
          return P->slabs[R.payloads[a].slab].sender < P->slabs[R.payloads[b].slab].sender;
        });
        R.pack_rank_begin.assign(P->egress.size() + 1, 0);
        R.unpack_rank_begin.assign(P->ingress.size() + 1, 0);
        uint32_t next_rank = 0;
        for (uint32_t k : by_sender) {
          const Payload& pl = R.payloads[k];
          const Slab& sl = P->slabs[pl.slab];
          while (next_rank <= sl.sender) R.pack_rank_begin[next_rank++] = (uint32_t)R.pack.tiles.size();
          slab_refs(sl, pl.rect, &src, &dsts);
          Ref bucket{-1, pl.bucket_off / ed, pl.rect.nc, 1};
          pk.add(src, std::vector<Ref>{bucket}, pl.rect.nr, pl.rect.nc);
          R.pack_ckpt.resize(R.pack.tiles.size(), sl.ckpt_index);
        }
        while (next_rank <= P->egress.size()) R.pack_rank_begin[next_rank++] = (uint32_t)R.pack.tiles.size();
        next_rank = 0;
        for (const Payload& pl : R.payloads) {
          const Slab& sl = P->slabs[pl.slab];
          while (next_rank <= sl.receiver) R.unpack_rank_begin[next_rank++] = (uint32_t)R.unpack.tiles.size();
          slab_refs(sl, pl.rect, &src, &dsts);
          Ref bucket{-1, pl.bucket_off / ed, pl.rect.nc, 1};
          up.add(bucket, dsts, pl.rect.nr, pl.rect.nc);
          R.unpack_ckpt.resize(R.unpack.tiles.size(), sl.ckpt_index);
        }
        while (next_rank <= P->ingress.size()) R.unpack_rank_begin[next_rank++] = (uint32_t)R.unpack.tiles.size();
        if (!pk.ok || !up.ok) return fail(WB_ERR_INVALID_ARG);
        assign_ctas(&R.pack, P->grid);
        assign_ctas(&R.unpack, P->grid);
        P->stats.n_tiles_pack += R.pack.tiles.size();
        P->stats.n_tiles_unpack += R.unpack.tiles.size();
        P->stats.bucket_bytes_total += R.bucket_bytes;
        P->stats.bucket_bytes_max = std::max<uint64_t>(P->stats.bucket_bytes_max, R.bucket_bytes);
      }
    }

    // ---- statistics ----------------------------------------------------------------------------------
    P->stats.n_rounds = P->rounds.size();
    P->stats.n_tiles_remap = P->remap.tiles.size();
    P->stats.grid_ctas = P->grid;
    P->stats.tile_bytes = P->opts.tile_bytes;
    P->stats.remap_cta_bytes_max = P->remap.bytes_max_cta;
    P->stats.remap_cta_bytes_mean = P->remap.bytes_total / std::max<uint32_t>(P->grid, 1);
    auto table_bytes = [&](const TileTable& t) {
      return t.tiles.size() * sizeof(DTile) + t.extras.size() * sizeof(DDst) +
             t.cta_begin.size() * sizeof(uint32_t);
    };
    P->stats.table_bytes = table_bytes(P->remap);
    for (const Round& R : P->rounds) P->stats.table_bytes += table_bytes(R.pack) + table_bytes(R.unpack);
    P->stats.build_seconds =
        std::chrono::duration<double>(std::chrono::steady_clock::now() - t_start).count();
  } catch (const std::bad_alloc&) {
    return fail(WB_ERR_OOM);
  }
  *out = P;
  return WB_OK;
}

extern "C" void wb_plan_free(wb_plan* plan) {
  if (!plan) return;
  wbi::release_device_tables(plan);
  delete plan;
}

extern "C" wb_status wb_plan_stats(const wb_plan* plan, wb_plan_stats_t* out) {
  if (!plan || !out) return WB_ERR_INVALID_ARG;
  *out = plan->stats;
  return WB_OK;
}

extern "C" wb_status wb_plan_rank_bytes(const wb_plan* plan, int side, uint32_t rank, uint64_t* out) {
  if (!plan || !out || (side != 0 && side != 1)) return WB_ERR_INVALID_ARG;
  const auto& v = side == 0 ? plan->egress : plan->ingress;
  if (rank >= v.size()) return WB_ERR_INVALID_ARG;
  *out = v[rank];
  return WB_OK;
}

extern "C" size_t wb_plan_num_rounds(const wb_plan* plan) { return plan ? plan->rounds.size() : 0; }

extern "C" size_t wb_plan_bucket_bytes(const wb_plan* plan, size_t round) {
  if (!plan || round >= plan->rounds.size()) return 0;
  return plan->rounds[round].bucket_bytes;
}

extern "C" wb_status wb_plan_bucket_entries(const wb_plan* plan, size_t round, wb_bucket_entry* out,
                                            size_t cap, size_t* n) {
  if (!plan || !n || round >= plan->rounds.size()) return WB_ERR_INVALID_ARG;
  const Round& R = plan->rounds[round];
  *n = R.payloads.size();
  if (!out) return WB_OK;
  for (size_t k = 0; k < R.payloads.size() && k < cap; ++k) {
    const Payload& p = R.payloads[k];
    const Slab& sl = plan->slabs[p.slab];
    wb_bucket_entry e{};
    e.sender = sl.sender;
    e.receiver = sl.receiver;
    e.ckpt_tensor = plan->dst.ckpts[sl.ckpt_index].id;
    e.r0 = p.rect.r0; e.c0 = p.rect.c0; e.nr = p.rect.nr; e.nc = p.rect.nc;
    e.bucket_off = p.bucket_off;
    e.dtype = plan->dst.dtype;
    e.n_dst = sl.dst_count;
    out[k] = e;
  }
  return WB_OK;
}

extern "C" wb_status wb_plan_bucket_regions(const wb_plan* plan, size_t round, wb_bucket_region* out, size_t cap,
                                            size_t* n) {
  if (!plan || !n || round >= plan->rounds.size()) return WB_ERR_INVALID_ARG;
  const Round& R = plan->rounds[round];
  *n = R.regions.size();
  if (!out) return WB_OK;
  for (size_t k = 0; k < R.regions.size() && k < cap; ++k) {
    const Region& g = R.regions[k];
    out[k] = wb_bucket_region{g.receiver, g.sender, g.off, g.bytes};
  }
  return WB_OK;
}

extern "C" wb_status wb_plan_num_ranks(const wb_plan* plan, uint32_t* n_trainer, uint32_t* n_rollout) {
  if (!plan || !n_trainer || !n_rollout) return WB_ERR_INVALID_ARG;
  *n_trainer = (uint32_t)plan->egress.size();
  *n_rollout = (uint32_t)plan->ingress.size();
  return WB_OK;
}

static const TileTable* pick_table(const wb_plan* plan, int which, size_t round) {
  if (which == WB_TABLE_REMAP) return &plan->remap;
  if (round >= plan->rounds.size()) return nullptr;
  if (which == WB_TABLE_PACK) return &plan->rounds[round].pack;
  if (which == WB_TABLE_UNPACK) return &plan->rounds[round].unpack;
  return nullptr;
}

extern "C" wb_status wb_plan_tiles(const wb_plan* plan, int which, size_t round, wb_tile_view* out,
                                   size_t cap, size_t* n) {
  if (!plan || !n) return WB_ERR_INVALID_ARG;
  const TileTable* T = pick_table(plan, which, round);
  if (!T) return WB_ERR_INVALID_ARG;
  size_t count = 0;
  for (const HTile& t : T->tiles) {
    for (uint32_t d = 0; d <= t.n_extra; ++d, ++count) {
      if (!out || count >= cap) continue;
      wb_tile_view v{};
      v.src_tensor = t.src_tensor; v.src_off = t.src_off;
      v.nr = t.nr; v.nc = t.nc; v.src_sr = t.ssr; v.src_sc = t.ssc;
      v.kind = t.kind; v.cta = t.cta;
      if (t.seam & kTileRowsBefore) v.flags |= WB_TILE_ROWS_BEFORE;
      if (t.seam & kTileRowsAfter) v.flags |= WB_TILE_ROWS_AFTER;
      if (d == 0) {
        v.dst_tensor = t.dst_tensor; v.dst_off = t.dst_off; v.dst_sr = t.dsr; v.dst_sc = t.dsc;
      } else {
        const HDst& x = T->extras[t.extra + d - 1];
        v.dst_tensor = x.tensor; v.dst_off = x.off; v.dst_sr = x.sr; v.dst_sc = x.sc;
        v.flags |= WB_TILE_FANOUT_CONT;
      }
      out[count] = v;
    }
  }
  *n = count;
  return WB_OK;
}

extern "C" wb_status wb_plan_rank_tiles(const wb_plan* plan, int which, size_t round, uint32_t rank, size_t* first,
                                        size_t* count) {
  if (!plan || !first || !count || round >= plan->rounds.size()) return WB_ERR_INVALID_ARG;
  if (which != WB_TABLE_PACK && which != WB_TABLE_UNPACK) return WB_ERR_INVALID_ARG;
  const Round& R = plan->rounds[round];
  const TileTable& T = which == WB_TABLE_PACK ? R.pack : R.unpack;
  const std::vector<uint32_t>& rb = which == WB_TABLE_PACK ? R.pack_rank_begin : R.unpack_rank_begin;
  if ((size_t)rank + 1 >= rb.size()) return WB_ERR_INVALID_ARG;
  // the listing has one entry per destination of a tile
  size_t a = 0, n = 0;
  for (uint32_t k = 0; k < rb[rank + 1]; ++k) (k < rb[rank] ? a : n) += 1 + T.tiles[k].n_extra;
  *first = a;
  *count = n;
  return WB_OK;
}

// =================================================================================================
// Verification by interval arithmetic, independent of how the tables were produced.
extern "C" wb_status wb_plan_verify(const wb_plan* plan) {
  if (!plan) return WB_ERR_INVALID_ARG;
  const wb_layout& S = plan->src;
  const wb_layout& D = plan->dst;
  try {
    // (1) slabs of one checkpoint tensor are pairwise disjoint: every id is read at most once
    {
      std::vector<uint32_t> idx(plan->slabs.size());
      std::iota(idx.begin(), idx.end(), 0);
      std::stable_sort(idx.begin(), idx.end(), [&](uint32_t a, uint32_t b) {
        const Slab& x = plan->slabs[a]; const Slab& y = plan->slabs[b];
        if (x.ckpt_index != y.ckpt_index) return x.ckpt_index < y.ckpt_index;
        return x.rect.r0 < y.rect.r0;
      });
      for (size_t i = 0; i < idx.size(); ++i) {
        const Slab& a = plan->slabs[idx[i]];
        for (size_t j = i + 1; j < idx.size(); ++j) {
          const Slab& b = plan->slabs[idx[j]];
          if (b.ckpt_index != a.ckpt_index || b.rect.r0 >= a.rect.r1()) break;
          if (intersect(a.rect, b.rect, nullptr)) return WB_ERR_INTERNAL;
        }
      }
    }
    // (2) every slab lies inside its source slice and inside each destination slice
    uint64_t written = 0, described = 0;
    for (const Slab& sl : plan->slabs) {
      Rect x;
      const NSlice& s = S.slices[sl.src_slice];
      if (S.ckpts[s.ckpt_index].id != D.ckpts[sl.ckpt_index].id) return WB_ERR_INTERNAL;
      if (!intersect(sl.rect, s.rect, &x) || x.area() != sl.rect.area()) return WB_ERR_INTERNAL;
      for (uint32_t d = 0; d < sl.dst_count; ++d) {
        const NSlice& t = D.slices[plan->slab_dsts[sl.dst_begin + d]];
        if (t.ckpt_index != sl.ckpt_index) return WB_ERR_INTERNAL;
        if (!intersect(sl.rect, t.rect, &x) || x.area() != sl.rect.area()) return WB_ERR_INTERNAL;
        written += sl.rect.area();
      }
    }
    for (const NSlice& t : D.slices) described += t.rect.area();
    if (written != described) return WB_ERR_INTERNAL;   // with (1): each described element once
    // (3) tables: inside their tensors, destinations disjoint, element totals match
    auto check_table = [&](const TileTable& T, bool src_bucket, bool dst_bucket, uint64_t bucket_elems,
                           uint64_t want_read, uint64_t want_written) -> bool {
      std::vector<Footprint> dstf, srcf;
      uint64_t rd = 0, wr = 0;
      if (T.cta_begin.size() != plan->grid + 1 || T.cta_begin.back() != T.tiles.size()) return false;
      for (size_t k = 0; k < T.tiles.size(); ++k) {
        const HTile& t = T.tiles[k];
        if (t.cta >= plan->grid || k < T.cta_begin[t.cta] || k >= T.cta_begin[t.cta + 1]) return false;
        auto inside = [&](int32_t tensor, bool bucket, const wb_layout& L, uint64_t off, uint32_t sr,
                          uint32_t sc) {
          uint64_t last = off + (uint64_t)(t.nr - 1) * sr + (uint64_t)(t.nc - 1) * sc;
          if (bucket) return tensor == -1 && last < bucket_elems;
          return tensor >= 0 && (size_t)tensor < L.tensors.size() && last < L.tensors[tensor].numel;
        };
        if (!inside(t.src_tensor, src_bucket, S, t.src_off, t.ssr, t.ssc)) return false;
        if (!inside(t.dst_tensor, dst_bucket, D, t.dst_off, t.dsr, t.dsc)) return false;
        srcf.push_back(footprint(t.src_tensor, t.src_off, t.nr, t.nc, t.ssr, t.ssc));
        dstf.push_back(footprint(t.dst_tensor, t.dst_off, t.nr, t.nc, t.dsr, t.dsc));
        rd += (uint64_t)t.nr * t.nc;
        wr += (uint64_t)t.nr * t.nc * (1 + t.n_extra);
        for (uint32_t d = 0; d < t.n_extra; ++d) {
          const HDst& x = T.extras[t.extra + d];
          if (!inside(x.tensor, dst_bucket, D, x.off, x.sr, x.sc)) return false;
          dstf.push_back(footprint(x.tensor, x.off, t.nr, t.nc, x.sr, x.sc));
        }
      }
      if (rd != want_read || wr != want_written) return false;
      if (any_overlap(dstf)) return false;
      if (any_overlap(srcf)) return false;
      return true;
    };
    if (!check_table(plan->remap, false, false, 0, plan->stats.src_elems_read, plan->stats.dst_elems_written))
      return WB_ERR_INTERNAL;
    uint64_t rd = 0, wr = 0;
    const uint32_t ed = D.dtype == WB_F32 ? 4 : 2;
    for (const Round& R : plan->rounds) {
      uint64_t elems = 0, elems_w = 0;
      for (const Payload& p : R.payloads) {
        elems += p.rect.area();
        elems_w += p.rect.area() * plan->slabs[p.slab].dst_count;
        if (p.bucket_off % 16 || p.bucket_off + p.rect.area() * ed > R.bucket_bytes) return WB_ERR_INTERNAL;
      }
      if (R.bucket_bytes > plan->opts.bucket_budget_bytes) return WB_ERR_INTERNAL;
      if (!check_table(R.pack, false, true, R.bucket_bytes / ed, elems, elems)) return WB_ERR_INTERNAL;
      if (!check_table(R.unpack, true, false, R.bucket_bytes / ed, elems, elems_w)) return WB_ERR_INTERNAL;
      // (4) rank partition: regions tile the bucket in order; a sender rank's pack tiles read only that
      // rank's tensors and write only its regions; a receiver rank's unpack tiles read only its regions
      {
        uint64_t end = 0;
        for (const Region& g : R.regions) {
          if (g.off % kRegionAlign || g.off < end || g.off + g.bytes > R.bucket_bytes) return WB_ERR_INTERNAL;
          end = g.off + g.bytes;
        }
        auto region_of = [&](uint64_t byte_lo, uint64_t byte_hi) -> const Region* {
          for (const Region& g : R.regions)
            if (byte_lo >= g.off && byte_hi <= g.off + g.bytes) return &g;
          return nullptr;
        };
        auto span = [&](uint64_t off, const HTile& t, uint32_t sr, uint32_t sc, uint64_t* lo, uint64_t* hi) {
          *lo = off * ed;
          *hi = (off + (uint64_t)(t.nr - 1) * sr + (uint64_t)(t.nc - 1) * sc + 1) * ed;
        };
        if (R.pack_rank_begin.size() != plan->egress.size() + 1 || R.pack_rank_begin.back() != R.pack.tiles.size())
          return WB_ERR_INTERNAL;
        if (R.unpack_rank_begin.size() != plan->ingress.size() + 1 || R.unpack_rank_begin.back() != R.unpack.tiles.size())
          return WB_ERR_INTERNAL;
        for (size_t rank = 0; rank + 1 < R.pack_rank_begin.size(); ++rank)
          for (uint32_t k = R.pack_rank_begin[rank]; k < R.pack_rank_begin[rank + 1]; ++k) {
            const HTile& t = R.pack.tiles[k];
            uint64_t lo, hi;
            span(t.dst_off, t, t.dsr, t.dsc, &lo, &hi);
            const Region* g = region_of(lo, hi);
            if (S.tensors[t.src_tensor].rank != rank || !g || g->sender != rank) return WB_ERR_INTERNAL;
          }
        for (size_t rank = 0; rank + 1 < R.unpack_rank_begin.size(); ++rank)
          for (uint32_t k = R.unpack_rank_begin[rank]; k < R.unpack_rank_begin[rank + 1]; ++k) {
            const HTile& t = R.unpack.tiles[k];
            uint64_t lo, hi;
            span(t.src_off, t, t.ssr, t.ssc, &lo, &hi);
            const Region* g = region_of(lo, hi);
            if (!g || g->receiver != rank) return WB_ERR_INTERNAL;
          }
      }
      rd += elems; wr += elems_w;
    }
    if (rd != plan->stats.src_elems_read || wr != plan->stats.dst_elems_written) return WB_ERR_INTERNAL;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  return WB_OK;
}


// =================================================================================================
// Three-stage routing, traffic accounting (Section 3.2).
extern "C" wb_status wb_route_account(const wb_plan* plan, const uint32_t* trainer_node, size_t n_trainer_ranks,
                                      const uint32_t* rollout_node, size_t n_rollout_ranks, double trainer_gbs,
                                      double node_gbs, wb_route_stats_t* out, uint64_t* node_rdma_ingress,
                                      uint64_t* node_required, size_t n_nodes) {
  if (!plan || !trainer_node || !rollout_node || !out || n_nodes == 0) return WB_ERR_INVALID_ARG;
  if (n_trainer_ranks < plan->egress.size() || n_rollout_ranks < plan->ingress.size()) return WB_ERR_INVALID_ARG;
  for (size_t r = 0; r < n_trainer_ranks; ++r) if (trainer_node[r] >= n_nodes) return WB_ERR_INVALID_ARG;
  for (size_t r = 0; r < n_rollout_ranks; ++r) if (rollout_node[r] >= n_nodes) return WB_ERR_INVALID_ARG;
  try {
    const uint64_t ed = plan->dst.dtype == WB_F32 ? 4 : 2;
    wb_route_stats_t st{};
    std::vector<uint64_t> t_egress(n_trainer_ranks, 0), r_rdma(n_rollout_ranks, 0);
    std::vector<uint64_t> node_in(n_nodes, 0), node_req(n_nodes, 0);
    std::vector<uint32_t> nodes, per_node;
    for (const Slab& sl : plan->slabs) {
      const uint64_t bytes = sl.rect.area() * ed;
      st.model_bytes += bytes;
      // stage 1: trainer rank -> designated receiver
      st.receive_bytes += bytes;
      t_egress[sl.sender] += bytes;
      const uint32_t home = rollout_node[sl.receiver];
      if (trainer_node[sl.sender] != home) { r_rdma[sl.receiver] += bytes; node_in[home] += bytes; }
      // the rollout nodes that need this slab, and how many of their ranks do
      nodes.clear(); per_node.clear();
      for (uint32_t d = 0; d < sl.dst_count; ++d) {
        const uint32_t rank = plan->dst.tensors[plan->dst.slices[plan->slab_dsts[sl.dst_begin + d]].tensor].rank;
        const uint32_t nd = rollout_node[rank];
        size_t k = 0;
        while (k < nodes.size() && nodes[k] != nd) ++k;
        if (k == nodes.size()) { nodes.push_back(nd); per_node.push_back(0); }
        per_node[k]++;
        // without exchange stages every rank pulls the slab itself
        if (trainer_node[sl.sender] != nd) st.direct_rdma_bytes += bytes;
      }
      for (size_t k = 0; k < nodes.size(); ++k) {
        node_req[nodes[k]] += bytes;
        if (nodes[k] != home) {               // stage 2: once into every other node that needs it
          st.external_bytes += bytes;
          node_in[nodes[k]] += bytes;
          // the designated receiver's counterpart takes it: the destination rank of that node
          // with the same position (in rank order) as the receiver has in its own node
          uint32_t pos = 0;
          std::vector<uint32_t> there;
          for (uint32_t d = 0; d < sl.dst_count; ++d) {
            const uint32_t rank = plan->dst.tensors[plan->dst.slices[plan->slab_dsts[sl.dst_begin + d]].tensor].rank;
            if (rollout_node[rank] == nodes[k]) there.push_back(rank);
            if (rollout_node[rank] == home && rank < sl.receiver) ++pos;
          }
          std::sort(there.begin(), there.end());
          r_rdma[there[pos % there.size()]] += bytes;
        }
        st.internal_bytes += bytes * (per_node[k] - 1);   // stage 3: the node's other ranks
      }
    }
    for (uint64_t v : t_egress) st.max_trainer_rank_egress = std::max(st.max_trainer_rank_egress, v);
    for (uint64_t v : r_rdma) st.max_rollout_rank_rdma_ingress = std::max(st.max_rollout_rank_rdma_ingress, v);
    double worst = 0;
    for (size_t v = 0; v < n_nodes; ++v) {
      st.max_node_rdma_ingress = std::max(st.max_node_rdma_ingress, node_in[v]);
      if (node_gbs > 0) worst = std::max(worst, node_req[v] / (node_gbs * 1e9));
      if (node_rdma_ingress) node_rdma_ingress[v] = node_in[v];
      if (node_required) node_required[v] = node_req[v];
    }
    if (trainer_gbs > 0) worst = std::max(worst, st.model_bytes / (trainer_gbs * 1e9));
    st.t_min_seconds = worst;
    *out = st;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  return WB_OK;
}
