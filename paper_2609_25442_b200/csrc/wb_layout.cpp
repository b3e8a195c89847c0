// Source-map ingestion (Section 3.1: a source map is a sequence of slice-copy operations,
// each optionally transposed).  Host only.
#include <algorithm>
#include <new>
#include <numeric>

#include "wb_internal.h"

using namespace wbi;

extern "C" const char* wb_status_str(wb_status s) {
  switch (s) {
    case WB_OK: return "ok";
    case WB_ERR_INVALID_ARG: return "invalid argument";
    case WB_ERR_DTYPE: return "unsupported or mixed dtype";
    case WB_ERR_SHAPE_MISMATCH: return "checkpoint tensor described with two shapes";
    case WB_ERR_OUT_OF_RANGE: return "slice out of range";
    case WB_ERR_DST_OVERLAP: return "destination element described twice";
    case WB_ERR_UNCOVERED: return "destination element not held by any source";
    case WB_ERR_BUCKET_TOO_SMALL: return "bucket budget too small";
    case WB_ERR_OOM: return "out of memory";
    case WB_ERR_CUDA: return "CUDA error";
    case WB_ERR_NOT_BOUND: return "plan not bound to device memory";
    case WB_ERR_INTERNAL: return "plan invariant violated";
    case WB_ERR_STATIC_LIMIT: return "tile table larger than the static scratch array";
    case WB_ERR_REPLICA_MISMATCH: return "trainer replicas of a checkpoint region differ";
  }
  return "unknown status";
}

extern "C" const char* wb_version(void) { return "wb 0.1 (sm_100a)"; }

static wb_status normalise(const wb_slice& s, const wb_tensor_desc& t, NSlice* out) {
  const uint64_t nr = s.nr, nc = s.nc;
  bool transposed;
  uint64_t pitch;
  if (nr == 1 && nc == 1) {
    transposed = false; pitch = 1;
  } else if (nc == 1) {            // one column of nr elements, spaced stride_r apart
    if (s.stride_r < 1) return WB_ERR_INVALID_ARG;
    if (s.stride_r == 1) { transposed = true; pitch = nr; }   // contiguous run along i
    else { transposed = false; pitch = (uint64_t)s.stride_r; }
  } else if (nr == 1) {            // one row of nc elements, spaced stride_c apart
    if (s.stride_c < 1) return WB_ERR_INVALID_ARG;
    if (s.stride_c == 1) { transposed = false; pitch = nc; }
    else { transposed = true; pitch = (uint64_t)s.stride_c; }
  } else if (s.stride_c == 1 && s.stride_r >= (int64_t)nc) {
    transposed = false; pitch = (uint64_t)s.stride_r;
  } else if (s.stride_r == 1 && s.stride_c >= (int64_t)nr) {
    transposed = true; pitch = (uint64_t)s.stride_c;
  } else {
    return WB_ERR_INVALID_ARG;
  }
  // last element touched
  const uint64_t outer = transposed ? nc : nr, inner = transposed ? nr : nc;
  if (outer > 1 && pitch >= (1ull << 32)) return WB_ERR_INVALID_ARG;   // a single run has no pitch
  // overflow-safe: outer, pitch < 2^63 / numel checks below
  const unsigned __int128 last = (unsigned __int128)s.local_off +
                                 (unsigned __int128)(outer - 1) * pitch + (inner - 1);
  if (last >= t.numel) return WB_ERR_OUT_OF_RANGE;
  out->tensor = s.tensor;
  out->off = s.local_off;
  out->pitch = pitch;
  out->transposed = transposed;
  out->rect = Rect{s.r0, s.c0, nr, nc};
  return WB_OK;
}

extern "C" wb_status wb_layout_describe(const wb_tensor_desc* tensors, size_t n_tensors,
                                        const wb_slice* slices, size_t n_slices,
                                        wb_layout** out) {
  if (!out || (!tensors && n_tensors) || (!slices && n_slices)) return WB_ERR_INVALID_ARG;
  if (n_tensors >= (1ull << 31) || n_slices >= (1ull << 32)) return WB_ERR_INVALID_ARG;
  wb_layout* L = new (std::nothrow) wb_layout();
  if (!L) return WB_ERR_OOM;
  try {
    L->tensors.assign(tensors, tensors + n_tensors);
    for (size_t i = 0; i < n_tensors; ++i) {
      if (tensors[i].dtype != WB_F32 && tensors[i].dtype != WB_BF16) { delete L; return WB_ERR_DTYPE; }
      if (i == 0) L->dtype = tensors[i].dtype;
      else if (tensors[i].dtype != L->dtype) { delete L; return WB_ERR_DTYPE; }
      L->n_ranks = std::max(L->n_ranks, tensors[i].rank + 1);
    }
    // checkpoint tensor ids -> compact indices, with one shape each
    std::vector<uint32_t> order;
    order.reserve(n_slices);
    for (size_t k = 0; k < n_slices; ++k) {
      const wb_slice& s = slices[k];
      if (s.reserved != 0 || s.tensor >= n_tensors) { delete L; return WB_ERR_INVALID_ARG; }
      if (s.nr == 0 || s.nc == 0) continue;
      // rectangle inside its checkpoint tensor (overflow-safe comparisons)
      if (s.r0 >= s.ckpt_rows || s.nr > s.ckpt_rows - s.r0 ||
          s.c0 >= s.ckpt_cols || s.nc > s.ckpt_cols - s.c0) { delete L; return WB_ERR_OUT_OF_RANGE; }
      if (s.ckpt_rows >= (1ull << 40) || s.ckpt_cols >= (1ull << 40)) { delete L; return WB_ERR_INVALID_ARG; }
      order.push_back((uint32_t)k);
    }
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
      return slices[a].ckpt_tensor < slices[b].ckpt_tensor;
    });
    L->slices.reserve(order.size());
    L->by_ckpt.resize(order.size());
    for (size_t p = 0; p < order.size(); ++p) {
      const wb_slice& s = slices[order[p]];
      if (L->ckpts.empty() || L->ckpts.back().id != s.ckpt_tensor) {
        L->ckpts.push_back(CkptInfo{s.ckpt_tensor, s.ckpt_rows, s.ckpt_cols, (uint32_t)p, 0});
      } else if (L->ckpts.back().rows != s.ckpt_rows || L->ckpts.back().cols != s.ckpt_cols) {
        delete L; return WB_ERR_SHAPE_MISMATCH;
      }
      L->ckpts.back().count++;
      NSlice ns{};
      wb_status st = normalise(s, tensors[s.tensor], &ns);
      if (st != WB_OK) { delete L; return st; }
      ns.ckpt_index = (uint32_t)(L->ckpts.size() - 1);
      L->slices.push_back(ns);
      L->by_ckpt[p] = (uint32_t)p;   // slices are stored already grouped by checkpoint tensor
    }
  } catch (const std::bad_alloc&) {
    delete L;
    return WB_ERR_OOM;
  }
  *out = L;
  return WB_OK;
}

extern "C" void wb_layout_free(wb_layout* layout) { delete layout; }

// A flat range of a row-major matrix in checkpoint coordinates: the rest of the first row, the full
// rows, the start of the last row (Section 3.1 slice copies of a flat shard).
extern "C" wb_status wb_layout_add_flat_range(uint32_t tensor, uint64_t local_off, uint64_t ckpt_tensor,
                                              uint64_t ckpt_rows, uint64_t ckpt_cols, uint64_t begin, uint64_t end,
                                              wb_slice* out, size_t cap, size_t* n_out) {
  if (!n_out || ckpt_cols == 0) return WB_ERR_INVALID_ARG;
  const unsigned __int128 numel = (unsigned __int128)ckpt_rows * ckpt_cols;
  if (begin > end || (unsigned __int128)end > numel) return WB_ERR_OUT_OF_RANGE;
  wb_slice tmp[3];
  size_t n = 0;
  auto rect = [&](uint64_t r0, uint64_t c0, uint64_t nr, uint64_t nc) {
    wb_slice s{};
    s.tensor = tensor;
    s.local_off = local_off + (r0 * ckpt_cols + c0 - begin);
    s.stride_r = (int64_t)nc;
    s.stride_c = 1;
    s.ckpt_tensor = ckpt_tensor; s.ckpt_rows = ckpt_rows; s.ckpt_cols = ckpt_cols;
    s.r0 = r0; s.c0 = c0; s.nr = nr; s.nc = nc;
    tmp[n++] = s;
  };
  if (end > begin) {
    uint64_t rb = begin / ckpt_cols, cb = begin % ckpt_cols;
    const uint64_t re = end / ckpt_cols, ce = end % ckpt_cols;
    if (rb == re) {
      rect(rb, cb, 1, end - begin);
    } else {
      if (cb) { rect(rb, cb, 1, ckpt_cols - cb); ++rb; }
      if (re > rb) rect(rb, 0, re - rb, ckpt_cols);
      if (ce) rect(re, 0, 1, ce);
    }
  }
  if (out) {
    if (cap < n) return WB_ERR_INVALID_ARG;
    for (size_t k = 0; k < n; ++k) out[k] = tmp[k];
  }
  *n_out = n;
  return WB_OK;
}
