// Internal data structures shared by the host planner and the CUDA executor.
#pragma once

#include <cstdint>
#include <cstddef>
#include <string>
#include <unordered_map>
#include <vector>

#include "wb.h"

namespace wbi {

struct Rect {
  uint64_t r0, c0, nr, nc;
  uint64_t area() const { return nr * nc; }
  uint64_t r1() const { return r0 + nr; }
  uint64_t c1() const { return c0 + nc; }
};

inline bool intersect(const Rect& a, const Rect& b, Rect* out) {
  uint64_t r0 = a.r0 > b.r0 ? a.r0 : b.r0;
  uint64_t c0 = a.c0 > b.c0 ? a.c0 : b.c0;
  uint64_t r1 = a.r1() < b.r1() ? a.r1() : b.r1();
  uint64_t c1 = a.c1() < b.c1() ? a.c1() : b.c1();
  if (r1 <= r0 || c1 <= c0) return false;
  if (out) *out = Rect{r0, c0, r1 - r0, c1 - c0};
  return true;
}

// A validated slice-copy operation.  Checkpoint element (r0+i, c0+j) is local element
// off + i*pitch + j (rows contiguous) or off + j*pitch + i (transposed: columns contiguous).
struct NSlice {
  uint32_t tensor;
  uint32_t ckpt_index;   // index into wb_layout::ckpts
  uint64_t off;
  uint64_t pitch;
  bool transposed;
  Rect rect;
  uint64_t elem(uint64_t r, uint64_t c) const {
    uint64_t i = r - rect.r0, j = c - rect.c0;
    return transposed ? off + j * pitch + i : off + i * pitch + j;
  }
  uint64_t sr() const { return transposed ? 1 : pitch; }
  uint64_t sc() const { return transposed ? pitch : 1; }
};

struct CkptInfo {
  uint64_t id, rows, cols;
  uint32_t first, count;   // range in wb_layout::by_ckpt
};

}  // namespace wbi

struct wb_layout {
  std::vector<wb_tensor_desc> tensors;
  std::vector<wbi::NSlice> slices;
  std::vector<wbi::CkptInfo> ckpts;        // sorted by id
  std::vector<uint32_t> by_ckpt;           // slice indices grouped by checkpoint tensor
  uint32_t dtype = 0;                      // uniform element type of the side
  uint32_t n_ranks = 0;
};

namespace wbi {

enum : uint32_t { KIND_ROWS = 0, KIND_TRANS = 1, KIND_ELEM = 2 };

// Which transposing tiles the executor stages through shared memory in chunks (the others are
// transposed by single warps): tiles that move at least kBatchTileBytes, with source rows of at least
// kTransMinPieceBytes and at least kTransMinRows of them, and one destination.  The planner needs
// the same rule: only between two staged tiles may a 16-byte destination window cross a seam.
#ifndef WB_TRANS_MIN_PIECE
#define WB_TRANS_MIN_PIECE 128
#endif
#ifndef WB_BATCH_TILE_BYTES
#define WB_BATCH_TILE_BYTES 8192
#endif
constexpr uint32_t kTransMinPieceBytes = WB_TRANS_MIN_PIECE;
constexpr uint32_t kTransMinRows = 16;
constexpr uint32_t kBatchTileBytes = WB_BATCH_TILE_BYTES;   // tiles moving less than this are batched, one warp per tile
inline bool staged_transposition(uint32_t kind, uint32_t n_extra, uint64_t nr, uint64_t nc, uint32_t es, uint32_t ed) {
  return kind == KIND_TRANS && n_extra == 0 && nc * es >= kTransMinPieceBytes && nr >= kTransMinRows &&
         nr * nc * (es + ed) >= kBatchTileBytes;
}

// Resident thread blocks per SM the executor kernel is compiled for; the planner's default
// grid is kNumSMs * kCtasPerSM so that one launch is exactly one wave on a B200.
constexpr uint32_t kNumSMs = 148;
constexpr uint32_t kCtasPerSM = 1;

// Host form of a tile: tensor indices and element offsets (resolved to addresses at bind).
struct HTile {
  int32_t src_tensor, dst_tensor;     // -1 = bucket
  uint64_t src_off, dst_off;          // elements
  uint32_t nr, nc;
  uint32_t ssr, ssc, dsr, dsc;        // element strides over (i, j)
  uint32_t kind;
  uint32_t n_extra, extra;            // fan-out destinations beyond the first
  uint32_t seam;                      // kTileRowsBefore | kTileRowsAfter (staged transposing tiles)
  uint32_t cta;
  uint64_t bytes;                     // bytes moved (read + all writes)
};

struct HDst {
  int32_t tensor;
  uint64_t off;
  uint32_t sr, sc;
};

// Device form.  `src` / `dst` are absolute device addresses for bound tensors, or byte
// offsets into the bucket for the side of a pack / unpack table that is the bucket (the
// kernel adds the bucket base to every tile of such a table).
struct alignas(16) DTile {
  uint64_t src;
  uint64_t dst;
  uint32_t nr, nc;
  uint32_t ssr, ssc;
  uint32_t dsr, dsc;
  uint32_t kind_extra;   // kind | n_extra << 8 | kTileHasMaps | kTileRowsBefore | kTileRowsAfter
  uint32_t extra;        // first fan-out record, or (kTileHasMaps) the tile's first tensor map
};
constexpr uint32_t kTileHasMaps = 1u << 16;
// A transposing slab cut into tiles along its rows: the tile above / below continues the same
// destination runs and is staged too.  A 16-byte destination window that straddles such a seam is
// written whole by the tile that holds its first row (which reads the few source rows it needs from
// the tile below); the tile below leaves those rows alone.  Without the flags either tile writes its
// part of the window with element stores.
constexpr uint32_t kTileRowsBefore = 1u << 17, kTileRowsAfter = 1u << 18;
static_assert(sizeof(DTile) == 48, "tile descriptor is three 16-byte words");

struct alignas(16) DDst {
  uint64_t dst;
  uint32_t sr, sc;
};
static_assert(sizeof(DDst) == 16, "");

struct TileTable {
  std::vector<HTile> tiles;           // ordered by thread block, then checkpoint order
  std::vector<HDst> extras;
  std::vector<uint32_t> cta_begin;    // grid + 1 offsets into tiles
  uint64_t bytes_max_cta = 0, bytes_total = 0;
  // device copies (owned by the plan; allocated at bind)
  DTile* d_tiles = nullptr;
  DDst* d_extras = nullptr;
  uint32_t* d_cta_begin = nullptr;
  uint32_t* d_sched = nullptr;        // {next tile, blocks done} for dynamic scheduling
  char* d_maps = nullptr;             // tensor maps (128 bytes each) of the tiles flagged kTileHasMaps
};

struct Slab {
  uint32_t ckpt_index;      // into the destination layout's ckpts
  Rect rect;
  uint32_t src_slice;       // into source layout slices
  uint32_t dst_begin, dst_count;   // into wb_plan::slab_dsts (destination slice indices)
  uint32_t sender, receiver;       // virtual ranks
};

// Two source slices that hold the same checkpoint rectangle (replicas).
struct ReplicaPair { uint32_t slice_a, slice_b; Rect rect; };

// Device form of a replica pair: element (i, j) of the rectangle at a + (i*a_sr + j*a_sc)*es etc.
struct alignas(16) DCompare {
  uint64_t a, b;
  uint32_t nr, nc;
  uint32_t a_sr, a_sc, b_sr, b_sc;
  uint32_t pad[2];
};
static_assert(sizeof(DCompare) == 48, "");

struct Payload {
  uint32_t slab;
  Rect rect;
  uint64_t bucket_off;      // bytes
};

// wb_remap_host: a group of consecutive remap tiles and the byte spans it touches per tensor.
struct HostSpan { uint32_t tensor; uint64_t off, bytes; };
struct HostGroup {
  uint32_t tile_begin = 0, tile_end = 0;
  std::vector<HostSpan> src, dst;
};

// One (receiver, sender) region of a round's bucket: the bytes virtual trainer rank `sender` packs for
// virtual rollout rank `receiver` (what an exchange between GPUs would carry from one to the other).
struct Region { uint32_t receiver, sender; uint64_t off, bytes; };

struct Round {
  std::vector<Payload> payloads;      // ordered by (receiver, sender), then checkpoint order
  uint64_t bucket_bytes = 0;
  TileTable pack, unpack;
  std::vector<Region> regions;        // in bucket order
  // pack tiles are grouped by sender rank, unpack tiles by (designated) receiver rank:
  // rank k's tiles are [x_rank_begin[k], x_rank_begin[k + 1])
  std::vector<uint32_t> pack_rank_begin, unpack_rank_begin;
  // checkpoint tensor (index into the destination layout's ckpts) of every pack / unpack tile: the
  // quantising kernels look the tensor's scale up by it
  std::vector<uint32_t> pack_ckpt, unpack_ckpt;
};

}  // namespace wbi

struct wb_plan {
  wb_layout src, dst;                   // private copies
  wb_plan_opts opts{};
  std::vector<wbi::Slab> slabs;
  std::vector<uint32_t> slab_dsts;
  std::vector<wbi::Round> rounds;
  std::vector<wbi::ReplicaPair> replica_pairs;
  wbi::TileTable remap;
  std::vector<uint64_t> egress, ingress;
  wb_plan_stats_t stats{};
  uint32_t grid = 0;
  // binding
  bool bound = false;
  int device = -1;
  std::vector<const void*> src_base;
  std::vector<void*> dst_base;
  void* d_arena = nullptr;              // one device allocation holding every table
  uint32_t* d_err = nullptr;            // sticky device error word (inside the arena)
  wbi::DCompare* d_compare = nullptr;   // replica pairs (inside the arena)
  unsigned long long* d_mismatch = nullptr;
  // wb_remap_host pipeline state (created on first use; streams and events are CUDA handles)
  std::vector<wbi::HostGroup> host_groups;
  void* h2d_stream = nullptr;
  void* d2h_stream = nullptr;
  std::vector<void*> host_events;
  size_t arena_bytes = 0;
  void* quant_tables = nullptr;         // work lists of the FP8 bucket quantisation (wb_quant.cu), built on first use
};

namespace wbi {
// implemented in wb_exec.cu
void release_device_tables(wb_plan* plan);
// the plan's two internal streams and at least n_events events (created on first use)
wb_status ensure_pipeline(wb_plan* plan, size_t n_events);
// true if the current device is the one the plan's tables and tensors were bound on (a launch from
// another device would dereference addresses of the bound one)
bool on_bound_device(const wb_plan* plan);
// implemented in wb_quant.cu
void release_quant_tables(wb_plan* plan);
}
