// Executor, part 2 of 3: the shared-memory rings, what the producer tells the workers about a slot,
// and the worker-side routines (staged rows, staged and warp-level transposition, short rows,
// element-wise tiles).  Included by wb_exec.cu only.
#pragma once
#include "wb_exec_prims.cuh"

namespace {
constexpr int kWorkers = kThreads - 32;       // warps 1.. convert staged chunks and run queued tiles
// Shared-memory rings (tuned on B200; the direct ring is very sensitive: 3 x 32 KiB moves 5 % more
// than 4 x 16 KiB).  Kernels whose element sizes differ never use the direct ring and give all of
// it to the worker ring: five slots of 44 KiB, 220 of the 227 KiB a block can have - a slot is busy
// for a load's latency plus the workers' time on it, so the ring's depth sets the rate of the staged
// classes that are not DRAM-bound (transposition chunks: 4 x 48 KiB -> 5 x 44 KiB, + 4 %).
#ifndef WB_DIRECT_STAGES
#define WB_DIRECT_STAGES 3
#endif
#ifndef WB_DIRECT_BYTES
#define WB_DIRECT_BYTES 32768
#endif
#ifndef WB_SLOTS_SAME
#define WB_SLOTS_SAME 4
#endif
#ifndef WB_SLOT_BYTES_SAME
#define WB_SLOT_BYTES_SAME 32768
#endif
#ifndef WB_SLOTS_CAST
#define WB_SLOTS_CAST 5
#endif
#ifndef WB_SLOT_BYTES_CAST
#define WB_SLOT_BYTES_CAST 45056
#endif
constexpr int kDirectStages = WB_DIRECT_STAGES;   // bulk ring of the direct (load -> store) path
constexpr int kDirectBytes = WB_DIRECT_BYTES;
constexpr int kMaxSlots = WB_SLOTS_SAME > WB_SLOTS_CAST ? WB_SLOTS_SAME : WB_SLOTS_CAST;
template <int ES, int ED> struct Rings {      // worker ring: staged chunks and queued tiles
  static constexpr int kSlots = ES == ED ? WB_SLOTS_SAME : WB_SLOTS_CAST;
  static constexpr int kSlotBytes = ES == ED ? WB_SLOT_BYTES_SAME : WB_SLOT_BYTES_CAST;
  static constexpr size_t kDirect = ES == ED ? (size_t)kDirectStages * kDirectBytes : 0;
  static constexpr size_t kDyn = kDirect + (size_t)kSlots * kSlotBytes;
};
constexpr int kWorkerWarps = kWorkers / 32;
#ifndef WB_STAGED_MIN_ROW_BYTES
#define WB_STAGED_MIN_ROW_BYTES 1024
#endif
constexpr size_t kStagedMinRowBytes = WB_STAGED_MIN_ROW_BYTES;   // shorter rows take the warp-level path

enum : uint32_t { MODE_END = 0, MODE_COOP = 1, MODE_ROWS = 2, MODE_BATCH = 3, MODE_TRANS = 4, MODE_TRANS_TMA = 5 };
// Staged transposition: a chunk is kTransChunkBytes of consecutive source columns (the
// 16-byte aligned superset of a row piece is one 16-byte asynchronous copy per lane of the producer
// warp - bulk copies this small are limited by their issue rate) by as many source rows as fit a slot.  Row r of the chunk lands at r * kTransPitch + 16 * ((r / NV) & 7) in the slot
// (NV = destination elements per 16 bytes): the pitch is a multiple of 128 bytes, so lanes that
// read the same column NV rows apart - neighbouring 16-byte windows of one destination run - hit
// different banks.  kTransHalo rows past the chunk's own rows complete its last window.
#ifndef WB_TRANS_PIECE
#define WB_TRANS_PIECE 512
#endif
constexpr uint32_t kTransPiece = WB_TRANS_PIECE;                      // bytes one warp instruction copies per row (aligned superset)
constexpr uint32_t kTransPitch = kTransPiece + 128;
// source bytes of a chunk's row pieces: at most kTransPiece - 16 (the aligned superset must fit);
// 480 makes 120 four-byte columns x 8 windows = 960 windows, two for each of the 480 worker threads
constexpr uint32_t kTransChunkBytes = 480;
static_assert(kTransChunkBytes + 16 <= kTransPiece, "the aligned superset of a row piece must fit the copy");
constexpr uint32_t kTransHalo = 8;
constexpr uint32_t kTransMinPiece = kTransMinPieceBytes;   // narrower tiles stay with the warp-level transposition
// Staged transposition fed by tensor-map (TMA) loads.  A tensor map wants a 16-byte aligned base and
// row pitches that are multiples of 16 bytes, which arbitrary tiles do not have.  But eight times any
// pitch of 2- or 4-byte elements is such a multiple: the rows of a tile are dealt to kTmaClasses = 8
// classes by row index mod 8, and class q gets a map of its own - base = the 16-byte boundary at or
// before the first element of row q, pitch = 8 x the tile's pitch.  A chunk is then eight loads (one box
// of kTmaInner bytes x (rows / 8) per class) instead of a per-lane copy for every 16 bytes.  Class q's box
// sits at q * (class stride) in the slot, its rows kTmaInner bytes apart: lanes that read one column
// eight rows apart (neighbouring windows of a 2-byte destination run) are 124 words apart, on different
// banks.
constexpr uint32_t kTmaClasses = 8;
#ifndef WB_TMA_CHUNK_BYTES
#define WB_TMA_CHUNK_BYTES 480
#endif
constexpr uint32_t kTmaChunkBytes = WB_TMA_CHUNK_BYTES;   // source bytes of a chunk's row pieces
constexpr uint32_t kTmaInner = kTmaChunkBytes + 16;       // box width in bytes: the aligned superset of a row piece
static_assert(kTmaInner % 32 == 16, "box rows must be an odd multiple of 16 bytes apart (bank spread)");
constexpr uint32_t kBatchMaxTiles = 120;

// What the producer tells the workers about one ring slot.
struct ChunkDesc {
  uint32_t mode;
  uint32_t tile;      // MODE_COOP / MODE_BATCH: index of the (first) tile to run; MODE_TRANS: the chunk's own rows
  uint32_t nr, nc;    // staged chunk: rows in the stage, elements per row
  uint32_t pitch;     // bytes between rows in the stage
  uint32_t pad;       // MODE_TRANS: 1 if the chunk holds the first rows of its destination runs
  uint64_t src;       // global address of the chunk's first source element (alignment arithmetic only)
  uint64_t dst;       // global address of the chunk's first destination element
  uint64_t sps;       // source row pitch in bytes
  uint64_t dps;       // destination pitch in bytes: between rows (ROWS) or between columns (TRANS)
  uint4 raw[3];       // MODE_COOP: the tile's descriptor, so that the workers need not fetch it from global memory
};

__device__ __forceinline__ uint32_t roundup16(uint32_t x) { return (x + 15u) & ~15u; }

struct TileFields {
  const char* s;
  char* d;
  uint32_t nr, nc, ssr, ssc, dsr, dsc, kind, n_extra, extra;
  bool tmaps;          // `extra` is the index of the tile's first tensor map (staged transposition by TMA)
  bool rows_before, rows_after;   // see kTileRowsBefore
};
__device__ __forceinline__ TileFields decode(const TileRegs& r, uint64_t src_add, uint64_t dst_add) {
  TileFields f;
  f.s = reinterpret_cast<const char*>(((uint64_t)r.a.y << 32 | r.a.x) + src_add);
  f.d = reinterpret_cast<char*>(((uint64_t)r.a.w << 32 | r.a.z) + dst_add);
  f.nr = r.b.x; f.nc = r.b.y; f.ssr = r.b.z; f.ssc = r.b.w;
  f.dsr = r.c.x; f.dsc = r.c.y;
  f.kind = r.c.z & 0xFF; f.n_extra = (r.c.z >> 8) & 0xFF; f.extra = r.c.w;
  f.tmaps = (r.c.z & kTileHasMaps) != 0;
  f.rows_before = (r.c.z & kTileRowsBefore) != 0;
  f.rows_after = (r.c.z & kTileRowsAfter) != 0;
  return f;
}

// A tile the producer thread can move by itself with bulk copies: same element size, rows that
// are long enough, and source / destination congruent modulo 16 bytes in every row.
template <int ES, int ED>
__device__ __forceinline__ bool direct_ok(const TileFields& f) {
  if (ES != ED || f.kind != KIND_ROWS || f.n_extra != 0) return false;
  if ((((uintptr_t)f.s ^ (uintptr_t)f.d) & 15u) != 0) return false;
  if (f.nr > 1 && (((((size_t)f.ssr - (size_t)f.dsr) * ES) & 15u) != 0 || (size_t)f.nc * ES < 1024)) return false;
  return (size_t)f.nc * ES >= 256;
}

// 16 bytes starting `s` bytes into the 32-byte concatenation of v0 and v1 (s a multiple of 2).
__device__ __forceinline__ uint4 shift16(uint4 v0, uint4 v1, uint32_t s) {
  const uint32_t sb = (s & 3u) * 8u;
  uint32_t w0, w1, w2, w3, w4;
  switch (s >> 2) {
    case 0: w0 = v0.x; w1 = v0.y; w2 = v0.z; w3 = v0.w; w4 = v1.x; break;
    case 1: w0 = v0.y; w1 = v0.z; w2 = v0.w; w3 = v1.x; w4 = v1.y; break;
    case 2: w0 = v0.z; w1 = v0.w; w2 = v1.x; w3 = v1.y; w4 = v1.z; break;
    default: w0 = v0.w; w1 = v1.x; w2 = v1.y; w3 = v1.z; w4 = v1.w; break;
  }
  return make_uint4(__funnelshift_r(w0, w1, sb), __funnelshift_r(w1, w2, sb),
                    __funnelshift_r(w2, w3, sb), __funnelshift_r(w3, w4, sb));
}

// One full destination vector (NV elements) from a staged row: `row` is the 16-byte aligned
// shared-memory base of the row, `o` the byte offset of the first source element in it.
template <int ES, int ED>
__device__ __forceinline__ uint4 staged_unit(const char* row, uint32_t o) {
  const uint4* q = reinterpret_cast<const uint4*>(row + (o & ~15u));
  const uint32_t s = o & 15u;
  if constexpr (ES == ED) {
    const uint4 v0 = q[0];
    if (s == 0) return v0;
    return shift16(v0, q[1], s);
  } else if constexpr (ES == 4) {   // 32 source bytes -> 16 destination bytes
    uint4 a = q[0], b = q[1];
    if (s != 0) {
      const uint4 c = q[2];
      a = shift16(a, b, s);
      b = shift16(b, c, s);
    }
    return make_uint4(f32x2_to_bf16x2(a.x, a.y), f32x2_to_bf16x2(a.z, a.w),
                      f32x2_to_bf16x2(b.x, b.y), f32x2_to_bf16x2(b.z, b.w));
  } else {                          // 8 source bytes -> 16 destination bytes
    uint4 a = q[0];
    if (s != 0) a = shift16(a, (s > 8) ? q[1] : a, s);
    return make_uint4(a.x << 16, a.x & 0xFFFF0000u, a.y << 16, a.y & 0xFFFF0000u);
  }
}

// Workers: rows staged in shared memory -> destination rows.  Every row is cut into 16-byte
// aligned destination slots; full slots are one vector store, ragged first/last slots are
// element stores.  Threads are independent (no barrier).  `t` is the rotated worker thread index.
template <int ES, int ED>
__device__ __forceinline__ void staged_rows(const ChunkDesc& d, const char* stage, uint32_t t) {
  using E = Elem<ES, ED>;
  constexpr uint32_t NV = 16 / ED;
  const uint32_t n = d.nc;
  const uint32_t smax = (n + 2 * NV - 2) / NV;     // slots a row can touch
  const uint32_t lead0 = (uint32_t)d.src & 15u, dlead = (uint32_t)d.sps & 15u;
  // the slots of all rows, numbered row by row, are dealt to the threads in order: neighbouring
  // lanes take neighbouring slots of a row, and no lane idles at the end of a row.  A thread's slots are
  // kWorkers apart; (row, slot in row) advances incrementally, so there is one division per chunk, not per slot
  const uint32_t dr = (uint32_t)kWorkers / smax, dk = (uint32_t)kWorkers - dr * smax;
  uint32_t r = t / smax, k = t - r * smax;
  for (; r < d.nr; r += dr, k += dk) {
    if (k >= smax) {
      k -= smax;
      if (++r >= d.nr) break;
    }
    const uint64_t D = d.dst + (uint64_t)r * d.dps;
    const uint32_t a = (uint32_t)(D & 15u) / ED;   // elements of slot 0 that precede the row
    const int32_t e0 = (int32_t)(k * NV) - (int32_t)a;
    if (e0 >= (int32_t)n) continue;
    const char* row = stage + r * d.pitch;
    const uint32_t lead = (lead0 + r * dlead) & 15u;
    if (e0 >= 0 && (uint32_t)e0 + NV <= n) {
      st16(reinterpret_cast<char*>((D & ~(uint64_t)15) + 16u * k), staged_unit<ES, ED>(row, lead + (uint32_t)e0 * ES));
    } else {
      const uint32_t lo = e0 < 0 ? 0u : (uint32_t)e0;
      const uint32_t hi = min(n, (uint32_t)(e0 + (int32_t)NV));
      for (uint32_t e = lo; e < hi; ++e)
        E::store(reinterpret_cast<char*>(D) + (size_t)e * ED, E::load(row + lead + e * ES));
    }
  }
}

// Raw source element from shared memory (32-bit shared-space address) and its cast.
template <int ES> __device__ __forceinline__ uint32_t lds_raw(uint32_t saddr) {
  uint32_t v;
  if constexpr (ES == 4) {
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(saddr));
  } else {
    uint16_t h;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(saddr));
    v = h;
  }
  return v;
}
template <int ES, int ED> __device__ __forceinline__ typename Elem<ES, ED>::V cast_raw(uint32_t raw) {
  if constexpr (ES == ED) return (typename Elem<ES, ED>::V)raw;
  else if constexpr (ES == 4) return f32_to_bf16(raw);
  else return raw << 16;
}
// A loop over compile-time indices (so that unrolled code can use immediate offsets).
template <int I> struct Idx { static constexpr int value = I; };
template <int I, int N, typename F> __device__ __forceinline__ void static_for(F&& fn) {
  if constexpr (I < N) {
    fn(Idx<I>{});
    static_for<I + 1, N>(fn);
  }
}

// two consecutive 2-byte destination elements packed in one word
template <int ES> __device__ __forceinline__ uint32_t pack_pair16(uint32_t lo, uint32_t hi) {
  if constexpr (ES == 4) return f32x2_to_bf16x2(lo, hi);
  else return lo | (hi << 16);
}

// Workers: transposing tile, dst[j*dsc + i] = cast(src[i*ssr + j]).  No block-wide step: every
// warp takes 32-column x RB-row blocks of the tile on its own.
//   phase A  lane = source column.  The warp reads row after row (32 consecutive elements per
//            load instruction, 16 loads in flight per lane, one batch ahead), casts, and writes
//            each value into its private patch of the ring slot, laid out as destination rows:
//            T[lane][row].
//   phase B  A run may start at any 2-/4-byte alignment in global memory; it is written in 16-byte
//            aligned windows, neighbouring lanes taking neighbouring windows of a run.  A block owns the windows that START in its
//            rows and reads up to NV-1 rows past its end to complete the last one, so neighbouring
//            blocks never share a window and almost every store is a full vector; only the two
//            ends of a whole run use element stores.
// The patch pitch is odd in 32-bit words, so lanes hit distinct banks in both phases.
template <int ES, int ED>
__device__ __forceinline__ void warp_transpose(const TileFields& f, char* patch, uint32_t patch_bytes,
                                               uint32_t warp, uint32_t nw, uint32_t lane) {
  // patch: this warp's private part of the ring slot; warp / nw: its share of the tile's blocks
  using E = Elem<ES, ED>;
  constexpr uint32_t NV = 16 / ED;
  constexpr uint32_t PER_WORD = 4 / ED;                     // destination elements per 32-bit word
  constexpr int UA = 16;                                    // rows per batch of loads
  // rows per block: as many as the warp's share of the slot allows next to the NV-1 halo rows
  // (multiple of 8, at most 64); no halo is needed when every run starts on a 16-byte boundary
  const uint32_t share = patch_bytes / 4;                    // words
  const bool aligned = (((uintptr_t)f.d | ((size_t)f.dsc * ED)) & 15u) == 0;
  // rows read past a block's end to complete its last window
  const uint32_t halo = aligned ? 0u : NV - 1, room = aligned ? 0u : 8u;
  const uint32_t rb = min(64u, ((share / 32 - 1) * PER_WORD - room) & ~7u);
  const uint32_t pitch_w = (rb + room) / PER_WORD + 1;      // odd: (rb+room)/PER_WORD is even
  const uint32_t tbase = smem_u32(patch);
  const uint32_t nbi = (f.nr + rb - 1) / rb, nbj = (f.nc + 31) / 32;
  const uint32_t nb = nbi * nbj;
  const size_t sps = (size_t)f.ssr * ES;
  if (warp >= nb) return;

  struct Block { uint32_t i0, j0, ni, nj, nl; };      // nl: rows loaded = own rows + halo
  auto block_of = [&](uint32_t b) {
    const uint32_t bi = b / nbj, bj = b - bi * nbj;
    const uint32_t i0 = bi * rb, ni = min(rb, f.nr - i0);
    return Block{i0, bj * 32, ni, min(32u, f.nc - bj * 32), min(ni + halo, f.nr - i0)};
  };
  // phase A, loads: UA rows of this lane's column into registers
  auto issue = [&](const Block& k, uint32_t r0, uint32_t (&dst)[UA]) {
    const char* src = f.s + ((size_t)(k.i0 + r0) * f.ssr + k.j0 + lane) * ES;
#pragma unroll
    for (int u = 0; u < UA; ++u) {
      dst[u] = 0;
      if (lane < k.nj && r0 + u < k.nl) {
        if constexpr (ES == 4) dst[u] = __ldcs(reinterpret_cast<const uint32_t*>(src + (size_t)u * sps));
        else dst[u] = __ldcs(reinterpret_cast<const uint16_t*>(src + (size_t)u * sps));
      }
    }
  };
  // phase A, stores: cast and write into the patch as destination row `lane`
  auto consume = [&](const Block& k, uint32_t r0, const uint32_t (&v)[UA]) {
    if (lane >= k.nj) return;
    const uint32_t trow = tbase + lane * pitch_w * 4;
    if constexpr (ED == 2) {
#pragma unroll
      for (int u = 0; u < UA; u += 2)
        if (r0 + u < k.nl)
          asm volatile("st.shared.u32 [%0], %1;" ::"r"(trow + (r0 + u) * 2), "r"(pack_pair16<ES>(v[u], v[u + 1])));
    } else {
#pragma unroll
      for (int u = 0; u < UA; ++u)
        if (r0 + u < k.nl)
          asm volatile("st.shared.u32 [%0], %1;" ::"r"(trow + (r0 + u) * 4), "r"((uint32_t)cast_raw<ES, ED>(v[u])));
    }
  };
  // phase B: the block's 16-byte windows (those that start inside its rows), numbered run by run,
  // are dealt to the lanes in order, so neighbouring lanes write neighbouring windows of one
  // destination run and a store instruction touches a few whole lines instead of 32 scattered
  // 16-byte pieces.
  auto phase_b = [&](const Block& k) {
    __syncwarp();
    const uint32_t wins = (k.ni + NV - 1) / NV;                    // windows per run, at most
    const uint32_t total = k.nj * wins;
    for (uint32_t idx = lane; idx < total; idx += 32) {
      const uint32_t j = idx / wins, w = idx - j * wins;
      char* run = f.d + (size_t)(k.j0 + j) * f.dsc * ED;            // element (j, 0) of the run
      const uint32_t a = (uint32_t)(((uintptr_t)run / ED + k.i0) & (NV - 1));   // offset of row i0 in its window
      const uint32_t lead = a ? NV - a : 0;                        // rows before the first window that starts here
      const uint32_t trow = tbase + j * pitch_w * 4;
      // those rows belong to the previous block's last window, except at the very start of the run
      if (w == 0 && k.i0 == 0)
        for (uint32_t e = 0; e < min(lead, k.ni); ++e)
          E::store(run + (size_t)e * ED, (typename E::V)lds_raw<ED>(trow + e * ED));
      const uint32_t e0 = lead + w * NV;
      if (e0 >= k.ni) continue;
      char* out = run + (size_t)(k.i0 + e0) * ED;                  // 16-byte aligned
      if (e0 + NV <= k.nl) {
        uint4 x;
        if constexpr (ED == 4) {
          x.x = lds_raw<4>(trow + (e0 + 0) * 4); x.y = lds_raw<4>(trow + (e0 + 1) * 4);
          x.z = lds_raw<4>(trow + (e0 + 2) * 4); x.w = lds_raw<4>(trow + (e0 + 3) * 4);
        } else {
          const uint32_t p = trow + (e0 >> 1) * 4;
          const uint32_t w0 = lds_raw<4>(p), w1 = lds_raw<4>(p + 4), w2 = lds_raw<4>(p + 8), w3 = lds_raw<4>(p + 12);
          if (e0 & 1) {
            const uint32_t w4 = lds_raw<4>(p + 16);
            x = make_uint4(__funnelshift_r(w0, w1, 16), __funnelshift_r(w1, w2, 16),
                           __funnelshift_r(w2, w3, 16), __funnelshift_r(w3, w4, 16));
          } else {
            x = make_uint4(w0, w1, w2, w3);
          }
        }
        st16(out, x);
      } else {
        // the run ends inside this window
        for (uint32_t e = e0; e < k.nl; ++e)
          E::store(run + (size_t)(k.i0 + e) * ED, (typename E::V)lds_raw<ED>(trow + e * ED));
      }
    }
    __syncwarp();
  };

  // The rows of a block are short pieces (128 bytes) a row pitch apart, and a lane holds only two
  // batches of loads, which is not enough memory parallelism to cover DRAM latency.  So the warp asks
  // for the block after next to be brought into L2 ahead of time (lane = row; the first and the last
  // byte of the piece - a request per sector was measured to cost more than it brings): that costs
  // no registers, and the loads then hit L2.
  auto prefetch = [&](uint32_t pb) {
    if (pb >= nb) return;
    const Block k = block_of(pb);
    for (uint32_t r = lane; r < k.nl; r += 32) {
      const char* row = f.s + ((size_t)(k.i0 + r) * f.ssr + k.j0) * ES;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(row));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(row + (size_t)(k.nj - 1) * ES));
    }
  };
  // The warp's batches in order; the loads of batch q+1 are issued before batch q is consumed, so
  // they are in flight during the shared-memory writes and during phase B.
  uint32_t b = warp, r0 = 0;
  Block blk = block_of(b);
  prefetch(b + nw);
  auto step = [&](uint32_t (&cur)[UA], uint32_t (&nxt)[UA]) -> bool {
    uint32_t b2 = b, r2 = r0 + UA;
    Block blk2 = blk;
    const bool same = r2 < blk.nl;
    if (!same) { b2 = b + nw; r2 = 0; }
    const bool more = same || b2 < nb;
    if (!same && more) { blk2 = block_of(b2); prefetch(b2 + nw); }
    if (more) issue(blk2, r2, nxt);
    consume(blk, r0, cur);
    if (!same) phase_b(blk);
    b = b2; r0 = r2; blk = blk2;
    return more;
  };
  uint32_t bufa[UA], bufb[UA];
  issue(blk, 0, bufa);
  for (;;) {
    if (!step(bufa, bufb)) break;
    if (!step(bufb, bufa)) break;
  }
}

// Workers: ROWS tile with short rows (dst[i*dsr + j] = cast(src[i*ssr + j]), nc small).  The tile is
// a flat sequence of nr*nc elements; every warp takes batches of 384 consecutive elements on its
// own.  Lane l loads elements l, l+32, ... of the batch (coalesced inside each row; row and column
// advance incrementally, no division per element), twelve loads in flight, one batch ahead.  If the
// destination rows are contiguous (dsr == nc) the cast values go through a private patch of a batch
// and leave as 16-byte vectors; otherwise each value is stored to its own row.
template <int ES, int ED>
__device__ __forceinline__ void warp_small_rows(const TileFields& f, char* patch_mem, uint32_t warp, uint32_t nw,
                                                uint32_t lane) {
  using E = Elem<ES, ED>;
  constexpr uint32_t NV = 16 / ED;
  constexpr int U = 12;          // loads in flight per lane (16 spills registers; 8 leaves rows of 520 B 10 % slower)
  constexpr uint32_t B = 32 * U;
  const uint32_t nc = f.nc, cnt = f.nr * f.nc;
  const bool packed = f.dsr == nc;
  // packed: elements before the first 16-byte boundary of the destination are stored one by one
  uint32_t head = 0;
  if (packed) {
    head = (uint32_t)((16u - ((uintptr_t)f.d & 15u)) & 15u) / ED;
    if (head > cnt) head = cnt;
    if (warp == 0 && lane < head) {
      const uint32_t i = lane / nc, j = lane - i * nc;
      E::store(f.d + (size_t)lane * ED, E::load(f.s + ((size_t)i * f.ssr + j) * ES));
    }
  }
  const uint32_t n_batches = (cnt - head + B - 1) / B;
  if (warp >= n_batches) return;
  const uint32_t q32 = 32 / nc, r32 = 32 % nc;
  const uint32_t patch = smem_u32(patch_mem);               // B * ED bytes of this warp's part of the slot
  // loads of batch b: raw source elements
  auto issue = [&](uint32_t b, uint32_t (&raw)[U]) {
    const uint32_t e0 = head + b * B + lane;
    uint32_t i = e0 / nc, j = e0 - i * nc;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      raw[u] = 0;
      if (e0 + 32u * u < cnt) {
        const char* p = f.s + ((size_t)i * f.ssr + j) * ES;
        if constexpr (ES == 4) raw[u] = __ldcs(reinterpret_cast<const uint32_t*>(p));
        else raw[u] = __ldcs(reinterpret_cast<const uint16_t*>(p));
      }
      i += q32; j += r32;
      if (j >= nc) { j -= nc; ++i; }
    }
  };
  auto consume = [&](uint32_t b, const uint32_t (&raw)[U]) {
    const uint32_t e0 = head + b * B;                       // first element of the batch
    const uint32_t n = min(B, cnt - e0);
    if (!packed) {
      uint32_t i = (e0 + lane) / nc, j = (e0 + lane) - i * nc;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (lane + 32u * u < n) E::store(f.d + ((size_t)i * f.dsr + j) * ED, cast_raw<ES, ED>(raw[u]));
        i += q32; j += r32;
        if (j >= nc) { j -= nc; ++i; }
      }
      return;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t at = patch + (lane + 32u * u) * ED;
      if constexpr (ED == 2) asm volatile("st.shared.u16 [%0], %1;" ::"r"(at), "h"((uint16_t)cast_raw<ES, ED>(raw[u])));
      else asm volatile("st.shared.u32 [%0], %1;" ::"r"(at), "r"((uint32_t)cast_raw<ES, ED>(raw[u])));
    }
    __syncwarp();
    char* out = f.d + (size_t)e0 * ED;                      // 16-byte aligned
    for (uint32_t v = lane; v * NV < n; v += 32) {
      if ((v + 1) * NV <= n) {
        uint4 x;
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(x.x), "=r"(x.y), "=r"(x.z), "=r"(x.w) : "r"(patch + v * 16));
        st16(out + (size_t)v * 16, x);
      } else {
        for (uint32_t e = v * NV; e < n; ++e)
          E::store(out + (size_t)e * ED, (typename E::V)lds_raw<ED>(patch + e * ED));
      }
    }
    __syncwarp();
  };
  uint32_t b = warp;
  auto step = [&](uint32_t (&cr)[U], uint32_t (&nx)[U]) -> bool {
    const uint32_t b2 = b + nw;
    const bool more = b2 < n_batches;
    if (more) issue(b2, nx);
    consume(b, cr);
    b = b2;
    return more;
  };
  uint32_t ra[U], rb2[U];
  issue(b, ra);
  for (;;) {
    if (!step(ra, rb2)) break;
    if (!step(rb2, ra)) break;
  }
}

// Element-wise execution of a tile by nth cooperating threads (this one is t): arbitrary strides, any
// number of destinations.  Only rare shapes come here (strided vectors, fan-out to replicas).
template <int ES, int ED>
__device__ __forceinline__ void coop_tile(const TileFields& f, const DDst* __restrict__ extras, uint64_t dst_add,
                                          uint32_t t, uint32_t nth) {
  using E = Elem<ES, ED>;
  const uint64_t cnt = (uint64_t)f.nr * f.nc;
  for (uint64_t e = t; e < cnt; e += nth) {
    const uint32_t i = (uint32_t)(e / f.nc), j = (uint32_t)(e - (uint64_t)i * f.nc);
    const typename E::V v = E::load(f.s + ((size_t)i * f.ssr + (size_t)j * f.ssc) * ES);
    E::store(f.d + ((size_t)i * f.dsr + (size_t)j * f.dsc) * ED, v);
    for (uint32_t x = 0; x < f.n_extra; ++x) {
      const DDst o = extras[f.extra + x];
      E::store(reinterpret_cast<char*>(o.dst + dst_add) + ((size_t)i * o.sr + (size_t)j * o.sc) * ED, v);
    }
  }
}

// Which tiles take the staged transposition, and how such a tile is cut into chunks: a chunk's columns
// x its own rows (+ halo), emitted columns outer, rows inner.
template <int ES> __device__ __host__ __forceinline__ bool staged_trans_ok(uint32_t kind, uint32_t n_extra, uint32_t nr, uint32_t nc) {
  return kind == KIND_TRANS && n_extra == 0 && (size_t)nc * ES >= kTransMinPiece && nr >= kTransMinRows;
}
template <int ES, int ED> struct TransGeom {
  // chunks staged by per-lane copies
  static constexpr uint32_t kOwn = (((uint32_t)Rings<ES, ED>::kSlotBytes / kTransPitch) - kTransHalo) & ~7u;
  static constexpr uint32_t kCols = kTransChunkBytes / ES;
  // chunks staged by tensor-map loads: the classes' boxes are kClassStride apart in a slot and hold as
  // many rows as fit
  static constexpr uint32_t kClassStride = ((uint32_t)Rings<ES, ED>::kSlotBytes / kTmaClasses) & ~127u;
  static constexpr uint32_t kBoxRows = kClassStride / kTmaInner;
  static constexpr uint32_t kOwnTma = kBoxRows * kTmaClasses - kTransHalo;
  static constexpr uint32_t kColsTma = kTmaChunkBytes / ES;
  static_assert(kTransHalo % kTmaClasses == 0 && kOwnTma % kTmaClasses == 0, "chunks start on a class-0 row");
  static_assert(kTmaInner / ES <= 256 && kBoxRows <= 256, "box dimensions are limited to 256 elements");
};

// Workers: a staged transposition chunk (rows of the source in shared memory, see kTransPitch)
// -> destination runs, dst[j*dps + i] = cast(chunk[i][j]).  A run may start at any 2-/4-byte
// alignment in global memory; it is written in 16-byte aligned windows.  The chunk owns the windows
// that START in its own rows and uses the halo rows to complete the last one, so neighbouring
// chunks never share a window; only the two ends of a whole run use element stores.  Windows are
// numbered run by run and dealt to the threads in order: neighbouring lanes write neighbouring
// windows of one run (whole lines per store instruction) and read different banks.
template <int ES, int ED>
__device__ __forceinline__ void staged_trans(const ChunkDesc& d, const char* stage, uint32_t t) {
  using E = Elem<ES, ED>;
  constexpr uint32_t NV = 16 / ED;
  const uint32_t own = d.tile, nl = d.nr;
  const uint32_t wins = (own + NV - 1) / NV;                   // windows per run, at most
  const uint32_t total = d.nc * wins;
  const uint32_t lead0 = (uint32_t)d.src & 15u, dlead = (uint32_t)d.sps & 15u;
  const uint32_t sbase = smem_u32(stage);
  constexpr uint32_t kSwzShift = ED == 2 ? 1 : 2;               // ((i / NV) & 7) << 4 == (i << shift) & 0x70
  auto elem = [&](uint32_t i, uint32_t j) -> uint32_t {         // raw source element (i, j) of the chunk
    return lds_raw<ES>(sbase + i * kTransPitch + ((i << kSwzShift) & 0x70u) + ((lead0 + i * dlead) & 15u) + j * ES);
  };
  const bool pow2 = (wins & (wins - 1)) == 0;
  const uint32_t wshift = 31u - __clz(wins);
  for (uint32_t idx = t; idx < total; idx += (uint32_t)kWorkers) {
    const uint32_t j = pow2 ? idx >> wshift : idx / wins, w = idx - j * wins;
    const uint64_t run = d.dst + (uint64_t)j * d.dps;           // destination element (j, first own row)
    const uint32_t a = (uint32_t)(run / ED) & (NV - 1);
    const uint32_t lead = a ? NV - a : 0;                       // rows before the first window that starts here
    // those rows belong to the previous chunk's last window, except at the very start of the run
    if (w == 0 && d.pad)
      for (uint32_t e = 0; e < min(lead, own); ++e)
        E::store(reinterpret_cast<char*>(run) + (size_t)e * ED, cast_raw<ES, ED>(elem(e, j)));
    const uint32_t e0 = lead + w * NV;
    if (e0 >= own) continue;
    char* out = reinterpret_cast<char*>(run) + (size_t)e0 * ED;   // 16-byte aligned
    if (e0 + NV <= nl) {
      uint32_t v[NV];
#pragma unroll
      for (uint32_t k = 0; k < NV; ++k) v[k] = elem(e0 + k, j);
      uint4 x;
      if constexpr (ED == 2)
        x = make_uint4(pack_pair16<ES>(v[0], v[1]), pack_pair16<ES>(v[2], v[3]), pack_pair16<ES>(v[4], v[5]),
                       pack_pair16<ES>(v[6], v[7]));
      else
        x = make_uint4((uint32_t)cast_raw<ES, ED>(v[0]), (uint32_t)cast_raw<ES, ED>(v[1]),
                       (uint32_t)cast_raw<ES, ED>(v[2]), (uint32_t)cast_raw<ES, ED>(v[3]));
      st16(out, x);
    } else {
      // the run ends inside this window
      for (uint32_t e = e0; e < nl; ++e)
        E::store(out + (size_t)(e - e0) * ED, cast_raw<ES, ED>(elem(e, j)));
    }
  }
}

// Workers: the same for a chunk that tensor-map loads brought in (eight per-class boxes, see
// kTmaClasses).  Row i of the chunk has class i mod 8 and is row i / 8 of its class's box.  `tab` is the
// shared-memory address of the producer's table for this chunk: entry (h, k), k < NV, is the offset of
// row e0 + k from (box row of e0) * kTmaInner for a window whose first row e0 has class h - it folds the
// class's box, the box row carry and the alignment remainder of the class's rows, so an element costs
// one add and one shared-memory load.  Windows are numbered run by run and dealt to the threads in
// order, as above; (run, window) of a thread advance incrementally.
template <int ES, int ED>
__device__ __forceinline__ void staged_trans_tma(const ChunkDesc& d, const char* stage, uint32_t t, uint32_t tab) {
  using E = Elem<ES, ED>;
  using TG = TransGeom<ES, ED>;
  constexpr uint32_t NV = 16 / ED;
  const uint32_t own = d.tile, nl = d.nr;
  const uint32_t wins = (own + NV - 1) / NV;                   // windows per run, at most
  const uint32_t sbase = smem_u32(stage);
  const uint32_t lead0 = (uint32_t)d.src & 15u, dlead = (uint32_t)d.sps & 15u;
  auto elem = [&](uint32_t i, uint32_t j) -> uint32_t {         // raw source element (i, j) of the chunk (ragged ends only)
    return lds_raw<ES>(sbase + (i % kTmaClasses) * TG::kClassStride + (i / kTmaClasses) * kTmaInner +
                       ((lead0 + i * dlead) & 15u) + j * ES);
  };
  const uint32_t dj = (uint32_t)kWorkers / wins, dw = (uint32_t)kWorkers - dj * wins;
  uint32_t j = t / wins, w = t - j * wins;
  for (; j < d.nc; j += dj, w += dw) {
    if (w >= wins) {
      w -= wins;
      if (++j >= d.nc) break;
    }
    const uint64_t run = d.dst + (uint64_t)j * d.dps;           // destination element (j, first own row)
    const uint32_t a = (uint32_t)(run / ED) & (NV - 1);
    const uint32_t lead = a ? NV - a : 0;                       // rows before the first window that starts here
    // those rows belong to the previous chunk's last window, except at the very start of the run
    if (w == 0 && d.pad)
      for (uint32_t e = 0; e < min(lead, own); ++e)
        E::store(reinterpret_cast<char*>(run) + (size_t)e * ED, cast_raw<ES, ED>(elem(e, j)));
    const uint32_t e0 = lead + w * NV;
    if (e0 >= own) continue;
    char* out = reinterpret_cast<char*>(run) + (size_t)e0 * ED;   // 16-byte aligned
    if (e0 + NV <= nl) {
      const uint32_t base = sbase + (e0 / kTmaClasses) * kTmaInner + j * ES;
      const uint32_t trow = tab + (e0 % kTmaClasses) * (NV * 4);
      uint32_t off[NV], v[NV];
#pragma unroll
      for (uint32_t q = 0; q < NV; q += 4)
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(off[q]), "=r"(off[q + 1]), "=r"(off[q + 2]), "=r"(off[q + 3]) : "r"(trow + q * 4));
#pragma unroll
      for (uint32_t k = 0; k < NV; ++k) v[k] = lds_raw<ES>(base + off[k]);
      uint4 x;
      if constexpr (ED == 2)
        x = make_uint4(pack_pair16<ES>(v[0], v[1]), pack_pair16<ES>(v[2], v[3]), pack_pair16<ES>(v[4], v[5]),
                       pack_pair16<ES>(v[6], v[7]));
      else
        x = make_uint4((uint32_t)cast_raw<ES, ED>(v[0]), (uint32_t)cast_raw<ES, ED>(v[1]),
                       (uint32_t)cast_raw<ES, ED>(v[2]), (uint32_t)cast_raw<ES, ED>(v[3]));
      st16(out, x);
    } else {
      // the run ends inside this window
      for (uint32_t e = e0; e < nl; ++e)
        E::store(out + (size_t)(e - e0) * ED, cast_raw<ES, ED>(elem(e, j)));
    }
  }
}

// Error codes written to the plan's device error word.
enum : uint32_t { ERR_NONE = 0, ERR_WAIT_LOAD = 1, ERR_WAIT_SLOT_EMPTY = 2, ERR_WAIT_SLOT_FULL = 3 };

}  // namespace
