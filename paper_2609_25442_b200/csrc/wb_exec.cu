// Device side of the weight-remap library: binding a plan to device memory and the
// persistent tile-walking kernel behind wb_remap / wb_pack / wb_unpack (sm_100a).
//
// One persistent launch (one thread block per SM) executes a whole tile table.  Blocks draw
// batches of consecutive tiles from a counter in device memory (or walk the byte-balanced range
// the planner computed, under WB_PLAN_STATIC_SCHEDULE); tiles are independent, so blocks never
// wait on each other.  Inside a block warp 0 is the producer and the other warps are workers:
//
//   direct   same element size, long rows, source and destination congruent mod 16 bytes:
//            lane 0 of the producer moves them by itself with bulk copies global -> shared ->
//            global through a small ring; the data never touches registers.
//   staged   other ROWS tiles with rows of at least kStagedMinRowBytes: the producer warp bulk-
//            loads the rows into a ring slot, the workers realign, cast and store 16 bytes at a time.
//   staged   transposing tiles: the producer warp copies chunks of source rows into a ring slot
//   transp.  (per-lane asynchronous copies, bank-swizzled rows), the workers write 16-byte windows
//            of the destination runs, neighbouring lanes on neighbouring windows of one run.
//   queued   everything else is handed to the workers by tile index, either one tile shared by all
//            worker warps or a run of small tiles, one warp per tile.
//
// Tile kinds
//   ROWS   nr runs of nc contiguous elements on both sides (nr == 1: one long run).
//   TRANS  source contiguous along j, destination contiguous along i: staged transposition, or
//          (narrow tiles) each warp transposes 32-column blocks through a private patch.
//   ELEM   anything else (strided vectors, fan-out to several destinations): element loop.
//
// Every wait in the kernel is bounded (see mbar_wait); a wait that runs out sets the plan's error
// word, which wb_plan_check reports.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "wb_internal.h"

using namespace wbi;

namespace {

#ifndef WB_THREADS
#define WB_THREADS 512
#endif
constexpr int kThreads = WB_THREADS;   // warp 0: producer; the other warps: workers

// ---------------------------------------------------------------------------------------------
// memory access helpers: streaming (evict-first) loads and stores, the data is touched once
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld16(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ uint2 ld8(const void* p) { return __ldcs(reinterpret_cast<const uint2*>(p)); }
__device__ __forceinline__ void st16(void* p, uint4 v) { __stcs(reinterpret_cast<uint4*>(p), v); }

// fp32 pair -> packed bf16 pair, round to nearest even (NaN -> 0x7FFF); `lo` lands in the low half
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(uint32_t lo, uint32_t hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(__uint_as_float(hi)), "f"(__uint_as_float(lo)));
  return r;
}
__device__ __forceinline__ uint16_t f32_to_bf16(uint32_t x) {
  uint16_t r;
  asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(__uint_as_float(x)));
  return r;
}

// One element: load raw bits, cast, store raw bits.
template <int ES, int ED> struct Elem;
template <> struct Elem<2, 2> {
  static __device__ __forceinline__ void copy(const char* s, char* d) {
    *reinterpret_cast<uint16_t*>(d) = *reinterpret_cast<const uint16_t*>(s);
  }
  using V = uint16_t;
  static __device__ __forceinline__ V load(const char* s) { return *reinterpret_cast<const uint16_t*>(s); }
  static __device__ __forceinline__ void store(char* d, V v) { *reinterpret_cast<uint16_t*>(d) = v; }
};
template <> struct Elem<4, 4> {
  using V = uint32_t;
  static __device__ __forceinline__ V load(const char* s) { return *reinterpret_cast<const uint32_t*>(s); }
  static __device__ __forceinline__ void store(char* d, V v) { *reinterpret_cast<uint32_t*>(d) = v; }
};
template <> struct Elem<4, 2> {
  using V = uint16_t;
  static __device__ __forceinline__ V load(const char* s) { return f32_to_bf16(*reinterpret_cast<const uint32_t*>(s)); }
  static __device__ __forceinline__ void store(char* d, V v) { *reinterpret_cast<uint16_t*>(d) = v; }
};
template <> struct Elem<2, 4> {
  using V = uint32_t;
  static __device__ __forceinline__ V load(const char* s) {
    return (uint32_t)(*reinterpret_cast<const uint16_t*>(s)) << 16;
  }
  static __device__ __forceinline__ void store(char* d, V v) { *reinterpret_cast<uint32_t*>(d) = v; }
};

// One 16-byte destination vector: NV elements, read with the widest aligned loads.
template <int ES, int ED> struct Unit;
template <> struct Unit<2, 2> {
  static constexpr int NV = 8, SRC_ALIGN = 16;
  uint4 a;
  __device__ __forceinline__ void load(const char* s) { a = ld16(s); }
  __device__ __forceinline__ uint4 out() const { return a; }
};
template <> struct Unit<4, 4> {
  static constexpr int NV = 4, SRC_ALIGN = 16;
  uint4 a;
  __device__ __forceinline__ void load(const char* s) { a = ld16(s); }
  __device__ __forceinline__ uint4 out() const { return a; }
};
template <> struct Unit<4, 2> {
  static constexpr int NV = 8, SRC_ALIGN = 16;
  uint4 a, b;
  __device__ __forceinline__ void load(const char* s) { a = ld16(s); b = ld16(s + 16); }
  __device__ __forceinline__ uint4 out() const {
    return make_uint4(f32x2_to_bf16x2(a.x, a.y), f32x2_to_bf16x2(a.z, a.w),
                      f32x2_to_bf16x2(b.x, b.y), f32x2_to_bf16x2(b.z, b.w));
  }
};
template <> struct Unit<2, 4> {
  static constexpr int NV = 4, SRC_ALIGN = 8;
  uint2 a;
  __device__ __forceinline__ void load(const char* s) { a = ld8(s); }
  __device__ __forceinline__ uint4 out() const {
    return make_uint4(a.x << 16, a.x & 0xFFFF0000u, a.y << 16, a.y & 0xFFFF0000u);
  }
};

// A 16-byte destination vector assembled from element loads (source not vector-aligned).
template <int ES, int ED>
__device__ __forceinline__ uint4 gather_unit(const char* s) {
  using E = Elem<ES, ED>;
  if constexpr (ED == 2) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      uint32_t lo = E::load(s + (2 * k) * ES), hi = E::load(s + (2 * k + 1) * ES);
      w[k] = lo | (hi << 16);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  } else {
    return make_uint4(E::load(s), E::load(s + ES), E::load(s + 2 * ES), E::load(s + 3 * ES));
  }
}

template <int ES, int ED> struct Unroll { static constexpr int U = (ES == 4 && ED == 2) ? 2 : 4; };

// Copy one run of n contiguous elements with `nth` cooperating threads (this thread is `t`).
template <int ES, int ED>
__device__ __forceinline__ void copy_run(const char* __restrict__ s, char* __restrict__ d, uint32_t n,
                                         uint32_t t, uint32_t nth) {
  using UN = Unit<ES, ED>;
  using E = Elem<ES, ED>;
  constexpr int NV = UN::NV;
  constexpr int U = Unroll<ES, ED>::U;
  // peel elements until the destination is 16-byte aligned
  uint32_t head = (uint32_t)((16u - ((uintptr_t)d & 15u)) & 15u) / ED;
  if (head > n) head = n;
  if (t < head) E::store(d + (size_t)t * ED, E::load(s + (size_t)t * ES));
  s += (size_t)head * ES;
  d += (size_t)head * ED;
  n -= head;
  const uint32_t nvec = n / NV;
  if (((uintptr_t)s & (UN::SRC_ALIGN - 1)) == 0) {
    for (uint32_t v0 = t; v0 < nvec; v0 += nth * U) {
      UN r[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint32_t v = v0 + u * nth;
        if (v < nvec) r[u].load(s + (size_t)v * (NV * ES));
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint32_t v = v0 + u * nth;
        if (v < nvec) st16(d + (size_t)v * 16, r[u].out());
      }
    }
  } else {
    for (uint32_t v = t; v < nvec; v += nth) st16(d + (size_t)v * 16, gather_unit<ES, ED>(s + (size_t)v * (NV * ES)));
  }
  const uint32_t tail = n - nvec * NV;
  if (t < tail) {
    const size_t e = (size_t)nvec * NV + t;
    E::store(d + e * ED, E::load(s + e * ES));
  }
}

struct TileRegs {
  uint4 a, b, c;
};

__device__ __forceinline__ TileRegs load_tile(const DTile* p) {
  const uint4* q = reinterpret_cast<const uint4*>(p);
  TileRegs r;
  r.a = __ldg(q);
  r.b = __ldg(q + 1);
  r.c = __ldg(q + 2);
  return r;
}

// ---------------------------------------------------------------------------------------------
// mbarrier / bulk-copy (TMA) primitives.  Every wait is bounded: after kSpinLimit failed
// polls the caller records an error code and leaves, so a lost signal cannot hang the GPU.
// ---------------------------------------------------------------------------------------------
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // 2 s

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One poll of the barrier.  (Giving try_wait an explicit suspend-time hint was measured to wake
// waiting warps late and cost 30 % of the staged paths' bandwidth, so the default is used.)
__device__ __forceinline__ bool mbar_try(uint32_t addr, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
  return ok != 0;
}
// Wait for the phase with the given parity to complete; gives up after `limit_ns`.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint64_t limit_ns = kWaitLimitNs) {
  const uint32_t addr = smem_u32(bar);
  if (mbar_try(addr, parity)) return true;
  const uint64_t t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(addr, parity)) return true;
    if ((it & 255u) == 0 && global_ns() - t0 > limit_ns) return false;
  }
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing ever signals.  The
// wait must give up after limit_ns, record its code and let the kernel end normally.
__global__ void wb_wait_probe_kernel(uint64_t limit_ns, uint32_t* __restrict__ err) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(&bar, 0, limit_ns)) atomicMax(err, 0x7Du);   // "timed out", distinct from the executor's codes
  }
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Per-thread asynchronous 16-byte copy global -> shared (both 16-byte aligned), and the arrival that
// signals an mbarrier once all earlier copies of the calling thread have landed (the pending count
// is raised by the instruction itself, so the barrier's initial count is not involved).
__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}
template <int OFF> __device__ __forceinline__ void cp_async16_at(uint32_t smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0+%2], [%1+%2], 16;" ::"r"(smem_dst), "l"(gsrc), "n"(OFF) : "memory");
}
__device__ __forceinline__ void cp_async_arrive(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.shared.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

constexpr int kWorkers = kThreads - 32;       // warps 1.. convert staged chunks and run queued tiles
// Shared-memory rings (tuned on B200; the direct ring is very sensitive: 3 x 32 KiB moves 5 % more
// than 4 x 16 KiB).  Kernels whose element sizes differ never use the direct ring and give all of
// it to the worker ring.
#ifndef WB_DIRECT_STAGES
#define WB_DIRECT_STAGES 3
#endif
#ifndef WB_DIRECT_BYTES
#define WB_DIRECT_BYTES 32768
#endif
#ifndef WB_SLOTS_SAME
#define WB_SLOTS_SAME 3
#endif
#ifndef WB_SLOT_BYTES_SAME
#define WB_SLOT_BYTES_SAME 32768
#endif
#ifndef WB_SLOTS_CAST
#define WB_SLOTS_CAST 4
#endif
#ifndef WB_SLOT_BYTES_CAST
#define WB_SLOT_BYTES_CAST 49152
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

enum : uint32_t { MODE_END = 0, MODE_COOP = 1, MODE_ROWS = 2, MODE_BATCH = 3, MODE_TRANS = 4 };
// Staged transposition: a chunk is up to kTransPiece - 16 bytes of consecutive source columns (the
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
constexpr uint32_t kTransHalo = 8;
#ifndef WB_TRANS_MIN_PIECE
#define WB_TRANS_MIN_PIECE 256
#endif
constexpr uint32_t kTransMinPiece = WB_TRANS_MIN_PIECE;   // narrower tiles stay with the warp-level transposition
constexpr uint32_t kTransMinRows = 16;
#ifndef WB_BATCH_TILE_BYTES
#define WB_BATCH_TILE_BYTES 8192
#endif
constexpr uint32_t kBatchTileBytes = WB_BATCH_TILE_BYTES;   // tiles moving less than this are batched, one warp per tile
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
};
__device__ __forceinline__ TileFields decode(const TileRegs& r, uint64_t src_add, uint64_t dst_add) {
  TileFields f;
  f.s = reinterpret_cast<const char*>(((uint64_t)r.a.y << 32 | r.a.x) + src_add);
  f.d = reinterpret_cast<char*>(((uint64_t)r.a.w << 32 | r.a.z) + dst_add);
  f.nr = r.b.x; f.nc = r.b.y; f.ssr = r.b.z; f.ssc = r.b.w;
  f.dsr = r.c.x; f.dsc = r.c.y;
  f.kind = r.c.z & 0xFF; f.n_extra = (r.c.z >> 8) & 0xFF; f.extra = r.c.w;
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
// element stores.  A group of G lanes (G = 32, 16 or 8 by row length) takes G consecutive slots
// of one row; groups are independent (no barrier).  `t` is the rotated worker thread index.
template <int ES, int ED>
__device__ __forceinline__ void staged_rows(const ChunkDesc& d, const char* stage, uint32_t t) {
  using E = Elem<ES, ED>;
  constexpr uint32_t NV = 16 / ED;
  const uint32_t n = d.nc;
  const uint32_t smax = (n + 2 * NV - 2) / NV;     // slots a row can touch
  const uint32_t gs = smax > 16 ? 5u : (smax > 8 ? 4u : 3u);
  const uint32_t G = 1u << gs;
  const uint32_t nb = (smax + G - 1) >> gs;        // slot blocks per row
  const uint32_t tasks = d.nr * nb;
  const uint32_t lead0 = (uint32_t)d.src & 15u, dlead = (uint32_t)d.sps & 15u;
  const uint32_t lig = t & (G - 1);
  for (uint32_t task = t >> gs; task < tasks; task += (uint32_t)kWorkers >> gs) {
    const uint32_t r = task / nb, k = (task - r * nb) * G + lig;
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
// Shared-memory word accesses at a compile-time offset from a 32-bit shared-space address, and a
// loop over compile-time indices (so that unrolled code uses immediate offsets).
template <int OFF> __device__ __forceinline__ uint32_t lds32_at(uint32_t base) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(base), "n"(OFF));
  return v;
}
template <int OFF> __device__ __forceinline__ void sts32_at(uint32_t base, uint32_t v) {
  asm volatile("st.shared.u32 [%0+%1], %2;" ::"r"(base), "n"(OFF), "r"(v));
}
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
  // rows read past a block's end to complete its last window: NV-1 are needed; with 2-byte
  // destinations 8 are read, which keeps the row count of a whole block a multiple of UA
  const uint32_t halo = aligned ? 0u : (ED == 2 ? 8u : NV - 1), room = aligned ? 0u : 8u;
  const uint32_t rb = min(64u, ((share / 32 - 1) * PER_WORD - room) & ~7u);
  const uint32_t pitch_w = (rb + room) / PER_WORD + 1;      // odd: (rb+room)/PER_WORD is even
  const uint32_t tbase = smem_u32(patch);
  const uint32_t nbi = (f.nr + rb - 1) / rb, nbj = (f.nc + 31) / 32;
  const uint32_t nb = nbi * nbj;
  const size_t sps = (size_t)f.ssr * ES;
  if (warp >= nb) return;

  // nl: rows loaded = own rows + halo.  full: every lane has a column and every batch all its rows,
  // so loads and shared-memory writes need no predicates; whole: in addition the block has all its
  // rows and halo and does not begin a run, so every window it owns is a full vector.
  struct Block { uint32_t i0, j0, ni, nj, nl; bool full, whole; };
  auto block_of = [&](uint32_t b) {
    const uint32_t bi = b / nbj, bj = b - bi * nbj;
    const uint32_t i0 = bi * rb, ni = min(rb, f.nr - i0);
    const uint32_t nj = min(32u, f.nc - bj * 32), nl = min(ni + halo, f.nr - i0);
    const bool full = nj == 32 && nl % UA == 0;
    return Block{i0, bj * 32, ni, nj, nl, full, full && nl == rb + halo && (aligned || i0 != 0)};
  };
  // phase A, loads: UA rows of this lane's column into registers
  auto issue = [&](const Block& k, uint32_t r0, uint32_t (&dst)[UA]) {
    const char* src = f.s + ((size_t)(k.i0 + r0) * f.ssr + k.j0 + lane) * ES;
    if (k.full) {
#pragma unroll
      for (int u = 0; u < UA; ++u, src += sps) {
        if constexpr (ES == 4) dst[u] = __ldcs(reinterpret_cast<const uint32_t*>(src));
        else dst[u] = __ldcs(reinterpret_cast<const uint16_t*>(src));
      }
      return;
    }
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
    if (k.full) {
      const uint32_t at = trow + r0 * ED;
      if constexpr (ED == 2)
        static_for<0, UA / 2>([&](auto uc) {
          constexpr int u = decltype(uc)::value * 2;
          sts32_at<u * 2>(at, pack_pair16<ES>(v[u], v[u + 1]));
        });
      else
        static_for<0, UA>([&](auto uc) {
          constexpr int u = decltype(uc)::value;
          sts32_at<u * 4>(at, (uint32_t)cast_raw<ES, ED>(v[u]));
        });
      return;
    }
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
    if (k.whole) {
      // lane = destination run; rb / NV full windows, the first one `lead` rows into the block
      char* run = f.d + (size_t)(k.j0 + lane) * f.dsc * ED;
      const uint32_t a = (uint32_t)(((uintptr_t)run / ED + k.i0) & (NV - 1));
      const uint32_t lead = a ? NV - a : 0;
      char* out = run + (size_t)(k.i0 + lead) * ED;
      const uint32_t trow = tbase + lane * pitch_w * 4;
      if constexpr (ED == 4) {
        uint32_t p = trow + lead * 4;
        for (uint32_t w = 0; w < rb / NV; ++w, p += 16, out += 16)
          st16(out, make_uint4(lds32_at<0>(p), lds32_at<4>(p), lds32_at<8>(p), lds32_at<12>(p)));
      } else if (aligned) {
        uint32_t p = trow;
        for (uint32_t w = 0; w < rb / NV; ++w, p += 16, out += 16)
          st16(out, make_uint4(lds32_at<0>(p), lds32_at<4>(p), lds32_at<8>(p), lds32_at<12>(p)));
      } else {
        uint32_t p = trow + (lead >> 1) * 4;
        const uint32_t sh = (lead & 1u) * 16u;                     // odd lead: windows straddle the words
        for (uint32_t w = 0; w < rb / NV; ++w, p += 16, out += 16) {
          const uint32_t w0 = lds32_at<0>(p), w1 = lds32_at<4>(p), w2 = lds32_at<8>(p), w3 = lds32_at<12>(p),
                         w4 = lds32_at<16>(p);
          st16(out, make_uint4(__funnelshift_r(w0, w1, sh), __funnelshift_r(w1, w2, sh),
                               __funnelshift_r(w2, w3, sh), __funnelshift_r(w3, w4, sh)));
        }
      }
      __syncwarp();
      return;
    }
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
  // for the block after next to be brought into L2 ahead of time (lane = row; every sector of the
  // piece): that costs no registers, and the loads then hit L2.
  auto prefetch = [&](uint32_t pb) {
#ifndef WB_NO_TRANS_PREFETCH
    if (pb >= nb) return;
    const Block k = block_of(pb);
    for (uint32_t r = lane; r < k.nl; r += 32) {
      const char* row = f.s + ((size_t)(k.i0 + r) * f.ssr + k.j0) * ES;
      const uint32_t bytes = k.nj * ES;                             // one request per 32-byte sector
      for (uint32_t o = 0; o < bytes; o += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(row + o));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(row + bytes - 1));
    }
#endif
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
// a flat sequence of nr*nc elements; every warp takes batches of 256 consecutive elements on its
// own.  Lane l loads elements l, l+32, ... of the batch (coalesced inside each row; row and column
// advance incrementally, no division per element), eight loads in flight, one batch ahead.  If the
// destination rows are contiguous (dsr == nc) the cast values go through a 512-byte private patch
// and leave as 16-byte vectors; otherwise each value is stored to its own row.
template <int ES, int ED>
__device__ __forceinline__ void warp_small_rows(const TileFields& f, char* patch_mem, uint32_t warp, uint32_t nw,
                                                uint32_t lane) {
  using E = Elem<ES, ED>;
  constexpr uint32_t NV = 16 / ED;
  constexpr int U = 8;
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

// Error codes written to the plan's device error word.
enum : uint32_t { ERR_NONE = 0, ERR_WAIT_LOAD = 1, ERR_WAIT_SLOT_EMPTY = 2, ERR_WAIT_SLOT_FULL = 3 };

// The persistent executor: one thread block per SM walks its range of the tile table.
//   warp 0   "producer".  Lane 0 moves direct tiles by itself through a ring of bulk (TMA) copies
//            global -> shared -> global.  For every other tile the warp feeds the worker ring:
//            either the tile's rows are staged into a ring slot with bulk loads (one per row, the
//            16-byte aligned superset of the row), or the tile index is queued as is.
//   warps 1.. "workers".  Take ring slots in order: convert staged rows (cast in registers,
//            realignment by funnel shifts, 16-byte vector stores), transpose staged blocks, or
//            run a queued tile cooperatively (element-wise fan-out and other rare shapes).
template <int ES, int ED>
__global__ void __launch_bounds__(kThreads, 1)
wb_exec_kernel(const DTile* __restrict__ tiles, const uint32_t* __restrict__ cta_begin,
               const DDst* __restrict__ extras, uint64_t src_add, uint64_t dst_add, uint32_t* __restrict__ err,
               uint32_t n_tiles, uint32_t* __restrict__ sched) {
  using E = Elem<ES, ED>;
  extern __shared__ __align__(128) char dyn_smem[];
  constexpr int kSlots = Rings<ES, ED>::kSlots;
  constexpr int kSlotBytes = Rings<ES, ED>::kSlotBytes;
  char* const ring = dyn_smem;                                         // kDirectStages x kDirectBytes
  char* const wring = dyn_smem + Rings<ES, ED>::kDirect;               // kSlots x kSlotBytes
  __shared__ __align__(8) uint64_t direct_full[kDirectStages];
  __shared__ __align__(8) uint64_t slot_full[kMaxSlots], slot_empty[kMaxSlots];
  __shared__ __align__(16) ChunkDesc desc[kMaxSlots];
  __shared__ char* q_dst[kDirectStages];        // direct ring: where each loaded stage goes
  __shared__ uint32_t q_bytes[kDirectStages];

  // Scheduling: with `sched` the blocks draw batches of consecutive tiles from a shared counter
  // (large batches first, shrinking towards the end); without it each block walks the fixed
  // range the planner assigned to it.
  const uint32_t begin = sched ? 0u : cta_begin[blockIdx.x], end = sched ? 0u : cta_begin[blockIdx.x + 1];
  if (!sched && begin >= end) return;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kDirectStages; ++i) mbar_init(&direct_full[i], 1);
    for (int i = 0; i < kSlots; ++i) { mbar_init(&slot_full[i], 1); mbar_init(&slot_empty[i], kWorkers / 32); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (threadIdx.x >= 32) {
    // ------------------------------- workers -------------------------------------------------
    const uint32_t t = threadIdx.x - 32;
    for (uint32_t n = 0;; ++n) {
      const uint32_t slot = n % kSlots;
      uint32_t ok = 1;
      if ((t & 31) == 0) ok = mbar_wait(&slot_full[slot], (n / kSlots) & 1);   // one poller per warp
      ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
      if (!ok) { if (t == 0) atomicMax(err, ERR_WAIT_SLOT_FULL); return; }
      const ChunkDesc d = desc[slot];
      if (d.mode == MODE_END) return;
      const char* stage = wring + (size_t)slot * kSlotBytes;
      // small chunks have fewer tasks than workers: rotate which warps take them
      uint32_t tr = t + (n * 256u) % kWorkers;
      if (tr >= (uint32_t)kWorkers) tr -= kWorkers;
      if (d.mode == MODE_ROWS) {
        staged_rows<ES, ED>(d, stage, tr);
      } else if (d.mode == MODE_TRANS) {
#ifndef WB_TRANS_SKIP_WORK
        staged_trans<ES, ED>(d, stage, tr);
#endif
      } else {
        // queued tiles: one big tile shared by all worker warps, or a run of small tiles with one
        // warp per tile
        const bool run = d.mode == MODE_BATCH;
        const uint32_t warp = tr >> 5, lane = t & 31;
        const uint32_t w = run ? 0u : warp, nw = run ? 1u : (uint32_t)kWorkerWarps;
        // every warp owns one fixed part of the slot as scratch, whatever kind of tile it runs
        constexpr uint32_t kPatchBytes = ((uint32_t)kSlotBytes / kWorkerWarps) & ~15u;
        char* patch = const_cast<char*>(stage) + warp * kPatchBytes;
        const uint32_t k0 = d.tile + (run ? warp : 0u), kend = d.tile + d.nr, kstep = run ? (uint32_t)kWorkerWarps : 1u;
        TileRegs regs;
        if (!run) { regs.a = d.raw[0]; regs.b = d.raw[1]; regs.c = d.raw[2]; }
        else if (k0 < kend) regs = load_tile(tiles + k0);
        for (uint32_t k = k0; k < kend; k += kstep) {
          const TileFields f = decode(regs, src_add, dst_add);
          if (k + kstep < kend) regs = load_tile(tiles + k + kstep);    // the next descriptor is on its way meanwhile
          if (f.n_extra == 0 && f.kind == KIND_TRANS) {
            warp_transpose<ES, ED>(f, patch, kPatchBytes, w, nw, lane);
          } else if (f.n_extra == 0 && f.kind == KIND_ROWS && (f.nr == 1 || (size_t)f.nc * ES >= kStagedMinRowBytes)) {
            for (uint32_t row = w; row < f.nr; row += nw)
              copy_run<ES, ED>(f.s + (size_t)row * f.ssr * ES, f.d + (size_t)row * f.dsr * ED, f.nc, lane, 32);
          } else if (f.n_extra == 0 && f.kind == KIND_ROWS && f.nr * (uint64_t)f.nc < (1ull << 31)) {
            warp_small_rows<ES, ED>(f, patch, w, nw, lane);
          } else {
            coop_tile<ES, ED>(f, extras, dst_add, w * 32 + lane, nw * 32);
          }
        }
      }
      __syncwarp();
      if ((t & 31) == 0) mbar_arrive(&slot_empty[slot]);
    }
  }

  // --------------------------------- producer warp -----------------------------------------------
  const uint32_t lane = threadIdx.x;
  uint32_t n_w = 0;                     // worker-ring slots handed out so far (warp-uniform)
  uint32_t n_load = 0, n_store = 0;     // direct ring positions (lane 0)
  bool failed = false;                  // warp-uniform

  // wait until the workers have released the slot that position n_w maps to
  auto acquire_slot = [&]() -> bool {
    uint32_t ok = 1;
    if (lane == 0 && n_w >= kSlots) ok = mbar_wait(&slot_empty[n_w % kSlots], ((n_w / kSlots) - 1) & 1);
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    if (!ok) { if (lane == 0) atomicMax(err, ERR_WAIT_SLOT_EMPTY); failed = true; }
    return ok != 0;
  };
  auto push_simple = [&](uint32_t mode, uint32_t tile, uint32_t count = 1, const TileRegs* regs = nullptr) {
    if (!acquire_slot()) return;
    const uint32_t slot = n_w % kSlots;
    if (lane == 0) {
      desc[slot].mode = mode;
      desc[slot].tile = tile;
      desc[slot].nr = count;
      if (regs) { desc[slot].raw[0] = regs->a; desc[slot].raw[1] = regs->b; desc[slot].raw[2] = regs->c; }
      mbar_arrive(&slot_full[slot]);    // release: the descriptor is visible to whoever sees the phase
    }
    ++n_w;
  };
  // stage R rows of n elements (row r starts at src + r*sps) into the next slot
  auto push_staged = [&](uint32_t mode, const char* src, char* dst, uint32_t R, uint32_t n, uint64_t sps,
                         uint64_t dps, uint32_t pitch) {
    if (!acquire_slot()) return;
    const uint32_t slot = n_w % kSlots;
    char* stage = wring + (size_t)slot * kSlotBytes;
    uint32_t mine = 0;
    for (uint32_t r = lane; r < R; r += 32)
      mine += roundup16((uint32_t)(((uintptr_t)src + (uint64_t)r * sps) & 15u) + n * ES);
    const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, mine);
    if (lane == 0) {
      ChunkDesc c;
      c.mode = mode; c.tile = 0; c.nr = R; c.nc = n; c.pitch = pitch; c.pad = 0;
      c.src = (uint64_t)(uintptr_t)src; c.dst = (uint64_t)(uintptr_t)dst; c.sps = sps; c.dps = dps;
      desc[slot] = c;
      mbar_expect_tx(&slot_full[slot], total);     // the producer's arrival + the bytes to come
    }
    __syncwarp();
    for (uint32_t r = lane; r < R; r += 32) {
      const uintptr_t a = (uintptr_t)src + (uint64_t)r * sps;
      bulk_load(stage + (size_t)r * pitch, reinterpret_cast<const void*>(a & ~(uintptr_t)15),
                roundup16((uint32_t)(a & 15u) + n * ES), &slot_full[slot]);
    }
    ++n_w;
  };
  // stage a transposition chunk: R row pieces of n elements, four lanes per row
  auto push_trans = [&](const char* src, char* dst, uint32_t R, uint32_t n, uint64_t sps, uint64_t dps,
                        uint32_t own, uint32_t first) {
    if (!acquire_slot()) return;
    const uint32_t slot = n_w % kSlots;
    const uint32_t stage = smem_u32(wring + (size_t)slot * kSlotBytes);
    if (lane == 0) {
      ChunkDesc c;
      c.mode = MODE_TRANS; c.tile = own; c.nr = R; c.nc = n; c.pitch = kTransPitch; c.pad = first;
      c.src = (uint64_t)(uintptr_t)src; c.dst = (uint64_t)(uintptr_t)dst; c.sps = sps; c.dps = dps;
      desc[slot] = c;
    }
    // Four lanes per row, eight rows per step: a lane copies every fourth 16-byte unit of its row
    // (immediate offsets), so the address arithmetic is paid once per eight rows.  This loop is the
    // producer's critical path: one warp feeds the whole block.
    constexpr uint32_t kSwzShift = ED == 2 ? 1 : 2;               // ((r / NV) & 7) << 4 == (r << shift) & 0x70
    const uint32_t nbytes = n * ES, q16 = (lane & 3u) * 16u;
    for (uint32_t r = lane >> 2; r < R; r += 8) {
      const uintptr_t a = (uintptr_t)src + (uint64_t)r * sps;
      const uint32_t need = (uint32_t)(a & 15u) + nbytes;         // bytes of the aligned superset that are needed
      const char* g = reinterpret_cast<const char*>(a & ~(uintptr_t)15) + q16;
      const uint32_t sm = stage + r * kTransPitch + ((r << kSwzShift) & 0x70u) + q16;
      static_for<0, (int)(kTransPiece / 64)>([&](auto kc) {
        constexpr int off = decltype(kc)::value * 64;
        if (q16 + (uint32_t)off < need) cp_async16_at<off>(sm, g);
      });
    }
    cp_async_arrive(&slot_full[slot]);
    __syncwarp();
    if (lane == 0) mbar_arrive(&slot_full[slot]);   // after every lane's pending arrival is counted
    ++n_w;
  };
  // direct ring (lane 0): store the oldest loaded chunk; one store behind, its stage is free again
  auto store_oldest = [&]() {
    const uint32_t st = n_store % kDirectStages;
    if (!mbar_wait(&direct_full[st], (n_store / kDirectStages) & 1)) { atomicMax(err, ERR_WAIT_LOAD); failed = true; return; }
    fence_async_smem();
    bulk_store(q_dst[st], ring + (size_t)st * kDirectBytes, q_bytes[st]);
    bulk_commit();
    ++n_store;
  };
  auto load_chunk = [&](const char* src, char* dst, uint32_t bytes) {
    while (!failed && n_load - n_store >= (uint32_t)kDirectStages - 1) { store_oldest(); bulk_wait_read_1(); }
    if (failed) return;
    const uint32_t st = n_load % kDirectStages;
    q_dst[st] = dst;
    q_bytes[st] = bytes;
    mbar_expect_tx(&direct_full[st], bytes);
    bulk_load(ring + (size_t)st * kDirectBytes, src, bytes, &direct_full[st]);
    ++n_load;
  };

  uint32_t bk = begin, bend = end;      // current batch [bk, bend)
  bool first = true;
  auto next_batch = [&]() -> bool {
    if (!sched) {
      const bool ok = first;
      first = false;
      return ok;
    }
    uint32_t s0 = n_tiles, b = 0;
    if (lane == 0) {
      const uint32_t cur = *reinterpret_cast<volatile uint32_t*>(&sched[0]);
      if (cur < n_tiles) {
        b = max(1u, (n_tiles - cur) / (gridDim.x * 4u));
        s0 = atomicAdd(&sched[0], b);
      }
    }
    s0 = __shfl_sync(0xFFFFFFFFu, s0, 0);
    b = __shfl_sync(0xFFFFFFFFu, b, 0);
    if (s0 >= n_tiles) return false;
    bk = s0;
    bend = min(s0 + b, n_tiles);
    return true;
  };

  uint32_t run0 = 0, run_n = 0;         // pending run of small tiles [run0, run0 + run_n)
  auto flush_run = [&]() {
    if (run_n) push_simple(MODE_BATCH, run0, run_n);
    run_n = 0;
  };
  while (!failed && next_batch()) {
  TileRegs nxt = load_tile(tiles + bk);
  for (uint32_t k = bk; k < bend && !failed; ++k) {
    const TileRegs cur = nxt;
    const TileFields f = decode(cur, src_add, dst_add);
    if (k + 1 < bend) nxt = load_tile(tiles + k + 1);
    // small tiles are handed over in runs and executed one warp per tile
    if ((uint64_t)f.nr * f.nc * (ES + ED * (1 + f.n_extra)) < kBatchTileBytes && !direct_ok<ES, ED>(f)) {
      if (run_n == 0) run0 = k;
      if (++run_n == kBatchMaxTiles) flush_run();
      continue;
    }
    flush_run();
    if (direct_ok<ES, ED>(f)) {
      if (lane == 0) {
        for (uint32_t i = 0; i < f.nr && !failed; ++i) {
          const char* s = f.s + (size_t)i * f.ssr * ES;
          char* d = f.d + (size_t)i * f.dsr * ED;
          size_t n = (size_t)f.nc * ES;
          // bytes before the first / after the last 16-byte boundary: element copies
          size_t head = (16u - ((uintptr_t)d & 15u)) & 15u;
          if (head > n) head = n;
          for (size_t b = 0; b < head; b += ES) E::store(d + b, E::load(s + b));
          s += head; d += head; n -= head;
          const size_t body = n & ~(size_t)15;
          for (size_t b = body; b < n; b += ES) E::store(d + b, E::load(s + b));
          for (size_t off = 0; off < body && !failed; off += kDirectBytes)
            load_chunk(s + off, d + off, (uint32_t)min((size_t)kDirectBytes, body - off));
        }
      }
      failed = __shfl_sync(0xFFFFFFFFu, (uint32_t)failed, 0) != 0;
    } else if (f.kind == KIND_ROWS && f.n_extra == 0 && (size_t)f.nc * ES >= kStagedMinRowBytes) {
      const uint32_t row_bytes = f.nc * ES + 16;                 // worst-case aligned superset of a row
      if (row_bytes <= (uint32_t)kSlotBytes) {
        const uint32_t pitch = roundup16(row_bytes);
        const uint32_t per = f.nr == 1 ? 1u : min(f.nr, (uint32_t)kSlotBytes / pitch);
        for (uint32_t r0 = 0; r0 < f.nr && !failed; r0 += per)
          push_staged(MODE_ROWS, f.s + (size_t)r0 * f.ssr * ES, f.d + (size_t)r0 * f.dsr * ED,
                      min(per, f.nr - r0), f.nc, (uint64_t)f.ssr * ES, (uint64_t)f.dsr * ED, pitch);
      } else {
        const uint32_t piece = ((uint32_t)kSlotBytes - 32) / ES / 64 * 64;   // elements per column piece
        for (uint32_t r = 0; r < f.nr && !failed; ++r)
          for (uint32_t c = 0; c < f.nc && !failed; c += piece)
            push_staged(MODE_ROWS, f.s + ((size_t)r * f.ssr + c) * ES, f.d + ((size_t)r * f.dsr + c) * ED, 1,
                        min(piece, f.nc - c), 0, 0, (uint32_t)kSlotBytes);
      }
    } else if (f.kind == KIND_TRANS && f.n_extra == 0 && (size_t)f.nc * ES >= kTransMinPiece && f.nr >= kTransMinRows) {
      // staged transposition: chunks of kTransPiece bytes of columns x kOwn rows (+ halo), rows fastest
      constexpr uint32_t kOwn = (((uint32_t)kSlotBytes / kTransPitch) - kTransHalo) & ~7u;
      constexpr uint32_t kCols = (kTransPiece - 16) / ES;
      // no halo when every destination run starts on a 16-byte boundary: windows never straddle chunks
      const uint32_t halo = ((((uintptr_t)f.d | ((size_t)f.dsc * ED)) & 15u) == 0 && kOwn % (16 / ED) == 0) ? 0u : kTransHalo;
      for (uint32_t j0 = 0; j0 < f.nc && !failed; j0 += kCols)
        for (uint32_t i0 = 0; i0 < f.nr && !failed; i0 += kOwn)
          push_trans(f.s + ((size_t)i0 * f.ssr + j0) * ES, f.d + ((size_t)j0 * f.dsc + i0) * ED,
                     min(kOwn + halo, f.nr - i0), min(kCols, f.nc - j0), (uint64_t)f.ssr * ES,
                     (uint64_t)f.dsc * ED, min(kOwn, f.nr - i0), i0 == 0 ? 1u : 0u);
    } else {
      push_simple(MODE_COOP, k, 1, &cur);   // narrow transposes, short rows, fan-out: the workers share the tile
    }
  }
  flush_run();          // runs do not cross scheduling batches: tile indices must stay consecutive
  }
  if (lane == 0) {
    while (!failed && n_store < n_load) store_oldest();
  }
  failed = __shfl_sync(0xFFFFFFFFu, (uint32_t)failed, 0) != 0;
  if (!failed) push_simple(MODE_END, 0);
  if (lane == 0) {
    bulk_wait_all();
    if (sched) {
      // the last block to finish re-arms the counters for the next launch of this table
      __threadfence();
      if (atomicAdd(&sched[1], 1u) == gridDim.x - 1) {
        sched[0] = 0;
        sched[1] = 0;
        __threadfence();
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// launch
// ---------------------------------------------------------------------------------------------

template <int ES, int ED>
cudaError_t launch_one(const wb_plan* plan, const TileTable& T, uint64_t src_add, uint64_t dst_add,
                       cudaStream_t stream, uint32_t tile_off, uint32_t tile_count, bool whole) {
  static bool configured[16] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 16 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(wb_exec_kernel<ES, ED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)Rings<ES, ED>::kDyn);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  wb_exec_kernel<ES, ED><<<dim3(plan->grid), dim3(kThreads), Rings<ES, ED>::kDyn, stream>>>(
      T.d_tiles + tile_off, T.d_cta_begin, T.d_extras, src_add, dst_add, plan->d_err, tile_count,
      (whole && (plan->opts.flags & WB_PLAN_STATIC_SCHEDULE)) ? nullptr : T.d_sched);
  return cudaGetLastError();
}

// Launch the executor on a tile table, or (tile_count != 0) on a contiguous range of its tiles; a
// range is always scheduled at run time, the fixed per-block ranges only describe whole tables.
wb_status launch_table(const wb_plan* plan, const TileTable& T, uint64_t src_add, uint64_t dst_add,
                       uint32_t es, uint32_t ed, cudaStream_t stream, uint32_t tile_off = 0,
                       uint32_t tile_count = 0) {
  if (T.tiles.empty()) return WB_OK;
  const bool whole = tile_count == 0;
  if (whole) tile_count = (uint32_t)T.tiles.size();
  cudaError_t e;
  if (es == 2 && ed == 2) e = launch_one<2, 2>(plan, T, src_add, dst_add, stream, tile_off, tile_count, whole);
  else if (es == 4 && ed == 4) e = launch_one<4, 4>(plan, T, src_add, dst_add, stream, tile_off, tile_count, whole);
  else if (es == 4 && ed == 2) e = launch_one<4, 2>(plan, T, src_add, dst_add, stream, tile_off, tile_count, whole);
  else e = launch_one<2, 4>(plan, T, src_add, dst_add, stream, tile_off, tile_count, whole);
  return e == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}

inline uint32_t esize(uint32_t dt) { return dt == WB_F32 ? 4u : 2u; }
inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

namespace wbi {
void release_device_tables(wb_plan* plan) {
  if (plan->d_arena) {
    cudaFree(plan->d_arena);
    plan->d_arena = nullptr;
  }
  for (void* e : plan->host_events) cudaEventDestroy(static_cast<cudaEvent_t>(e));
  plan->host_events.clear();
  if (plan->h2d_stream) cudaStreamDestroy(static_cast<cudaStream_t>(plan->h2d_stream));
  if (plan->d2h_stream) cudaStreamDestroy(static_cast<cudaStream_t>(plan->d2h_stream));
  plan->h2d_stream = plan->d2h_stream = nullptr;
  plan->bound = false;
}
}  // namespace wbi

extern "C" int wb_launches_per_call(void) { return 1; }

extern "C" wb_status wb_plan_bind(wb_plan* plan, const void* const* src_base, size_t n_src,
                                  void* const* dst_base, size_t n_dst) {
  if (!plan || !src_base || !dst_base) return WB_ERR_INVALID_ARG;
  if (n_src != plan->src.tensors.size() || n_dst != plan->dst.tensors.size()) return WB_ERR_INVALID_ARG;
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype);
  for (size_t i = 0; i < n_src; ++i)
    if (!src_base[i] || ((uintptr_t)src_base[i] % es)) return WB_ERR_INVALID_ARG;
  for (size_t i = 0; i < n_dst; ++i)
    if (!dst_base[i] || ((uintptr_t)dst_base[i] % ed)) return WB_ERR_INVALID_ARG;
  try {
    plan->src_base.assign(src_base, src_base + n_src);
    plan->dst_base.assign(dst_base, dst_base + n_dst);
    // lay every table out in one arena
    std::vector<TileTable*> tabs{&plan->remap};
    for (Round& R : plan->rounds) { tabs.push_back(&R.pack); tabs.push_back(&R.unpack); }
    size_t bytes = 0;
    for (TileTable* T : tabs)
      bytes += up256(T->tiles.size() * sizeof(DTile)) + up256(T->extras.size() * sizeof(DDst)) +
               up256(T->cta_begin.size() * sizeof(uint32_t)) + 256;
    const size_t err_off = up256(bytes);
    const size_t cmp_off = err_off + 256;
    bytes = up256(cmp_off + plan->replica_pairs.size() * sizeof(DCompare) + 256);
    std::vector<char> host(bytes, 0);
    if (!plan->d_arena || plan->arena_bytes != bytes) {
      wbi::release_device_tables(plan);
      if (cudaMalloc(&plan->d_arena, bytes) != cudaSuccess) { plan->d_arena = nullptr; return WB_ERR_OOM; }
      plan->arena_bytes = bytes;
    }
    if (cudaGetDevice(&plan->device) != cudaSuccess) return WB_ERR_CUDA;
    char* dbase = static_cast<char*>(plan->d_arena);
    plan->d_err = reinterpret_cast<uint32_t*>(dbase + err_off);
    plan->d_mismatch = reinterpret_cast<unsigned long long*>(dbase + err_off + 64);
    plan->d_compare = reinterpret_cast<DCompare*>(dbase + cmp_off);
    {
      DCompare* hc = reinterpret_cast<DCompare*>(host.data() + cmp_off);
      for (size_t k = 0; k < plan->replica_pairs.size(); ++k) {
        const ReplicaPair& rp = plan->replica_pairs[k];
        const NSlice& a = plan->src.slices[rp.slice_a];
        const NSlice& b = plan->src.slices[rp.slice_b];
        DCompare c{};
        c.a = (uint64_t)(uintptr_t)plan->src_base[a.tensor] + a.elem(rp.rect.r0, rp.rect.c0) * es;
        c.b = (uint64_t)(uintptr_t)plan->src_base[b.tensor] + b.elem(rp.rect.r0, rp.rect.c0) * es;
        c.nr = (uint32_t)rp.rect.nr; c.nc = (uint32_t)rp.rect.nc;
        c.a_sr = (uint32_t)a.sr(); c.a_sc = (uint32_t)a.sc(); c.b_sr = (uint32_t)b.sr(); c.b_sc = (uint32_t)b.sc();
        hc[k] = c;
      }
    }
    size_t off = 0;
    for (size_t ti = 0; ti < tabs.size(); ++ti) {
      TileTable* T = tabs[ti];
      // the side of a pack (odd index) / unpack (even index > 0) table that is the bucket keeps
      // byte offsets; the kernel adds the bucket base
      const uint32_t tes = (ti != 0 && ti % 2 == 0) ? ed : es;   // unpack reads bucket (dst dtype)
      auto addr = [&](int32_t tensor, uint64_t elem_off, bool is_src) -> uint64_t {
        if (tensor < 0) return elem_off * (is_src ? tes : ed);
        return is_src ? (uint64_t)(uintptr_t)plan->src_base[tensor] + elem_off * tes
                      : (uint64_t)(uintptr_t)plan->dst_base[tensor] + elem_off * ed;
      };
      T->d_tiles = reinterpret_cast<DTile*>(dbase + off);
      DTile* ht = reinterpret_cast<DTile*>(host.data() + off);
      for (size_t k = 0; k < T->tiles.size(); ++k) {
        const HTile& h = T->tiles[k];
        DTile dt{};
        dt.src = addr(h.src_tensor, h.src_off, true);
        dt.dst = addr(h.dst_tensor, h.dst_off, false);
        dt.nr = h.nr; dt.nc = h.nc; dt.ssr = h.ssr; dt.ssc = h.ssc; dt.dsr = h.dsr; dt.dsc = h.dsc;
        dt.kind_extra = h.kind | (h.n_extra << 8);
        dt.extra = h.extra;
        ht[k] = dt;
      }
      off += up256(T->tiles.size() * sizeof(DTile));
      T->d_extras = reinterpret_cast<DDst*>(dbase + off);
      DDst* hx = reinterpret_cast<DDst*>(host.data() + off);
      for (size_t k = 0; k < T->extras.size(); ++k) {
        const HDst& h = T->extras[k];
        hx[k] = DDst{addr(h.tensor, h.off, false), h.sr, h.sc};
      }
      off += up256(T->extras.size() * sizeof(DDst));
      T->d_cta_begin = reinterpret_cast<uint32_t*>(dbase + off);
      std::memcpy(host.data() + off, T->cta_begin.data(), T->cta_begin.size() * sizeof(uint32_t));
      off += up256(T->cta_begin.size() * sizeof(uint32_t));
      T->d_sched = reinterpret_cast<uint32_t*>(dbase + off);   // {next tile, blocks done}, zero
      off += 256;
    }
    if (cudaMemcpy(plan->d_arena, host.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess)
      return WB_ERR_CUDA;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  plan->bound = true;
  return WB_OK;
}

// Replica consistency: the planner reads a replicated region from one holder only, which is valid
// because replicas carry the same bits.  This debug pass compares every replica pair element by
// element and counts the differences.
template <typename T>
__global__ void wb_compare_kernel(const DCompare* __restrict__ ops, uint32_t n_ops,
                                  unsigned long long* __restrict__ mismatches) {
  unsigned long long bad = 0;
  for (uint32_t k = blockIdx.x; k < n_ops; k += gridDim.x) {
    const DCompare c = ops[k];
    const T* a = reinterpret_cast<const T*>(c.a);
    const T* b = reinterpret_cast<const T*>(c.b);
    const unsigned long long n = (unsigned long long)c.nr * c.nc;
    for (unsigned long long e = threadIdx.x; e < n; e += blockDim.x) {
      const unsigned long long i = e / c.nc, j = e - i * c.nc;
      if (a[i * c.a_sr + j * c.a_sc] != b[i * c.b_sr + j * c.b_sc]) ++bad;
    }
  }
  if (bad) atomicAdd(mismatches, bad);
}

extern "C" wb_status wb_plan_check_replicas(const wb_plan* plan, uint64_t* n_mismatches, void* cuda_stream) {
  if (!plan) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long bad = 0;
  const uint32_t n = (uint32_t)plan->replica_pairs.size();
  if (n) {
    if (cudaMemsetAsync(plan->d_mismatch, 0, sizeof(unsigned long long), stream) != cudaSuccess) return WB_ERR_CUDA;
    const uint32_t grid = n < 148u * 8 ? n : 148u * 8;
    if (esize(plan->src.dtype) == 4) wb_compare_kernel<uint32_t><<<grid, 256, 0, stream>>>(plan->d_compare, n, plan->d_mismatch);
    else wb_compare_kernel<uint16_t><<<grid, 256, 0, stream>>>(plan->d_compare, n, plan->d_mismatch);
    if (cudaGetLastError() != cudaSuccess) return WB_ERR_CUDA;
    if (cudaMemcpyAsync(&bad, plan->d_mismatch, sizeof(bad), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return WB_ERR_CUDA;
  }
  if (n_mismatches) *n_mismatches = bad;
  return bad ? WB_ERR_REPLICA_MISMATCH : WB_OK;
}

extern "C" wb_status wb_wait_probe(uint32_t limit_ms, void* cuda_stream) {
  if (limit_ms == 0 || limit_ms > 2000) return WB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t* d_err = nullptr;
  uint32_t err = 0;
  if (cudaMalloc(&d_err, sizeof(uint32_t)) != cudaSuccess) return WB_ERR_OOM;
  cudaError_t e = cudaMemsetAsync(d_err, 0, sizeof(uint32_t), stream);
  if (e == cudaSuccess) {
    wb_wait_probe_kernel<<<1, 32, 0, stream>>>((uint64_t)limit_ms * 1000000ull, d_err);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&err, d_err, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  cudaFree(d_err);
  if (e != cudaSuccess) return WB_ERR_CUDA;
  return err == 0x7Du ? WB_ERR_INTERNAL : WB_OK;
}

extern "C" wb_status wb_plan_check(const wb_plan* plan) {
  if (!plan) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  uint32_t e = 0;
  if (cudaMemcpy(&e, plan->d_err, sizeof(e), cudaMemcpyDeviceToHost) != cudaSuccess) return WB_ERR_CUDA;
  return e == 0 ? WB_OK : WB_ERR_INTERNAL;
}

extern "C" wb_status wb_remap(const wb_plan* plan, void* cuda_stream) {
  if (!plan) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  return launch_table(plan, plan->remap, 0, 0, esize(plan->src.dtype), esize(plan->dst.dtype),
                      static_cast<cudaStream_t>(cuda_stream));
}

extern "C" wb_status wb_pack(const wb_plan* plan, size_t round, void* bucket, void* cuda_stream) {
  if (!plan || !bucket || round >= plan->rounds.size() || ((uintptr_t)bucket & 15u)) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  return launch_table(plan, plan->rounds[round].pack, 0, (uint64_t)(uintptr_t)bucket,
                      esize(plan->src.dtype), esize(plan->dst.dtype), static_cast<cudaStream_t>(cuda_stream));
}

extern "C" wb_status wb_unpack(const wb_plan* plan, size_t round, const void* bucket, void* cuda_stream) {
  if (!plan || !bucket || round >= plan->rounds.size() || ((uintptr_t)bucket & 15u)) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  return launch_table(plan, plan->rounds[round].unpack, (uint64_t)(uintptr_t)bucket, 0,
                      esize(plan->dst.dtype), esize(plan->dst.dtype), static_cast<cudaStream_t>(cuda_stream));
}

// Internal streams and events shared by the multi-stream entry points (created on first use,
// destroyed with the device tables).
static wb_status ensure_pipeline(wb_plan* plan, size_t n_events) {
  if (!plan->h2d_stream) {
    cudaStream_t a, b;
    if (cudaStreamCreateWithFlags(&a, cudaStreamNonBlocking) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaStreamCreateWithFlags(&b, cudaStreamNonBlocking) != cudaSuccess) { cudaStreamDestroy(a); return WB_ERR_CUDA; }
    plan->h2d_stream = a;
    plan->d2h_stream = b;
  }
  while (plan->host_events.size() < n_events) {
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return WB_ERR_CUDA;
    plan->host_events.push_back(e);
  }
  return WB_OK;
}

// wb_transfer_rounds: all rounds of the two-pass path with two buckets in flight (Section 3.2:
// consecutive rounds overlap; Section 4: a depth-2 buffer system).  Packing runs on one internal
// stream and assembly on another; pack(r) waits for unpack(r-2), which frees bucket r mod 2, and
// unpack(r) waits for pack(r).  On one GPU the two persistent kernels compete for the same SMs, so
// what overlaps is the tail of one launch with the head of the next.
extern "C" wb_status wb_transfer_rounds(const wb_plan* plan_c, void* bucket0, void* bucket1, uint32_t flags,
                                        void* cuda_stream) {
  if (!plan_c || !bucket0 || ((uintptr_t)bucket0 & 15u) || (flags & ~WB_ROUNDS_SERIAL)) return WB_ERR_INVALID_ARG;
  const bool serial = flags & WB_ROUNDS_SERIAL;
  if (!serial && (!bucket1 || ((uintptr_t)bucket1 & 15u) || bucket1 == bucket0)) return WB_ERR_INVALID_ARG;
  if (!plan_c->bound) return WB_ERR_NOT_BOUND;
  wb_plan* plan = const_cast<wb_plan*>(plan_c);     // lazily built pipeline state, not the plan itself
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype);
  const size_t R = plan->rounds.size();
  if (R == 0) return WB_OK;
  if (serial) {
    for (size_t r = 0; r < R; ++r) {
      wb_status st = launch_table(plan, plan->rounds[r].pack, 0, (uint64_t)(uintptr_t)bucket0, es, ed, stream);
      if (st == WB_OK) st = launch_table(plan, plan->rounds[r].unpack, (uint64_t)(uintptr_t)bucket0, 0, ed, ed, stream);
      if (st != WB_OK) return st;
    }
    return WB_OK;
  }
  try {
    wb_status st = ensure_pipeline(plan, 2 * R + 1);
    if (st != WB_OK) return st;
    cudaStream_t ps = static_cast<cudaStream_t>(plan->h2d_stream), us = static_cast<cudaStream_t>(plan->d2h_stream);
    auto packed = [&](size_t r) { return static_cast<cudaEvent_t>(plan->host_events[2 * r]); };
    auto unpacked = [&](size_t r) { return static_cast<cudaEvent_t>(plan->host_events[2 * r + 1]); };
    cudaEvent_t start = static_cast<cudaEvent_t>(plan->host_events[2 * R]);
    // both internal streams start after whatever the caller already queued on its stream
    if (cudaEventRecord(start, stream) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaStreamWaitEvent(ps, start, 0) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaStreamWaitEvent(us, start, 0) != cudaSuccess) return WB_ERR_CUDA;
    for (size_t r = 0; r < R; ++r) {
      const uint64_t bucket = (uint64_t)(uintptr_t)((r & 1) ? bucket1 : bucket0);
      if (r >= 2 && cudaStreamWaitEvent(ps, unpacked(r - 2), 0) != cudaSuccess) return WB_ERR_CUDA;
      st = launch_table(plan, plan->rounds[r].pack, 0, bucket, es, ed, ps);
      if (st != WB_OK) return st;
      if (cudaEventRecord(packed(r), ps) != cudaSuccess) return WB_ERR_CUDA;
      if (cudaStreamWaitEvent(us, packed(r), 0) != cudaSuccess) return WB_ERR_CUDA;
      st = launch_table(plan, plan->rounds[r].unpack, bucket, 0, ed, ed, us);
      if (st != WB_OK) return st;
      if (cudaEventRecord(unpacked(r), us) != cudaSuccess) return WB_ERR_CUDA;
    }
    // the caller's stream completes when the last assembly has (the assembly stream is in order
    // and its last kernel waited for the last pack)
    if (cudaStreamWaitEvent(stream, unpacked(R - 1), 0) != cudaSuccess) return WB_ERR_CUDA;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  return WB_OK;
}

// wb_remap_host pipelines the transfer over PCIe: the remap table is cut into groups of
// consecutive tiles; group g's source spans go host -> device on one copy stream, its tiles run
// on the caller's stream, its destination spans go device -> host on a second copy stream, so
// uploads, the kernel and downloads of neighbouring groups overlap (PCIe is full duplex).  A span
// is the bounding element interval a group touches in one tensor; spans of different groups may
// overlap, which only copies some bytes twice: the later download of an element always follows
// the kernel that wrote it.
static wb_status build_host_groups(wb_plan* plan) {
  const TileTable& T = plan->remap;
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype);
  uint64_t total = 0;
  for (const HTile& t : T.tiles) total += t.bytes;
  const uint64_t target = std::max<uint64_t>(256ull << 20, total / 24);
  plan->host_groups.clear();
  HostGroup g{};
  uint64_t acc = 0;
  std::vector<std::pair<uint64_t, uint64_t>> smin(plan->src.tensors.size()), dmin(plan->dst.tensors.size());
  std::vector<uint32_t> stouched, dtouched;
  auto reset = [&]() {
    for (uint32_t i : stouched) smin[i] = {UINT64_MAX, 0};
    for (uint32_t i : dtouched) dmin[i] = {UINT64_MAX, 0};
    stouched.clear(); dtouched.clear();
  };
  for (auto& p : smin) p = {UINT64_MAX, 0};
  for (auto& p : dmin) p = {UINT64_MAX, 0};
  auto touch = [&](std::vector<std::pair<uint64_t, uint64_t>>& v, std::vector<uint32_t>& list, int32_t tensor,
                   uint64_t off, uint32_t nr, uint32_t nc, uint32_t sr, uint32_t sc) {
    const uint64_t last = off + (uint64_t)(nr - 1) * sr + (uint64_t)(nc - 1) * sc;
    auto& p = v[tensor];
    if (p.first == UINT64_MAX) list.push_back((uint32_t)tensor);
    p.first = std::min(p.first, off);
    p.second = std::max(p.second, last + 1);
  };
  auto flush = [&](uint32_t end_tile) {
    g.tile_end = end_tile;
    for (uint32_t i : stouched) g.src.push_back(HostSpan{i, smin[i].first * es, (smin[i].second - smin[i].first) * es});
    for (uint32_t i : dtouched) g.dst.push_back(HostSpan{i, dmin[i].first * ed, (dmin[i].second - dmin[i].first) * ed});
    plan->host_groups.push_back(g);
    g = HostGroup{};
    g.tile_begin = end_tile;
    reset();
    acc = 0;
  };
  for (uint32_t k = 0; k < T.tiles.size(); ++k) {
    const HTile& t = T.tiles[k];
    touch(smin, stouched, t.src_tensor, t.src_off, t.nr, t.nc, t.ssr, t.ssc);
    touch(dmin, dtouched, t.dst_tensor, t.dst_off, t.nr, t.nc, t.dsr, t.dsc);
    for (uint32_t x = 0; x < t.n_extra; ++x) {
      const HDst& o = T.extras[t.extra + x];
      touch(dmin, dtouched, o.tensor, o.off, t.nr, t.nc, o.sr, o.sc);
    }
    acc += t.bytes;
    if (acc >= target) flush(k + 1);
  }
  if (acc > 0 || plan->host_groups.empty()) flush((uint32_t)T.tiles.size());
  return WB_OK;
}

extern "C" wb_status wb_remap_host(const wb_plan* plan_c, const void* const* host_src, size_t n_src,
                                   void* const* host_dst, size_t n_dst, void* cuda_stream) {
  if (!plan_c || !host_src || !host_dst) return WB_ERR_INVALID_ARG;
  if (!plan_c->bound) return WB_ERR_NOT_BOUND;
  if (n_src != plan_c->src.tensors.size() || n_dst != plan_c->dst.tensors.size()) return WB_ERR_INVALID_ARG;
  for (size_t i = 0; i < n_src; ++i) if (!host_src[i]) return WB_ERR_INVALID_ARG;
  for (size_t i = 0; i < n_dst; ++i) if (!host_dst[i]) return WB_ERR_INVALID_ARG;
  wb_plan* plan = const_cast<wb_plan*>(plan_c);     // lazily built pipeline state, not the plan itself
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype);
  try {
    if (plan->host_groups.empty()) build_host_groups(plan);
    const size_t G = plan->host_groups.size();
    { wb_status pst = ensure_pipeline(plan, 2 * G + 2); if (pst != WB_OK) return pst; }
    cudaStream_t up = static_cast<cudaStream_t>(plan->h2d_stream), down = static_cast<cudaStream_t>(plan->d2h_stream);
    auto ev = [&](size_t i) { return static_cast<cudaEvent_t>(plan->host_events[i]); };
    // the copy streams start after whatever the caller already queued on its stream
    if (cudaEventRecord(ev(2 * G), stream) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaStreamWaitEvent(up, ev(2 * G), 0) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaStreamWaitEvent(down, ev(2 * G), 0) != cudaSuccess) return WB_ERR_CUDA;
    for (size_t g = 0; g < G; ++g) {
      const HostGroup& hg = plan->host_groups[g];
      for (const HostSpan& sp : hg.src)
        if (cudaMemcpyAsync(static_cast<char*>(const_cast<void*>(plan->src_base[sp.tensor])) + sp.off,
                            static_cast<const char*>(host_src[sp.tensor]) + sp.off, sp.bytes,
                            cudaMemcpyHostToDevice, up) != cudaSuccess) return WB_ERR_CUDA;
      if (cudaEventRecord(ev(2 * g), up) != cudaSuccess) return WB_ERR_CUDA;
      if (cudaStreamWaitEvent(stream, ev(2 * g), 0) != cudaSuccess) return WB_ERR_CUDA;
      wb_status st = launch_table(plan, plan->remap, 0, 0, es, ed, stream, hg.tile_begin, hg.tile_end - hg.tile_begin);
      if (st != WB_OK) return st;
      if (cudaEventRecord(ev(2 * g + 1), stream) != cudaSuccess) return WB_ERR_CUDA;
      if (cudaStreamWaitEvent(down, ev(2 * g + 1), 0) != cudaSuccess) return WB_ERR_CUDA;
      for (const HostSpan& sp : hg.dst)
        if (cudaMemcpyAsync(static_cast<char*>(host_dst[sp.tensor]) + sp.off,
                            static_cast<const char*>(plan->dst_base[sp.tensor]) + sp.off, sp.bytes,
                            cudaMemcpyDeviceToHost, down) != cudaSuccess) return WB_ERR_CUDA;
    }
    // the caller's stream completes when the last download has
    if (cudaEventRecord(ev(2 * G + 1), down) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaStreamWaitEvent(stream, ev(2 * G + 1), 0) != cudaSuccess) return WB_ERR_CUDA;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  return WB_OK;
}


// =================================================================================================
// wb_remap_static: the fused remap for callers that must not allocate device memory.
//
// The executor kernel needs scratch beyond the caller's tensors: the tile table it walks and an
// error word.  wb_plan_bind puts those in a cudaMalloc'd arena.  This entry point instead keeps
// them in the fixed array below, which every GPU that loads the library holds until the process
// exits.  It never calls cudaMalloc, cudaFree or any allocating routine.
// =================================================================================================
static __device__ __align__(256) unsigned char g_static_scratch[WB_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxStaticDevices = 64;
void* g_static_ptr[kMaxStaticDevices] = {};     // device address of g_static_scratch, per device
unsigned char g_static_stage[WB_STATIC_SCRATCH_BYTES];   // host image of the scratch, built per call
struct SpinLock {
  std::atomic_flag f = ATOMIC_FLAG_INIT;
  void lock() { while (f.test_and_set(std::memory_order_acquire)) {} }
  void unlock() { f.clear(std::memory_order_release); }
} g_static_lock;

// Set-up, once per device, with that device current: resolve the array's device address (in host
// code the array's name is only a stand-in, not a device address) and let the kernels use their
// dynamic shared memory.
template <int ES, int ED>
cudaError_t static_setup_kernel() {
  return cudaFuncSetAttribute(wb_exec_kernel<ES, ED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)Rings<ES, ED>::kDyn);
}
wb_status static_setup(int dev) {
  if (g_static_ptr[dev]) return WB_OK;
  void* ptr = nullptr;
  if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return WB_ERR_CUDA;
  if (static_setup_kernel<2, 2>() != cudaSuccess || static_setup_kernel<4, 4>() != cudaSuccess ||
      static_setup_kernel<4, 2>() != cudaSuccess || static_setup_kernel<2, 4>() != cudaSuccess)
    return WB_ERR_CUDA;
  g_static_ptr[dev] = ptr;
  return WB_OK;
}
}  // namespace

extern "C" wb_status wb_remap_static(const wb_plan* plan, const void* const* src_base, size_t n_src,
                                     void* const* dst_base, size_t n_dst, uint32_t flags, void* cuda_stream) {
  if (!plan || !src_base || !dst_base || (flags & ~WB_STATIC_SYNC_CHECK)) return WB_ERR_INVALID_ARG;
  if (n_src != plan->src.tensors.size() || n_dst != plan->dst.tensors.size()) return WB_ERR_INVALID_ARG;
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype);
  for (size_t i = 0; i < n_src; ++i)
    if (!src_base[i] || ((uintptr_t)src_base[i] % es)) return WB_ERR_INVALID_ARG;
  for (size_t i = 0; i < n_dst; ++i)
    if (!dst_base[i] || ((uintptr_t)dst_base[i] % ed)) return WB_ERR_INVALID_ARG;
  const TileTable& T = plan->remap;
  if (T.tiles.empty()) return WB_OK;
  // layout of the scratch: [error word | tiles | fan-out records | per-block tile ranges]
  const size_t off_tiles = 256;
  const size_t off_extras = off_tiles + up256(T.tiles.size() * sizeof(DTile));
  const size_t off_begin = off_extras + up256(T.extras.size() * sizeof(DDst));
  const size_t total = off_begin + up256(T.cta_begin.size() * sizeof(uint32_t));
  if (total > (size_t)WB_STATIC_SCRATCH_BYTES) return WB_ERR_STATIC_LIMIT;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxStaticDevices) return WB_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  g_static_lock.lock();
  wb_status st = static_setup(dev);
  if (st != WB_OK) { g_static_lock.unlock(); return st; }
  char* dbase = static_cast<char*>(g_static_ptr[dev]);
  // the array keeps the previous call's contents: rebuild everything this launch reads, and
  // zero the error word and the scheduling counters (first 256 bytes)
  std::memset(g_static_stage, 0, off_tiles);
  DTile* ht = reinterpret_cast<DTile*>(g_static_stage + off_tiles);
  for (size_t k = 0; k < T.tiles.size(); ++k) {
    const HTile& h = T.tiles[k];
    DTile dt{};
    dt.src = (uint64_t)(uintptr_t)src_base[h.src_tensor] + h.src_off * es;
    dt.dst = (uint64_t)(uintptr_t)dst_base[h.dst_tensor] + h.dst_off * ed;
    dt.nr = h.nr; dt.nc = h.nc; dt.ssr = h.ssr; dt.ssc = h.ssc; dt.dsr = h.dsr; dt.dsc = h.dsc;
    dt.kind_extra = h.kind | (h.n_extra << 8);
    dt.extra = h.extra;
    ht[k] = dt;
  }
  DDst* hx = reinterpret_cast<DDst*>(g_static_stage + off_extras);
  for (size_t k = 0; k < T.extras.size(); ++k) {
    const HDst& h = T.extras[k];
    hx[k] = DDst{(uint64_t)(uintptr_t)dst_base[h.tensor] + h.off * ed, h.sr, h.sc};
  }
  std::memcpy(g_static_stage + off_begin, T.cta_begin.data(), T.cta_begin.size() * sizeof(uint32_t));
  // pageable source: the runtime has taken its copy of the image when this returns, so the host
  // image can be reused by the next call
  cudaError_t e = cudaMemcpyAsync(dbase, g_static_stage, total, cudaMemcpyHostToDevice, stream);
  g_static_lock.unlock();
  if (e != cudaSuccess) return WB_ERR_CUDA;

  const DTile* d_tiles = reinterpret_cast<const DTile*>(dbase + off_tiles);
  const DDst* d_extras = reinterpret_cast<const DDst*>(dbase + off_extras);
  const uint32_t* d_begin = reinterpret_cast<const uint32_t*>(dbase + off_begin);
  uint32_t* d_err = reinterpret_cast<uint32_t*>(dbase);
  uint32_t* d_sched = (plan->opts.flags & WB_PLAN_STATIC_SCHEDULE) ? nullptr : reinterpret_cast<uint32_t*>(dbase + 64);
  const uint32_t n_tiles = (uint32_t)T.tiles.size();
  const dim3 grid(plan->grid), block(kThreads);
  if (es == 2 && ed == 2) wb_exec_kernel<2, 2><<<grid, block, Rings<2, 2>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched);
  else if (es == 4 && ed == 4) wb_exec_kernel<4, 4><<<grid, block, Rings<4, 4>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched);
  else if (es == 4 && ed == 2) wb_exec_kernel<4, 2><<<grid, block, Rings<4, 2>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched);
  else wb_exec_kernel<2, 4><<<grid, block, Rings<2, 4>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched);
  if (cudaGetLastError() != cudaSuccess) return WB_ERR_CUDA;
  if (flags & WB_STATIC_SYNC_CHECK) {
    uint32_t err = 0;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaMemcpy(&err, d_err, sizeof(err), cudaMemcpyDeviceToHost) != cudaSuccess) return WB_ERR_CUDA;
    if (err) return WB_ERR_INTERNAL;
  }
  return WB_OK;
}
