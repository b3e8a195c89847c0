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
//   staged   transposing tiles: the producer warp brings chunks of source rows into a ring slot - eight
//   transp.  2-D tensor-map (TMA) loads per chunk where wb_plan_bind could encode maps (the fused table),
//            per-lane asynchronous copies into bank-swizzled rows otherwise; the workers write 16-byte
//            windows of the destination runs, neighbouring lanes on neighbouring windows of one run.
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
//
// Files: wb_exec_prims.cuh (access, cast, mbarrier and copy primitives), wb_exec_workers.cuh (rings,
// slot descriptors, worker routines), wb_exec_kernel.cuh (the kernel), this file (launch, binding
// and the extern "C" entry points).
#include <cuda.h>            // CUtensorMap and its enums only: the encoder is looked up at run time
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "wb_internal.h"

using namespace wbi;

#include "wb_exec_kernel.cuh"

namespace {

// ---------------------------------------------------------------------------------------------
// launch
// ---------------------------------------------------------------------------------------------

template <int ES, int ED>
cudaError_t launch_one(const wb_plan* plan, const TileTable& T, uint64_t src_add, uint64_t dst_add,
                       cudaStream_t stream, uint32_t tile_off, uint32_t tile_count, bool whole) {
  // the kernel needs more dynamic shared memory than the default limit: raise it once per device
  // (on every launch for device ordinals beyond the table)
  static std::atomic<bool> configured[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
  const bool tracked = dev >= 0 && dev < 64;
  if (!tracked || !configured[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(wb_exec_kernel<ES, ED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)Rings<ES, ED>::kDyn);
    if (e != cudaSuccess) return e;
    if (tracked) configured[dev].store(true, std::memory_order_release);
  }
  wb_exec_kernel<ES, ED><<<dim3(plan->grid), dim3(kThreads), Rings<ES, ED>::kDyn, stream>>>(
      T.d_tiles + tile_off, T.d_cta_begin, T.d_extras, src_add, dst_add, plan->d_err, tile_count,
      (whole && (plan->opts.flags & WB_PLAN_STATIC_SCHEDULE)) ? nullptr : T.d_sched, T.d_maps);
  return cudaGetLastError();
}

// Launch the executor on a tile table, or (tile_count != 0) on a contiguous range of its tiles; a
// range is always scheduled at run time, the fixed per-block ranges only describe whole tables.
wb_status launch_table(const wb_plan* plan, const TileTable& T, uint64_t src_add, uint64_t dst_add,
                       uint32_t es, uint32_t ed, cudaStream_t stream, uint32_t tile_off = 0,
                       uint32_t tile_count = 0) {
  if (T.tiles.empty()) return WB_OK;
  if (!wbi::on_bound_device(plan)) return WB_ERR_INVALID_ARG;
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

// ---------------------------------------------------------------------------------------------
// tensor maps of the staged transposition (see kTmaClasses)
// ---------------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// The driver's encoder, through the runtime (the library does not link the driver); null if this
// driver has none, and the tables then keep the per-lane copies.
EncodeTiledFn tensor_map_encoder() {
  static std::atomic<EncodeTiledFn> cached{nullptr};
  static std::atomic<bool> looked{false};
  if (!looked.load(std::memory_order_acquire)) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult res = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) != cudaSuccess ||
        res != cudaDriverEntryPointSuccess)
      fn = nullptr;
    (void)cudaGetLastError();
    cached.store(reinterpret_cast<EncodeTiledFn>(fn), std::memory_order_release);
    looked.store(true, std::memory_order_release);
  }
  return cached.load(std::memory_order_acquire);
}

// limits of a tensor map: pitches below 2^40 bytes, extents up to 2^32 elements (any tile meets the second)
bool pitch_ok(const HTile& h, uint32_t es) { return (uint64_t)h.ssr * es * kTmaClasses < (1ull << 40); }

// Does tile h of a table whose source elements have `es` bytes (destination `ed`) get tensor maps?
bool tile_wants_maps(const HTile& h, uint32_t es) {
  if (h.src_tensor < 0) return false;       // the bucket's address is only known at launch
  return es == 4 ? staged_trans_ok<4>(h.kind, h.n_extra, h.nr, h.nc) : staged_trans_ok<2>(h.kind, h.n_extra, h.nr, h.nc);
}

// The kTmaClasses maps of one tile: class q covers tile rows q, q + 8, ...; its base is the 16-byte
// boundary at or before the first element of row q, its rows are 8 tile pitches apart, and its width is
// the 16-byte aligned superset of a tile row, so a load never touches memory outside the supersets
// of the tile's rows (coordinates beyond read as zero).
template <int ES, int ED>
bool encode_tile_maps(EncodeTiledFn encode, uint64_t tile_src, const HTile& h, CUtensorMap* out) {
  const uint64_t pitch = (uint64_t)h.ssr * ES;
  for (uint32_t q = 0; q < kTmaClasses; ++q) {
    const uint64_t a = tile_src + q * pitch, lead = a & 15u;
    // rows the tile may read: its own and, across a seam, the first of the tile below (see kTileRowsAfter)
    const uint64_t rows = h.nr + ((h.seam & kTileRowsAfter) ? 16 / ED - 1 : 0);
    cuuint64_t dims[2] = {(lead + (uint64_t)h.nc * ES + 15) / 16 * 16 / ES, (rows - q + kTmaClasses - 1) / kTmaClasses};
    cuuint64_t strides[1] = {pitch * kTmaClasses};
    cuuint32_t box[2] = {kTmaInner / ES, TransGeom<ES, ED>::kBoxRows};
    cuuint32_t estr[2] = {1, 1};
    if (encode(&out[q], ES == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_UINT16, 2,
               reinterpret_cast<void*>(a - lead), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

}  // namespace

namespace wbi {
bool on_bound_device(const wb_plan* plan) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == plan->device;
}
void release_device_tables(wb_plan* plan) {
  release_quant_tables(plan);
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
  wbi::release_quant_tables(plan);      // they hold addresses of the previous binding
  try {
    plan->src_base.assign(src_base, src_base + n_src);
    plan->dst_base.assign(dst_base, dst_base + n_dst);
    // lay every table out in one arena
    std::vector<TileTable*> tabs{&plan->remap};
    for (Round& R : plan->rounds) { tabs.push_back(&R.pack); tabs.push_back(&R.unpack); }
    // tensor maps: the transposing tiles of the fused remap table whose rows get staged (the source
    // of an unpack table is the bucket, whose address arrives with the launch)
    EncodeTiledFn encode = (plan->opts.flags & WB_PLAN_NO_TENSOR_MAPS) ? nullptr : tensor_map_encoder();
    size_t n_map_tiles = 0;
    if (encode)
      for (const HTile& h : plan->remap.tiles) n_map_tiles += tile_wants_maps(h, es) && pitch_ok(h, es);
    size_t bytes = 0;
    for (TileTable* T : tabs)
      bytes += up256(T->tiles.size() * sizeof(DTile)) + up256(T->extras.size() * sizeof(DDst)) +
               up256(T->cta_begin.size() * sizeof(uint32_t)) + 256;
    const size_t maps_off = up256(bytes);
    bytes = maps_off + n_map_tiles * kTmaClasses * sizeof(CUtensorMap);
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
      T->d_maps = nullptr;
      DTile* ht = reinterpret_cast<DTile*>(host.data() + off);
      size_t n_maps = 0;       // maps of this table written so far
      for (size_t k = 0; k < T->tiles.size(); ++k) {
        const HTile& h = T->tiles[k];
        DTile dt{};
        dt.src = addr(h.src_tensor, h.src_off, true);
        dt.dst = addr(h.dst_tensor, h.dst_off, false);
        dt.nr = h.nr; dt.nc = h.nc; dt.ssr = h.ssr; dt.ssc = h.ssc; dt.dsr = h.dsr; dt.dsc = h.dsc;
        dt.kind_extra = h.kind | (h.n_extra << 8) | h.seam;
        dt.extra = h.extra;
        if (ti == 0 && encode && tile_wants_maps(h, es) && pitch_ok(h, es)) {
          CUtensorMap* hm = reinterpret_cast<CUtensorMap*>(host.data() + maps_off) + n_maps;
          const bool ok = es == 4 ? (ed == 4 ? encode_tile_maps<4, 4>(encode, dt.src, h, hm) : encode_tile_maps<4, 2>(encode, dt.src, h, hm))
                                  : (ed == 4 ? encode_tile_maps<2, 4>(encode, dt.src, h, hm) : encode_tile_maps<2, 2>(encode, dt.src, h, hm));
          if (ok) {                           // a refused map leaves the tile on the per-lane copies
            dt.kind_extra |= kTileHasMaps;
            dt.extra = (uint32_t)n_maps;
            n_maps += kTmaClasses;
          }
        }
        ht[k] = dt;
      }
      if (ti == 0 && n_maps) T->d_maps = dbase + maps_off;
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
  if (!wbi::on_bound_device(plan)) return WB_ERR_INVALID_ARG;
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
  if (!wbi::on_bound_device(plan)) return WB_ERR_INVALID_ARG;
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

// The tiles of a set of virtual ranks: maximal runs of consecutive ranks are contiguous tile ranges of
// the round's table (the planner groups pack tiles by sender and unpack tiles by receiver).
static wb_status launch_ranks(const wb_plan* plan, const TileTable& T, const std::vector<uint32_t>& rank_begin,
                              const uint32_t* ranks, size_t n_ranks, uint64_t src_add, uint64_t dst_add, uint32_t es,
                              uint32_t ed, cudaStream_t stream) {
  if (!ranks && n_ranks) return WB_ERR_INVALID_ARG;
  const size_t side_ranks = rank_begin.size() - 1;
  try {
    std::vector<uint32_t> sorted(ranks, ranks + n_ranks);
    for (uint32_t r : sorted) if (r >= side_ranks) return WB_ERR_INVALID_ARG;
    std::sort(sorted.begin(), sorted.end());
    sorted.erase(std::unique(sorted.begin(), sorted.end()), sorted.end());
    for (size_t a = 0; a < sorted.size();) {
      size_t b = a + 1;
      while (b < sorted.size() && sorted[b] == sorted[b - 1] + 1) ++b;
      const uint32_t t0 = rank_begin[sorted[a]], t1 = rank_begin[sorted[b - 1] + 1];
      if (t1 > t0) {
        wb_status st = launch_table(plan, T, src_add, dst_add, es, ed, stream, t0, t1 - t0);
        if (st != WB_OK) return st;
      }
      a = b;
    }
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  return WB_OK;
}

extern "C" wb_status wb_pack_ranks(const wb_plan* plan, size_t round, const uint32_t* ranks, size_t n_ranks,
                                   void* bucket, void* cuda_stream) {
  if (!plan || !bucket || round >= plan->rounds.size() || ((uintptr_t)bucket & 15u)) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  const Round& R = plan->rounds[round];
  return launch_ranks(plan, R.pack, R.pack_rank_begin, ranks, n_ranks, 0, (uint64_t)(uintptr_t)bucket,
                      esize(plan->src.dtype), esize(plan->dst.dtype), static_cast<cudaStream_t>(cuda_stream));
}

extern "C" wb_status wb_unpack_ranks(const wb_plan* plan, size_t round, const uint32_t* ranks, size_t n_ranks,
                                     const void* bucket, void* cuda_stream) {
  if (!plan || !bucket || round >= plan->rounds.size() || ((uintptr_t)bucket & 15u)) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  const Round& R = plan->rounds[round];
  return launch_ranks(plan, R.unpack, R.unpack_rank_begin, ranks, n_ranks, (uint64_t)(uintptr_t)bucket, 0,
                      esize(plan->dst.dtype), esize(plan->dst.dtype), static_cast<cudaStream_t>(cuda_stream));
}

// Internal streams and events shared by the multi-stream entry points (created on first use,
// destroyed with the device tables).
namespace wbi {
wb_status ensure_pipeline(wb_plan* plan, size_t n_events) {
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
}  // namespace wbi
using wbi::ensure_pipeline;

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
  const uint64_t target = plan->opts.host_group_kib ? (uint64_t)plan->opts.host_group_kib << 10
                                                    : std::max<uint64_t>(256ull << 20, total / 24);
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
    // a transposing tile flagged kTileRowsAfter also reads the first rows of the tile below (the window
    // that straddles the seam), which may belong to a later group
    touch(smin, stouched, t.src_tensor, t.src_off, t.nr + ((t.seam & kTileRowsAfter) ? 16 / ed - 1 : 0), t.nc, t.ssr, t.ssc);
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
  // The table is uploaded from one shared host image: a captured copy would read that image again at
  // every replay, with whatever a later call left there.  Refuse instead of recording that.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) return WB_ERR_CUDA;
  if (cap != cudaStreamCaptureStatusNone) return WB_ERR_INVALID_ARG;
  // One lock covers building the image, the upload and the launch: two host threads that call on
  // the same stream must not interleave as copy A, copy B, kernel B, kernel A (kernel A would walk
  // B's table).
  struct Guard {
    SpinLock& l;
    explicit Guard(SpinLock& x) : l(x) { l.lock(); }
    ~Guard() { l.unlock(); }
  } guard(g_static_lock);
  wb_status st = static_setup(dev);
  if (st != WB_OK) return st;
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
    dt.kind_extra = h.kind | (h.n_extra << 8) | h.seam;
    dt.extra = h.extra;
    ht[k] = dt;
  }
  DDst* hx = reinterpret_cast<DDst*>(g_static_stage + off_extras);
  for (size_t k = 0; k < T.extras.size(); ++k) {
    const HDst& h = T.extras[k];
    hx[k] = DDst{(uint64_t)(uintptr_t)dst_base[h.tensor] + h.off * ed, h.sr, h.sc};
  }
  std::memcpy(g_static_stage + off_begin, T.cta_begin.data(), T.cta_begin.size() * sizeof(uint32_t));
  // pageable source: the runtime has taken its copy of the image when this returns (the call
  // blocks the host for that long), so the host image can be reused by the next call
  if (cudaMemcpyAsync(dbase, g_static_stage, total, cudaMemcpyHostToDevice, stream) != cudaSuccess) return WB_ERR_CUDA;

  const DTile* d_tiles = reinterpret_cast<const DTile*>(dbase + off_tiles);
  const DDst* d_extras = reinterpret_cast<const DDst*>(dbase + off_extras);
  const uint32_t* d_begin = reinterpret_cast<const uint32_t*>(dbase + off_begin);
  uint32_t* d_err = reinterpret_cast<uint32_t*>(dbase);
  uint32_t* d_sched = (plan->opts.flags & WB_PLAN_STATIC_SCHEDULE) ? nullptr : reinterpret_cast<uint32_t*>(dbase + 64);
  const uint32_t n_tiles = (uint32_t)T.tiles.size();
  const dim3 grid(plan->grid), block(kThreads);
  if (es == 2 && ed == 2) wb_exec_kernel<2, 2><<<grid, block, Rings<2, 2>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched, nullptr);
  else if (es == 4 && ed == 4) wb_exec_kernel<4, 4><<<grid, block, Rings<4, 4>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched, nullptr);
  else if (es == 4 && ed == 2) wb_exec_kernel<4, 2><<<grid, block, Rings<4, 2>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched, nullptr);
  else wb_exec_kernel<2, 4><<<grid, block, Rings<2, 4>::kDyn, stream>>>(d_tiles, d_begin, d_extras, 0, 0, d_err, n_tiles, d_sched, nullptr);
  if (cudaGetLastError() != cudaSuccess) return WB_ERR_CUDA;
  if (flags & WB_STATIC_SYNC_CHECK) {
    uint32_t err = 0;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return WB_ERR_CUDA;
    if (cudaMemcpy(&err, d_err, sizeof(err), cudaMemcpyDeviceToHost) != cudaSuccess) return WB_ERR_CUDA;
    if (err) return WB_ERR_INTERNAL;
  }
  return WB_OK;
}

