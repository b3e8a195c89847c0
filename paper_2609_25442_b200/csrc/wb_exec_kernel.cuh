// Executor, part 3 of 3: the persistent kernel (producer warp + worker warps).  Included by wb_exec.cu only.
#pragma once
#include "wb_exec_workers.cuh"

namespace {
// The persistent executor: one thread block per SM walks its range of the tile table.
//   warp 0   "producer".  Lane 0 moves direct tiles by itself through a ring of bulk (TMA) copies
//            global -> shared -> global.  For every other tile the warp feeds the worker ring:
//            either the tile's rows are staged into a ring slot with bulk loads (one per row, the
//            16-byte aligned superset of the row; transposing tiles: eight tensor-map loads per chunk,
//            or per-lane asynchronous copies where the table has no tensor maps), or the tile index
//            is queued as is.
//   warps 1.. "workers".  Take ring slots in order: convert staged rows (cast in registers,
//            realignment by funnel shifts, 16-byte vector stores), transpose staged blocks, or
//            run a queued tile cooperatively (element-wise fan-out and other rare shapes).
template <int ES, int ED>
__global__ void __launch_bounds__(kThreads, 1)
wb_exec_kernel(const DTile* __restrict__ tiles, const uint32_t* __restrict__ cta_begin,
               const DDst* __restrict__ extras, uint64_t src_add, uint64_t dst_add, uint32_t* __restrict__ err,
               uint32_t n_tiles, uint32_t* __restrict__ sched, const char* __restrict__ tmaps) {
  using E = Elem<ES, ED>;
  using TG = TransGeom<ES, ED>;
  extern __shared__ __align__(128) char dyn_smem[];
  constexpr int kSlots = Rings<ES, ED>::kSlots;
  constexpr int kSlotBytes = Rings<ES, ED>::kSlotBytes;
  char* const ring = dyn_smem;                                         // kDirectStages x kDirectBytes
  char* const wring = dyn_smem + Rings<ES, ED>::kDirect;               // kSlots x kSlotBytes
  __shared__ __align__(8) uint64_t direct_full[kDirectStages];
  __shared__ __align__(8) uint64_t slot_full[kMaxSlots], slot_empty[kMaxSlots];
  __shared__ __align__(16) ChunkDesc desc[kMaxSlots];
  __shared__ __align__(16) uint32_t trans_tab[kMaxSlots][kTmaClasses * (16 / ED)];   // see staged_trans (tensor-map chunks)
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
        staged_trans<ES, ED>(d, stage, tr);
      } else if (d.mode == MODE_TRANS_TMA) {
        staged_trans_tma<ES, ED>(d, stage, tr, smem_u32(trans_tab[slot]));
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
  uint64_t tab_keys = 0;                // 8 bits per slot: what trans_tab[slot] was computed for (0: nothing yet)
  static_assert(kMaxSlots <= 8, "one 8-bit key per slot");
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
  // the same chunk by tensor-map loads: lane q fetches the box of row class q (rows q, q + 8, ... of the
  // chunk; `tile_src` is the tile's first element, (i0, j0) the chunk's position in the tile)
  auto push_trans_tma = [&](uint32_t map0, const char* tile_src, uint32_t i0, uint32_t j0, char* dst, uint32_t R,
                            uint32_t n, uint64_t sps, uint64_t dps, uint32_t own, uint32_t first) {
    if (!acquire_slot()) return;
    const uint32_t slot = n_w % kSlots;
    char* stage = wring + (size_t)slot * kSlotBytes;
    // where the rows of a destination window are in the slot: entry (h, k) is the offset of row
    // e0 + k relative to the box row of e0, for a window whose first row e0 has class h.  It depends
    // on the alignment of the rows only, so the chunks of a column of tiles find it in place
    const uint32_t lead0 = (uint32_t)(((uintptr_t)tile_src + (uint64_t)j0 * ES) & 15u), dlead = (uint32_t)sps & 15u;
    const uint32_t key = 0x80u | (lead0 >> 1 << 3) | (dlead >> 1);       // both are even and below 16
    if (((tab_keys >> (8 * slot)) & 0xFFu) != key) {
      tab_keys = (tab_keys & ~(0xFFull << (8 * slot))) | ((uint64_t)key << (8 * slot));
      constexpr uint32_t NV = 16 / ED;
      for (uint32_t e = lane; e < kTmaClasses * NV; e += 32) {
        const uint32_t hk = e / NV + e % NV, cls = hk % kTmaClasses;
        trans_tab[slot][e] = cls * TG::kClassStride + ((lead0 + cls * dlead) & 15u) + (hk / kTmaClasses) * kTmaInner;
      }
      __syncwarp();
    }
    if (lane == 0) {
      ChunkDesc c;
      c.mode = MODE_TRANS_TMA; c.tile = own; c.nr = R; c.nc = n; c.pitch = kTmaInner; c.pad = first;
      c.src = (uint64_t)(uintptr_t)tile_src + (uint64_t)i0 * sps + (uint64_t)j0 * ES;
      c.dst = (uint64_t)(uintptr_t)dst; c.sps = sps; c.dps = dps;
      desc[slot] = c;
      // every box counts in full, whatever part of it lies outside the tile
      mbar_expect_tx(&slot_full[slot], kTmaClasses * TG::kBoxRows * kTmaInner);
    }
    __syncwarp();
    if (lane < kTmaClasses) {
      // the class's map starts at the 16-byte boundary at or before the first element of tile row `lane`
      const uint32_t lead = (uint32_t)(((uintptr_t)tile_src + (uint64_t)lane * sps) & 15u);
      const uint32_t x = ((lead + j0 * ES) >> 4) * (16 / ES);
      tensor_load_2d(stage + lane * TG::kClassStride, tmaps + (size_t)(map0 + lane) * 128, x, i0 / kTmaClasses,
                     &slot_full[slot]);
    }
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
    } else if (staged_trans_ok<ES>(f.kind, f.n_extra, f.nr, f.nc)) {
      // staged transposition: chunks of kTransPiece bytes of columns x kOwn rows (+ halo), rows fastest
      const uint32_t kOwn = f.tmaps ? TG::kOwnTma : TG::kOwn;
      const uint32_t kCols = f.tmaps ? TG::kColsTma : TG::kCols;
      constexpr uint32_t NV = 16 / ED;
      // no halo when every destination run starts on a 16-byte boundary: windows never straddle chunks
      // (nor the seam to the tile below, if this tile's rows are whole windows)
      const uint32_t halo = ((((uintptr_t)f.d | ((size_t)f.dsc * ED)) & 15u) == 0 && kOwn % NV == 0 &&
                             (!f.rows_after || f.nr % NV == 0)) ? 0u : kTransHalo;
      // source rows this tile may read: its own, and - to complete the window that straddles the seam -
      // the first rows of the tile below
      const uint32_t avail = f.nr + (f.rows_after ? NV - 1 : 0u);
      // the rows before a run's first window are written here only at the top of a slab's column
      // equal column shares per chunk (no thin last chunk), a multiple of four columns
      const uint32_t n_col = (f.nc + kCols - 1) / kCols;
      const uint32_t cols = min(kCols, (((f.nc + n_col - 1) / n_col) + 3u) & ~3u);
      if (f.tmaps) {
        // the descriptors of the next tile's maps are on their way while this tile is loaded
        if (k + 1 < bend && lane < kTmaClasses && (nxt.c.z & kTileHasMaps))
          tensor_map_prefetch(tmaps + (size_t)(nxt.c.w + lane) * 128);
        for (uint32_t j0 = 0; j0 < f.nc && !failed; j0 += cols)
          for (uint32_t i0 = 0; i0 < f.nr && !failed; i0 += kOwn)
            push_trans_tma(f.extra, f.s, i0, j0, f.d + ((size_t)j0 * f.dsc + i0) * ED, min(kOwn + halo, avail - i0),
                           min(cols, f.nc - j0), (uint64_t)f.ssr * ES, (uint64_t)f.dsc * ED, min(kOwn, f.nr - i0),
                           (i0 == 0 && !f.rows_before) ? 1u : 0u);
      } else {
        for (uint32_t j0 = 0; j0 < f.nc && !failed; j0 += cols)
          for (uint32_t i0 = 0; i0 < f.nr && !failed; i0 += kOwn)
            push_trans(f.s + ((size_t)i0 * f.ssr + j0) * ES, f.d + ((size_t)j0 * f.dsc + i0) * ED,
                       min(kOwn + halo, avail - i0), min(cols, f.nc - j0), (uint64_t)f.ssr * ES,
                       (uint64_t)f.dsc * ED, min(kOwn, f.nr - i0), (i0 == 0 && !f.rows_before) ? 1u : 0u);
      }
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

}  // namespace
