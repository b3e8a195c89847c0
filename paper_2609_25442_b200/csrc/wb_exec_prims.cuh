// Executor, part 1 of 3: element access and cast helpers, the tile descriptor loader, and the bounded
// mbarrier / bulk-copy (TMA) / asynchronous-copy primitives.  Included by wb_exec.cu only.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

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

// Tiled 2-D tensor-map (TMA) load: the box at element coordinates (x, y) of the tensor that `map`
// describes (a 128-byte CUtensorMap in global memory) lands densely at smem_dst (128-byte aligned)
// and completes on the mbarrier with the box's full byte count.  x * element size must be a
// multiple of 16 bytes.  Coordinates outside the tensor read as zero without touching memory.
__device__ __forceinline__ void tensor_load_2d(void* smem_dst, const void* map, uint32_t x, uint32_t y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tensor_map_prefetch(const void* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
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

}  // namespace
