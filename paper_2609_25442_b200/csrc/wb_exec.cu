// Device side of the weight-remap library: binding a plan to device memory and the
// persistent tile-walking kernel behind wb_remap / wb_pack / wb_unpack (sm_100a).
//
// One launch executes a whole tile table.  Each thread block owns a contiguous range of
// tiles (balanced by bytes at plan time) and walks it; tiles are independent, so there is
// no inter-block communication and nothing a block ever waits on.
//
// Tile kinds
//   ROWS   nr runs of nc contiguous elements on both sides (nr == 1: one long run).
//          16-byte vector loads and stores with the cast done in registers; unaligned
//          heads/tails are peeled per run; rows whose pitches keep every run 16-byte
//          aligned are flattened into one vector index space.
//   TRANS  source contiguous along j, destination contiguous along i: staged through a
//          padded shared-memory block so that both sides stay coalesced.
//   ELEM   anything else (strided vectors, fan-out): one element per thread.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "wb_internal.h"

using namespace wbi;

namespace {

constexpr int kThreads = 256;
constexpr int kMinBlocksPerSM = wbi::kCtasPerSM;

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

template <int ES, int ED> struct Unroll { static constexpr int U = (ES == 4 && ED == 2) ? 4 : 8; };

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

// Rows whose every run starts 16-byte aligned on both sides: one flat vector index space.
template <int ES, int ED>
__device__ __forceinline__ void copy_rows_aligned(const char* __restrict__ s, char* __restrict__ d,
                                                  uint32_t nr, uint32_t nc, uint32_t sp, uint32_t dp,
                                                  uint32_t t, uint32_t nth) {
  using UN = Unit<ES, ED>;
  using E = Elem<ES, ED>;
  constexpr int NV = UN::NV;
  constexpr int U = Unroll<ES, ED>::U;
  const uint32_t vpr = nc / NV;
  const uint32_t total = nr * vpr;
  const size_t sps = (size_t)sp * ES, dps = (size_t)dp * ED;
  for (uint32_t v0 = t; v0 < total; v0 += nth * U) {
    UN r[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t v = v0 + u * nth;
      if (v < total) {
        const uint32_t row = v / vpr, cv = v - row * vpr;
        r[u].load(s + row * sps + (size_t)cv * (NV * ES));
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t v = v0 + u * nth;
      if (v < total) {
        const uint32_t row = v / vpr, cv = v - row * vpr;
        st16(d + row * dps + (size_t)cv * 16, r[u].out());
      }
    }
  }
  const uint32_t rem = nc - vpr * NV;   // ragged row ends
  if (rem) {
    const uint32_t cnt = nr * rem;
    for (uint32_t e = t; e < cnt; e += nth) {
      const uint32_t row = e / rem, c = vpr * NV + (e - row * rem);
      E::store(d + row * dps + (size_t)c * ED, E::load(s + row * sps + (size_t)c * ES));
    }
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

constexpr int kTB = 64;   // transpose block edge

template <int ES, int ED>
__global__ void __launch_bounds__(kThreads, kMinBlocksPerSM)
wb_exec_kernel(const DTile* __restrict__ tiles, const uint32_t* __restrict__ cta_begin,
               const DDst* __restrict__ extras, uint64_t src_add, uint64_t dst_add) {
  using E = Elem<ES, ED>;
  __shared__ typename E::V smem[kTB][kTB + (ED == 2 ? 2 : 1)];
  const uint32_t t = threadIdx.x;
  uint32_t k = cta_begin[blockIdx.x];
  const uint32_t end = cta_begin[blockIdx.x + 1];
  if (k >= end) return;
  TileRegs nxt = load_tile(tiles + k);
  for (; k < end; ++k) {
    const TileRegs cur = nxt;
    if (k + 1 < end) nxt = load_tile(tiles + k + 1);
    const char* s = reinterpret_cast<const char*>(((uint64_t)cur.a.y << 32 | cur.a.x) + src_add);
    char* d = reinterpret_cast<char*>(((uint64_t)cur.a.w << 32 | cur.a.z) + dst_add);
    const uint32_t nr = cur.b.x, nc = cur.b.y, ssr = cur.b.z, ssc = cur.b.w;
    const uint32_t dsr = cur.c.x, dsc = cur.c.y;
    const uint32_t kind = cur.c.z & 0xFF, n_extra = (cur.c.z >> 8) & 0xFF, extra = cur.c.w;

    if (kind == KIND_ROWS && n_extra == 0) {
      if (nr == 1) {
        copy_run<ES, ED>(s, d, nc, t, kThreads);
      } else {
        const bool aligned = (((uintptr_t)d & 15u) == 0) && ((((size_t)dsr * ED) & 15u) == 0) &&
                             (((uintptr_t)s & (Unit<ES, ED>::SRC_ALIGN - 1)) == 0) &&
                             ((((size_t)ssr * ES) & (Unit<ES, ED>::SRC_ALIGN - 1)) == 0);
        if (aligned) {
          copy_rows_aligned<ES, ED>(s, d, nr, nc, ssr, dsr, t, kThreads);
        } else if (nc >= 128) {
          const uint32_t lane = t & 31, warp = t >> 5;
          for (uint32_t row = warp; row < nr; row += kThreads / 32)
            copy_run<ES, ED>(s + (size_t)row * ssr * ES, d + (size_t)row * dsr * ED, nc, lane, 32);
        } else {
          const uint32_t cnt = nr * nc;
          for (uint32_t e = t; e < cnt; e += kThreads) {
            const uint32_t i = e / nc, j = e - i * nc;
            E::store(d + ((size_t)i * dsr + j) * ED, E::load(s + ((size_t)i * ssr + j) * ES));
          }
        }
      }
    } else if (kind == KIND_TRANS && n_extra == 0) {
      // dst[j*dsc + i] = src[i*ssr + j]; 64x64 blocks through shared memory
      for (uint32_t i0 = 0; i0 < nr; i0 += kTB) {
        for (uint32_t j0 = 0; j0 < nc; j0 += kTB) {
          const uint32_t bi = min((uint32_t)kTB, nr - i0), bj = min((uint32_t)kTB, nc - j0);
          // load: threads sweep j fastest (coalesced on the source)
          for (uint32_t e = t; e < bi * kTB; e += kThreads) {
            const uint32_t i = e / kTB, j = e % kTB;
            if (j < bj) smem[i][j] = E::load(s + ((size_t)(i0 + i) * ssr + (j0 + j)) * ES);
          }
          __syncthreads();
          // store: threads sweep i fastest (coalesced on the destination)
          for (uint32_t e = t; e < bj * kTB; e += kThreads) {
            const uint32_t j = e / kTB, i = e % kTB;
            if (i < bi) E::store(d + ((size_t)(j0 + j) * dsc + (i0 + i)) * ED, smem[i][j]);
          }
          __syncthreads();
        }
      }
    } else {
      // element-wise: arbitrary strides, any number of destinations
      const uint32_t cnt = nr * nc;
      for (uint32_t e = t; e < cnt; e += kThreads) {
        const uint32_t i = e / nc, j = e - i * nc;
        const typename E::V v = E::load(s + ((size_t)i * ssr + (size_t)j * ssc) * ES);
        E::store(d + ((size_t)i * dsr + (size_t)j * dsc) * ED, v);
        for (uint32_t x = 0; x < n_extra; ++x) {
          const DDst o = extras[extra + x];
          E::store(reinterpret_cast<char*>(o.dst + dst_add) + ((size_t)i * o.sr + (size_t)j * o.sc) * ED, v);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// launch
// ---------------------------------------------------------------------------------------------
wb_status launch_table(const wb_plan* plan, const TileTable& T, uint64_t src_add, uint64_t dst_add,
                       uint32_t es, uint32_t ed, cudaStream_t stream) {
  if (T.tiles.empty()) return WB_OK;
  const dim3 grid(plan->grid), block(kThreads);
  if (es == 2 && ed == 2)
    wb_exec_kernel<2, 2><<<grid, block, 0, stream>>>(T.d_tiles, T.d_cta_begin, T.d_extras, src_add, dst_add);
  else if (es == 4 && ed == 4)
    wb_exec_kernel<4, 4><<<grid, block, 0, stream>>>(T.d_tiles, T.d_cta_begin, T.d_extras, src_add, dst_add);
  else if (es == 4 && ed == 2)
    wb_exec_kernel<4, 2><<<grid, block, 0, stream>>>(T.d_tiles, T.d_cta_begin, T.d_extras, src_add, dst_add);
  else
    wb_exec_kernel<2, 4><<<grid, block, 0, stream>>>(T.d_tiles, T.d_cta_begin, T.d_extras, src_add, dst_add);
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
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
               up256(T->cta_begin.size() * sizeof(uint32_t));
    bytes = up256(bytes + 256);
    std::vector<char> host(bytes, 0);
    if (!plan->d_arena || plan->arena_bytes != bytes) {
      wbi::release_device_tables(plan);
      if (cudaMalloc(&plan->d_arena, bytes) != cudaSuccess) { plan->d_arena = nullptr; return WB_ERR_OOM; }
      plan->arena_bytes = bytes;
    }
    if (cudaGetDevice(&plan->device) != cudaSuccess) return WB_ERR_CUDA;
    char* dbase = static_cast<char*>(plan->d_arena);
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
    }
    if (cudaMemcpy(plan->d_arena, host.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess)
      return WB_ERR_CUDA;
  } catch (const std::bad_alloc&) {
    return WB_ERR_OOM;
  }
  plan->bound = true;
  return WB_OK;
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

extern "C" wb_status wb_remap_host(const wb_plan* plan, const void* const* host_src, size_t n_src,
                                   void* const* host_dst, size_t n_dst, void* cuda_stream) {
  if (!plan || !host_src || !host_dst) return WB_ERR_INVALID_ARG;
  if (!plan->bound) return WB_ERR_NOT_BOUND;
  if (n_src != plan->src.tensors.size() || n_dst != plan->dst.tensors.size()) return WB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype);
  for (size_t i = 0; i < n_src; ++i) {
    if (!host_src[i]) return WB_ERR_INVALID_ARG;
    if (cudaMemcpyAsync(const_cast<void*>(plan->src_base[i]), host_src[i], plan->src.tensors[i].numel * es,
                        cudaMemcpyHostToDevice, stream) != cudaSuccess) return WB_ERR_CUDA;
  }
  wb_status st = wb_remap(plan, cuda_stream);
  if (st != WB_OK) return st;
  for (size_t i = 0; i < n_dst; ++i) {
    if (!host_dst[i]) return WB_ERR_INVALID_ARG;
    if (cudaMemcpyAsync(host_dst[i], plan->dst_base[i], plan->dst.tensors[i].numel * ed,
                        cudaMemcpyDeviceToHost, stream) != cudaSuccess) return WB_ERR_CUDA;
  }
  return WB_OK;
}
