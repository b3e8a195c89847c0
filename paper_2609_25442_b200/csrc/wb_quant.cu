// FP8 quantisation of transfer buckets (Section 5 of the paper, "Parameter precision mismatch":
// trainer tensors are quantised before the transfer, which needs the full tensor gathered first).
// The paper fixes no rule; the one built here: FP8 E4M3, one scale per checkpoint tensor,
// s = amax / 448 and r = 448 / amax with amax the tensor's largest magnitude in the destination dtype
// (the gather becomes a maximum over every trainer shard of the tensor), q = e4m3(x * r) with round
// to nearest even and saturation, x' = cast(value(q) * s).  The rule is total: a quotient amax / 448
// that rounds to zero becomes the smallest subnormal, and a tensor whose r is not finite (amax below
// 448 / FLT_MAX, or NaN) is encoded as q = e4m3(x / s) instead, so zeros stay zeros whatever the
// tensor's magnitude.
//
//   wb_absmax            one pass over the de-duplicated trainer regions -> amax per checkpoint tensor
//   wb_bucket_quantize   a packed round's bucket (destination dtype) -> FP8 bucket, same element offsets
//   wb_bucket_dequantize the inverse on the rollout side, before wb_unpack
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "wb_internal.h"

using namespace wbi;

namespace {

// A 2-D region of one trainer tensor: n0 runs of n1 contiguous elements, run i at a + i * s0 elements.
struct alignas(16) AmaxItem {
  uint64_t a;
  uint32_t n0, n1;
  uint64_t s0;
  uint32_t ckpt, pad;
};
// A contiguous piece of a bucket: n elements from element offset `off`, scaled with amax[ckpt].
struct alignas(16) QuantItem {
  uint64_t off;
  uint32_t n, ckpt;
};

constexpr uint32_t kItemElems = 1u << 18;   // work items are cut to about this many elements

inline uint32_t esize(uint32_t dt) { return dt == WB_F32 ? 4u : 2u; }

__device__ __forceinline__ uint32_t f32_to_bf16_bits(uint32_t x) {
  uint16_t r;
  asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(__uint_as_float(x)));
  return r;
}
// two fp32 -> two E4M3 codes (lo in the low byte), round to nearest even, saturating
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
// two E4M3 codes -> two fp32 (exact, through fp16)
__device__ __forceinline__ float2 e4m3x2_to_f32x2(uint32_t two) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)two));
  float lo, hi;
  asm("{ .reg .b16 l, h; mov.b32 {l, h}, %2; cvt.f32.f16 %0, l; cvt.f32.f16 %1, h; }" : "=f"(lo), "=f"(hi) : "r"(h2));
  return make_float2(lo, hi);
}
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float scale_of(const float* __restrict__ amax, uint32_t ckpt) {
  const float a = __ldg(amax + ckpt);
  if (a == 0.f) return 1.f;
  const float s = __fdiv_rn(a, 448.f);
  return s == 0.f ? __uint_as_float(1u) : s;      // never zero for a tensor that is not: 2^-149
}
__device__ __forceinline__ float rscale_of(const float* __restrict__ amax, uint32_t ckpt) {
  const float a = __ldg(amax + ckpt);
  return a == 0.f ? 1.f : __fdiv_rn(448.f, a);
}

// Sign-cleared fp32 pattern of one source element / of the elements packed in a 32-bit word.
template <int ES> __device__ __forceinline__ uint32_t abs_elem(const char* p) {
  if (ES == 4) return *reinterpret_cast<const uint32_t*>(p) & 0x7FFFFFFFu;
  return ((uint32_t)*reinterpret_cast<const uint16_t*>(p) << 16) & 0x7FFFFFFFu;
}
template <int ES> __device__ __forceinline__ uint32_t abs_word(uint32_t w) {
  if (ES == 4) return w & 0x7FFFFFFFu;
  return max((w << 16) & 0x7FFFFFFFu, w & 0x7FFF0000u);
}

// One work item (tile) at a time for the whole block, drawn from a counter in device memory.
__device__ __forceinline__ uint32_t next_tile(uint32_t* counter, uint32_t* slot) {
  __syncthreads();                                   // everyone is done with the previous value
  if (threadIdx.x == 0) *slot = atomicAdd(counter, 1u);
  __syncthreads();
  return *slot;
}

// amax: magnitudes are compared as unsigned integers of the sign-cleared fp32 patterns (a NaN wins).
// A warp takes a run; the part between 16-byte boundaries is read with 16-byte loads, four in
// flight per lane, the ends element by element.  Items whose runs are short (a column piece of a
// wider matrix) are read as one flat sequence of n0 * n1 elements instead, a lane taking every 32nd
// element (coalesced inside each run; run and column advance incrementally) with eight loads in
// flight: one run per warp and round trip would leave the memory idle.  Eight blocks per SM.
template <int ES, int ED>
__global__ void __launch_bounds__(256, 8)
wb_absmax_kernel(const AmaxItem* __restrict__ items, uint32_t n_items, uint32_t* __restrict__ amax,
                 uint32_t* __restrict__ counter) {
  __shared__ uint32_t warp_max[8];
  __shared__ uint32_t slot;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr uint32_t PER = 16 / ES;
  for (uint32_t k = next_tile(counter, &slot); k < n_items; k = next_tile(counter, &slot)) {
    const AmaxItem it = items[k];
    uint32_t m = 0;
    constexpr uint32_t kShortRunBytes = 1024;
    const bool short_runs = it.n0 > 1 && it.n1 * ES < kShortRunBytes;
    if (short_runs) {
      constexpr int U = 8;
      const uint32_t n1 = it.n1, total = it.n0 * n1;       // an item has about kItemElems elements
      const uint32_t q32 = 32 / n1, r32 = 32 % n1;
      for (uint32_t e0 = warp * (32 * U); e0 < total; e0 += 8 * 32 * U) {
        uint32_t i = (e0 + lane) / n1, j = (e0 + lane) - i * n1;
        uint32_t x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          x[u] = 0;
          if (e0 + lane + 32u * u < total)
            x[u] = abs_elem<ES>(reinterpret_cast<const char*>(it.a) + ((size_t)i * it.s0 + j) * ES);
          i += q32; j += r32;
          if (j >= n1) { j -= n1; ++i; }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) m = max(m, x[u]);
      }
    }
    // the warps share the item's runs in segments of kSeg elements (a flat shard is one long run)
    constexpr uint32_t kSeg = 8192;
    const uint32_t segs = (it.n1 + kSeg - 1) / kSeg;
    for (uint32_t t = warp; t < it.n0 * segs && !short_runs; t += 8) {
      const uint32_t i = t / segs, sg = t - i * segs;
      const char* row = reinterpret_cast<const char*>(it.a) + ((size_t)i * it.s0 + (size_t)sg * kSeg) * ES;
      const uint32_t n1 = min(kSeg, it.n1 - sg * kSeg);
      const uint32_t head = min(n1, (uint32_t)(((16u - ((uintptr_t)row & 15u)) & 15u) / ES));
      if (lane < head) m = max(m, abs_elem<ES>(row + lane * ES));
      const uint4* body = reinterpret_cast<const uint4*>(row + head * ES);
      const uint32_t nv = (n1 - head) / PER;
      for (uint32_t v0 = 0; v0 < nv; v0 += 32 * 4) {
        uint4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t v = v0 + lane + 32u * u;
          x[u] = v < nv ? __ldcs(body + v) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
          m = max(max(m, abs_word<ES>(x[u].x)), max(max(abs_word<ES>(x[u].y), abs_word<ES>(x[u].z)), abs_word<ES>(x[u].w)));
      }
      const uint32_t done = head + nv * PER;
      if (done + lane < n1) m = max(m, abs_elem<ES>(row + (size_t)(done + lane) * ES));
    }
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if (lane == 0) warp_max[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < 8; ++w) m = max(m, warp_max[w]);
      // the maximum of the destination-dtype values: rounding is monotonic, so round the maximum
      if (ES == 4 && ED == 2) m = f32_to_bf16_bits(m) << 16;
      if (m) atomicMax(amax + it.ckpt, m);
    }
  }
}

// bucket (ED-byte elements) -> FP8 codes at the same element offsets; eight elements per thread step
template <int ED>
__global__ void __launch_bounds__(256)
wb_quantize_kernel(const QuantItem* __restrict__ items, uint32_t n_items, const char* __restrict__ bucket,
                   uint8_t* __restrict__ q, const float* __restrict__ amax) {
  for (uint32_t k = blockIdx.x; k < n_items; k += gridDim.x) {
    const QuantItem it = items[k];
    const float r = rscale_of(amax, it.ckpt);
    const char* x = bucket + it.off * ED;
    uint8_t* out = q + it.off;
    const uint32_t body = it.n & ~7u;
    if (!isfinite(r)) {
      // tiny magnitudes (448 / amax overflows) or a NaN maximum: divide by the scale, element by element
      const float s = scale_of(amax, it.ckpt);
      for (uint32_t e = threadIdx.x; e < it.n; e += blockDim.x) {
        float f;
        if (ED == 2) f = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(x)[e] << 16);
        else f = reinterpret_cast<const float*>(x)[e];
        out[e] = (uint8_t)(f32x2_to_e4m3x2(__fdiv_rn(f, s), 0.f) & 0xFFu);
      }
      continue;
    }
#pragma unroll 2
    for (uint32_t e = threadIdx.x * 8; e < body; e += blockDim.x * 8) {
      float f[8];
      if (ED == 2) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(x + (size_t)e * 2));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          f[2 * p] = __uint_as_float(w[p] << 16);
          f[2 * p + 1] = __uint_as_float(w[p] & 0xFFFF0000u);
        }
      } else {
        const float4 a = __ldcs(reinterpret_cast<const float4*>(x + (size_t)e * 4));
        const float4 b = __ldcs(reinterpret_cast<const float4*>(x + (size_t)e * 4) + 1);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
      }
      uint32_t c[4];
#pragma unroll
      for (int p = 0; p < 4; ++p) c[p] = f32x2_to_e4m3x2(__fmul_rn(f[2 * p], r), __fmul_rn(f[2 * p + 1], r));
      // two-byte buckets start payloads on multiples of 8 elements, four-byte buckets on multiples of 4
      if (ED == 2) {
        __stcs(reinterpret_cast<uint2*>(out + e), make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16)));
      } else {
        __stcs(reinterpret_cast<uint32_t*>(out + e), c[0] | (c[1] << 16));
        __stcs(reinterpret_cast<uint32_t*>(out + e) + 1, c[2] | (c[3] << 16));
      }
    }
    for (uint32_t e = body + threadIdx.x; e < it.n; e += blockDim.x) {
      float f;
      if (ED == 2) f = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(x)[e] << 16);
      else f = reinterpret_cast<const float*>(x)[e];
      out[e] = (uint8_t)(f32x2_to_e4m3x2(__fmul_rn(f, r), 0.f) & 0xFFu);
    }
  }
}

// FP8 codes -> bucket (ED-byte elements): value(q) * s, rounded to the destination dtype
template <int ED>
__global__ void __launch_bounds__(256)
wb_dequantize_kernel(const QuantItem* __restrict__ items, uint32_t n_items, const uint8_t* __restrict__ q,
                     char* __restrict__ bucket, const float* __restrict__ amax) {
  for (uint32_t k = blockIdx.x; k < n_items; k += gridDim.x) {
    const QuantItem it = items[k];
    const float s = scale_of(amax, it.ckpt);
    const uint8_t* in = q + it.off;
    char* x = bucket + it.off * ED;
    const uint32_t body = it.n & ~7u;
    for (uint32_t e = threadIdx.x * 8; e < body; e += blockDim.x * 8) {
      uint2 c;
      if (ED == 2) {
        c = __ldcs(reinterpret_cast<const uint2*>(in + e));
      } else {
        c.x = __ldcs(reinterpret_cast<const uint32_t*>(in + e));
        c.y = __ldcs(reinterpret_cast<const uint32_t*>(in + e) + 1);
      }
      float f[8];
      const uint32_t two[4] = {c.x & 0xFFFFu, c.x >> 16, c.y & 0xFFFFu, c.y >> 16};
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        const float2 v = e4m3x2_to_f32x2(two[p]);
        f[2 * p] = __fmul_rn(v.x, s);
        f[2 * p + 1] = __fmul_rn(v.y, s);
      }
      if (ED == 2) {
        __stcs(reinterpret_cast<uint4*>(x + (size_t)e * 2),
               make_uint4(f32x2_to_bf16x2(f[0], f[1]), f32x2_to_bf16x2(f[2], f[3]), f32x2_to_bf16x2(f[4], f[5]),
                          f32x2_to_bf16x2(f[6], f[7])));
      } else {
        __stcs(reinterpret_cast<float4*>(x + (size_t)e * 4), make_float4(f[0], f[1], f[2], f[3]));
        __stcs(reinterpret_cast<float4*>(x + (size_t)e * 4) + 1, make_float4(f[4], f[5], f[6], f[7]));
      }
    }
    for (uint32_t e = body + threadIdx.x; e < it.n; e += blockDim.x) {
      const float f = __fmul_rn(e4m3x2_to_f32x2(in[e]).x, s);
      if (ED == 2) reinterpret_cast<uint16_t*>(x)[e] = (uint16_t)(f32x2_to_bf16x2(f, 0.f) & 0xFFFFu);
      else reinterpret_cast<float*>(x)[e] = f;
    }
  }
}


// ---------------------------------------------------------------------------------------------------
// Fused forms: wb_pack_fp8 writes E4M3 codes straight into the FP8 bucket while it packs, wb_unpack_fp8
// reads codes and writes the rollout tensors in their dtype.  Same arithmetic as the separate kernels
// (cast to the destination dtype, multiply by r or divide by s, encode; decode, multiply by s, cast), so
// the results are bit-identical; the 2- or 4-byte bucket and the two extra passes over it disappear.
// They walk the round's ordinary tile tables.  A thread block draws one tile at a time from a counter
// and its 256 threads share the tile.
// ---------------------------------------------------------------------------------------------------
struct TileQ {
  const char* s;
  char* d;
  uint32_t nr, nc, ssr, ssc, dsr, dsc, kind, n_extra, extra;
};
__device__ __forceinline__ TileQ load_tile_q(const DTile* __restrict__ p) {
  const DTile t = *p;
  TileQ f;
  f.s = reinterpret_cast<const char*>(t.src);
  f.d = reinterpret_cast<char*>(t.dst);
  f.nr = t.nr; f.nc = t.nc; f.ssr = t.ssr; f.ssc = t.ssc; f.dsr = t.dsr; f.dsc = t.dsc;
  f.kind = t.kind_extra & 0xFF; f.n_extra = (t.kind_extra >> 8) & 0xFF; f.extra = t.extra;
  return f;
}
// The value the bucket would hold (destination dtype), as fp32, from the raw source element.
template <int ES, int EDP> __device__ __forceinline__ float bucket_value(uint32_t raw) {
  if (ES == 2) return __uint_as_float(raw << 16);                              // bf16 widens exactly
  if (EDP == 2) return __uint_as_float(f32_to_bf16_bits(raw) << 16);           // fp32 rounded to bf16
  return __uint_as_float(raw);
}
struct Scale { float r, s; bool by_division; };
__device__ __forceinline__ Scale scale_for(const float* __restrict__ amax, uint32_t ckpt) {
  Scale sc;
  sc.r = rscale_of(amax, ckpt);
  sc.s = scale_of(amax, ckpt);
  sc.by_division = !isfinite(sc.r);
  return sc;
}
__device__ __forceinline__ float scaled(float f, const Scale& sc) {
  return sc.by_division ? __fdiv_rn(f, sc.s) : __fmul_rn(f, sc.r);
}
template <int ES, int EDP> __device__ __forceinline__ uint8_t quant_elem(const char* p, const Scale& sc) {
  const uint32_t raw = ES == 4 ? *reinterpret_cast<const uint32_t*>(p) : (uint32_t)*reinterpret_cast<const uint16_t*>(p);
  return (uint8_t)(f32x2_to_e4m3x2(scaled(bucket_value<ES, EDP>(raw), sc), 0.f) & 0xFFu);
}
template <int EDP> __device__ __forceinline__ void dequant_store(char* d, uint32_t code, float s) {
  const float f = __fmul_rn(e4m3x2_to_f32x2(code).x, s);
  if (EDP == 2) *reinterpret_cast<uint16_t*>(d) = (uint16_t)(f32x2_to_bf16x2(f, 0.f) & 0xFFFFu);
  else *reinterpret_cast<float*>(d) = f;
}

template <int ES, int EDP>
__global__ void __launch_bounds__(256)
wb_pack_fp8_kernel(const DTile* __restrict__ tiles, const uint32_t* __restrict__ tile_ckpt, uint32_t n_tiles,
                   uint8_t* __restrict__ q, const float* __restrict__ amax, uint32_t* __restrict__ counter) {
  __shared__ uint32_t slot;
  for (uint32_t k = next_tile(counter, &slot); k < n_tiles; k = next_tile(counter, &slot)) {
    const TileQ f = load_tile_q(tiles + k);
    const Scale sc = scale_for(amax, __ldg(tile_ckpt + k));
    uint8_t* const out = q + (uintptr_t)f.d / EDP;           // the table holds byte offsets of the EDP-byte bucket
    if (f.kind == KIND_ROWS && f.nc >= 16384 && !sc.by_division) {
      // long rows: the 8-element groups between the first and the last 8-byte boundary of the code row are
      // taken four at a time per thread (four independent 16-byte loads in flight); the ends one by one
      for (uint32_t i = 0; i < f.nr; ++i) {
        uint8_t* drow = out + (size_t)i * f.dsr;
        const char* srow = f.s + (size_t)i * f.ssr * ES;
        const uint32_t head = (uint32_t)((8u - ((uintptr_t)drow & 7u)) & 7u);
        const uint32_t ngrp = (f.nc - head) >> 3;
        const uint32_t done = head + ngrp * 8;
        if (threadIdx.x < head) drow[threadIdx.x] = quant_elem<ES, EDP>(srow + (size_t)threadIdx.x * ES, sc);
        if (threadIdx.x >= 32 && threadIdx.x - 32 < f.nc - done)
          drow[done + threadIdx.x - 32] = quant_elem<ES, EDP>(srow + (size_t)(done + threadIdx.x - 32) * ES, sc);
        const char* sb = srow + (size_t)head * ES;
        uint8_t* db = drow + head;
        if (((uintptr_t)sb & 15u) == 0) {
          constexpr int U = 4;
          for (uint32_t g0 = threadIdx.x; g0 < ngrp; g0 += blockDim.x * U) {
            uint4 x[U], y[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const uint32_t g = g0 + u * blockDim.x;
              if (g < ngrp) {
                x[u] = __ldcs(reinterpret_cast<const uint4*>(sb + (size_t)g * 8 * ES));
                if (ES == 4) y[u] = __ldcs(reinterpret_cast<const uint4*>(sb + (size_t)g * 8 * ES) + 1);
              }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const uint32_t g = g0 + u * blockDim.x;
              if (g >= ngrp) continue;
              float v[8];
              if (ES == 2) {
                const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                  v[2 * p] = bucket_value<ES, EDP>(w[p] & 0xFFFFu);
                  v[2 * p + 1] = bucket_value<ES, EDP>(w[p] >> 16);
                }
              } else {
                const uint32_t w[8] = {x[u].x, x[u].y, x[u].z, x[u].w, y[u].x, y[u].y, y[u].z, y[u].w};
#pragma unroll
                for (int p = 0; p < 8; ++p) v[p] = bucket_value<ES, EDP>(w[p]);
              }
              uint32_t c[4];
#pragma unroll
              for (int p = 0; p < 4; ++p) c[p] = f32x2_to_e4m3x2(__fmul_rn(v[2 * p], sc.r), __fmul_rn(v[2 * p + 1], sc.r));
              __stcs(reinterpret_cast<uint2*>(db + (size_t)g * 8), make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16)));
            }
          }
        } else {
          for (uint32_t g = threadIdx.x; g < ngrp; g += blockDim.x) {
            uint32_t c[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) {
              const char* e = sb + ((size_t)g * 8 + 2 * p) * ES;
              c[p] = (uint32_t)quant_elem<ES, EDP>(e, sc) | ((uint32_t)quant_elem<ES, EDP>(e + ES, sc) << 8);
            }
            __stcs(reinterpret_cast<uint2*>(db + (size_t)g * 8), make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16)));
          }
        }
      }
    } else if (f.kind == KIND_ROWS) {
      // rows of nc contiguous elements on both sides; each row is cut into 8-byte groups of the code row
      const uint32_t gmax = (f.nc + 14) >> 3;
      const uint32_t total = f.nr * gmax;
      for (uint32_t idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const uint32_t i = f.nr == 1 ? 0u : idx / gmax, g = idx - i * gmax;
        uint8_t* drow = out + (size_t)i * f.dsr;
        const char* srow = f.s + (size_t)i * f.ssr * ES;
        const int a = (int)((uintptr_t)drow & 7u);
        const int e0 = (int)(g * 8) - a;
        if (e0 >= (int)f.nc) continue;
        const char* sp = srow + (ptrdiff_t)e0 * ES;
        if (e0 >= 0 && (uint32_t)e0 + 8 <= f.nc) {
          float v[8];
          if (((uintptr_t)sp & 15u) == 0) {
            if (ES == 2) {
              const uint4 x = __ldcs(reinterpret_cast<const uint4*>(sp));
              const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
              for (int p = 0; p < 4; ++p) {
                v[2 * p] = bucket_value<ES, EDP>(w[p] & 0xFFFFu);
                v[2 * p + 1] = bucket_value<ES, EDP>(w[p] >> 16);
              }
            } else {
              const uint4 x = __ldcs(reinterpret_cast<const uint4*>(sp)), y = __ldcs(reinterpret_cast<const uint4*>(sp) + 1);
              const uint32_t w[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
#pragma unroll
              for (int p = 0; p < 8; ++p) v[p] = bucket_value<ES, EDP>(w[p]);
            }
          } else {
#pragma unroll
            for (int p = 0; p < 8; ++p) {
              const uint32_t raw = ES == 4 ? *reinterpret_cast<const uint32_t*>(sp + p * ES)
                                           : (uint32_t)*reinterpret_cast<const uint16_t*>(sp + p * ES);
              v[p] = bucket_value<ES, EDP>(raw);
            }
          }
          uint32_t c[4];
#pragma unroll
          for (int p = 0; p < 4; ++p) c[p] = f32x2_to_e4m3x2(scaled(v[2 * p], sc), scaled(v[2 * p + 1], sc));
          __stcs(reinterpret_cast<uint2*>(drow + e0), make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16)));
        } else {
          const int lo = e0 < 0 ? 0 : e0, hi = min((int)f.nc, e0 + 8);
          for (int e = lo; e < hi; ++e) drow[e] = quant_elem<ES, EDP>(srow + (size_t)e * ES, sc);
        }
      }
    } else {
      // transposed or strided sources: element by element (trainer layouts rarely have them)
      const uint64_t cnt = (uint64_t)f.nr * f.nc;
      for (uint64_t e = threadIdx.x; e < cnt; e += blockDim.x) {
        const uint32_t i = (uint32_t)(e / f.nc), j = (uint32_t)(e - (uint64_t)i * f.nc);
        out[(size_t)i * f.dsr + (size_t)j * f.dsc] = quant_elem<ES, EDP>(f.s + ((size_t)i * f.ssr + (size_t)j * f.ssc) * ES, sc);
      }
    }
  }
}

template <int EDP>
__global__ void __launch_bounds__(256)
wb_unpack_fp8_kernel(const DTile* __restrict__ tiles, const uint32_t* __restrict__ tile_ckpt, const DDst* __restrict__ extras,
                     uint32_t n_tiles, const uint8_t* __restrict__ q, const float* __restrict__ amax,
                     uint32_t* __restrict__ counter) {
  constexpr uint32_t NV = 16 / EDP;                           // destination elements per 16-byte store
  constexpr uint32_t kTB = 64;                                // transposition block: kTB x kTB elements
  __shared__ uint32_t slot;
  __shared__ __align__(16) char tbuf[kTB * (kTB * EDP + 16)];
  for (uint32_t k = next_tile(counter, &slot); k < n_tiles; k = next_tile(counter, &slot)) {
    const TileQ f = load_tile_q(tiles + k);
    const float s = scale_of(amax, __ldg(tile_ckpt + k));
    const uint8_t* const in = q + (uintptr_t)f.s / EDP;
    if (f.n_extra == 0 && f.kind == KIND_ROWS && f.nc >= 16384) {
      // long rows: the NV-element groups between the first and the last 16-byte boundary of the destination row,
      // four per thread at a time; the ends one by one
      for (uint32_t i = 0; i < f.nr; ++i) {
        char* drow = f.d + (size_t)i * f.dsr * EDP;
        const uint8_t* srow = in + (size_t)i * f.ssr;
        const uint32_t head = (uint32_t)(((16u - ((uintptr_t)drow & 15u)) & 15u) / EDP);
        const uint32_t ngrp = (f.nc - head) / NV;
        const uint32_t done = head + ngrp * NV;
        if (threadIdx.x < head) dequant_store<EDP>(drow + (size_t)threadIdx.x * EDP, srow[threadIdx.x], s);
        if (threadIdx.x >= 32 && threadIdx.x - 32 < f.nc - done)
          dequant_store<EDP>(drow + (size_t)(done + threadIdx.x - 32) * EDP, srow[done + threadIdx.x - 32], s);
        const uint8_t* sb = srow + head;
        char* db = drow + (size_t)head * EDP;
        const bool vec = ((uintptr_t)sb & (NV - 1)) == 0;
        constexpr int U = 4;
        for (uint32_t g0 = threadIdx.x; g0 < ngrp; g0 += blockDim.x * U) {
          uint32_t lo[U], hi[U];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const uint32_t g = g0 + u * blockDim.x;
            lo[u] = hi[u] = 0;
            if (g < ngrp) {
              const uint8_t* sp = sb + (size_t)g * NV;
              if (vec) {
                if (NV == 8) { const uint2 c = __ldcs(reinterpret_cast<const uint2*>(sp)); lo[u] = c.x; hi[u] = c.y; }
                else lo[u] = __ldcs(reinterpret_cast<const uint32_t*>(sp));
              } else {
                lo[u] = sp[0] | (sp[1] << 8) | (sp[2] << 16) | ((uint32_t)sp[3] << 24);
                if (NV == 8) hi[u] = sp[4] | (sp[5] << 8) | (sp[6] << 16) | ((uint32_t)sp[7] << 24);
              }
            }
          }
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const uint32_t g = g0 + u * blockDim.x;
            if (g >= ngrp) continue;
            const float2 v0 = e4m3x2_to_f32x2(lo[u] & 0xFFFFu), v1 = e4m3x2_to_f32x2(lo[u] >> 16);
            if (NV == 8) {
              const float2 v2 = e4m3x2_to_f32x2(hi[u] & 0xFFFFu), v3 = e4m3x2_to_f32x2(hi[u] >> 16);
              __stcs(reinterpret_cast<uint4*>(db + (size_t)g * 16),
                     make_uint4(f32x2_to_bf16x2(__fmul_rn(v0.x, s), __fmul_rn(v0.y, s)), f32x2_to_bf16x2(__fmul_rn(v1.x, s), __fmul_rn(v1.y, s)),
                                f32x2_to_bf16x2(__fmul_rn(v2.x, s), __fmul_rn(v2.y, s)), f32x2_to_bf16x2(__fmul_rn(v3.x, s), __fmul_rn(v3.y, s))));
            } else {
              __stcs(reinterpret_cast<float4*>(db + (size_t)g * 16),
                     make_float4(__fmul_rn(v0.x, s), __fmul_rn(v0.y, s), __fmul_rn(v1.x, s), __fmul_rn(v1.y, s)));
            }
          }
        }
      }
    } else if (f.n_extra == 0 && f.kind == KIND_ROWS) {
      const uint32_t gmax = (f.nc + 2 * NV - 2) / NV;
      const uint32_t total = f.nr * gmax;
      for (uint32_t idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const uint32_t i = f.nr == 1 ? 0u : idx / gmax, g = idx - i * gmax;
        char* drow = f.d + (size_t)i * f.dsr * EDP;
        const uint8_t* srow = in + (size_t)i * f.ssr;
        const int a = (int)(((uintptr_t)drow & 15u) / EDP);
        const int e0 = (int)(g * NV) - a;
        if (e0 >= (int)f.nc) continue;
        if (e0 >= 0 && (uint32_t)e0 + NV <= f.nc) {
          const uint8_t* sp = srow + e0;
          uint32_t lo, hi = 0;
          if (((uintptr_t)sp & (NV - 1)) == 0) {
            if (NV == 8) { const uint2 c = __ldcs(reinterpret_cast<const uint2*>(sp)); lo = c.x; hi = c.y; }
            else lo = __ldcs(reinterpret_cast<const uint32_t*>(sp));
          } else {
            lo = sp[0] | (sp[1] << 8) | (sp[2] << 16) | ((uint32_t)sp[3] << 24);
            if (NV == 8) hi = sp[4] | (sp[5] << 8) | (sp[6] << 16) | ((uint32_t)sp[7] << 24);
          }
          const float2 v0 = e4m3x2_to_f32x2(lo & 0xFFFFu), v1 = e4m3x2_to_f32x2(lo >> 16);
          if (NV == 8) {
            const float2 v2 = e4m3x2_to_f32x2(hi & 0xFFFFu), v3 = e4m3x2_to_f32x2(hi >> 16);
            __stcs(reinterpret_cast<uint4*>(drow + (size_t)e0 * EDP),
                   make_uint4(f32x2_to_bf16x2(__fmul_rn(v0.x, s), __fmul_rn(v0.y, s)), f32x2_to_bf16x2(__fmul_rn(v1.x, s), __fmul_rn(v1.y, s)),
                              f32x2_to_bf16x2(__fmul_rn(v2.x, s), __fmul_rn(v2.y, s)), f32x2_to_bf16x2(__fmul_rn(v3.x, s), __fmul_rn(v3.y, s))));
          } else {
            __stcs(reinterpret_cast<float4*>(drow + (size_t)e0 * EDP),
                   make_float4(__fmul_rn(v0.x, s), __fmul_rn(v0.y, s), __fmul_rn(v1.x, s), __fmul_rn(v1.y, s)));
          }
        } else {
          const int lo = e0 < 0 ? 0 : e0, hi = min((int)f.nc, e0 + (int)NV);
          for (int e = lo; e < hi; ++e) dequant_store<EDP>(drow + (size_t)e * EDP, srow[e], s);
        }
      }
    } else if (f.n_extra == 0 && f.kind == KIND_TRANS) {
      // dst[j * dsc + i] = value(src[i * ssr + j]): blocks of kTB x kTB codes go through shared memory, where
      // block row i is written as column i of a [kTB][kTB] array of destination elements, and leave as
      // 16-byte pieces of the destination runs (element stores where a run is not 16-byte aligned)
      constexpr uint32_t kPitch = kTB * EDP + 16;
      const uint32_t bi = (f.nr + kTB - 1) / kTB, bj = (f.nc + kTB - 1) / kTB;
      for (uint32_t b = 0; b < bi * bj; ++b) {
        const uint32_t i0 = (b % bi) * kTB, j0 = (b / bi) * kTB;                // rows fastest: runs continue
        const uint32_t ni = min(kTB, f.nr - i0), nj = min(kTB, f.nc - j0);
        __syncthreads();
        // a thread takes 16 neighbouring codes of one block row (one or four loads), decodes them and writes them
        // down a column of the shared array
        for (uint32_t e = threadIdx.x; e < ni * 4; e += blockDim.x) {
          const uint32_t i = e >> 2, c0 = (e & 3u) * 16u;
          if (c0 >= nj) continue;
          const uint8_t* sp = in + (size_t)(i0 + i) * f.ssr + j0 + c0;
          const uint32_t nn = min(16u, nj - c0);
          uint32_t w[4] = {0, 0, 0, 0};
          if (nn == 16 && ((uintptr_t)sp & 3u) == 0) {
#pragma unroll
            for (int p = 0; p < 4; ++p) w[p] = __ldcs(reinterpret_cast<const uint32_t*>(sp) + p);
          } else {
            for (uint32_t p = 0; p < nn; ++p) w[p >> 2] |= (uint32_t)sp[p] << (8 * (p & 3));
          }
#pragma unroll
          for (int p = 0; p < 8; ++p) {
            const float2 v = e4m3x2_to_f32x2((w[p >> 1] >> (16 * (p & 1))) & 0xFFFFu);
            char* at = tbuf + (c0 + 2 * p) * kPitch + i * EDP;
            if (2u * p < nn) {
              if (EDP == 2) *reinterpret_cast<uint16_t*>(at) = (uint16_t)(f32x2_to_bf16x2(__fmul_rn(v.x, s), 0.f) & 0xFFFFu);
              else *reinterpret_cast<float*>(at) = __fmul_rn(v.x, s);
            }
            if (2u * p + 1 < nn) {
              if (EDP == 2) *reinterpret_cast<uint16_t*>(at + kPitch) = (uint16_t)(f32x2_to_bf16x2(__fmul_rn(v.y, s), 0.f) & 0xFFFFu);
              else *reinterpret_cast<float*>(at + kPitch) = __fmul_rn(v.y, s);
            }
          }
        }
        __syncthreads();
        // run j of the block: ni consecutive destination elements from f.d + ((j0 + j) * dsc + i0) * EDP, written in
        // 16-byte aligned windows of the destination (a window that the block covers fully is one vector store,
        // assembled from the shared array at whatever offset the run's alignment gives)
        const uint32_t wins = (ni + 2 * NV - 2) / NV;
        for (uint32_t idx = threadIdx.x; idx < nj * wins; idx += blockDim.x) {
          const uint32_t j = idx / wins, w = idx - j * wins;
          char* run = f.d + ((size_t)(j0 + j) * f.dsc + i0) * EDP;
          const int a = (int)(((uintptr_t)run & 15u) / EDP);
          const int e0 = (int)(w * NV) - a;
          if (e0 >= (int)ni) continue;
          const char* sm = tbuf + j * kPitch;
          if (e0 >= 0 && (uint32_t)e0 + NV <= ni) {
            uint4 x;
            if (EDP == 2) {
              const uint16_t* h = reinterpret_cast<const uint16_t*>(sm) + e0;
              x = make_uint4(h[0] | ((uint32_t)h[1] << 16), h[2] | ((uint32_t)h[3] << 16), h[4] | ((uint32_t)h[5] << 16),
                             h[6] | ((uint32_t)h[7] << 16));
            } else {
              const uint32_t* h = reinterpret_cast<const uint32_t*>(sm) + e0;
              x = make_uint4(h[0], h[1], h[2], h[3]);
            }
            *reinterpret_cast<uint4*>(run + (size_t)e0 * EDP) = x;
          } else {
            const int lo = e0 < 0 ? 0 : e0, hi = min((int)ni, e0 + (int)NV);
            for (int e = lo; e < hi; ++e) {
              if (EDP == 2) *reinterpret_cast<uint16_t*>(run + (size_t)e * 2) = *reinterpret_cast<const uint16_t*>(sm + (size_t)e * 2);
              else *reinterpret_cast<uint32_t*>(run + (size_t)e * 4) = *reinterpret_cast<const uint32_t*>(sm + (size_t)e * 4);
            }
          }
        }
      }
    } else {
      // strided vectors and fan-out to several rollout tensors: element by element
      const uint64_t cnt = (uint64_t)f.nr * f.nc;
      for (uint64_t e = threadIdx.x; e < cnt; e += blockDim.x) {
        const uint32_t i = (uint32_t)(e / f.nc), j = (uint32_t)(e - (uint64_t)i * f.nc);
        const uint32_t code = in[(size_t)i * f.ssr + (size_t)j * f.ssc];
        dequant_store<EDP>(f.d + ((size_t)i * f.dsr + (size_t)j * f.dsc) * EDP, code, s);
        for (uint32_t x = 0; x < f.n_extra; ++x) {
          const DDst o = extras[f.extra + x];
          dequant_store<EDP>(reinterpret_cast<char*>(o.dst) + ((size_t)i * o.sr + (size_t)j * o.sc) * EDP, code, s);
        }
      }
    }
  }
}

// Work lists, built on first use and kept with the plan's device tables.
struct QuantTables {
  void* d_mem = nullptr;
  AmaxItem* d_amax = nullptr;
  uint32_t n_amax = 0;
  std::vector<QuantItem*> d_round;
  std::vector<uint32_t> n_round;
  // fused quantising pack / dequantising unpack: checkpoint index of every tile, one tile counter per launch
  std::vector<uint32_t*> d_pack_ckpt, d_unpack_ckpt;
  uint32_t* d_counters = nullptr;         // 2 per round: [2r] pack, [2r + 1] unpack; then one for the amax pass
};

wb_status build_tables(wb_plan* plan) {
  if (plan->quant_tables) return WB_OK;
  const uint32_t es = esize(plan->src.dtype);
  std::vector<AmaxItem> amax;
  for (const Slab& sl : plan->slabs) {
    const NSlice& s = plan->src.slices[sl.src_slice];
    const uint64_t base = (uint64_t)(uintptr_t)plan->src_base[s.tensor] + s.elem(sl.rect.r0, sl.rect.c0) * es;
    // runs along the contiguous direction of the slice (columns, or rows when it is transposed)
    const uint64_t n0 = s.transposed ? sl.rect.nc : sl.rect.nr, n1 = s.transposed ? sl.rect.nr : sl.rect.nc;
    const uint64_t per = n1 >= kItemElems ? 1 : kItemElems / n1;      // runs per item
    for (uint64_t i = 0; i < n0; i += per)
      for (uint64_t j = 0; j < n1; j += 1u << 30) {                    // run lengths fit 32 bits
        AmaxItem it{};
        it.a = base + (i * s.pitch + j) * es;
        it.n0 = (uint32_t)std::min<uint64_t>(per, n0 - i);
        it.n1 = (uint32_t)std::min<uint64_t>(1u << 30, n1 - j);
        it.s0 = s.pitch;
        it.ckpt = sl.ckpt_index;
        amax.push_back(it);
      }
  }
  std::vector<std::vector<QuantItem>> rounds(plan->rounds.size());
  const uint32_t ed = esize(plan->dst.dtype);
  for (size_t r = 0; r < plan->rounds.size(); ++r)
    for (const Payload& p : plan->rounds[r].payloads) {
      const uint64_t n = p.rect.nr * p.rect.nc, off = p.bucket_off / ed;
      for (uint64_t e = 0; e < n; e += kItemElems)
        rounds[r].push_back(QuantItem{off + e, (uint32_t)std::min<uint64_t>(kItemElems, n - e),
                                      plan->slabs[p.slab].ckpt_index});
    }
  auto up256 = [](size_t x) { return (x + 255) / 256 * 256; };
  size_t bytes = amax.size() * sizeof(AmaxItem) + 256;
  for (auto& v : rounds) bytes += v.size() * sizeof(QuantItem) + 256;
  for (const Round& R : plan->rounds) bytes += up256(R.pack_ckpt.size() * 4) + up256(R.unpack_ckpt.size() * 4);
  bytes += up256(plan->rounds.size() * 8 + 8) + 256;
  auto* T = new (std::nothrow) QuantTables;
  if (!T) return WB_ERR_OOM;
  if (cudaMalloc(&T->d_mem, bytes) != cudaSuccess) { delete T; return WB_ERR_OOM; }
  std::vector<char> host(bytes, 0);
  size_t off = 0;
  T->d_amax = reinterpret_cast<AmaxItem*>(static_cast<char*>(T->d_mem) + off);
  T->n_amax = (uint32_t)amax.size();
  if (!amax.empty()) std::memcpy(host.data() + off, amax.data(), amax.size() * sizeof(AmaxItem));
  off += (amax.size() * sizeof(AmaxItem) + 255) / 256 * 256;
  for (auto& v : rounds) {
    T->d_round.push_back(reinterpret_cast<QuantItem*>(static_cast<char*>(T->d_mem) + off));
    T->n_round.push_back((uint32_t)v.size());
    if (!v.empty()) std::memcpy(host.data() + off, v.data(), v.size() * sizeof(QuantItem));
    off += (v.size() * sizeof(QuantItem) + 255) / 256 * 256;
  }
  for (const Round& R : plan->rounds) {
    T->d_pack_ckpt.push_back(reinterpret_cast<uint32_t*>(static_cast<char*>(T->d_mem) + off));
    if (!R.pack_ckpt.empty()) std::memcpy(host.data() + off, R.pack_ckpt.data(), R.pack_ckpt.size() * 4);
    off += up256(R.pack_ckpt.size() * 4);
    T->d_unpack_ckpt.push_back(reinterpret_cast<uint32_t*>(static_cast<char*>(T->d_mem) + off));
    if (!R.unpack_ckpt.empty()) std::memcpy(host.data() + off, R.unpack_ckpt.data(), R.unpack_ckpt.size() * 4);
    off += up256(R.unpack_ckpt.size() * 4);
  }
  T->d_counters = reinterpret_cast<uint32_t*>(static_cast<char*>(T->d_mem) + off);
  off += up256(plan->rounds.size() * 8 + 8);
  if (cudaMemcpy(T->d_mem, host.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaFree(T->d_mem);
    delete T;
    return WB_ERR_CUDA;
  }
  plan->quant_tables = T;
  return WB_OK;
}

inline uint32_t grid_for(uint32_t n_items) { return n_items < 148u * 8 ? (n_items ? n_items : 1u) : 148u * 8; }

}  // namespace

namespace wbi {
void release_quant_tables(wb_plan* plan) {
  auto* T = static_cast<QuantTables*>(plan->quant_tables);
  if (!T) return;
  cudaFree(T->d_mem);
  delete T;
  plan->quant_tables = nullptr;
}
}  // namespace wbi

extern "C" size_t wb_plan_num_ckpts(const wb_plan* plan) { return plan ? plan->dst.ckpts.size() : 0; }

extern "C" wb_status wb_plan_ckpt_ids(const wb_plan* plan, uint64_t* out, size_t cap) {
  if (!plan || !out || cap < plan->dst.ckpts.size()) return WB_ERR_INVALID_ARG;
  for (size_t k = 0; k < plan->dst.ckpts.size(); ++k) out[k] = plan->dst.ckpts[k].id;
  return WB_OK;
}

extern "C" size_t wb_plan_qbucket_bytes(const wb_plan* plan, size_t round) {
  if (!plan || round >= plan->rounds.size()) return 0;
  return plan->rounds[round].bucket_bytes / esize(plan->dst.dtype);
}

extern "C" wb_status wb_absmax(const wb_plan* plan_c, float* amax, void* cuda_stream) {
  if (!plan_c || !amax) return WB_ERR_INVALID_ARG;
  if (!plan_c->bound) return WB_ERR_NOT_BOUND;
  if (!on_bound_device(plan_c)) return WB_ERR_INVALID_ARG;
  wb_plan* plan = const_cast<wb_plan*>(plan_c);      // lazily built work lists, not the plan itself
  wb_status st = WB_OK;
  try { st = build_tables(plan); } catch (const std::bad_alloc&) { return WB_ERR_OOM; }
  if (st != WB_OK) return st;
  auto* T = static_cast<QuantTables*>(plan->quant_tables);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(amax, 0, plan->dst.ckpts.size() * sizeof(float), stream) != cudaSuccess) return WB_ERR_CUDA;
  if (T->n_amax == 0) return WB_OK;
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype), grid = grid_for(T->n_amax);
  uint32_t* out = reinterpret_cast<uint32_t*>(amax);
  uint32_t* counter = T->d_counters + 2 * plan->rounds.size();      // the slot after the rounds' counters
  if (cudaMemsetAsync(counter, 0, sizeof(uint32_t), stream) != cudaSuccess) return WB_ERR_CUDA;
  if (es == 4 && ed == 2) wb_absmax_kernel<4, 2><<<grid, 256, 0, stream>>>(T->d_amax, T->n_amax, out, counter);
  else if (es == 4) wb_absmax_kernel<4, 4><<<grid, 256, 0, stream>>>(T->d_amax, T->n_amax, out, counter);
  else wb_absmax_kernel<2, 2><<<grid, 256, 0, stream>>>(T->d_amax, T->n_amax, out, counter);   // bf16 widens exactly
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}

static wb_status quant_common(const wb_plan* plan_c, size_t round, const void* a, const void* b, const float* amax,
                              QuantTables** T) {
  if (!plan_c || !a || !b || !amax || round >= plan_c->rounds.size()) return WB_ERR_INVALID_ARG;
  if (((uintptr_t)a & 15u) || ((uintptr_t)b & 15u)) return WB_ERR_INVALID_ARG;
  if (!plan_c->bound) return WB_ERR_NOT_BOUND;
  if (!on_bound_device(plan_c)) return WB_ERR_INVALID_ARG;
  wb_plan* plan = const_cast<wb_plan*>(plan_c);
  wb_status st = WB_OK;
  try { st = build_tables(plan); } catch (const std::bad_alloc&) { return WB_ERR_OOM; }
  if (st != WB_OK) return st;
  *T = static_cast<QuantTables*>(plan->quant_tables);
  return WB_OK;
}

extern "C" wb_status wb_bucket_quantize(const wb_plan* plan, size_t round, const void* bucket, void* qbucket,
                                        const float* amax, void* cuda_stream) {
  QuantTables* T = nullptr;
  const wb_status st = quant_common(plan, round, bucket, qbucket, amax, &T);
  if (st != WB_OK) return st;
  const uint32_t n = T->n_round[round];
  if (n == 0) return WB_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (esize(plan->dst.dtype) == 2)
    wb_quantize_kernel<2><<<grid_for(n), 256, 0, stream>>>(T->d_round[round], n, static_cast<const char*>(bucket),
                                                           static_cast<uint8_t*>(qbucket), amax);
  else
    wb_quantize_kernel<4><<<grid_for(n), 256, 0, stream>>>(T->d_round[round], n, static_cast<const char*>(bucket),
                                                           static_cast<uint8_t*>(qbucket), amax);
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}

extern "C" wb_status wb_bucket_dequantize(const wb_plan* plan, size_t round, const void* qbucket, void* bucket,
                                          const float* amax, void* cuda_stream) {
  QuantTables* T = nullptr;
  const wb_status st = quant_common(plan, round, qbucket, bucket, amax, &T);
  if (st != WB_OK) return st;
  const uint32_t n = T->n_round[round];
  if (n == 0) return WB_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (esize(plan->dst.dtype) == 2)
    wb_dequantize_kernel<2><<<grid_for(n), 256, 0, stream>>>(T->d_round[round], n, static_cast<const uint8_t*>(qbucket),
                                                             static_cast<char*>(bucket), amax);
  else
    wb_dequantize_kernel<4><<<grid_for(n), 256, 0, stream>>>(T->d_round[round], n, static_cast<const uint8_t*>(qbucket),
                                                             static_cast<char*>(bucket), amax);
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}


// Fused quantising pack / dequantising unpack (see the kernels above).
extern "C" wb_status wb_pack_fp8(const wb_plan* plan, size_t round, void* qbucket, const float* amax, void* cuda_stream) {
  QuantTables* T = nullptr;
  const wb_status st = quant_common(plan, round, qbucket, qbucket, amax, &T);
  if (st != WB_OK) return st;
  const TileTable& tab = plan->rounds[round].pack;
  const uint32_t n = (uint32_t)tab.tiles.size();
  if (n == 0) return WB_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t* counter = T->d_counters + 2 * round;
  if (cudaMemsetAsync(counter, 0, sizeof(uint32_t), stream) != cudaSuccess) return WB_ERR_CUDA;
  const uint32_t grid = n < 148u * 6 ? n : 148u * 6;
  const uint32_t es = esize(plan->src.dtype), ed = esize(plan->dst.dtype);
  uint8_t* q = static_cast<uint8_t*>(qbucket);
  if (es == 4 && ed == 2) wb_pack_fp8_kernel<4, 2><<<grid, 256, 0, stream>>>(tab.d_tiles, T->d_pack_ckpt[round], n, q, amax, counter);
  else if (es == 4) wb_pack_fp8_kernel<4, 4><<<grid, 256, 0, stream>>>(tab.d_tiles, T->d_pack_ckpt[round], n, q, amax, counter);
  else if (ed == 2) wb_pack_fp8_kernel<2, 2><<<grid, 256, 0, stream>>>(tab.d_tiles, T->d_pack_ckpt[round], n, q, amax, counter);
  else wb_pack_fp8_kernel<2, 4><<<grid, 256, 0, stream>>>(tab.d_tiles, T->d_pack_ckpt[round], n, q, amax, counter);
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}

extern "C" wb_status wb_unpack_fp8(const wb_plan* plan, size_t round, const void* qbucket, const float* amax,
                                   void* cuda_stream) {
  QuantTables* T = nullptr;
  const wb_status st = quant_common(plan, round, qbucket, qbucket, amax, &T);
  if (st != WB_OK) return st;
  const TileTable& tab = plan->rounds[round].unpack;
  const uint32_t n = (uint32_t)tab.tiles.size();
  if (n == 0) return WB_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t* counter = T->d_counters + 2 * round + 1;
  if (cudaMemsetAsync(counter, 0, sizeof(uint32_t), stream) != cudaSuccess) return WB_ERR_CUDA;
  const uint32_t grid = n < 148u * 6 ? n : 148u * 6;
  const uint8_t* q = static_cast<const uint8_t*>(qbucket);
  if (esize(plan->dst.dtype) == 2) wb_unpack_fp8_kernel<2><<<grid, 256, 0, stream>>>(tab.d_tiles, T->d_unpack_ckpt[round], tab.d_extras, n, q, amax, counter);
  else wb_unpack_fp8_kernel<4><<<grid, 256, 0, stream>>>(tab.d_tiles, T->d_unpack_ckpt[round], tab.d_extras, n, q, amax, counter);
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}

// All rounds of the quantised two-pass path with two bucket pairs in flight, like wb_transfer_rounds:
// the packing stream runs amax, then per round pack -> quantise; the assembly stream dequantise -> unpack.
extern "C" wb_status wb_transfer_rounds_fp8(const wb_plan* plan_c, void* bucket0, void* bucket1, void* qbucket0,
                                            void* qbucket1, float* amax, void* cuda_stream) {
  if (!plan_c || !bucket0 || !bucket1 || !qbucket0 || !qbucket1 || !amax) return WB_ERR_INVALID_ARG;
  if (bucket0 == bucket1 || qbucket0 == qbucket1) return WB_ERR_INVALID_ARG;
  if ((((uintptr_t)bucket0 | (uintptr_t)bucket1 | (uintptr_t)qbucket0 | (uintptr_t)qbucket1) & 15u)) return WB_ERR_INVALID_ARG;
  if (!plan_c->bound) return WB_ERR_NOT_BOUND;
  wb_plan* plan = const_cast<wb_plan*>(plan_c);      // lazily built pipeline state, not the plan itself
  const size_t R = plan->rounds.size();
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  wb_status st = WB_OK;
  try { st = ensure_pipeline(plan, 2 * R + 1); } catch (const std::bad_alloc&) { return WB_ERR_OOM; }
  if (st != WB_OK) return st;
  cudaStream_t ps = static_cast<cudaStream_t>(plan->h2d_stream), us = static_cast<cudaStream_t>(plan->d2h_stream);
  auto packed = [&](size_t r) { return static_cast<cudaEvent_t>(plan->host_events[2 * r]); };
  auto unpacked = [&](size_t r) { return static_cast<cudaEvent_t>(plan->host_events[2 * r + 1]); };
  cudaEvent_t start = static_cast<cudaEvent_t>(plan->host_events[2 * R]);
  if (cudaEventRecord(start, stream) != cudaSuccess) return WB_ERR_CUDA;
  if (cudaStreamWaitEvent(ps, start, 0) != cudaSuccess || cudaStreamWaitEvent(us, start, 0) != cudaSuccess) return WB_ERR_CUDA;
  if ((st = wb_absmax(plan, amax, ps)) != WB_OK) return st;
  for (size_t r = 0; r < R; ++r) {
    void* b = (r & 1) ? bucket1 : bucket0;
    void* q = (r & 1) ? qbucket1 : qbucket0;
    if (r >= 2 && cudaStreamWaitEvent(ps, unpacked(r - 2), 0) != cudaSuccess) return WB_ERR_CUDA;
    if ((st = wb_pack(plan, r, b, ps)) != WB_OK) return st;
    if ((st = wb_bucket_quantize(plan, r, b, q, amax, ps)) != WB_OK) return st;
    if (cudaEventRecord(packed(r), ps) != cudaSuccess || cudaStreamWaitEvent(us, packed(r), 0) != cudaSuccess) return WB_ERR_CUDA;
    // (the transfer of q would happen here)
    if ((st = wb_bucket_dequantize(plan, r, q, b, amax, us)) != WB_OK) return st;
    if ((st = wb_unpack(plan, r, b, us)) != WB_OK) return st;
    if (cudaEventRecord(unpacked(r), us) != cudaSuccess) return WB_ERR_CUDA;
  }
  // with no rounds the amax pass is all there is: the caller's stream waits for the packing stream
  cudaEvent_t last = R ? unpacked(R - 1) : start;
  if (R == 0 && cudaEventRecord(start, ps) != cudaSuccess) return WB_ERR_CUDA;
  if (cudaStreamWaitEvent(stream, last, 0) != cudaSuccess) return WB_ERR_CUDA;
  return WB_OK;
}

// The quantised transfer with the fused kernels: amax, then per round wb_pack_fp8 on the packing stream and
// wb_unpack_fp8 on the assembly stream, two FP8 buckets in flight (no 2- or 4-byte bucket at all).
extern "C" wb_status wb_transfer_rounds_fp8_fused(const wb_plan* plan_c, void* qbucket0, void* qbucket1, float* amax,
                                                  void* cuda_stream) {
  if (!plan_c || !qbucket0 || !qbucket1 || !amax || qbucket0 == qbucket1) return WB_ERR_INVALID_ARG;
  if ((((uintptr_t)qbucket0 | (uintptr_t)qbucket1) & 15u)) return WB_ERR_INVALID_ARG;
  if (!plan_c->bound) return WB_ERR_NOT_BOUND;
  wb_plan* plan = const_cast<wb_plan*>(plan_c);      // lazily built pipeline state, not the plan itself
  const size_t R = plan->rounds.size();
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  wb_status st = WB_OK;
  try { st = ensure_pipeline(plan, 2 * R + 1); } catch (const std::bad_alloc&) { return WB_ERR_OOM; }
  if (st != WB_OK) return st;
  cudaStream_t ps = static_cast<cudaStream_t>(plan->h2d_stream), us = static_cast<cudaStream_t>(plan->d2h_stream);
  auto packed = [&](size_t r) { return static_cast<cudaEvent_t>(plan->host_events[2 * r]); };
  auto unpacked = [&](size_t r) { return static_cast<cudaEvent_t>(plan->host_events[2 * r + 1]); };
  cudaEvent_t start = static_cast<cudaEvent_t>(plan->host_events[2 * R]);
  if (cudaEventRecord(start, stream) != cudaSuccess) return WB_ERR_CUDA;
  if (cudaStreamWaitEvent(ps, start, 0) != cudaSuccess || cudaStreamWaitEvent(us, start, 0) != cudaSuccess) return WB_ERR_CUDA;
  if ((st = wb_absmax(plan, amax, ps)) != WB_OK) return st;
  for (size_t r = 0; r < R; ++r) {
    void* q = (r & 1) ? qbucket1 : qbucket0;
    if (r >= 2 && cudaStreamWaitEvent(ps, unpacked(r - 2), 0) != cudaSuccess) return WB_ERR_CUDA;
    if ((st = wb_pack_fp8(plan, r, q, amax, ps)) != WB_OK) return st;
    if (cudaEventRecord(packed(r), ps) != cudaSuccess || cudaStreamWaitEvent(us, packed(r), 0) != cudaSuccess) return WB_ERR_CUDA;
    // (the transfer of q would happen here)
    if ((st = wb_unpack_fp8(plan, r, q, amax, us)) != WB_OK) return st;
    if (cudaEventRecord(unpacked(r), us) != cudaSuccess) return WB_ERR_CUDA;
  }
  cudaEvent_t last = R ? unpacked(R - 1) : start;
  if (R == 0 && cudaEventRecord(start, ps) != cudaSuccess) return WB_ERR_CUDA;
  if (cudaStreamWaitEvent(stream, last, 0) != cudaSuccess) return WB_ERR_CUDA;
  return WB_OK;
}
