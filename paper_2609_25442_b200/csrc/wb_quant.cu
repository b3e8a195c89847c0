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

// amax: magnitudes are compared as unsigned integers of the sign-cleared fp32 patterns (a NaN wins).
// A warp takes a run; the part between 16-byte boundaries is read with 16-byte loads, four in
// flight per lane, the ends element by element.
template <int ES, int ED>
__global__ void __launch_bounds__(256)
wb_absmax_kernel(const AmaxItem* __restrict__ items, uint32_t n_items, uint32_t* __restrict__ amax) {
  __shared__ uint32_t warp_max[8];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr uint32_t PER = 16 / ES;
  for (uint32_t k = blockIdx.x; k < n_items; k += gridDim.x) {
    const AmaxItem it = items[k];
    uint32_t m = 0;
    // the warps share the item's runs in segments of kSeg elements (a flat shard is one long run)
    constexpr uint32_t kSeg = 8192;
    const uint32_t segs = (it.n1 + kSeg - 1) / kSeg;
    for (uint32_t t = warp; t < it.n0 * segs; t += 8) {
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
    __syncthreads();
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

// Work lists, built on first use and kept with the plan's device tables.
struct QuantTables {
  void* d_mem = nullptr;
  AmaxItem* d_amax = nullptr;
  uint32_t n_amax = 0;
  std::vector<QuantItem*> d_round;
  std::vector<uint32_t> n_round;
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
  size_t bytes = amax.size() * sizeof(AmaxItem) + 256;
  for (auto& v : rounds) bytes += v.size() * sizeof(QuantItem) + 256;
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
  if (es == 4 && ed == 2) wb_absmax_kernel<4, 2><<<grid, 256, 0, stream>>>(T->d_amax, T->n_amax, out);
  else if (es == 4) wb_absmax_kernel<4, 4><<<grid, 256, 0, stream>>>(T->d_amax, T->n_amax, out);
  else wb_absmax_kernel<2, 2><<<grid, 256, 0, stream>>>(T->d_amax, T->n_amax, out);   // bf16 widens exactly
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
