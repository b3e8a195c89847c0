// Source-map extraction, device part (Section 3.1 and Appendix B of the paper): the second-order
// difference diff2 of an identifier field, with compaction of its non-zero entries.
//
// diff2 = diff1 o diff1 with diff1(A)[i,j] = A[i,j] - A[i-1,j] - A[i,j-1] + A[i-1,j-1] and A = 0 for
// negative indices, i.e. the causal 3x3 stencil with weights [1,-2,1] x [1,-2,1].  Over a rectangle
// that one slice-copy operation filled the field is affine, so only a constant number of entries
// around the rectangle's corners survive; those are appended to a caller-provided list.
#include <cuda_runtime.h>

#include <cstdint>

#include "wb.h"

namespace {

template <int KIND> __device__ __forceinline__ long long field_at(const void* f, unsigned long long idx);
template <> __device__ __forceinline__ long long field_at<WB_ID_I64>(const void* f, unsigned long long idx) {
  return __ldg(static_cast<const long long*>(f) + idx);
}
template <> __device__ __forceinline__ long long field_at<WB_ID_U16>(const void* f, unsigned long long idx) {
  return (long long)__ldg(static_cast<const unsigned short*>(f) + idx);
}
template <> __device__ __forceinline__ long long field_at<WB_ID_F32>(const void* f, unsigned long long idx) {
  return (long long)__float2ll_rn(__ldg(static_cast<const float*>(f) + idx));
}
template <> __device__ __forceinline__ long long field_at<WB_ID_BF16>(const void* f, unsigned long long idx) {
  const unsigned int bits = (unsigned int)__ldg(static_cast<const unsigned short*>(f) + idx) << 16;
  return (long long)__float2ll_rn(__uint_as_float(bits));
}

// One thread per element, grid-stride over the row-major field.  A thread reads the 3x3 causal
// neighbourhood (the neighbours are L1/L2 hits: DRAM sees every element about once) and, if the
// stencil is non-zero, takes a slot in the output list; slots are claimed once per warp.
template <int KIND>
__global__ void __launch_bounds__(256)
wb_diff2_kernel(const void* __restrict__ field, unsigned long long rows, unsigned long long cols,
                wb_diff2_entry* __restrict__ out, unsigned long long cap, unsigned long long* __restrict__ count) {
  const unsigned long long n = rows * cols;
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  const unsigned lane = threadIdx.x & 31;
  // whole warps iterate together so that the ballot below always has all lanes
  for (unsigned long long base = (unsigned long long)blockIdx.x * blockDim.x + (threadIdx.x & ~31u); base < n;
       base += stride) {
    const unsigned long long e = base + lane;
    long long d = 0;
    unsigned long long i = 0, j = 0;
    if (e < n) {
      i = e / cols;
      j = e - i * cols;
      long long acc[3] = {0, 0, 0};       // [1,-2,1] along j for rows i, i-1, i-2
#pragma unroll
      for (int a = 0; a < 3; ++a) {
        if (i >= (unsigned long long)a) {
          const unsigned long long r = e - (unsigned long long)a * cols;
          long long v = field_at<KIND>(field, r);
          if (j >= 1) v -= 2 * field_at<KIND>(field, r - 1);
          if (j >= 2) v += field_at<KIND>(field, r - 2);
          acc[a] = v;
        }
      }
      d = acc[0] - 2 * acc[1] + acc[2];
    }
    const unsigned mask = __ballot_sync(0xFFFFFFFFu, d != 0);
    if (mask) {
      unsigned long long slot0 = 0;
      if (lane == 0) slot0 = atomicAdd(count, (unsigned long long)__popc(mask));
      slot0 = __shfl_sync(0xFFFFFFFFu, slot0, 0);
      if (d != 0) {
        const unsigned long long slot = slot0 + __popc(mask & ((1u << lane) - 1));
        if (slot < cap) out[slot] = wb_diff2_entry{i, j, d};
      }
    }
  }
}

}  // namespace

extern "C" wb_status wb_diff2_nonzeros(const void* field, uint32_t id_kind, uint64_t rows, uint64_t cols,
                                       wb_diff2_entry* out, uint64_t cap, uint64_t* count, void* cuda_stream) {
  if (!field || !count || (!out && cap) || id_kind > WB_ID_BF16) return WB_ERR_INVALID_ARG;
  if (rows == 0 || cols == 0) return WB_OK;
  if (rows > (1ull << 40) || cols > (1ull << 40) || rows * cols > (1ull << 48)) return WB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const unsigned long long n = rows * cols;
  const unsigned long long want = (n + 255) / 256;
  const unsigned grid = (unsigned)(want < 148ull * 16 ? want : 148ull * 16);
  auto* cnt = reinterpret_cast<unsigned long long*>(count);
  switch (id_kind) {
    case WB_ID_I64: wb_diff2_kernel<WB_ID_I64><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
    case WB_ID_U16: wb_diff2_kernel<WB_ID_U16><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
    case WB_ID_F32: wb_diff2_kernel<WB_ID_F32><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
    default: wb_diff2_kernel<WB_ID_BF16><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
  }
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}
