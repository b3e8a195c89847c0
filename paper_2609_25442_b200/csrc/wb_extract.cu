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

// A warp task is a strip of kStrip = 32*kV columns marched down up to kRowsPerTask rows.  Lane l
// owns columns c0 + l + 32 k (k < kV), so each of its kV loads per row is a fully coalesced warp
// access and all kV are in flight together.  The two values to the left of a column come from
// lanes l-1 and l-2 by shuffle (from the previous k for lanes 0 and 1; from memory at the strip's
// left edge), and the horizontal second difference h(i,j) = A(i,j) - 2 A(i,j-1) + A(i,j-2) of the
// two rows above stays in registers, so diff2(i,j) = h(i,j) - 2 h(i-1,j) + h(i-2,j) costs one
// global load per element (plus two halo rows per task).  Non-zeros are rare: a warp vote skips
// the compaction for almost every row.
constexpr int kRowsPerTask = 64;
constexpr int kV = 8;
constexpr int kStrip = 32 * kV;

template <int KIND>
__device__ __forceinline__ void row_h(const void* field, unsigned long long row_base, unsigned long long cols,
                                      unsigned long long c0, unsigned lane, long long h[kV]) {
  long long a[kV];
#pragma unroll
  for (int k = 0; k < kV; ++k) {
    const unsigned long long c = c0 + lane + 32u * k;
    a[k] = c < cols ? field_at<KIND>(field, row_base + c) : 0;
  }
  // halo: the two columns left of the strip (read by lanes 0 and 1, both end up needing them)
  long long e1 = 0, e2 = 0;                                  // A[c0-1], A[c0-2]
  if (lane < 2) {
    if (c0 >= 1) e1 = field_at<KIND>(field, row_base + c0 - 1);
    if (c0 >= 2) e2 = field_at<KIND>(field, row_base + c0 - 2);
  }
  long long prev30 = e2, prev31 = e1;                          // "lanes 30 / 31 of k-1"; uniform per warp below
  prev30 = __shfl_sync(0xFFFFFFFFu, prev30, 0);
  prev31 = __shfl_sync(0xFFFFFFFFu, prev31, 0);
#pragma unroll
  for (int k = 0; k < kV; ++k) {
    long long l1 = __shfl_up_sync(0xFFFFFFFFu, a[k], 1), l2 = __shfl_up_sync(0xFFFFFFFFu, a[k], 2);
    if (lane == 0) { l1 = prev31; l2 = prev30; }
    if (lane == 1) l2 = prev31;
    h[k] = a[k] - 2 * l1 + l2;
    prev30 = __shfl_sync(0xFFFFFFFFu, a[k], 30);
    prev31 = __shfl_sync(0xFFFFFFFFu, a[k], 31);
  }
}

template <int KIND>
__global__ void __launch_bounds__(256)
wb_diff2_kernel(const void* __restrict__ field, unsigned long long rows, unsigned long long cols,
                wb_diff2_entry* __restrict__ out, unsigned long long cap, unsigned long long* __restrict__ count) {
  const unsigned lane = threadIdx.x & 31;
  const unsigned long long strips = (cols + kStrip - 1) / kStrip, blocks = (rows + kRowsPerTask - 1) / kRowsPerTask;
  const unsigned long long n_tasks = strips * blocks;
  const unsigned long long warp0 = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const unsigned long long n_warps = ((unsigned long long)gridDim.x * blockDim.x) >> 5;
  for (unsigned long long task = warp0; task < n_tasks; task += n_warps) {
    const unsigned long long rb = task / strips, cs = task - rb * strips;   // neighbouring warps: neighbouring strips
    const unsigned long long i0 = rb * kRowsPerTask;
    const unsigned long long i1 = i0 + kRowsPerTask < rows ? i0 + kRowsPerTask : rows;
    const unsigned long long c0 = cs * kStrip;
    long long hm1[kV], hm2[kV];
#pragma unroll
    for (int k = 0; k < kV; ++k) hm1[k] = hm2[k] = 0;
    if (i0 >= 2) row_h<KIND>(field, (i0 - 2) * cols, cols, c0, lane, hm2);
    if (i0 >= 1) row_h<KIND>(field, (i0 - 1) * cols, cols, c0, lane, hm1);
    for (unsigned long long i = i0; i < i1; ++i) {
      long long h[kV], d[kV];
      row_h<KIND>(field, i * cols, cols, c0, lane, h);
      long long any = 0;
#pragma unroll
      for (int k = 0; k < kV; ++k) {
        d[k] = (c0 + lane + 32u * k < cols) ? h[k] - 2 * hm1[k] + hm2[k] : 0;
        hm2[k] = hm1[k];
        hm1[k] = h[k];
        any |= d[k];
      }
      if (__any_sync(0xFFFFFFFFu, any != 0)) {
#pragma unroll
        for (int k = 0; k < kV; ++k) {
          const unsigned mask = __ballot_sync(0xFFFFFFFFu, d[k] != 0);
          if (!mask) continue;
          unsigned long long slot0 = 0;
          if (lane == 0) slot0 = atomicAdd(count, (unsigned long long)__popc(mask));
          slot0 = __shfl_sync(0xFFFFFFFFu, slot0, 0);
          if (d[k] != 0) {
            const unsigned long long slot = slot0 + __popc(mask & ((1u << lane) - 1));
            if (slot < cap) out[slot] = wb_diff2_entry{i, c0 + lane + 32u * k, d[k]};
          }
        }
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
  const unsigned long long tasks = ((cols + kStrip - 1) / kStrip) * ((rows + kRowsPerTask - 1) / kRowsPerTask);
  const unsigned long long want = (tasks + 7) / 8;                 // 8 warps per block
  const unsigned grid = (unsigned)(want < 148ull * 8 ? want : 148ull * 8);
  auto* cnt = reinterpret_cast<unsigned long long*>(count);
  switch (id_kind) {
    case WB_ID_I64: wb_diff2_kernel<WB_ID_I64><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
    case WB_ID_U16: wb_diff2_kernel<WB_ID_U16><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
    case WB_ID_F32: wb_diff2_kernel<WB_ID_F32><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
    default: wb_diff2_kernel<WB_ID_BF16><<<grid, 256, 0, stream>>>(field, rows, cols, out, cap, cnt); break;
  }
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}
