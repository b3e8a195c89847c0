// Source-map extraction, device part (Section 3.1 and Appendix B of the paper): the second-order
// difference diff2 of an identifier field, with compaction of its non-zero entries.
//
// diff2 = diff1 o diff1 with diff1(A)[i,j] = A[i,j] - A[i-1,j] - A[i,j-1] + A[i-1,j-1] and A = 0 for
// negative indices, i.e. the causal 3x3 stencil with weights [1,-2,1] x [1,-2,1].  Over a rectangle
// that one slice-copy operation filled the field is affine, so only a constant number of entries
// around the rectangle's corners survive; those are appended to a caller-provided list.
#include <cuda_runtime.h>

#include <cstdint>
#include <new>
#include <vector>

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

// A warp task is a strip of kStrip = 32 * kQ * kG columns marched down up to kRowsPerTask rows.
// In each of the kG groups a lane owns kQ = 4 adjacent columns, c0 + 128 g + 4 l + {0..3}, which it
// fetches with one or two vector loads, so only its leftmost two columns need values from another
// lane (one rotating shuffle per group hands lane l-1's last two columns to lane l; lane 0 takes
// the strip's left halo in group 0 and what the rotation brought round from lane 31 after that).
//
// diff2 is separable.  The kernel applies the vertical second difference first,
//   v(i,j) = A(i,j) - 2 A(i-1,j) + A(i-2,j),      diff2(i,j) = v(i,j) - 2 v(i,j-1) + v(i,j-2),
// because v needs no other lane (the two rows above stay in registers) and vanishes wherever three
// consecutive rows belong to one slice-copy operation: a warp vote then skips the horizontal step
// for almost every row.  A field with a single row (a flat shard) has v = A and goes straight to
// the horizontal step.  The loads of the next row visit (the next row, or the first row of the
// warp's next task) are issued before the current row is consumed.
constexpr int kRowsPerTask = 64;
constexpr int kQ = 4;
constexpr int kG = 2;
constexpr int kV = kQ * kG;
constexpr int kStrip = 32 * kV;

template <int KIND> struct FieldElem;
template <> struct FieldElem<WB_ID_I64> { static constexpr int kBytes = 8; };
template <> struct FieldElem<WB_ID_U16> { static constexpr int kBytes = 2; };
template <> struct FieldElem<WB_ID_F32> { static constexpr int kBytes = 4; };
template <> struct FieldElem<WB_ID_BF16> { static constexpr int kBytes = 2; };

__device__ __forceinline__ long long bf16_bits_to_ll(unsigned int b) {
  return (long long)__float2ll_rn(__uint_as_float(b << 16));
}

// Four adjacent elements starting at element index idx, the address known to be aligned for the
// vector access of the kind.
template <int KIND> __device__ __forceinline__ void load_quad(const void* f, unsigned long long idx, long long x[kQ]);
template <> __device__ __forceinline__ void load_quad<WB_ID_I64>(const void* f, unsigned long long idx, long long x[kQ]) {
  const longlong2* p = reinterpret_cast<const longlong2*>(static_cast<const long long*>(f) + idx);
  const longlong2 a = __ldg(p), b = __ldg(p + 1);
  x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
}
template <> __device__ __forceinline__ void load_quad<WB_ID_U16>(const void* f, unsigned long long idx, long long x[kQ]) {
  const uint2 a = __ldg(reinterpret_cast<const uint2*>(static_cast<const unsigned short*>(f) + idx));
  x[0] = a.x & 0xFFFFu; x[1] = a.x >> 16; x[2] = a.y & 0xFFFFu; x[3] = a.y >> 16;
}
template <> __device__ __forceinline__ void load_quad<WB_ID_F32>(const void* f, unsigned long long idx, long long x[kQ]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(f) + idx));
  x[0] = __float2ll_rn(a.x); x[1] = __float2ll_rn(a.y); x[2] = __float2ll_rn(a.z); x[3] = __float2ll_rn(a.w);
}
template <> __device__ __forceinline__ void load_quad<WB_ID_BF16>(const void* f, unsigned long long idx, long long x[kQ]) {
  const uint2 a = __ldg(reinterpret_cast<const uint2*>(static_cast<const unsigned short*>(f) + idx));
  x[0] = bf16_bits_to_ll(a.x & 0xFFFFu); x[1] = bf16_bits_to_ll(a.x >> 16);
  x[2] = bf16_bits_to_ll(a.y & 0xFFFFu); x[3] = bf16_bits_to_ll(a.y >> 16);
}

// One row of a strip as a lane holds it: its kV elements and (lane 0) the two elements left of
// the strip.
struct RowRegs {
  long long a[kV];
  long long e1, e2;                                            // A[c0-1], A[c0-2]
};

template <int KIND>
__device__ __forceinline__ void row_load(const void* field, unsigned long long row_base, unsigned long long cols,
                                         unsigned long long c0, unsigned lane, RowRegs& r) {
  // vector accesses need the quad's first element on a multiple of the vector size; every quad of
  // a row starts at a column that is a multiple of 4, so one test covers the row
  constexpr unsigned long long kVecElems = FieldElem<KIND>::kBytes == 8 ? 2 : 4;
  const unsigned long long first = (unsigned long long)(reinterpret_cast<uintptr_t>(field) / FieldElem<KIND>::kBytes) + row_base;
  const bool vec = first % kVecElems == 0;
#pragma unroll
  for (int g = 0; g < kG; ++g) {
    const unsigned long long c = c0 + 128u * g + 4u * lane;
    if (vec && c + kQ <= cols) {
      load_quad<KIND>(field, row_base + c, &r.a[kQ * g]);
    } else {
#pragma unroll
      for (int q = 0; q < kQ; ++q) r.a[kQ * g + q] = c + q < cols ? field_at<KIND>(field, row_base + c + q) : 0;
    }
  }
  r.e1 = r.e2 = 0;
  if (lane == 0) {
    if (c0 >= 1) r.e1 = field_at<KIND>(field, row_base + c0 - 1);
    if (c0 >= 2) r.e2 = field_at<KIND>(field, row_base + c0 - 2);
  }
}

// Horizontal second difference of one row of values v (with halo ve1 = v[c0-1], ve2 = v[c0-2] in
// lane 0), and compaction of its non-zero entries.
__device__ __forceinline__ void put_entry(wb_diff2_entry* out, unsigned long long slot, unsigned long long row,
                                          unsigned long long col, long long value, unsigned) {
  out[slot] = wb_diff2_entry{row, col, value};
}
__device__ __forceinline__ void put_entry(wb_diff2_tagged_entry* out, unsigned long long slot, unsigned long long row,
                                          unsigned long long col, long long value, unsigned tag) {
  out[slot] = wb_diff2_tagged_entry{row, col, value, tag, 0u};
}

template <typename Entry>
__device__ __forceinline__ void emit_row(const long long v[kV], long long ve1, long long ve2, unsigned long long row,
                                         unsigned long long c0, unsigned long long cols, unsigned lane,
                                         Entry* __restrict__ out, unsigned long long cap,
                                         unsigned long long* __restrict__ count, unsigned tag = 0) {
  const unsigned from = (lane + 31u) & 31u;
  long long carry1 = ve1, carry2 = ve2;                        // lane 0: the two values left of the group
#pragma unroll
  for (int g = 0; g < kG; ++g) {
    const long long* x = &v[kQ * g];
    long long l1 = __shfl_sync(0xFFFFFFFFu, x[3], from), l2 = __shfl_sync(0xFFFFFFFFu, x[2], from);
    if (lane == 0) {                                           // received lane 31's pair: the next group's halo
      const long long n1 = l1, n2 = l2;
      l1 = carry1; l2 = carry2;
      carry1 = n1; carry2 = n2;
    }
    long long d[kQ];
    d[0] = x[0] - 2 * l1 + l2;
    d[1] = x[1] - 2 * x[0] + l1;
    d[2] = x[2] - 2 * x[1] + x[0];
    d[3] = x[3] - 2 * x[2] + x[1];
    const unsigned long long c = c0 + 128u * g + 4u * lane;
    int n = 0;
#pragma unroll
    for (int q = 0; q < kQ; ++q) {
      if (c + q >= cols) d[q] = 0;
      n += d[q] != 0;
    }
    if (!__any_sync(0xFFFFFFFFu, n != 0)) continue;
    // exclusive prefix of the lanes' counts, one atomic for the warp
    int incl = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= (unsigned)o) incl += t;
    }
    const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    unsigned long long slot0 = 0;
    if (lane == 0) slot0 = atomicAdd(count, (unsigned long long)total);
    slot0 = __shfl_sync(0xFFFFFFFFu, slot0, 0);
    unsigned long long slot = slot0 + (unsigned)(incl - n);
#pragma unroll
    for (int q = 0; q < kQ; ++q)
      if (d[q] != 0) {
        if (slot < cap) put_entry(out, slot, row, c + q, d[q], tag);
        ++slot;
      }
  }
}

// The sequence of row visits of a warp: for each of its tasks the two rows above the task, which
// only prime the registers (rows -2 and -1 of the field read as zeros), then the task's own rows.
struct Visit {
  unsigned long long task;
  int row, i0, i1;                                             // fields with several rows: rows, cols < 2^31
  unsigned c0;
};

__device__ __forceinline__ void visit_begin(Visit& v, unsigned long long task, unsigned strips, unsigned rows,
                                            unsigned rows_per_task) {
  const unsigned long long rb = task / strips;                 // neighbouring warps: neighbouring strips
  v.task = task;
  v.i0 = (int)((unsigned)rb * rows_per_task);
  v.i1 = (unsigned)v.i0 + rows_per_task < rows ? (int)((unsigned)v.i0 + rows_per_task) : (int)rows;
  v.c0 = (unsigned)(task - rb * strips) * kStrip;
  v.row = v.i0 - 2;
}

template <int KIND>
__device__ __forceinline__ void visit_load(const void* field, const Visit& v, unsigned long long cols, unsigned lane,
                                           RowRegs& r) {
  if (v.row >= 0) {
    row_load<KIND>(field, (unsigned long long)v.row * cols, cols, v.c0, lane, r);
  } else {
#pragma unroll
    for (int k = 0; k < kV; ++k) r.a[k] = 0;
    r.e1 = r.e2 = 0;
  }
}

// The rows a warp holds live in a ring of register sets addressed by the position in an unrolled
// loop (current row, the row being fetched and the two rows above), so advancing a row moves no registers.
template <int KIND, typename Entry>
__global__ void __launch_bounds__(256, 2)
wb_diff2_kernel(const void* __restrict__ field, unsigned long long rows, unsigned long long cols,
                unsigned long long rows_per_task, Entry* __restrict__ out, unsigned long long cap,
                unsigned long long* __restrict__ count, unsigned tag) {
  constexpr int kRing = 4;
  const unsigned lane = threadIdx.x & 31;
  const unsigned strips = (unsigned)((cols + kStrip - 1) / kStrip);
  const unsigned long long n_tasks = (unsigned long long)strips * ((rows + rows_per_task - 1) / rows_per_task);
  const unsigned long long warp0 = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const unsigned n_warps = (gridDim.x * blockDim.x) >> 5;
  if (warp0 >= n_tasks) return;
  Visit v, w;
  visit_begin(v, warp0, strips, (unsigned)rows, (unsigned)rows_per_task);
  RowRegs R[kRing];
  visit_load<KIND>(field, v, cols, lane, R[0]);
  for (;;) {
#pragma unroll
    for (int s = 0; s < kRing; ++s) {
      const RowRegs& cur = R[s];
      w = v;                                                   // the visit after this one
      bool more = true;
      if (++w.row == w.i1) {
        more = w.task + n_warps < n_tasks;
        if (more) visit_begin(w, w.task + n_warps, strips, (unsigned)rows, (unsigned)rows_per_task);
      }
      if (more) visit_load<KIND>(field, w, cols, lane, R[(s + 1) % kRing]);
      if (v.row >= v.i0) {
        const RowRegs& p1 = R[(s + kRing - 1) % kRing];
        const RowRegs& p2 = R[(s + kRing - 2) % kRing];
        long long vv[kV];
        bool nz = false;
#pragma unroll
        for (int k = 0; k < kV; ++k) {
          vv[k] = cur.a[k] - 2 * p1.a[k] + p2.a[k];
          nz |= vv[k] != 0;
        }
        const long long ve1 = cur.e1 - 2 * p1.e1 + p2.e1, ve2 = cur.e2 - 2 * p1.e2 + p2.e2;
        nz |= (ve1 | ve2) != 0;
        if (__any_sync(0xFFFFFFFFu, nz))
          emit_row(vv, ve1, ve2, (unsigned long long)v.row, v.c0, cols, lane, out, cap, count, tag);
      }
      if (!more) return;
      v = w;
    }
  }
}

// A field with one row (a flat shard): diff2 is the second difference along the row, every task is
// one strip, and a warp alternates between two register sets so that the next strip is in flight
// while the current one is consumed.
template <int KIND, typename Entry>
__global__ void __launch_bounds__(256, 3)
wb_diff2_row_kernel(const void* __restrict__ field, unsigned long long cols, Entry* __restrict__ out,
                    unsigned long long cap, unsigned long long* __restrict__ count, unsigned tag) {
  const unsigned lane = threadIdx.x & 31;
  const unsigned long long stride = (((unsigned long long)gridDim.x * blockDim.x) >> 5) * kStrip;
  unsigned long long c0 = ((((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5)) * kStrip;
  if (c0 >= cols) return;
  RowRegs r0, r1;
  row_load<KIND>(field, 0, cols, c0, lane, r0);
  for (;;) {
    const unsigned long long c1 = c0 + stride;
    if (c1 < cols) row_load<KIND>(field, 0, cols, c1, lane, r1);
    emit_row(r0.a, r0.e1, r0.e2, 0, c0, cols, lane, out, cap, count, tag);
    if (c1 >= cols) return;
    c0 = c1 + stride;
    if (c0 < cols) row_load<KIND>(field, 0, cols, c0, lane, r0);
    emit_row(r1.a, r1.e1, r1.e2, 0, c1, cols, lane, out, cap, count, tag);
    if (c0 >= cols) return;
  }
}

// ---- many fields in one launch ---------------------------------------------------------------------
// A model has thousands of local tensors, most of them small: one launch per tensor is bound by launch
// latency.  Here the tasks (strip x block of kRowsPerTask rows) of all fields form one list; a warp
// finds the field of a task by bisection over the fields' first task numbers and walks the task with
// the two rows above it primed, the next row's loads in flight.
// fields of at least this many elements are launched on their own by the batched entry point
constexpr unsigned long long kBatchLargeField = 1ull << 24;

struct BatchField {
  const void* field;
  unsigned long long rows, cols, task_begin;
  unsigned id_kind, tag;
};

template <int KIND>
__device__ __forceinline__ void batch_task(const BatchField& f, unsigned long long local, unsigned lane,
                                           wb_diff2_tagged_entry* __restrict__ out, unsigned long long cap,
                                           unsigned long long* __restrict__ count) {
  const unsigned long long strips = (f.cols + kStrip - 1) / kStrip;
  const unsigned long long rb = local / strips, c0 = (local - rb * strips) * kStrip;
  const unsigned long long i0 = rb * kRowsPerTask, i1 = i0 + kRowsPerTask < f.rows ? i0 + kRowsPerTask : f.rows;
  RowRegs p2, p1, cur, nxt;
#pragma unroll
  for (int k = 0; k < kV; ++k) p1.a[k] = p2.a[k] = 0;
  p1.e1 = p1.e2 = p2.e1 = p2.e2 = 0;
  if (i0 >= 2) row_load<KIND>(f.field, (i0 - 2) * f.cols, f.cols, c0, lane, p2);
  if (i0 >= 1) row_load<KIND>(f.field, (i0 - 1) * f.cols, f.cols, c0, lane, p1);
  row_load<KIND>(f.field, i0 * f.cols, f.cols, c0, lane, cur);
  for (unsigned long long i = i0; i < i1; ++i) {
    if (i + 1 < i1) row_load<KIND>(f.field, (i + 1) * f.cols, f.cols, c0, lane, nxt);
    long long vv[kV];
    bool nz = false;
#pragma unroll
    for (int k = 0; k < kV; ++k) {
      vv[k] = cur.a[k] - 2 * p1.a[k] + p2.a[k];
      nz |= vv[k] != 0;
    }
    const long long ve1 = cur.e1 - 2 * p1.e1 + p2.e1, ve2 = cur.e2 - 2 * p1.e2 + p2.e2;
    nz |= (ve1 | ve2) != 0;
    if (__any_sync(0xFFFFFFFFu, nz)) emit_row(vv, ve1, ve2, i, c0, f.cols, lane, out, cap, count, f.tag);
    p2 = p1;
    p1 = cur;
    cur = nxt;
  }
}

__global__ void __launch_bounds__(256, 2)
wb_diff2_batch_kernel(const BatchField* __restrict__ fields, unsigned n_fields, unsigned long long n_tasks,
                      wb_diff2_tagged_entry* __restrict__ out, unsigned long long cap,
                      unsigned long long* __restrict__ count) {
  const unsigned lane = threadIdx.x & 31;
  const unsigned long long warp0 = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const unsigned long long n_warps = ((unsigned long long)gridDim.x * blockDim.x) >> 5;
  for (unsigned long long task = warp0; task < n_tasks; task += n_warps) {
    unsigned lo = 0, hi = n_fields - 1;                        // last field whose first task is <= task
    while (lo < hi) {
      const unsigned mid = (lo + hi + 1) >> 1;
      if (fields[mid].task_begin <= task) lo = mid; else hi = mid - 1;
    }
    const BatchField f = fields[lo];
    const unsigned long long local = task - f.task_begin;
    switch (f.id_kind) {
      case WB_ID_I64: batch_task<WB_ID_I64>(f, local, lane, out, cap, count); break;
      case WB_ID_U16: batch_task<WB_ID_U16>(f, local, lane, out, cap, count); break;
      case WB_ID_F32: batch_task<WB_ID_F32>(f, local, lane, out, cap, count); break;
      default: batch_task<WB_ID_BF16>(f, local, lane, out, cap, count); break;
    }
  }
}

}  // namespace

namespace {
// One field, one launch of the tuned kernels (entries of type Entry, all carrying `tag`).
template <typename Entry>
cudaError_t launch_field(const void* field, uint32_t id_kind, uint64_t rows, uint64_t cols, Entry* out, uint64_t cap,
                         unsigned long long* cnt, unsigned tag, cudaStream_t stream) {
  // Tasks are dealt to warps round robin, so the rows per task are chosen to give every warp the
  // same number of tasks (about kRowsPerTask rows each) instead of leaving a last, partly filled turn.
  const unsigned long long strips = (cols + kStrip - 1) / kStrip;
  const unsigned long long resident = 148ull * (rows == 1 ? 3 : 2);   // blocks the registers let an SM hold
  const unsigned long long n_warps = resident * 8;                      // 8 warps per block
  unsigned long long rows_per_task = rows < (unsigned long long)kRowsPerTask ? rows : kRowsPerTask;
  if (strips * ((rows + rows_per_task - 1) / rows_per_task) > n_warps) {
    unsigned long long turns = (strips * rows + n_warps * kRowsPerTask / 2) / (n_warps * kRowsPerTask);
    if (turns == 0) turns = 1;
    const unsigned long long row_blocks = (turns * n_warps) / strips;   // tasks <= turns * n_warps
    if (row_blocks >= 1) rows_per_task = (rows + row_blocks - 1) / row_blocks;
  }
  const unsigned long long tasks = strips * ((rows + rows_per_task - 1) / rows_per_task);
  const unsigned long long want = (tasks + 7) / 8;
  const unsigned grid = (unsigned)(want < resident ? want : resident);
#define WB_DIFF2_LAUNCH(KIND)                                                                                  \
  do {                                                                                                        \
    if (rows == 1) wb_diff2_row_kernel<KIND, Entry><<<grid, 256, 0, stream>>>(field, cols, out, cap, cnt, tag);  \
    else wb_diff2_kernel<KIND, Entry><<<grid, 256, 0, stream>>>(field, rows, cols, rows_per_task, out, cap, cnt, tag); \
  } while (0)
  switch (id_kind) {
    case WB_ID_I64: WB_DIFF2_LAUNCH(WB_ID_I64); break;
    case WB_ID_U16: WB_DIFF2_LAUNCH(WB_ID_U16); break;
    case WB_ID_F32: WB_DIFF2_LAUNCH(WB_ID_F32); break;
    default: WB_DIFF2_LAUNCH(WB_ID_BF16); break;
  }
#undef WB_DIFF2_LAUNCH
  return cudaGetLastError();
}
inline bool field_size_ok(uint64_t rows, uint64_t cols) {
  if (rows > (1ull << 40) || cols > (1ull << 40) || rows * cols > (1ull << 48)) return false;
  return !(rows > 1 && (rows >= (1ull << 31) || cols >= (1ull << 31)));
}
}  // namespace

extern "C" wb_status wb_diff2_nonzeros(const void* field, uint32_t id_kind, uint64_t rows, uint64_t cols,
                                       wb_diff2_entry* out, uint64_t cap, uint64_t* count, void* cuda_stream) {
  if (!field || !count || (!out && cap) || id_kind > WB_ID_BF16) return WB_ERR_INVALID_ARG;
  if (rows == 0 || cols == 0) return WB_OK;
  if (!field_size_ok(rows, cols)) return WB_ERR_INVALID_ARG;
  return launch_field(field, id_kind, rows, cols, out, cap, reinterpret_cast<unsigned long long*>(count), 0u,
                      static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}

extern "C" size_t wb_diff2_batch_scratch_bytes(size_t n_fields) { return n_fields * sizeof(BatchField); }

extern "C" wb_status wb_diff2_nonzeros_batch(const wb_diff2_field* fields, size_t n_fields, void* scratch,
                                             size_t scratch_bytes, wb_diff2_tagged_entry* out, uint64_t cap,
                                             uint64_t* count, void* cuda_stream) {
  if (!count || (!out && cap) || (n_fields && (!fields || !scratch))) return WB_ERR_INVALID_ARG;
  if (n_fields == 0) return WB_OK;
  if (n_fields > (1u << 30) || scratch_bytes < n_fields * sizeof(BatchField) || ((uintptr_t)scratch & 15u))
    return WB_ERR_INVALID_ARG;
  std::vector<BatchField> host;
  try { host.reserve(n_fields); } catch (const std::bad_alloc&) { return WB_ERR_OOM; }
  unsigned long long tasks = 0;
  for (size_t k = 0; k < n_fields; ++k) {
    const wb_diff2_field& f = fields[k];
    if (f.id_kind > WB_ID_BF16) return WB_ERR_INVALID_ARG;
    if (f.rows == 0 || f.cols == 0) continue;                  // empty fields have no tasks
    if (!f.field || !field_size_ok(f.rows, f.cols)) return WB_ERR_INVALID_ARG;
    if (f.rows * f.cols >= kBatchLargeField) continue;          // launched on its own below
    host.push_back(BatchField{f.field, f.rows, f.cols, tasks, f.id_kind, f.tag});
    tasks += ((f.cols + kStrip - 1) / kStrip) * ((f.rows + kRowsPerTask - 1) / kRowsPerTask);
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  auto* cnt = reinterpret_cast<unsigned long long*>(count);
  // large fields: the tuned single-field kernels keep the memory system busy by themselves
  for (size_t k = 0; k < n_fields; ++k) {
    const wb_diff2_field& f = fields[k];
    if (f.rows == 0 || f.cols == 0 || f.rows * f.cols < kBatchLargeField) continue;
    if (launch_field(f.field, f.id_kind, f.rows, f.cols, out, cap, cnt, f.tag, stream) != cudaSuccess) return WB_ERR_CUDA;
  }
  if (host.empty()) return WB_OK;
  // the descriptors are copied before the call returns (pageable source), so `host` may go out of scope
  if (cudaMemcpyAsync(scratch, host.data(), host.size() * sizeof(BatchField), cudaMemcpyHostToDevice, stream) != cudaSuccess)
    return WB_ERR_CUDA;
  const unsigned long long want = (tasks + 7) / 8;
  const unsigned grid = (unsigned)(want < 148ull * 2 ? want : 148ull * 2);
  wb_diff2_batch_kernel<<<grid, 256, 0, stream>>>(static_cast<const BatchField*>(scratch), (unsigned)host.size(), tasks, out,
                                                  cap, cnt);
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}
