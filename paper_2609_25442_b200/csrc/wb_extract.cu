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

// ---- large, vector-aligned fields: rows fed through a ring of bulk (TMA) copies ---------------------------
// The register-fed kernels above keep one row of loads in flight per warp, which leaves the memory system
// half idle.  Here a producer thread streams row pieces of kRingRowBytes into a ring of shared-memory stages
// with cp.async.bulk (completion on an mbarrier), so the bytes in flight do not depend on registers, and
// eight consumer warps difference out of shared memory: a thread owns 16 bytes of every row piece, i.e.
// 16 / sizeof(element) adjacent columns, and marches down the rows of its unit with the two rows above in
// registers.  As above the vertical second difference comes first and a warp vote skips everything else
// for almost every row; a row that has a non-zero vertical difference somewhere in the warp takes the
// horizontal step, neighbours' values by shuffle.  The warps' parts of a row overlap by one thread: lane 0
// re-reads the 16 bytes that the last lane of the warp before it owns (for the first warp of a strip, the 16
// bytes left of the strip, which the producer loads as a halo), takes part in the vote and hands its values
// to lane 1, but emits nothing - so a non-zero vertical difference in one warp's last columns is seen by
// the warp whose first columns it affects.
// A field with one row is cut into segments of one stage each (one bulk copy per segment, 16 bytes of left
// halo) and differenced along the row.  Every wait is bounded; a wait that runs out marks the count with
// kRingFailed and the block leaves.
constexpr int kRingStages = 3;
constexpr int kRingRows = 8;
constexpr int kRingRowBytes = 4096;                 // a row of a stage: 16 bytes of left halo + the strip's piece
constexpr int kRingStripBytes = 8 * 31 * 16;        // 2-D fields: 31 emitting threads per warp, 16 bytes each
constexpr int kRingPitch = kRingRowBytes + 16;
constexpr int kRingStageBytes = kRingRows * kRingPitch;
constexpr int kRingConsumers = 256;
constexpr unsigned long long kRingFailed = 1ull << 62;
constexpr unsigned long long kRingWaitNs = 2000000000ull;

__device__ __forceinline__ unsigned ring_smem(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ring_bar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ring_smem(bar)), "r"(count));
}
__device__ __forceinline__ void ring_bar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ring_smem(bar)) : "memory");
}
__device__ __forceinline__ void ring_bar_expect(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(ring_smem(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool ring_bar_wait(unsigned long long* bar, unsigned parity) {
  const unsigned addr = ring_smem(bar);
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return true;
    if ((it & 255u) == 0) {
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (t0 == 0) t0 = now;
      else if (now - t0 > kRingWaitNs) return false;
    }
  }
}
__device__ __forceinline__ void ring_bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(ring_smem(smem_dst)), "l"(gsrc), "r"(bytes), "r"(ring_smem(bar)) : "memory");
}

// The 16 bytes a thread owns, as kNE integers.  Only int64 ids need 64-bit arithmetic: the values of the other
// kinds are below 2^24, so their second differences (at most 16 times a value) fit 32 bits.
template <int KIND> struct RingElems {
  static constexpr int kNE = 16 / FieldElem<KIND>::kBytes;
  using V = int;
};
template <> struct RingElems<WB_ID_I64> {
  static constexpr int kNE = 2;
  using V = long long;
};
template <int KIND> __device__ __forceinline__ void ring_unpack(const uint4& w, typename RingElems<KIND>::V (&x)[RingElems<KIND>::kNE]);
template <> __device__ __forceinline__ void ring_unpack<WB_ID_I64>(const uint4& w, long long (&x)[2]) {
  x[0] = (long long)(((unsigned long long)w.y << 32) | w.x);
  x[1] = (long long)(((unsigned long long)w.w << 32) | w.z);
}
template <> __device__ __forceinline__ void ring_unpack<WB_ID_F32>(const uint4& w, int (&x)[4]) {
  x[0] = __float2int_rn(__uint_as_float(w.x)); x[1] = __float2int_rn(__uint_as_float(w.y));
  x[2] = __float2int_rn(__uint_as_float(w.z)); x[3] = __float2int_rn(__uint_as_float(w.w));
}
template <> __device__ __forceinline__ void ring_unpack<WB_ID_U16>(const uint4& w, int (&x)[8]) {
  const unsigned v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int p = 0; p < 4; ++p) { x[2 * p] = (int)(v[p] & 0xFFFFu); x[2 * p + 1] = (int)(v[p] >> 16); }
}
template <> __device__ __forceinline__ void ring_unpack<WB_ID_BF16>(const uint4& w, int (&x)[8]) {
  const unsigned v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    x[2 * p] = __float2int_rn(__uint_as_float(v[p] << 16));
    x[2 * p + 1] = __float2int_rn(__uint_as_float(v[p] & 0xFFFF0000u));
  }
}

template <typename Entry>
__device__ __forceinline__ void ring_emit(Entry* __restrict__ out, unsigned long long cap, unsigned long long* __restrict__ count,
                                          unsigned long long row, unsigned long long col, long long value, unsigned tag) {
  const unsigned long long slot = atomicAdd(count, 1ull);
  if (slot < cap) put_entry(out, slot, row, col, value, tag);
}

template <int KIND, typename Entry>
__global__ void __launch_bounds__(kRingConsumers + 32, 2)
wb_diff2_ring_kernel(const void* __restrict__ field, unsigned long long rows, unsigned long long cols,
                     unsigned long long rows_per_unit, Entry* __restrict__ out, unsigned long long cap,
                     unsigned long long* __restrict__ count, unsigned tag) {
  constexpr int ES = FieldElem<KIND>::kBytes, NE = RingElems<KIND>::kNE;
  constexpr unsigned long long W = kRingStripBytes / ES;                  // columns of a strip
  extern __shared__ __align__(128) char ring_smem_buf[];
  __shared__ __align__(8) unsigned long long full[kRingStages], empty[kRingStages];
  if (threadIdx.x == 0) {
    for (int k = 0; k < kRingStages; ++k) { ring_bar_init(&full[k], 1); ring_bar_init(&empty[k], kRingConsumers / 32); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const unsigned long long strips = (cols + W - 1) / W, row_units = (rows + rows_per_unit - 1) / rows_per_unit;
  const unsigned long long n_units = strips * row_units;
  if (threadIdx.x >= kRingConsumers) {
    // ---- producer: one thread streams the row pieces of this block's units
    if (threadIdx.x != kRingConsumers) return;
    unsigned n = 0;
    for (unsigned long long u = blockIdx.x; u < n_units; u += gridDim.x) {
      const unsigned long long strip = u % strips, ru = u / strips, c0 = strip * W;
      const unsigned halo = c0 ? 16u : 0u;                              // the 16 bytes left of the strip
      const unsigned bytes = (unsigned)((cols - c0 < W ? cols - c0 : W) * ES) + halo;
      const unsigned long long i_begin = ru * rows_per_unit, i_end = i_begin + rows_per_unit < rows ? i_begin + rows_per_unit : rows;
      for (unsigned long long r = i_begin >= 2 ? i_begin - 2 : 0; r < i_end; r += kRingRows, ++n) {
        const unsigned nrow = (unsigned)(i_end - r < (unsigned long long)kRingRows ? i_end - r : kRingRows);
        const unsigned st = n % kRingStages;
        if (n >= (unsigned)kRingStages && !ring_bar_wait(&empty[st], ((n / kRingStages) - 1) & 1)) { atomicMax(count, kRingFailed); return; }
        ring_bar_expect(&full[st], nrow * bytes);
        for (unsigned k = 0; k < nrow; ++k)
          ring_bulk_load(ring_smem_buf + (size_t)st * kRingStageBytes + (size_t)k * kRingPitch + 16 - halo,
                         static_cast<const char*>(field) + ((r + k) * cols + c0) * ES - halo, bytes, &full[st]);
      }
    }
    return;
  }
  // ---- consumers
  const unsigned t = threadIdx.x, lane = t & 31;
  unsigned n = 0;
  for (unsigned long long u = blockIdx.x; u < n_units; u += gridDim.x) {
    const unsigned long long strip = u % strips, ru = u / strips, c0 = strip * W;
    const unsigned long long wcols = cols - c0 < W ? cols - c0 : W;
    const unsigned long long i_begin = ru * rows_per_unit, i_end = i_begin + rows_per_unit < rows ? i_begin + rows_per_unit : rows;
    // window g of a row: g = 0 is the halo left of the strip, g >= 1 the strip's bytes [16 (g-1), 16 g);
    // warp w takes windows 31 w .. 31 w + 31, its lane 0 sharing a window with the warp before
    const unsigned g = (t >> 5) * 31 + lane;
    const bool active = g == 0 ? c0 != 0 : (unsigned long long)(g - 1) * NE < wcols;
    const unsigned long long j0 = c0 + (unsigned long long)g * NE - NE;   // this thread's first column (lane 0 of warp 0: left of the strip)
    using V = typename RingElems<KIND>::V;
    V p1[NE], p2[NE];
#pragma unroll
    for (int q = 0; q < NE; ++q) p1[q] = p2[q] = 0;
    for (unsigned long long r = i_begin >= 2 ? i_begin - 2 : 0; r < i_end; r += kRingRows, ++n) {
      const unsigned nrow = (unsigned)(i_end - r < (unsigned long long)kRingRows ? i_end - r : kRingRows);
      const unsigned st = n % kRingStages;
      unsigned ok = 1;
      if (lane == 0) ok = ring_bar_wait(&full[st], (n / kRingStages) & 1);
      ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
      if (!ok) { if (t == 0) atomicMax(count, kRingFailed); return; }
      const char* base = ring_smem_buf + (size_t)st * kRingStageBytes + (size_t)g * 16;
      for (unsigned k = 0; k < nrow; ++k) {
        const unsigned long long i = r + k;
        V cur[NE], v[NE];
#pragma unroll
        for (int q = 0; q < NE; ++q) cur[q] = 0;
        if (active) ring_unpack<KIND>(*reinterpret_cast<const uint4*>(base + (size_t)k * kRingPitch), cur);
        bool nz = false;
#pragma unroll
        for (int q = 0; q < NE; ++q) {
          v[q] = cur[q] - 2 * p1[q] + p2[q];
          nz |= v[q] != 0;
          p2[q] = p1[q];
          p1[q] = cur[q];
        }
        if (i < i_begin) continue;                                        // the two rows above the unit only prime
        if (!__any_sync(0xFFFFFFFFu, nz)) continue;
        // horizontal step: the two values left of this thread's columns come from the lane below, or from
        // global memory for the first lane of the warp
        const V l1 = __shfl_up_sync(0xFFFFFFFFu, v[NE - 1], 1), l2 = __shfl_up_sync(0xFFFFFFFFu, v[NE - 2], 1);
        if (!active || lane == 0) continue;                               // lane 0 only lends its values to lane 1
#pragma unroll
        for (int q = 0; q < NE; ++q) {
          const V a1 = q >= 1 ? v[q - 1] : l1, a2 = q >= 2 ? v[q - 2] : (q == 1 ? l1 : l2);
          const V d = v[q] - 2 * a1 + a2;
          if (d != 0) ring_emit(out, cap, count, i, j0 + q, (long long)d, tag);
        }
      }
      __syncwarp();
      if (lane == 0) ring_bar_arrive(&empty[st]);
    }
  }
}

// One-row fields: segments of one stage each.
template <int KIND, typename Entry>
__global__ void __launch_bounds__(kRingConsumers + 32, 2)
wb_diff2_ring_row_kernel(const void* __restrict__ field, unsigned long long cols, Entry* __restrict__ out,
                         unsigned long long cap, unsigned long long* __restrict__ count, unsigned tag) {
  constexpr int ES = FieldElem<KIND>::kBytes, NE = RingElems<KIND>::kNE;
  constexpr unsigned long long kSegBytes = (unsigned long long)kRingRows * kRingRowBytes;   // 32 KiB of the row per stage
  extern __shared__ __align__(128) char ring_smem_buf[];
  __shared__ __align__(8) unsigned long long full[kRingStages], empty[kRingStages];
  if (threadIdx.x == 0) {
    for (int k = 0; k < kRingStages; ++k) { ring_bar_init(&full[k], 1); ring_bar_init(&empty[k], kRingConsumers / 32); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const unsigned long long total = cols * ES, n_seg = (total + kSegBytes - 1) / kSegBytes;
  if (threadIdx.x >= kRingConsumers) {
    if (threadIdx.x != kRingConsumers) return;
    unsigned n = 0;
    for (unsigned long long sg = blockIdx.x; sg < n_seg; sg += gridDim.x, ++n) {
      const unsigned long long b0 = sg * kSegBytes;
      const unsigned bytes = (unsigned)(total - b0 < kSegBytes ? total - b0 : kSegBytes);
      const unsigned halo = sg ? 16u : 0u;
      const unsigned st = n % kRingStages;
      if (n >= (unsigned)kRingStages && !ring_bar_wait(&empty[st], ((n / kRingStages) - 1) & 1)) { atomicMax(count, kRingFailed); return; }
      ring_bar_expect(&full[st], bytes + halo);
      // the segment lands 16 bytes into the stage; its left halo, when there is one, right before it
      ring_bulk_load(ring_smem_buf + (size_t)st * kRingStageBytes + 16 - halo, static_cast<const char*>(field) + b0 - halo,
                     bytes + halo, &full[st]);
    }
    return;
  }
  const unsigned t = threadIdx.x, lane = t & 31;
  unsigned n = 0;
  for (unsigned long long sg = blockIdx.x; sg < n_seg; sg += gridDim.x, ++n) {
    const unsigned long long b0 = sg * kSegBytes;
    const unsigned bytes = (unsigned)(total - b0 < kSegBytes ? total - b0 : kSegBytes);
    const unsigned st = n % kRingStages;
    unsigned ok = 1;
    if (lane == 0) ok = ring_bar_wait(&full[st], (n / kRingStages) & 1);
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    if (!ok) { if (t == 0) atomicMax(count, kRingFailed); return; }
    const char* data = ring_smem_buf + (size_t)st * kRingStageBytes + 16;
    for (unsigned off = t * 16; off < bytes; off += kRingConsumers * 16) {
      using V = typename RingElems<KIND>::V;
      V x[NE], p[NE];
      ring_unpack<KIND>(*reinterpret_cast<const uint4*>(data + off), x);
#pragma unroll
      for (int q = 0; q < NE; ++q) p[q] = 0;
      if (b0 + off >= 16) ring_unpack<KIND>(*reinterpret_cast<const uint4*>(data + off - 16), p);
      const unsigned long long j0 = (b0 + off) / ES;
#pragma unroll
      for (int q = 0; q < NE; ++q) {
        const V a1 = q >= 1 ? x[q - 1] : p[NE - 1], a2 = q >= 2 ? x[q - 2] : p[NE - 2 + q];
        const V d = x[q] - 2 * a1 + a2;
        if (d != 0) ring_emit(out, cap, count, 0, j0 + q, (long long)d, tag);
      }
    }
    __syncwarp();
    if (lane == 0) ring_bar_arrive(&empty[st]);
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
  // Large fields whose rows start on 16-byte boundaries go through the bulk-copy ring.
  {
    const unsigned es = id_kind == WB_ID_I64 ? 8u : (id_kind == WB_ID_F32 ? 4u : 2u);
    const bool aligned = ((uintptr_t)field & 15u) == 0 && (cols * es) % 16 == 0;
    if (aligned && rows * cols * es >= (4ull << 20) && (rows == 1 || cols * es >= 2048)) {
      const size_t dyn = (size_t)kRingStages * kRingStageBytes;
      const unsigned blocks = 148 * 2;
      cudaError_t e = cudaSuccess;
      if (rows == 1) {
        const unsigned long long n_seg = (cols * es + (unsigned long long)kRingRows * kRingRowBytes - 1) / ((unsigned long long)kRingRows * kRingRowBytes);
        const unsigned grid = (unsigned)(n_seg < blocks ? n_seg : blocks);
#define WB_RING_ROW(KIND)                                                                                                 \
  do {                                                                                                                    \
    e = cudaFuncSetAttribute(wb_diff2_ring_row_kernel<KIND, Entry>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); \
    if (e == cudaSuccess) wb_diff2_ring_row_kernel<KIND, Entry><<<grid, kRingConsumers + 32, dyn, stream>>>(field, cols, out, cap, cnt, tag); \
  } while (0)
        switch (id_kind) {
          case WB_ID_I64: WB_RING_ROW(WB_ID_I64); break;
          case WB_ID_U16: WB_RING_ROW(WB_ID_U16); break;
          case WB_ID_F32: WB_RING_ROW(WB_ID_F32); break;
          default: WB_RING_ROW(WB_ID_BF16); break;
        }
#undef WB_RING_ROW
      } else {
        // units of one strip x rows_per_unit rows, about eight per block; two extra rows per unit prime the
        // vertical difference
        const unsigned long long strips = (cols * es + kRingStripBytes - 1) / kRingStripBytes;
        unsigned long long row_units = (blocks * 8ull + strips - 1) / strips;
        if (row_units > (rows + 63) / 64) row_units = (rows + 63) / 64;       // at least 64 rows per unit
        if (row_units < 1) row_units = 1;
        const unsigned long long rpu = (rows + row_units - 1) / row_units;
        const unsigned long long n_units = strips * ((rows + rpu - 1) / rpu);
        const unsigned grid = (unsigned)(n_units < blocks ? n_units : blocks);
#define WB_RING_2D(KIND)                                                                                                  \
  do {                                                                                                                    \
    e = cudaFuncSetAttribute(wb_diff2_ring_kernel<KIND, Entry>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);   \
    if (e == cudaSuccess) wb_diff2_ring_kernel<KIND, Entry><<<grid, kRingConsumers + 32, dyn, stream>>>(field, rows, cols, rpu, out, cap, cnt, tag); \
  } while (0)
        switch (id_kind) {
          case WB_ID_I64: WB_RING_2D(WB_ID_I64); break;
          case WB_ID_U16: WB_RING_2D(WB_ID_U16); break;
          case WB_ID_F32: WB_RING_2D(WB_ID_F32); break;
          default: WB_RING_2D(WB_ID_BF16); break;
        }
#undef WB_RING_2D
      }
      return e != cudaSuccess ? e : cudaGetLastError();
    }
  }
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

// =================================================================================================
// Chunk passes with carries (Algorithm 1, inner loop; Appendix B, "Difference encoding", last two
// paragraphs).  The paper sketches this step only; the construction built here:
//
//   ids = sum_k 2^(bk) A_k, so diff2(ids) = sum_k 2^(bk) diff2(A_k) is evaluated like a multi-digit
//   addition, least significant chunk first.  Pass k forms D = diff2(A_k) + Gamma, Gamma the carry out
//   of pass k-1, and splits it (EmitCarry) into the balanced b-bit digit Z in [-2^(b-1), 2^(b-1)) and
//   the carry C = (D - Z) / 2^b.  Z is zero wherever diff2(ids) is, so NonZeros(Z) has O(N_c) entries.
//   C is non-zero wherever chunk k wraps, every s = 2^(b(k+1)) consecutive ids of a run; it goes to
//   the host as NonZeros(StridedDiff1(C)),
//       G[x] = C[x] - C[x - s] - C[x - s cols] + C[x - s - s cols]     (x = i cols + j, C = 0 before the tensor),
//   Eq. diff1 with the left neighbour s elements back in flat order and the upper neighbour s rows up,
//   which cancels the periodic pattern.  ExpandCarry inverts it on the device before the next pass:
//   the records are scattered into a zeroed one-byte-per-element field, then summed over every s-th
//   element of the flat order and over every s-th row.
//
// The carry field of the tensor lives in caller-provided scratch (one byte per element: |C| <= 17),
// is overwritten in place by the pass (D at x needs Gamma at x only) and differenced by a last kernel.
// =================================================================================================
namespace {

constexpr unsigned kCarryBlocks = 148 * 8;
constexpr unsigned long long kCarryAuxEntries = 1ull << 16;        // partial column sums of the strided prefix

__global__ void wb_carry_scatter_kernel(const wb_diff2_entry* __restrict__ rec, unsigned long long n_rec,
                                        unsigned long long rows, unsigned long long cols, signed char* __restrict__ y) {
  for (unsigned long long k = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; k < n_rec;
       k += (unsigned long long)gridDim.x * blockDim.x) {
    const wb_diff2_entry e = rec[k];
    if (e.row < rows && e.col < cols) y[e.row * cols + e.col] = (signed char)e.value;
  }
}

// y[x] += y[x - t] for all x, as the column-wise running sum of the [H, t] row-major view of y.  The H
// rows are cut into nblk blocks of hb rows; a thread owns four adjacent columns (one 32-bit word) of
// one block.  phase 0: block sums -> part; phase 1 (one block of rows only needs phase 2): exclusive
// scan of part over the blocks; phase 2: running sums written back, starting from the scanned offset.
// t is a multiple of 4 and y is padded to a multiple of 4 bytes.
__device__ __forceinline__ void add4(int (&acc)[4], unsigned w) {
  acc[0] += (signed char)(w & 0xFF); acc[1] += (signed char)((w >> 8) & 0xFF);
  acc[2] += (signed char)((w >> 16) & 0xFF); acc[3] += (signed char)(w >> 24);
}
__global__ void wb_strided_prefix_kernel(signed char* __restrict__ y, unsigned long long n4, unsigned long long t,
                                         unsigned long long H, unsigned long long hb, unsigned long long nblk,
                                         int* __restrict__ part, int phase) {
  const unsigned long long tw = t / 4;                         // words per row of the view
  const unsigned long long total = phase == 1 ? tw : nblk * tw;
  for (unsigned long long id = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; id < total;
       id += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned long long blk = phase == 1 ? 0 : id / tw, w = id - blk * tw;
    if (phase == 1) {
      int run[4] = {0, 0, 0, 0};
      for (unsigned long long b = 0; b < nblk; ++b) {
        int4* p = reinterpret_cast<int4*>(part) + b * tw + w;
        const int4 v = *p;
        *p = make_int4(run[0], run[1], run[2], run[3]);
        run[0] += v.x; run[1] += v.y; run[2] += v.z; run[3] += v.w;
      }
      continue;
    }
    int acc[4] = {0, 0, 0, 0};
    if (phase == 2 && nblk > 1) {
      const int4 v = reinterpret_cast<const int4*>(part)[blk * tw + w];
      acc[0] = v.x; acc[1] = v.y; acc[2] = v.z; acc[3] = v.w;
    }
    const unsigned long long h0 = blk * hb, h1 = h0 + hb < H ? h0 + hb : H;
    for (unsigned long long h = h0; h < h1; ++h) {
      const unsigned long long x = h * t + 4 * w;
      if (x >= n4) break;
      unsigned* p = reinterpret_cast<unsigned*>(y + x);
      add4(acc, *p);
      if (phase == 2)
        *p = (unsigned)(acc[0] & 0xFF) | ((unsigned)(acc[1] & 0xFF) << 8) | ((unsigned)(acc[2] & 0xFF) << 16) |
             ((unsigned)(acc[3] & 0xFF) << 24);
    }
    if (phase == 0) reinterpret_cast<int4*>(part)[blk * tw + w] = make_int4(acc[0], acc[1], acc[2], acc[3]);
  }
}

// Gamma at one element from the sorted carry records (see wb_carry_sort_kernel): ExpandCarry in closed
// form.  C = prefix over every s-th element of the flat order, then over every s-th row, of G, so a record
// (x_r, g) reaches x when x - x_r = m s with m >= 0, once for every split m = a + c cols (a, c >= 0) if the
// row stride applies, i.e. floor(m / cols) + 1 times, else once.
struct CarryRec { unsigned long long x; long long g; };
struct CarryIndex {
  const unsigned* first;          // 257 offsets into rec, by x mod 256
  const unsigned char* has;       // 32 bytes: bit r set if some record has x mod 256 == r
  const CarryRec* rec;
  unsigned long long s, cols;
  unsigned s_shift;
  int use_up;
};
__device__ __forceinline__ int gamma_at(const CarryIndex& ci, unsigned long long x) {
  const unsigned r = (unsigned)x & 255u;
  int acc = 0;
  for (unsigned k = __ldg(ci.first + r), e = __ldg(ci.first + r + 1); k < e; ++k) {
    const unsigned long long xr = __ldg(&ci.rec[k].x);
    if (x < xr || ((x - xr) & (ci.s - 1)) != 0) continue;
    const unsigned long long m = (x - xr) >> ci.s_shift;
    const long long mult = ci.use_up ? (long long)(m / ci.cols) + 1 : 1;
    acc += (int)(__ldg(&ci.rec[k].g) * mult);
  }
  return acc;
}

// Sort the carry records by x mod 256 (one block): counts, offsets, placement.
__global__ void __launch_bounds__(256)
wb_carry_sort_kernel(const wb_diff2_entry* __restrict__ rec, unsigned n_rec, unsigned long long cols,
                     unsigned* __restrict__ first, unsigned char* __restrict__ has, CarryRec* __restrict__ sorted) {
  __shared__ unsigned bin[257], cur[256];
  bin[threadIdx.x] = 0;
  if (threadIdx.x == 0) bin[256] = 0;
  __syncthreads();
  for (unsigned k = threadIdx.x; k < n_rec; k += 256) atomicAdd(&bin[(unsigned)(rec[k].row * cols + rec[k].col) & 255u], 1u);
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned run = 0;
    for (int r = 0; r < 256; ++r) { const unsigned c = bin[r]; bin[r] = run; run += c; }
    bin[256] = run;
  }
  __syncthreads();
  cur[threadIdx.x] = bin[threadIdx.x];
  first[threadIdx.x] = bin[threadIdx.x];
  if (threadIdx.x == 0) first[256] = bin[256];
  if (threadIdx.x < 32) {
    unsigned char m = 0;
    for (int q = 0; q < 8; ++q) m |= (unsigned char)((bin[threadIdx.x * 8 + q + 1] > bin[threadIdx.x * 8 + q]) << q);
    has[threadIdx.x] = m;
  }
  __syncthreads();
  for (unsigned k = threadIdx.x; k < n_rec; k += 256) {
    const unsigned long long x = rec[k].row * cols + rec[k].col;
    sorted[atomicAdd(&cur[(unsigned)x & 255u], 1u)] = CarryRec{x, rec[k].value};
  }
}

// Eight adjacent elements / the two elements before them, as integers (chunk values are below 2^16).
template <int KIND> __device__ __forceinline__ void load8(const void* f, unsigned long long idx, int (&x)[8]);
template <> __device__ __forceinline__ void load8<WB_ID_U16>(const void* f, unsigned long long idx, int (&x)[8]) {
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(static_cast<const unsigned short*>(f) + idx));
  x[0] = a.x & 0xFFFF; x[1] = a.x >> 16; x[2] = a.y & 0xFFFF; x[3] = a.y >> 16;
  x[4] = a.z & 0xFFFF; x[5] = a.z >> 16; x[6] = a.w & 0xFFFF; x[7] = a.w >> 16;
}
__device__ __forceinline__ int bf16_bits_to_int(unsigned b) { return __float2int_rn(__uint_as_float(b << 16)); }
template <> __device__ __forceinline__ void load8<WB_ID_BF16>(const void* f, unsigned long long idx, int (&x)[8]) {
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(static_cast<const unsigned short*>(f) + idx));
  x[0] = bf16_bits_to_int(a.x & 0xFFFF); x[1] = bf16_bits_to_int(a.x >> 16);
  x[2] = bf16_bits_to_int(a.y & 0xFFFF); x[3] = bf16_bits_to_int(a.y >> 16);
  x[4] = bf16_bits_to_int(a.z & 0xFFFF); x[5] = bf16_bits_to_int(a.z >> 16);
  x[6] = bf16_bits_to_int(a.w & 0xFFFF); x[7] = bf16_bits_to_int(a.w >> 16);
}
template <> __device__ __forceinline__ void load8<WB_ID_F32>(const void* f, unsigned long long idx, int (&x)[8]) {
  const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(f) + idx);
  const float4 a = __ldg(p), b = __ldg(p + 1);
  x[0] = __float2int_rn(a.x); x[1] = __float2int_rn(a.y); x[2] = __float2int_rn(a.z); x[3] = __float2int_rn(a.w);
  x[4] = __float2int_rn(b.x); x[5] = __float2int_rn(b.y); x[6] = __float2int_rn(b.z); x[7] = __float2int_rn(b.w);
}
template <> __device__ __forceinline__ void load8<WB_ID_I64>(const void* f, unsigned long long idx, int (&x)[8]) {
  const longlong2* p = reinterpret_cast<const longlong2*>(static_cast<const long long*>(f) + idx);
#pragma unroll
  for (int q = 0; q < 4; ++q) { const longlong2 a = __ldg(p + q); x[2 * q] = (int)a.x; x[2 * q + 1] = (int)a.y; }
}

// The pass proper, one element (any shape, any alignment): D = diff2(A)(i, j) + Gamma[x]; digit and carry;
// the carry goes to carry[x]; a non-zero digit is appended to the list.
// mode 0: no carry-in; 1: Gamma from the sorted records; 2: Gamma expanded in carry[] beforehand.
template <int KIND>
__device__ __forceinline__ void chunk_elem(const void* __restrict__ field, unsigned long long cols, unsigned b, int mode,
                                           const CarryIndex& ci, signed char* __restrict__ carry, unsigned long long x,
                                           wb_diff2_entry* __restrict__ out, unsigned long long cap,
                                           unsigned long long* __restrict__ count) {
  const unsigned long long i = x / cols, j = x - i * cols;
  long long v[3];
#pragma unroll
  for (int dj = 0; dj < 3; ++dj) {
    v[dj] = 0;
    if (j >= (unsigned)dj) {
      const unsigned long long at = x - dj;
      v[dj] = field_at<KIND>(field, at);
      if (i >= 1) v[dj] -= 2 * field_at<KIND>(field, at - cols);
      if (i >= 2) v[dj] += field_at<KIND>(field, at - 2 * cols);
    }
  }
  long long d = v[0] - 2 * v[1] + v[2];
  if (mode == 1) d += gamma_at(ci, x);
  else if (mode == 2) d += carry[x];
  const long long half = 1ll << (b - 1), mask = (1ll << b) - 1;
  const long long z = ((d + half) & mask) - half;
  carry[x] = (signed char)((d - z) >> b);
  if (z != 0) {
    const unsigned long long slot = atomicAdd(count, 1ull);
    if (slot < cap) out[slot] = wb_diff2_entry{i, j, z};
  }
}

template <int KIND>
__global__ void __launch_bounds__(256)
wb_chunk_pass_kernel(const void* __restrict__ field, unsigned long long rows, unsigned long long cols, unsigned b,
                     int mode, CarryIndex ci, signed char* __restrict__ carry, wb_diff2_entry* __restrict__ out,
                     unsigned long long cap, unsigned long long* __restrict__ count) {
  const unsigned long long n = rows * cols;
  for (unsigned long long x = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; x < n;
       x += (unsigned long long)gridDim.x * blockDim.x)
    chunk_elem<KIND>(field, cols, b, mode, ci, carry, x, out, cap, count);
}

// The same for fields whose rows start on vector boundaries (cols a multiple of 8, or a single row; base
// 16-byte aligned): a thread takes eight adjacent elements of one row with vector loads of the rows
// i, i-1, i-2 (the rows above were read shortly before by other threads and come from L2) and the two
// elements left of them, computes in 32-bit integers, and stores the eight carries as one 8-byte word.
template <int KIND>
__global__ void __launch_bounds__(256)
wb_chunk_pass8_kernel(const void* __restrict__ field, unsigned long long rows, unsigned long long cols, unsigned b,
                      int mode, CarryIndex ci, signed char* __restrict__ carry, wb_diff2_entry* __restrict__ out,
                      unsigned long long cap, unsigned long long* __restrict__ count) {
  const unsigned long long n = rows * cols, n8 = (n + 7) / 8;
  const int half = 1 << (b - 1), mask = (1 << b) - 1;
  for (unsigned long long q = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; q < n8;
       q += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned long long x0 = q * 8;
    if (x0 + 8 > n) {                                           // ragged end of a single-row field
      for (unsigned long long x = x0; x < n; ++x) chunk_elem<KIND>(field, cols, b, mode, ci, carry, x, out, cap, count);
      continue;
    }
    const unsigned long long i = rows == 1 ? 0ull : x0 / cols, j0 = x0 - i * cols;
    int v[8], l[2] = {0, 0};                                    // vertical second differences; l = columns j0-2, j0-1
    load8<KIND>(field, x0, v);
    if (j0) { l[0] = (int)field_at<KIND>(field, x0 - 2); l[1] = (int)field_at<KIND>(field, x0 - 1); }
    if (i >= 1) {
      int u[8];
      load8<KIND>(field, x0 - cols, u);
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] -= 2 * u[k];
      if (j0) { l[0] -= 2 * (int)field_at<KIND>(field, x0 - cols - 2); l[1] -= 2 * (int)field_at<KIND>(field, x0 - cols - 1); }
    }
    if (i >= 2) {
      int u[8];
      load8<KIND>(field, x0 - 2 * cols, u);
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] += u[k];
      if (j0) { l[0] += (int)field_at<KIND>(field, x0 - 2 * cols - 2); l[1] += (int)field_at<KIND>(field, x0 - 2 * cols - 1); }
    }
    int d[8];
    d[0] = v[0] - 2 * l[1] + l[0];
    d[1] = v[1] - 2 * v[0] + l[1];
#pragma unroll
    for (int k = 2; k < 8; ++k) d[k] = v[k] - 2 * v[k - 1] + v[k - 2];
    if (mode == 1) {
      const unsigned bits = __ldg(ci.has + ((x0 >> 3) & 31u));
      if (bits) {
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (bits >> k & 1u) d[k] += gamma_at(ci, x0 + k);
      }
    } else if (mode == 2) {
      const uint2 g = *reinterpret_cast<const uint2*>(carry + x0);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        d[k] += (signed char)((g.x >> (8 * k)) & 0xFF);
        d[4 + k] += (signed char)((g.y >> (8 * k)) & 0xFF);
      }
    }
    unsigned lo = 0, hi = 0;
    bool any = false;
    int z[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      z[k] = ((d[k] + half) & mask) - half;
      const unsigned c = (unsigned)((d[k] - z[k]) >> b) & 0xFFu;
      if (k < 4) lo |= c << (8 * k); else hi |= c << (8 * (k - 4));
      any |= z[k] != 0;
    }
    *reinterpret_cast<uint2*>(carry + x0) = make_uint2(lo, hi);
    if (any) {
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (z[k] != 0) {
          const unsigned long long slot = atomicAdd(count, 1ull);
          if (slot < cap) out[slot] = wb_diff2_entry{i, j0 + k, (long long)z[k]};
        }
    }
  }
}

// One-row fields (flat shards): a thread takes sixteen adjacent elements, two 16-byte-per-eight loads in flight
// plus the two elements before them, and stores the sixteen carries as one 16-byte word.
template <int KIND>
__global__ void __launch_bounds__(256)
wb_chunk_row16_kernel(const void* __restrict__ field, unsigned long long n, unsigned b, int mode, CarryIndex ci,
                      signed char* __restrict__ carry, wb_diff2_entry* __restrict__ out, unsigned long long cap,
                      unsigned long long* __restrict__ count) {
  const unsigned long long n16 = (n + 15) / 16;
  const int half = 1 << (b - 1), mask = (1 << b) - 1;
  for (unsigned long long q = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; q < n16;
       q += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned long long x0 = q * 16;
    if (x0 + 16 > n) {                                          // ragged end
      for (unsigned long long x = x0; x < n; ++x) chunk_elem<KIND>(field, n, b, mode, ci, carry, x, out, cap, count);
      continue;
    }
    int v[18];                                                  // v[0], v[1]: the two elements before the group
    load8<KIND>(field, x0, reinterpret_cast<int(&)[8]>(v[2]));
    load8<KIND>(field, x0 + 8, reinterpret_cast<int(&)[8]>(v[10]));
    v[0] = v[1] = 0;
    if (x0) { v[0] = (int)field_at<KIND>(field, x0 - 2); v[1] = (int)field_at<KIND>(field, x0 - 1); }
    int d[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) d[k] = v[k + 2] - 2 * v[k + 1] + v[k];
    if (mode == 1) {
      const unsigned bits = (unsigned)__ldg(ci.has + ((x0 >> 3) & 31u)) | ((unsigned)__ldg(ci.has + (((x0 >> 3) + 1) & 31u)) << 8);
      if (bits) {
#pragma unroll
        for (int k = 0; k < 16; ++k)
          if (bits >> k & 1u) d[k] += gamma_at(ci, x0 + k);
      }
    } else if (mode == 2) {
      const uint4 g = *reinterpret_cast<const uint4*>(carry + x0);
      const unsigned w[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
      for (int k = 0; k < 16; ++k) d[k] += (signed char)((w[k >> 2] >> (8 * (k & 3))) & 0xFF);
    }
    unsigned c[4] = {0, 0, 0, 0};
    unsigned nzmask = 0;
    int z[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      z[k] = ((d[k] + half) & mask) - half;
      c[k >> 2] |= ((unsigned)((d[k] - z[k]) >> b) & 0xFFu) << (8 * (k & 3));
      nzmask |= (unsigned)(z[k] != 0) << k;
    }
    *reinterpret_cast<uint4*>(carry + x0) = make_uint4(c[0], c[1], c[2], c[3]);
    if (nzmask) {
#pragma unroll
      for (int k = 0; k < 16; ++k)
        if (nzmask >> k & 1u) {
          const unsigned long long slot = atomicAdd(count, 1ull);
          if (slot < cap) out[slot] = wb_diff2_entry{0, x0 + k, (long long)z[k]};
        }
    }
  }
}

// NonZeros(StridedDiff1(C)) for the carry field C (one byte per element, padded to a multiple of 16 bytes):
// a thread takes sixteen adjacent elements, two such groups per step; s and s cols are multiples of 16, so the
// neighbours are aligned 16-byte words.
__device__ __forceinline__ void sub16(int (&g)[16], uint4 w, int sign) {
  const unsigned v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int p = 0; p < 4; ++p)
#pragma unroll
    for (int k = 0; k < 4; ++k) g[4 * p + k] += sign * (signed char)((v[p] >> (8 * k)) & 0xFF);
}
__global__ void __launch_bounds__(256)
wb_strided_diff_kernel(const signed char* __restrict__ c, unsigned long long n, unsigned long long cols,
                       unsigned long long s, unsigned long long up, int use_s, int use_up,
                       wb_diff2_entry* __restrict__ out, unsigned long long cap, unsigned long long* __restrict__ count) {
  const unsigned long long n16 = (n + 15) / 16, stride = (unsigned long long)gridDim.x * blockDim.x;
  const uint4 zero = make_uint4(0, 0, 0, 0);
  for (unsigned long long q0 = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; q0 < n16; q0 += 2 * stride) {
    uint4 w[2][4];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const unsigned long long q = q0 + u * stride, x0 = q * 16;
      const bool in = q < n16;
      w[u][0] = in ? *reinterpret_cast<const uint4*>(c + x0) : zero;
      w[u][1] = in && use_s && x0 >= s ? *reinterpret_cast<const uint4*>(c + x0 - s) : zero;
      w[u][2] = in && use_up && x0 >= up ? *reinterpret_cast<const uint4*>(c + x0 - up) : zero;
      w[u][3] = in && use_s && use_up && x0 >= s + up ? *reinterpret_cast<const uint4*>(c + x0 - s - up) : zero;
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const unsigned long long x0 = (q0 + u * stride) * 16;
      // all four words zero: nothing to do (almost every group)
      const unsigned any = w[u][0].x | w[u][0].y | w[u][0].z | w[u][0].w | w[u][1].x | w[u][1].y | w[u][1].z | w[u][1].w |
                           w[u][2].x | w[u][2].y | w[u][2].z | w[u][2].w | w[u][3].x | w[u][3].y | w[u][3].z | w[u][3].w;
      if (!any) continue;
      int g[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) g[k] = 0;
      sub16(g, w[u][0], 1); sub16(g, w[u][1], -1); sub16(g, w[u][2], -1); sub16(g, w[u][3], 1);
#pragma unroll
      for (int k = 0; k < 16; ++k)
        if (g[k] != 0 && x0 + k < n) {
          const unsigned long long slot = atomicAdd(count, 1ull);
          if (slot < cap) out[slot] = wb_diff2_entry{(x0 + k) / cols, (x0 + k) % cols, (long long)g[k]};
        }
    }
  }
}

// 2^(b(k+1)) or "beyond any field" (bit 62) when that does not fit
inline unsigned long long carry_stride(unsigned b, unsigned k) {
  const unsigned long long sh = (unsigned long long)b * (k + 1);
  return sh >= 62 ? (1ull << 62) : (1ull << sh);
}

cudaError_t strided_prefix(signed char* y, unsigned long long n4, unsigned long long t, int* part, cudaStream_t stream) {
  if (t >= n4) return cudaSuccess;
  const unsigned long long H = (n4 + t - 1) / t, tw = t / 4;
  unsigned long long nblk = kCarryAuxEntries / t;               // so that nblk * t entries fit the partial sums
  if (nblk < 1) nblk = 1;
  if (nblk > H) nblk = H;
  const unsigned long long hb = (H + nblk - 1) / nblk;
  nblk = (H + hb - 1) / hb;
  const unsigned long long work = nblk * tw;
  const unsigned grid = (unsigned)((work + 255) / 256 < kCarryBlocks ? (work + 255) / 256 : kCarryBlocks);
  if (nblk > 1) {
    wb_strided_prefix_kernel<<<grid, 256, 0, stream>>>(y, n4, t, H, hb, nblk, part, 0);
    wb_strided_prefix_kernel<<<(unsigned)((tw + 255) / 256 < kCarryBlocks ? (tw + 255) / 256 : kCarryBlocks), 256, 0, stream>>>(
        y, n4, t, H, hb, nblk, part, 1);
  }
  wb_strided_prefix_kernel<<<grid, 256, 0, stream>>>(y, n4, t, H, hb, nblk, part, 2);
  return cudaGetLastError();
}

}  // namespace

extern "C" size_t wb_diff2_chunk_scratch_bytes(uint64_t rows, uint64_t cols) {
  const unsigned long long n16 = (rows * cols + 15) / 16 * 16;
  return (size_t)(n16 + kCarryAuxEntries * sizeof(int));
}

extern "C" wb_status wb_diff2_chunk_pass(const void* field, uint32_t id_kind, uint64_t rows, uint64_t cols,
                                         uint32_t chunk_bits, uint32_t pass, const wb_diff2_entry* carry_in,
                                         uint64_t n_carry_in, void* scratch, size_t scratch_bytes, wb_diff2_entry* z_out,
                                         uint64_t z_cap, uint64_t* z_count, wb_diff2_entry* carry_out, uint64_t carry_cap,
                                         uint64_t* carry_count, void* cuda_stream) {
  if (!field || !scratch || !z_count || !carry_count || (!z_out && z_cap) || (!carry_out && carry_cap)) return WB_ERR_INVALID_ARG;
  if (id_kind > WB_ID_BF16 || (chunk_bits != 8 && chunk_bits != 16) || pass >= 8) return WB_ERR_INVALID_ARG;
  if ((n_carry_in && !carry_in) || (pass == 0 && n_carry_in) || ((uintptr_t)scratch & 15u)) return WB_ERR_INVALID_ARG;
  if (rows == 0 || cols == 0) return WB_OK;
  if (!field_size_ok(rows, cols) || rows * cols > (1ull << 40)) return WB_ERR_INVALID_ARG;
  if (scratch_bytes < wb_diff2_chunk_scratch_bytes(rows, cols)) return WB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const unsigned long long n = rows * cols, n16 = (n + 15) / 16 * 16;
  signed char* carry = static_cast<signed char*>(scratch);
  int* part = reinterpret_cast<int*>(carry + n16);
  auto* zc = reinterpret_cast<unsigned long long*>(z_count);
  auto* cc = reinterpret_cast<unsigned long long*>(carry_count);
  // ExpandCarry(H_Gamma[pass - 1]): a short record list is sorted and evaluated in closed form inside the
  // pass (mode 1); a long one is expanded into the scratch field first (mode 2)
  constexpr unsigned long long kSparseMax = (kCarryAuxEntries * sizeof(int) - 2048) / sizeof(CarryRec);
  const unsigned long long s_in = pass ? carry_stride(chunk_bits, pass - 1) : 0;
  const int mode = n_carry_in == 0 ? 0 : (n_carry_in <= kSparseMax ? 1 : 2);
  CarryIndex ci{};
  if (mode == 1) {
    unsigned* first = reinterpret_cast<unsigned*>(part);
    unsigned char* has = reinterpret_cast<unsigned char*>(part) + 1536;
    CarryRec* sorted = reinterpret_cast<CarryRec*>(reinterpret_cast<char*>(part) + 2048);
    wb_carry_sort_kernel<<<1, 256, 0, stream>>>(carry_in, (unsigned)n_carry_in, cols, first, has, sorted);
    if (cudaGetLastError() != cudaSuccess) return WB_ERR_CUDA;
    ci.first = first; ci.has = has; ci.rec = sorted;
    ci.s = s_in; ci.cols = cols; ci.use_up = s_in < rows;
    ci.s_shift = chunk_bits * pass < 62u ? chunk_bits * pass : 62u;      // matches carry_stride
  } else if (mode == 2) {
    if (cudaMemsetAsync(carry, 0, n16, stream) != cudaSuccess) return WB_ERR_CUDA;
    const unsigned g = (unsigned)((n_carry_in + 255) / 256 < kCarryBlocks ? (n_carry_in + 255) / 256 : kCarryBlocks);
    wb_carry_scatter_kernel<<<g, 256, 0, stream>>>(carry_in, n_carry_in, rows, cols, carry);
    if (cudaGetLastError() != cudaSuccess) return WB_ERR_CUDA;
    if (strided_prefix(carry, n16, s_in, part, stream) != cudaSuccess) return WB_ERR_CUDA;
    if (s_in < rows && strided_prefix(carry, n16, s_in * cols, part, stream) != cudaSuccess) return WB_ERR_CUDA;
  }
  const bool vec = ((uintptr_t)field % 16u) == 0 && (rows == 1 || cols % 8 == 0);
  const unsigned long long work = vec ? (rows == 1 ? (n + 15) / 16 : (n + 7) / 8) : n;
  const unsigned grid = (unsigned)((work + 255) / 256 < kCarryBlocks ? (work + 255) / 256 : kCarryBlocks);
#define WB_CHUNK_LAUNCH(KIND)                                                                                        \
  do {                                                                                                               \
    if (vec && rows == 1) wb_chunk_row16_kernel<KIND><<<grid, 256, 0, stream>>>(field, n, chunk_bits, mode, ci, carry, z_out, z_cap, zc); \
    else if (vec) wb_chunk_pass8_kernel<KIND><<<grid, 256, 0, stream>>>(field, rows, cols, chunk_bits, mode, ci, carry, z_out, z_cap, zc); \
    else wb_chunk_pass_kernel<KIND><<<grid, 256, 0, stream>>>(field, rows, cols, chunk_bits, mode, ci, carry, z_out, z_cap, zc);      \
  } while (0)
  switch (id_kind) {
    case WB_ID_I64: WB_CHUNK_LAUNCH(WB_ID_I64); break;
    case WB_ID_U16: WB_CHUNK_LAUNCH(WB_ID_U16); break;
    case WB_ID_F32: WB_CHUNK_LAUNCH(WB_ID_F32); break;
    default: WB_CHUNK_LAUNCH(WB_ID_BF16); break;
  }
#undef WB_CHUNK_LAUNCH
  if (cudaGetLastError() != cudaSuccess) return WB_ERR_CUDA;
  const unsigned long long s_out = carry_stride(chunk_bits, pass);
  const unsigned long long sd_blocks = ((n + 15) / 16 + 511) / 512;             // two groups of 16 per thread and step
  const unsigned grid8 = (unsigned)(sd_blocks < kCarryBlocks ? (sd_blocks ? sd_blocks : 1) : kCarryBlocks);
  wb_strided_diff_kernel<<<grid8, 256, 0, stream>>>(carry, n, cols, s_out, s_out < rows ? s_out * cols : 0, s_out < n,
                                                   s_out < rows, carry_out, carry_cap, cc);
  return cudaGetLastError() == cudaSuccess ? WB_OK : WB_ERR_CUDA;
}
