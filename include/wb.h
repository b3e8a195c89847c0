/*
 * wb.h -- C ABI of the B200 weight-remap library.
 *
 * The library moves every model parameter element from a trainer's sharded layout into a
 * rollout (inference) engine's layout, casting on the way, without reading any source
 * element twice.  It follows the weight-transfer method of the WeightBridge paper:
 *
 *   - Section 3.1: each side's layout is a *source map*, a list of slice-copy operations
 *     (optionally transposed) that say which checkpoint elements a worker's local tensors
 *     hold.  Two local elements correspond iff the same checkpoint element supplies both.
 *   - Section 3.2: a planner turns the correspondence into a non-redundant plan
 *     (replicas on the trainer side each send a distinct slice; replicas on the rollout
 *     side are fed from one copy), splits the model into roughly equal rounds that fit a
 *     transfer-buffer budget, and an executor runs the plan every iteration with one
 *     batched packing kernel (trainer side) and one batched assembly kernel (rollout side)
 *     per round.
 *
 * Here all virtual trainer and rollout ranks are regions of ONE GPU's memory, so the wire
 * between packing and assembly is a device buffer ("bucket"), and a fused path
 * (wb_remap) goes from trainer tensors to rollout tensors directly.
 *
 * Conventions
 *   - Every function returns a wb_status and never throws or aborts.  On error the
 *     out-parameters are left untouched and nothing is launched.
 *   - "host" / "device" is stated for every pointer.  The caller owns all weight memory,
 *     all buckets and the CUDA stream; layouts and plans are opaque, owned by the library
 *     and released with their _free function.
 *   - A plan is immutable after wb_plan_bind and is reused for every model version
 *     (Section 3: the plan is computed once, in `connect`, and executed per update).
 *   - wb_pack / wb_unpack / wb_remap are asynchronous on the given stream, allocate
 *     nothing and copy nothing between host and device.
 *   - Local-tensor elements that no slice describes (e.g. FSDP padding) are never read on
 *     the source side and never written on the destination side.
 *   - Replicated source elements are assumed bit-identical.
 */
#ifndef WB_H_
#define WB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  WB_OK = 0,
  WB_ERR_INVALID_ARG = 1,      /* NULL pointer, bad index, unsupported strides              */
  WB_ERR_DTYPE = 2,            /* unknown dtype, or mixed dtypes on one side                 */
  WB_ERR_SHAPE_MISMATCH = 3,   /* one checkpoint tensor described with two different shapes  */
  WB_ERR_OUT_OF_RANGE = 4,     /* a slice leaves its checkpoint tensor or its local tensor   */
  WB_ERR_DST_OVERLAP = 5,      /* a destination element is described by two slices           */
  WB_ERR_UNCOVERED = 6,        /* a destination element needs a checkpoint id no source holds*/
  WB_ERR_BUCKET_TOO_SMALL = 7, /* the bucket budget cannot hold a single payload chunk       */
  WB_ERR_OOM = 8,              /* host or device allocation failed                           */
  WB_ERR_CUDA = 9,             /* a CUDA runtime call failed                                 */
  WB_ERR_NOT_BOUND = 10,       /* execution requested before wb_plan_bind                    */
  WB_ERR_INTERNAL = 11,        /* a plan invariant does not hold (wb_plan_verify)            */
  WB_ERR_STATIC_LIMIT = 12,    /* the plan's tile table exceeds WB_STATIC_SCRATCH_BYTES       */
  WB_ERR_REPLICA_MISMATCH = 13 /* two trainer replicas of a checkpoint region differ          */
} wb_status;

typedef enum { WB_F32 = 0, WB_BF16 = 1 } wb_dtype;

/* One local tensor of a virtual rank (a flat array of `numel` elements). */
typedef struct {
  uint32_t rank;   /* virtual rank that owns it (used for per-rank accounting and buckets) */
  uint32_t dtype;  /* wb_dtype */
  uint64_t numel;
} wb_tensor_desc;

/* One slice-copy operation of a source map (Section 3.1).  The rectangle
 * [r0, r0+nr) x [c0, c0+nc) of checkpoint tensor `ckpt_tensor` -- viewed as a row-major
 * ckpt_rows x ckpt_cols matrix; vectors are [1, n]; N-D tensors collapse leading dims --
 * lives in local tensor `tensor` (an index into the layout's tensor table); checkpoint
 * element (r0+i, c0+j) is local element local_off + i*stride_r + j*stride_c.
 * Supported stride shapes: rows contiguous (stride_c == 1, stride_r >= nc) or, for a
 * transposed copy, columns contiguous (stride_r == 1, stride_c >= nr); a stride whose
 * extent is 1 is ignored.  Zero-area slices are ignored. */
typedef struct {
  uint32_t tensor;
  uint32_t reserved;      /* must be 0 */
  uint64_t local_off;
  int64_t  stride_r;
  int64_t  stride_c;
  uint64_t ckpt_tensor;
  uint64_t ckpt_rows;
  uint64_t ckpt_cols;
  uint64_t r0, c0, nr, nc;
} wb_slice;

typedef struct wb_layout wb_layout;
typedef struct wb_plan wb_plan;

/* Planner options; zero-initialise for defaults. */
typedef struct {
  uint64_t bucket_budget_bytes; /* bytes of transfer buffer one round may use; 0 = 4 GiB
                                   (the paper's default RDMA budget, Appendix D)           */
  uint32_t tile_bytes;          /* target bytes moved (read + written) per tile; 0 = auto   */
  uint32_t grid_ctas;           /* thread blocks per launch; 0 = auto (multiple of 148 SMs) */
  uint32_t flags;               /* WB_PLAN_* bits                                           */
  uint32_t host_group_kib;      /* wb_remap_host: KiB moved (read + written) per pipeline stage;
                                   0 = auto (1/24 of the transfer, at least 256 MiB)        */
} wb_plan_opts;

#define WB_PLAN_NO_REPLICA_SPLIT 1u /* read replicated source regions from the lowest rank
                                       only instead of a distinct slice per replica        */
#define WB_PLAN_STATIC_SCHEDULE 2u  /* every thread block walks the fixed, byte-balanced tile
                                       range the planner gave it, instead of drawing batches
                                       of tiles from a shared counter at run time          */
#define WB_PLAN_NO_TENSOR_MAPS 4u   /* wb_plan_bind builds no tensor maps: wb_remap stages the
                                       source rows of transposing tiles with per-lane copies
                                       (as wb_unpack and wb_remap_static always do) instead
                                       of tensor-map (TMA) loads                           */

typedef struct {
  uint64_t n_ckpt_tensors;      /* checkpoint tensors the destination consumes              */
  uint64_t n_slabs;             /* one-to-one (or one-to-k fan-out) copy rectangles          */
  uint64_t n_fanout_slabs;      /* slabs with more than one destination                      */
  uint64_t n_rounds;
  uint64_t n_tiles_remap;
  uint64_t n_tiles_pack;        /* summed over rounds                                        */
  uint64_t n_tiles_unpack;
  uint64_t src_elems_read;      /* distinct checkpoint elements read == source elements read */
  uint64_t dst_elems_written;
  uint64_t src_bytes_read;
  uint64_t dst_bytes_written;
  uint64_t replica_elems_skipped; /* source elements never read because a replica supplies them */
  uint64_t bucket_bytes_total;  /* payload + alignment padding, summed over rounds           */
  uint64_t bucket_bytes_max;    /* largest round                                             */
  uint64_t table_bytes;         /* device bytes of all tile tables                           */
  uint64_t remap_cta_bytes_max; /* bytes moved by the most loaded thread block (remap)       */
  uint64_t remap_cta_bytes_mean;
  uint32_t grid_ctas;
  uint32_t tile_bytes;
  double   build_seconds;       /* wall time of wb_plan_build                                */
} wb_plan_stats_t;

/* One payload of a round's bucket: the checkpoint rectangle it carries, row-major in the
 * destination dtype, starting `bucket_off` bytes into the bucket (16-byte aligned). */
typedef struct {
  uint32_t sender;        /* virtual trainer rank the bytes come from                       */
  uint32_t receiver;      /* virtual rollout rank the payload is addressed to               */
  uint64_t ckpt_tensor;
  uint64_t r0, c0, nr, nc;
  uint64_t bucket_off;
  uint32_t dtype;         /* wb_dtype of the payload (== destination dtype)                 */
  uint32_t n_dst;         /* rollout tensors this payload is written to by wb_unpack        */
} wb_bucket_entry;

/* Host view of one tile of a tile table (for verification on the host).  A tile copies
 * dst[dst_off + i*dst_sr + j*dst_sc] = cast(src[src_off + i*src_sr + j*src_sc]) for
 * i < nr, j < nc; a tensor index of -1 means the bucket, with offsets in elements of the
 * bucket dtype.  A fan-out tile appears once per destination; entries after the first
 * carry WB_TILE_FANOUT_CONT and re-use the first entry's source read. */
typedef struct {
  int32_t  src_tensor, dst_tensor;
  uint64_t src_off, dst_off;
  uint32_t nr, nc;
  uint32_t src_sr, src_sc, dst_sr, dst_sc;
  uint32_t kind;          /* kernel path hint: 0 rows, 1 transpose, 2 element-wise          */
  uint32_t flags;
  uint32_t cta;           /* thread block the tile is assigned to                           */
  uint32_t reserved;
} wb_tile_view;

#define WB_TILE_FANOUT_CONT 1u
/* A transposing slab cut into tiles along its rows: the tile holding the rows just before / after
 * this one continues the same destination runs.  The executor then writes a 16-byte destination
 * vector that straddles the seam from the tile that holds its first row (reading the up to 7 source
 * rows it needs from the tile after), and the tile after leaves those rows to it; the table as a
 * whole still writes every element once.  Both tiles of a seam belong to one (sender, receiver) pair. */
#define WB_TILE_ROWS_BEFORE 2u
#define WB_TILE_ROWS_AFTER 4u

enum { WB_TABLE_REMAP = 0, WB_TABLE_PACK = 1, WB_TABLE_UNPACK = 2 };

/* ---- layouts (host only) --------------------------------------------------------------
 * wb_layout_describe: ingest one side's source map (Section 3.1: a list of slice-copy
 * operations, any of which may also transpose).  `tensors` and `slices` are host
 * arrays, copied.  Checks indices, dtypes, stride shapes, that every slice stays inside its
 * checkpoint tensor and its local tensor, and that a checkpoint tensor has one shape.
 * Errors: INVALID_ARG, DTYPE, SHAPE_MISMATCH, OUT_OF_RANGE, OOM. */
wb_status wb_layout_describe(const wb_tensor_desc* tensors, size_t n_tensors,
                             const wb_slice* slices, size_t n_slices, wb_layout** out);
void wb_layout_free(wb_layout* layout);

/* wb_layout_add_flat_range (host, pure arithmetic): the slice-copy operations of one piece of a
 * flat shard (Section 3.1: a source map is a list of slice copies over the checkpoint's 2-D views).
 * A trainer that keeps parameters flattened (FSDP-style flat shards) holds, of the row-major
 * ckpt_rows x ckpt_cols checkpoint tensor `ckpt_tensor`, the flat element range [begin, end)
 * contiguously in local tensor `tensor` from element `local_off` on.  In checkpoint coordinates that
 * range is at most three rectangles - the rest of the first row, the full rows, the start of the
 * last row.  Writes them to out[0 .. cap) as wb_slice records (row-contiguous: stride_c = 1,
 * stride_r = the rectangle's width), in ascending flat order, ready to be
 * appended to the slice list given to wb_layout_describe, and stores their number (0..3) in *n_out;
 * with out == NULL only the number is computed.  An empty range gives 0 slices.
 * Errors: INVALID_ARG (n_out NULL, ckpt_cols 0, cap too small for the slices needed), OUT_OF_RANGE
 * (begin > end or end > ckpt_rows * ckpt_cols). */
wb_status wb_layout_add_flat_range(uint32_t tensor, uint64_t local_off, uint64_t ckpt_tensor,
                                   uint64_t ckpt_rows, uint64_t ckpt_cols, uint64_t begin, uint64_t end,
                                   wb_slice* out, size_t cap, size_t* n_out);

/* ---- planning (host only, no CUDA call) -------------------------------------------------
 * wb_plan_build: Section 3.2.  Intersects the two source maps per checkpoint tensor
 * (element correspondence), de-duplicates replicas on both sides so that every consumed
 * checkpoint element is read exactly once (trainer replicas each supply a distinct slice;
 * rollout replicas are written by fan-out from one read), cuts the resulting slabs into
 * load-balanced tiles assigned to thread blocks, and partitions the model into rounds whose
 * buckets fit `bucket_budget_bytes`.  `trainer` is the source side, `rollout` the
 * destination side; swap them for the inverse transfer.  `opts` may be NULL.
 * Errors: INVALID_ARG, DTYPE, SHAPE_MISMATCH, DST_OVERLAP, UNCOVERED, BUCKET_TOO_SMALL, OOM. */
wb_status wb_plan_build(const wb_layout* trainer, const wb_layout* rollout,
                        const wb_plan_opts* opts, wb_plan** out);
void wb_plan_free(wb_plan* plan);

/* wb_plan_verify: re-derives, by interval arithmetic over the slabs only, that destination
 * spans are pairwise disjoint and cover every described destination element, that source
 * spans of different slabs are disjoint in checkpoint coordinates (each id read once), and
 * that every tile of every table stays inside its tensors / bucket.  INTERNAL on failure. */
wb_status wb_plan_verify(const wb_plan* plan);
wb_status wb_plan_stats(const wb_plan* plan, wb_plan_stats_t* out /* host */);
/* Bytes a virtual rank sends (side 0: trainer egress, source dtype) or receives
 * (side 1: rollout ingress through buckets, destination dtype).  Section 3.2: trainers
 * collectively transmit exactly one copy of the model. */
wb_status wb_plan_rank_bytes(const wb_plan* plan, int side, uint32_t rank, uint64_t* out);

size_t wb_plan_num_rounds(const wb_plan* plan);
size_t wb_plan_bucket_bytes(const wb_plan* plan, size_t round);   /* 0 if round is invalid */
/* Directory of a round's bucket.  Writes up to `cap` entries to `out` (host, may be NULL)
 * and the total count to *n. */
wb_status wb_plan_bucket_entries(const wb_plan* plan, size_t round, wb_bucket_entry* out,
                                 size_t cap, size_t* n);
/* One (receiver, sender) region of a round's bucket (Section 3.2: packing builds one contiguous buffer
 * per receiver; here the receivers' buffers are laid end to end, and inside a receiver's buffer each
 * sender has its own 256-byte aligned piece).  Region k of wb_plan_bucket_regions covers bucket bytes
 * [off, off + bytes): everything virtual trainer rank `sender` packs for virtual rollout rank `receiver`
 * in this round.  Regions are listed in bucket order and do not overlap.  In a deployment with the
 * virtual ranks spread over several GPUs, region (r, s) is what travels from the GPU of s to the GPU
 * of r between wb_pack_ranks and wb_unpack_ranks; the sizes are fixed by the plan. */
typedef struct {
  uint32_t receiver, sender;
  uint64_t off, bytes;
} wb_bucket_region;
wb_status wb_plan_bucket_regions(const wb_plan* plan, size_t round, wb_bucket_region* out, size_t cap,
                                 size_t* n);
/* Number of virtual ranks on each side (highest rank named by a tensor + 1). */
wb_status wb_plan_num_ranks(const wb_plan* plan, uint32_t* n_trainer, uint32_t* n_rollout);
/* Host view of a tile table (`which` = WB_TABLE_*; `round` ignored for WB_TABLE_REMAP). */
wb_status wb_plan_tiles(const wb_plan* plan, int which, size_t round, wb_tile_view* out,
                        size_t cap, size_t* n);

/* ---- binding (device memory; synchronous; allocates the plan's device tables) ------------
 * src_base[i] / dst_base[i]: DEVICE address of trainer / rollout local tensor i, aligned to
 * its element size (16-byte alignment lets the kernels use their widest path).  Host
 * arrays of device pointers, copied.  May be called again to re-bind.  The bound regions
 * must not alias each other.  The kernels fetch whole 16-byte units: they may READ (never write)
 * the up to 15 bytes between a run's first / last element and the enclosing 16-byte boundaries,
 * which always lie inside the same device allocation (allocations are at least 256-byte granular).
 * For the transposing tiles of the fused table whose rows are staged through shared memory the call
 * also encodes tensor maps of the bound source addresses (8 x 128 bytes per tile, in the same device
 * allocation; the driver's cuTensorMapEncodeTiled is looked up at run time, and without it - or under
 * WB_PLAN_NO_TENSOR_MAPS - the kernels copy those rows lane by lane instead).
 * Errors: INVALID_ARG, OOM, CUDA. */
wb_status wb_plan_bind(wb_plan* plan, const void* const* src_base, size_t n_src,
                       void* const* dst_base, size_t n_dst);

/* ---- execution (device; asynchronous on `cuda_stream`, a cudaStream_t or NULL) -----------
 * Each of wb_remap / wb_pack / wb_unpack is a single kernel launch on `cuda_stream` and can be captured
 * into a CUDA graph once it has been called outside capture (the first call sets a kernel attribute).
 * wb_remap: the fused path, trainer tensors -> rollout tensors in one persistent launch:
 * dst[x] = cast(src[y]) for every corresponding pair (Section 3.1), fp32 -> bf16 by
 * round-to-nearest-even, same dtype = bit copy.
 * wb_pack: Section 3.2 packing kernel: this round's source slabs -> checkpoint-format
 * payloads in `bucket` (device, >= wb_plan_bucket_bytes(round), 16-byte aligned), cast
 * applied here so the bucket carries destination-dtype bytes.
 * wb_unpack: Section 3.2 assembly kernel: payloads of `bucket` -> rollout tensors (fused
 * qkv / gate_up concatenation, head regrouping, expert stacking, transposition, fan-out).
 * The device that was current at wb_plan_bind must be current for every call that launches on the plan
 * (INVALID_ARG otherwise: the tables hold that device's addresses).
 * One launch of a tile table at a time: the run-time tile scheduler keeps its counters per table in the
 * plan's device memory, so two calls on the same plan whose GPU work can overlap (different streams
 * with no ordering between them) must not use the same table - wb_remap twice, or wb_pack / wb_unpack
 * of the same round twice.  Calls ordered on one stream, or by events, are fine.
 * Errors: INVALID_ARG, NOT_BOUND, CUDA. */
wb_status wb_remap(const wb_plan* plan, void* cuda_stream);
wb_status wb_pack(const wb_plan* plan, size_t round, void* bucket, void* cuda_stream);
wb_status wb_unpack(const wb_plan* plan, size_t round, const void* bucket, void* cuda_stream);

/* wb_pack_ranks / wb_unpack_ranks: the part of a round that a subset of the virtual ranks executes
 * (Section 3.2: every trainer worker packs its own shards, every rollout worker assembles its own
 * parameters; the receive stage moves each sender's buffer to its receiver in between).
 * wb_pack_ranks runs the packing tiles of the trainer ranks listed in `ranks` (host array, n_ranks
 * entries, any order, duplicates ignored): it reads only those ranks' tensors and writes only the
 * (receiver, sender) regions whose sender is listed.  wb_unpack_ranks runs the assembly tiles whose
 * payload is addressed to a listed rollout rank: it reads only the regions whose receiver is listed and
 * writes those payloads to every rollout tensor that needs them - the listed ranks' own tensors and,
 * for a replicated checkpoint region, the other replicas' tensors (on one GPU a plain store; across
 * GPUs that store is the exchange among replicas).  Packing all trainer ranks in any grouping fills the
 * same bucket as wb_pack; assembling all rollout ranks in any grouping equals wb_unpack.  The tiles of
 * consecutive ranks form one launch; a list with gaps takes one launch per run of consecutive ranks.
 * Same stream, bucket and re-entrancy rules as wb_pack / wb_unpack.
 * Errors: INVALID_ARG (also: a rank beyond the side's rank count), NOT_BOUND, CUDA. */
wb_status wb_pack_ranks(const wb_plan* plan, size_t round, const uint32_t* ranks, size_t n_ranks, void* bucket,
                        void* cuda_stream);
wb_status wb_unpack_ranks(const wb_plan* plan, size_t round, const uint32_t* ranks, size_t n_ranks,
                          const void* bucket, void* cuda_stream);

/* Which entries of the wb_plan_tiles listing of a round's WB_TABLE_PACK / WB_TABLE_UNPACK table belong to
 * virtual rank `rank` (a trainer rank for the pack table, a rollout rank for the unpack table): entries
 * [*first, *first + *count).  For checking the partition on the host.  Errors: INVALID_ARG. */
wb_status wb_plan_rank_tiles(const wb_plan* plan, int which, size_t round, uint32_t rank, size_t* first,
                             size_t* count);

/* wb_plan_check: synchronises with the device and reports whether any launch on this plan
 * recorded an error (the kernels bound every internal wait; a wait that ran out sets a
 * sticky error word instead of hanging).  OK, NOT_BOUND, CUDA, or INTERNAL. */
wb_status wb_plan_check(const wb_plan* plan);

/* wb_plan_check_replicas (device, synchronous): the plan reads a replicated checkpoint region from
 * one trainer replica only (Section 3.2: together the trainers send a single copy of the model),
 * which presumes the replicas are bit-identical.  This debug pass compares every pair of replicas
 * the source layout declares, element by element, on the bound tensors.  *n_mismatches (host, may
 * be NULL) receives the number of differing elements.  OK, REPLICA_MISMATCH, NOT_BOUND, CUDA. */
wb_status wb_plan_check_replicas(const wb_plan* plan, uint64_t* n_mismatches, void* cuda_stream);

/* wb_wait_probe: self-test of the kernels' bounded waits.  Launches one thread that waits on a
 * barrier nothing ever signals, with a limit of limit_ms (1..2000) milliseconds, and synchronises.
 * Returns WB_ERR_INTERNAL when the wait gave up as designed (the expected outcome), WB_OK if it
 * did not have to, CUDA / OOM on runtime errors.  The context stays usable afterwards. */
wb_status wb_wait_probe(uint32_t limit_ms, void* cuda_stream);

/* wb_transfer_rounds: every round of the two-pass path, pipelined (Section 3.2: consecutive
 * rounds overlap; Section 4: with two buffers per side, neighbouring rounds run at the same
 * time).  Round r packs into bucket r mod 2 on one internal stream and is assembled from it on
 * a second internal stream; pack(r) waits until unpack(r-2) has released that bucket, unpack(r)
 * waits for pack(r).  Equivalent to wb_pack + wb_unpack for rounds 0..R-1 in order; the rollout
 * tensors end up as after wb_remap.  Work starts after what `cuda_stream` already holds and
 * `cuda_stream` completes after the last assembly.  Returns without synchronising.
 * bucket0 / bucket1: DEVICE, distinct, each >= max over rounds of wb_plan_bucket_bytes, 16-byte
 * aligned, caller-owned.  flags: WB_ROUNDS_SERIAL runs pack(0), unpack(0), pack(1), ... on
 * `cuda_stream` alone through bucket0 (bucket1 may be NULL) - the unpipelined baseline.
 * Creates two streams and a few events on first use; not reentrant per plan (shares them with
 * wb_remap_host).  Errors: INVALID_ARG, NOT_BOUND, CUDA, OOM. */
#define WB_ROUNDS_SERIAL 1u
wb_status wb_transfer_rounds(const wb_plan* plan, void* bucket0, void* bucket1, uint32_t flags,
                             void* cuda_stream);

/* ---- FP8 quantisation of a round's bucket (device; asynchronous on `cuda_stream`) -----------------
 * Section 5 ("Parameter precision mismatch") sketches it: trainer tensors are quantised before the
 * transfer, which needs the full tensor, so every round starts with the trainers gathering the
 * shards of the tensors to be quantised.  The paper fixes no rule.  The one
 * built: FP8 E4M3 (largest finite value 448), one scale per checkpoint tensor, s = amax / 448 and
 * r = 448 / amax in fp32 (s = r = 1 if amax = 0; an s that rounds to zero becomes 2^-149), amax =
 * the tensor's largest magnitude in the destination dtype; q = e4m3(x * r), fp32 multiplication,
 * round to nearest even, saturating, NaN -> 0x7F; a tensor whose r is not finite (amax below
 * 448 / FLT_MAX, about 1.3e-36) is encoded as q = e4m3(x / s) instead, so that zeros stay zeros and
 * nothing turns NaN whatever the magnitudes; x' = cast_dst(value(q) * s).  Checkpoint tensors are numbered 0 .. wb_plan_num_ckpts-1 in ascending
 * order of their ids (wb_plan_ckpt_ids).
 * wb_absmax: the gather, as a maximum: one pass over the de-duplicated trainer regions of the bound
 *   tensors; amax (DEVICE, wb_plan_num_ckpts floats) is zeroed and then filled.  A tensor that holds a
 *   NaN gets a NaN amax (magnitudes are compared as sign-cleared bit patterns).
 * wb_bucket_quantize: `bucket` (DEVICE, as written by wb_pack for `round`) -> `qbucket` (DEVICE,
 *   wb_plan_qbucket_bytes(round) bytes, one byte per element at the same element offset; padding is
 *   never written).  wb_bucket_dequantize: the inverse, into a bucket wb_unpack can consume.
 *   Both buffers 16-byte aligned, caller-owned.  Work lists are built and uploaded on first use
 *   (one device allocation, released with the plan's device tables).
 * Errors: INVALID_ARG, NOT_BOUND, OOM, CUDA. */
size_t wb_plan_num_ckpts(const wb_plan* plan);
wb_status wb_plan_ckpt_ids(const wb_plan* plan, uint64_t* out /* host */, size_t cap);
size_t wb_plan_qbucket_bytes(const wb_plan* plan, size_t round);   /* 0 if round is invalid */
wb_status wb_absmax(const wb_plan* plan, float* amax, void* cuda_stream);
wb_status wb_bucket_quantize(const wb_plan* plan, size_t round, const void* bucket, void* qbucket,
                             const float* amax, void* cuda_stream);
wb_status wb_bucket_dequantize(const wb_plan* plan, size_t round, const void* qbucket, void* bucket,
                               const float* amax, void* cuda_stream);
/* wb_transfer_rounds_fp8: wb_absmax and then every round of pack -> quantise | dequantise -> unpack with
 * two bucket pairs in flight on the plan's two internal streams, ordered like wb_transfer_rounds
 * (round r uses bucket r mod 2 and qbucket r mod 2; the transfer of the FP8 bucket would sit between
 * the two halves).  Buffers DEVICE, 16-byte aligned, pairwise distinct: buckets >= the largest
 * wb_plan_bucket_bytes, qbuckets >= the largest wb_plan_qbucket_bytes, amax wb_plan_num_ckpts floats.
 * Work starts after what `cuda_stream` already holds; `cuda_stream` completes after the last assembly.
 * Errors: INVALID_ARG, NOT_BOUND, OOM, CUDA. */
wb_status wb_transfer_rounds_fp8(const wb_plan* plan, void* bucket0, void* bucket1, void* qbucket0, void* qbucket1,
                                 float* amax, void* cuda_stream);

/* The fused forms of the quantised transfer (Section 5: the trainers quantise before the transfer, so the
 * wire carries FP8).  wb_pack_fp8 is wb_pack + wb_bucket_quantize in one kernel: this round's source slabs
 * go straight into `qbucket` as E4M3 codes (DEVICE, wb_plan_qbucket_bytes(round) bytes, 16-byte aligned; one
 * byte per element at the element offsets of wb_plan_bucket_entries; padding never written).  wb_unpack_fp8 is
 * wb_bucket_dequantize + wb_unpack: codes -> rollout tensors in their dtype, with the same concatenation,
 * regrouping, stacking, transposition and fan-out as wb_unpack.  Same arithmetic as the separate calls, so
 * qbucket and the rollout tensors are bit-identical to theirs; the 2- or 4-byte bucket and two passes over it
 * are saved.  amax: DEVICE, as filled by wb_absmax.  Asynchronous on `cuda_stream`; one launch of a round's
 * pack (unpack) at a time (each has one tile counter, zeroed in stream order before the launch).
 * wb_transfer_rounds_fp8_fused: wb_absmax, then every round of wb_pack_fp8 | wb_unpack_fp8 with two FP8
 * buckets in flight on the plan's two internal streams, ordered like wb_transfer_rounds.
 * Errors: INVALID_ARG, NOT_BOUND, OOM, CUDA. */
wb_status wb_pack_fp8(const wb_plan* plan, size_t round, void* qbucket, const float* amax, void* cuda_stream);
wb_status wb_unpack_fp8(const wb_plan* plan, size_t round, const void* qbucket, const float* amax, void* cuda_stream);
wb_status wb_transfer_rounds_fp8_fused(const wb_plan* plan, void* qbucket0, void* qbucket1, float* amax,
                                       void* cuda_stream);

/* wb_remap_host: the same transfer for callers whose weights are in HOST memory.  The remap
 * is cut into groups of consecutive tiles; for each group the trainer bytes it reads are copied
 * host -> bound device regions on an internal copy stream, its tiles run on `cuda_stream`, and the
 * rollout bytes it wrote are copied back on a second internal copy stream, so uploads, kernel
 * and downloads of neighbouring groups overlap.  Returns without synchronising; `cuda_stream`
 * completes after the last download.  Creates two streams and a few events on first use.
 * host_src[i] / host_dst[i]: HOST addresses (page-locked for real asynchrony) of the tensors
 * in table order.  Elements no slice describes are neither uploaded nor downloaded reliably:
 * treat padding in host_dst as unspecified.  Errors: INVALID_ARG, NOT_BOUND, CUDA, OOM. */
wb_status wb_remap_host(const wb_plan* plan, const void* const* host_src, size_t n_src,
                        void* const* host_dst, size_t n_dst, void* cuda_stream);

/* wb_remap_static: wb_remap for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a deployment convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a rollout engine that has
 * already handed all free HBM to its KV-cache pool, a weight update triggered from inside a
 * region where the allocator must not be entered, a process whose memory budget is fixed at
 * start-up.  wb_plan_bind allocates a device arena for the tile tables, so such callers cannot
 * use it.  Here the tables and the error word live in a fixed array of
 * WB_STATIC_SCRATCH_BYTES (4 MiB) that is part of the library image: every GPU that loads the
 * library holds those 4 MiB until the process exits, and nothing is ever allocated or freed.
 * The function calls no cudaMalloc / cudaFree / allocating routine, and the plan need not be
 * bound.
 *
 * plan      built by wb_plan_build (host object; its remap table is used)
 * src_base  host array of n_src DEVICE addresses of the trainer tensors, in table order
 * dst_base  host array of n_dst DEVICE addresses of the rollout tensors; the caller still owns
 *           and passes all inputs and outputs
 * flags     0, or WB_STATIC_SYNC_CHECK: synchronise the stream after the launch and return
 *           WB_ERR_INTERNAL if a bounded wait inside the kernel ran out
 *
 * Limits and rules:
 *   - A plan whose remap table (48 B per tile + 16 B per fan-out record + 4 B per thread block
 *     + 512 B) does not fit in 4 MiB -- about 87,000 tiles, e.g. 40 GB moved at the default
 *     512 KiB tile size -- is refused with WB_ERR_STATIC_LIMIT and nothing is launched; build
 *     the plan with a larger tile_bytes, or use wb_plan_bind + wb_remap.
 *   - The first call on each device resolves the array's device address and configures the
 *     kernels (no allocation).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents: each
 *     call rewrites the table it needs and zeroes the error word, in stream order.  Two calls
 *     whose GPU work can overlap (different streams without an ordering between them) race on
 *     the array; order them on one stream or with events.  Host-side preparation, the upload of
 *     the table and the launch are serialised internally, so host threads that call on one stream
 *     cannot interleave.
 *   - The table (up to 4 MiB) is uploaded from ordinary host memory: the call blocks the host
 *     until the runtime has staged it.  A call on a stream that is being captured is refused with
 *     WB_ERR_INVALID_ARG (a replay would upload whatever a later call left in the staging image).
 *   - A bounded wait that ran out inside the kernel is reported only by a call made with
 *     WB_STATIC_SYNC_CHECK (there is no bound plan whose wb_plan_check could be asked).
 * Errors: INVALID_ARG, STATIC_LIMIT, CUDA, INTERNAL (only with WB_STATIC_SYNC_CHECK). */
#define WB_STATIC_SCRATCH_BYTES (4u << 20)
#define WB_STATIC_SYNC_CHECK 1u
wb_status wb_remap_static(const wb_plan* plan, const void* const* src_base, size_t n_src,
                          void* const* dst_base, size_t n_dst, uint32_t flags, void* cuda_stream);

/* ---- three-stage routing over nodes: traffic accounting (Section 3.2, Eq. 1) ------------------
 * With virtual ranks placed on nodes, a plan's slabs define the paper's three stages: *receive*
 * (each slab travels from its trainer rank to its designated rollout rank -- replicas of a tensor
 * are the designated receivers of distinct slices), *external exchange* (every other rollout node
 * that needs the slab gets it once, over RDMA, from the designated receiver) and *internal
 * exchange* (the remaining ranks of a node copy it over NVLink).  Nothing is moved: this returns
 * the byte counts the stages would carry, to check the plan against the paper's traffic claims --
 * trainers send exactly one model copy M, node v receives exactly its de-duplicated volume M_v over
 * RDMA -- and the lower bound T_min = max(M / B_T, max_v M_v / B_v) of Eq. 1.
 * Bytes are destination-dtype bytes (wb_pack casts before the wire). */
typedef struct {
  uint64_t model_bytes;            /* M: every consumed checkpoint element once                    */
  uint64_t receive_bytes;          /* stage 1, trainers -> designated receivers                    */
  uint64_t external_bytes;         /* stage 2, between rollout nodes (RDMA)                        */
  uint64_t internal_bytes;         /* stage 3, inside rollout nodes (NVLink)                       */
  uint64_t direct_rdma_bytes;      /* without the exchange stages: every rank pulls all it needs   */
  uint64_t max_trainer_rank_egress;
  uint64_t max_rollout_rank_rdma_ingress;
  uint64_t max_node_rdma_ingress;
  double   t_min_seconds;          /* Eq. 1 with the bandwidths given                              */
} wb_route_stats_t;
/* trainer_node[r] / rollout_node[r]: node of virtual trainer / rollout rank r (host arrays; node ids
 * are small integers, trainer and rollout nodes share one numbering).  trainer_gbs = aggregate
 * trainer egress bandwidth B_T, node_gbs = ingress bandwidth B_v of a rollout node, in GB/s.
 * node_rdma_ingress / node_required (host, n_nodes entries each, may be NULL) receive, per node, the
 * RDMA bytes entering it in stages 1+2 and M_v.  Errors: INVALID_ARG. */
wb_status wb_route_account(const wb_plan* plan, const uint32_t* trainer_node, size_t n_trainer_ranks,
                           const uint32_t* rollout_node, size_t n_rollout_ranks, double trainer_gbs,
                           double node_gbs, wb_route_stats_t* out, uint64_t* node_rdma_ingress,
                           uint64_t* node_required, size_t n_nodes);

/* ---- source-map extraction (Section 3.1, Appendix B / Algorithm 1) ---------------------------
 * A worker's source map can be recovered from its black-box load_weights instead of being
 * written by hand: fill the checkpoint with position ids (1-based, so 0 = "no source"), load,
 * and analyse the id field each local tensor ends up with.  The field is not shipped to the
 * host: its second-order difference diff2 (Appendix B, Eq. diff1/diff2) is non-zero only around
 * the corners of the rectangles the slice-copy operations filled.  For parameters narrower than
 * the ids the probe is repeated per b-bit id chunk and the sparse results are recombined. */
typedef struct { uint64_t row, col; int64_t value; } wb_diff2_entry;
enum { WB_ID_I64 = 0,   /* field of int64                                              */
       WB_ID_U16 = 1,   /* raw 16-bit patterns (a 16-bit chunk held in a bf16 tensor)   */
       WB_ID_F32 = 2,   /* fp32 holding an integer value (below 2^24, where fp32 is exact)  */
       WB_ID_BF16 = 3   /* bf16 holding an integer value (8-bit chunks are exact)        */ };

/* wb_diff2_nonzeros (device, asynchronous on cuda_stream): diff2 of the rows x cols row-major
 * field at `field` (DEVICE), read as `id_kind`.  Every non-zero entry is appended to `out`
 * (DEVICE, `cap` entries) in no particular order; *count (DEVICE uint64, zeroed by the caller)
 * receives the number found, which may exceed cap (the surplus is dropped: retry with a larger
 * list).  `field` needs only the alignment of its element type; rows whose start is aligned for
 * 16-byte (8-byte for 16-bit kinds) accesses are read with vector loads; a field of 4 MiB or more whose
 * rows all start on 16-byte boundaries is streamed through a ring of bulk copies.  Every wait inside the
 * kernels is bounded: a count of 2^62 or more reports that one ran out (nothing hangs; the list is then
 * incomplete).  Limits: rows * cols <= 2^48; a field of several rows has rows, cols < 2^31.
 * Errors: INVALID_ARG, CUDA. */
wb_status wb_diff2_nonzeros(const void* field, uint32_t id_kind, uint64_t rows, uint64_t cols,
                            wb_diff2_entry* out, uint64_t cap, uint64_t* count, void* cuda_stream);
/* wb_diff2_nonzeros_batch: the same for many fields in ONE launch (a model has thousands of local
 * tensors, most of them small; a launch per tensor is bound by launch latency - the per-tensor
 * overhead Section 3.2 warns about).  `fields`: HOST array of n_fields descriptors (`field` DEVICE);
 * every entry found in field k carries fields[k].tag.  `scratch`: DEVICE, 16-byte aligned, at least
 * wb_diff2_batch_scratch_bytes(n_fields) bytes, must stay valid until the kernel has run.  `out`
 * (DEVICE, `cap` entries, one list for all fields, no particular order) and *count (DEVICE uint64,
 * zeroed by the caller) as above.  Fields with rows or cols = 0 are skipped.  Errors: INVALID_ARG,
 * OOM, CUDA. */
typedef struct wb_diff2_field {
  const void* field;
  uint64_t rows, cols;
  uint32_t id_kind;
  uint32_t tag;
} wb_diff2_field;
typedef struct wb_diff2_tagged_entry {
  uint64_t row, col;
  int64_t value;
  uint32_t tag, reserved;
} wb_diff2_tagged_entry;
size_t wb_diff2_batch_scratch_bytes(size_t n_fields);
wb_status wb_diff2_nonzeros_batch(const wb_diff2_field* fields, size_t n_fields, void* scratch, size_t scratch_bytes,
                                  wb_diff2_tagged_entry* out, uint64_t cap, uint64_t* count, void* cuda_stream);
/* wb_diff2_chunk_pass (device, asynchronous on cuda_stream): one pass of Algorithm 1's inner loop for one
 * local tensor, with carries, so that O(N_c) entries per pass reach the host even for 8-bit chunks
 * (Appendix B: diff2 of a truncated chunk overflows at regularly spaced positions; the overflow is carried
 * into the next chunk, and a strided difference cancels the periodic pattern).  The paper sketches the
 * step only; what this computes:
 *   D = diff2(field) + Gamma          field = chunk `pass` of the ids as load_weights left it (values in
 *                                     [0, 2^chunk_bits)), Gamma = ExpandCarry(carry_in), 0 for pass 0
 *   D = Z + 2^chunk_bits C            EmitCarry: Z the balanced digit in [-2^(b-1), 2^(b-1)), C the carry
 *   z_out    <- NonZeros(Z)           H_Z[pass]: the pass-th balanced digit of every entry of diff2(ids)
 *   carry_out <- NonZeros(StridedDiff1(C))   H_Gamma[pass], with s = 2^(chunk_bits (pass + 1)), x = i cols + j:
 *                                     G[x] = C[x] - C[x - s] - C[x - s cols] + C[x - s - s cols]
 *   ExpandCarry inverts StridedDiff1 of the previous pass (s = 2^(chunk_bits pass)).
 * Feeding the z_out lists of passes 0 .. K-1 to wb_diff2_recombine gives diff2 of the full ids when
 * K chunk_bits >= bits(16 max id) + 1 (then the last carry_out list is empty).
 * field: DEVICE, rows x cols, read as id_kind.  carry_in: DEVICE list of the previous pass's carry_out
 * entries for this tensor (n_carry_in of them; NULL / 0 for pass 0 or an empty list).  scratch: DEVICE,
 * 16-byte aligned, wb_diff2_chunk_scratch_bytes(rows, cols) bytes (one byte per element plus 256 KiB),
 * contents irrelevant before and after.  z_out / carry_out (DEVICE, z_cap / carry_cap entries, no
 * particular order) and *z_count / *carry_count (DEVICE uint64, zeroed by the caller) as for
 * wb_diff2_nonzeros.  Several kernels per call.  Limits: chunk_bits 8 or 16, pass < 8, rows * cols <= 2^40.
 * Errors: INVALID_ARG, CUDA. */
size_t wb_diff2_chunk_scratch_bytes(uint64_t rows, uint64_t cols);
wb_status wb_diff2_chunk_pass(const void* field, uint32_t id_kind, uint64_t rows, uint64_t cols, uint32_t chunk_bits,
                              uint32_t pass, const wb_diff2_entry* carry_in, uint64_t n_carry_in, void* scratch,
                              size_t scratch_bytes, wb_diff2_entry* z_out, uint64_t z_cap, uint64_t* z_count,
                              wb_diff2_entry* carry_out, uint64_t carry_cap, uint64_t* carry_count, void* cuda_stream);
/* wb_diff2_recombine (host): Algorithm 1, Recombine.  sum_k 2^(chunk_bits*k) * passes[k], merged
 * by position, zeros dropped, sorted by (row, col).  Writes up to cap entries, *n_out = total. */
wb_status wb_diff2_recombine(const wb_diff2_entry* const* passes, const size_t* counts, size_t n_passes,
                             uint32_t chunk_bits, wb_diff2_entry* out, size_t cap, size_t* n_out);
/* wb_scan_slices (host): Algorithm 1, ScanSliceMappings.  From the diff2 entries of one local
 * tensor viewed as rows x cols (starting `elem_off` elements into local tensor `tensor`) recover
 * the slice-copy operations as wb_slice records.  The checkpoint is given as n_ckpt tensors with
 * shapes ckpt_rows[t] x ckpt_cols[t] whose first element has id ckpt_base[t] + 1 (ckpt_base has
 * n_ckpt + 1 entries, the last being the total element count).  Writes up to cap slices,
 * *n_out = total.  INVALID_ARG if the field is not piecewise affine in the two shapes a slice
 * copy produces; OUT_OF_RANGE for entries outside the view. */
wb_status wb_scan_slices(const wb_diff2_entry* nz, size_t n, uint64_t rows, uint64_t cols,
                         const uint64_t* ckpt_base, const uint64_t* ckpt_rows, const uint64_t* ckpt_cols,
                         size_t n_ckpt, uint32_t tensor, uint64_t elem_off, wb_slice* out, size_t cap,
                         size_t* n_out);

/* Number of kernels wb_remap / wb_pack / wb_unpack launch per call (always 1). */
int wb_launches_per_call(void);

const char* wb_status_str(wb_status s);
const char* wb_version(void);

#ifdef __cplusplus
}
#endif
#endif /* WB_H_ */
