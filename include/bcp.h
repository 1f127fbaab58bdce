/*
 * bcp.h - C ABI of the B200 load-time checkpoint resharding engine.
 *
 * The library implements the device-side hot path of load-time resharding as the
 * ByteCheckpoint paper (arXiv 2407.20143) states the problem:
 *
 *   - every tensor has a fully qualified name (FQN) and a global shape
 *     (Sec. 3.2, "Model and optimizer states");
 *   - every saved or wanted shard is an index tuple (fqn, nD_offsets, nD_lengths)
 *     inside that global shape: the ShardMeta (Sec. 3.2);
 *   - a ByteMeta gives the byte start offset and length of the shard inside its
 *     storage file (Sec. 3.2, "Checkpoint representation");
 *   - an irregular shard (a 1-D slice of a flattened tensor, as ZeRO / FSDP produce)
 *     is represented by several regular ShardMeta entries
 *     (Sec. 3.2, "Decomposing irregular tensors");
 *   - at load time each new shard is matched against the saved shards and the
 *     matching segments are copied into it (Sec. 3.3, Step 2 and Step 5).
 *
 * A "storage file" is a device buffer here (a blob); all source ranks and all target
 * ranks are separate buffers, normally on ONE GPU (source blobs may also be another GPU's
 * memory mapped into this process: bcp_ipc_*).  The engine moves raw bytes unchanged, unless
 * bcp_plan_opts.convert asks for a binary32 <-> bfloat16 conversion of some tensors.
 *
 * Conventions
 *   - Every function returns an int: BCP_OK (0) or a negative bcp_status.  A failing
 *     call leaves its outputs untouched and launches nothing.  bcp_last_error()
 *     returns a thread-local, NUL-terminated description of the last failure on the
 *     calling thread (valid until that thread's next failing call).
 *   - "host" pointers are ordinary CPU memory; "device" pointers are addresses in the
 *     memory of the CUDA device that is current when the call is made.
 *   - `stream` arguments are CUDA stream handles (cudaStream_t) passed as void*;
 *     NULL is the legacy default stream.
 *   - Nothing here throws, aborts or traps the device.
 *   - Threads: a plan, a stager and the fixed scratch of bcp_pack_static each serve one
 *     call at a time; different plans may be used from different threads concurrently.
 *     bcp_pack / bcp_unpack serialise themselves (their cache of work lists is shared).
 *   - Source and target buffers of one call must not overlap: sources are read through the
 *     read-only data path.
 */
#ifndef BCP_H_
#define BCP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BCP_MAX_NDIM 8

#if defined(__GNUC__)
#define BCP_API __attribute__((visibility("default")))
#else
#define BCP_API
#endif

typedef enum {
  BCP_OK = 0,
  BCP_ERR_INVALID = -1,   /* null pointer, bad ndim/itemsize/kind, negative length, box outside the
                             global shape, byte_length != element count * itemsize, bad option    */
  BCP_ERR_MISMATCH = -2,  /* entries of one FQN disagree on itemsize, dtype_tag, ndim or global shape */
  BCP_ERR_OVERLAP = -3,   /* two source entries of one FQN hold the same element                 */
  BCP_ERR_UNCOVERED = -4, /* some element of a target entry is held by no source entry           */
  BCP_ERR_BOUNDS = -5,    /* a byte range reaches past the size given for its buffer              */
  BCP_ERR_DST_ALIAS = -6, /* two target entries write overlapping byte ranges of one buffer       */
  BCP_ERR_CUDA = -7,      /* a CUDA runtime call failed (message carries the CUDA error string)   */
  BCP_ERR_NOMEM = -8,     /* host allocation failed                                               */
  BCP_ERR_DEVICE_TIMEOUT = -9, /* a bounded device-side wait gave up (TMA path only); the targets of
                                  that execution are incomplete                                     */
  BCP_ERR_CAPACITY = -10  /* an output array supplied by the caller is too small                  */
} bcp_status;

typedef enum { BCP_BOX = 0, BCP_FLAT_SLICE = 1 } bcp_kind;

/*
 * One entry of the paper's TensorShardToBasicByteMap (Sec. 3.2): ShardMeta
 * (fqn, offsets, lengths) + the part of BasicMeta that matters for raw bytes
 * (itemsize, dtype_tag) + ByteMeta (buf_index, byte_offset, byte_length).
 *
 * Layout of the bytes (the paper gives only offset and length): the entry's elements are
 * stored densely in C (row-major) order.
 *   BCP_BOX        : the box offsets[0..ndim) + lengths[0..ndim) of the global tensor.
 *   BCP_FLAT_SLICE : elements [flat_begin, flat_end) of the C-order flattening of the
 *                    box offsets/lengths (the rank's local tensor), i.e. an irregular
 *                    shard; the library decomposes it into regular boxes itself.
 * ndim == 0 is a scalar (one element).  Zero-volume entries are legal and produce no work.
 */
typedef struct {
  const char* fqn;      /* host, NUL-terminated, caller-owned; read only during bcp_plan       */
  uint32_t itemsize;    /* bytes per element: 1, 2, 4 or 8                                      */
  uint32_t dtype_tag;   /* opaque dtype identity; must agree across all entries of an FQN       */
  uint32_t ndim;        /* 0..BCP_MAX_NDIM                                                      */
  uint32_t kind;        /* bcp_kind                                                             */
  int64_t global_shape[BCP_MAX_NDIM];
  int64_t offsets[BCP_MAX_NDIM];
  int64_t lengths[BCP_MAX_NDIM];
  int64_t flat_begin;   /* BCP_FLAT_SLICE only; 0 <= flat_begin <= flat_end <= prod(lengths)    */
  int64_t flat_end;
  uint32_t buf_index;   /* source: which blob; target: which target-rank buffer                 */
  uint32_t reserved;    /* must be 0                                                            */
  uint64_t byte_offset; /* ByteMeta start inside that buffer                                    */
  uint64_t byte_length; /* ByteMeta length = element count * itemsize                           */
} bcp_shard_meta;

/* Planner / launch options.  Zero in any field selects the default written beside it. */
typedef struct {
  uint32_t tile_bytes;     /* payload of one CTA-wide work unit, multiple of 4096.  0 default: 65536, except that
                              16-byte aligned contiguous runs of a plan without DP replicas are cut at 32768  */
  uint32_t small_bytes;    /* work units with a payload below this go to the warp path; default 4096  */
  uint32_t block_threads;  /* threads per CTA of the register kernel: 256, 512 or 1024; default 512     */
  uint32_t ctas_per_sm;    /* register path: persistent CTAs per SM; default 2 (4 with worker 2)       */
  uint32_t order;          /* 1 units that read the same source bytes (replicas of a target shard) side by side,
                              so that they are staged once and hit L2: the lists are in source-address order,
                              and the staged units are then rearranged group by group into the order of each
                              group's first target address; 2 order by target address (the pieces of one
                              stretch of a target are written at about the same time; replicas are not
                              grouped); 3 plain source-address order (replicas side by side, nothing
                              rearranged); 0 default: 2 when every source byte is wanted once, else 1 if
                              the plan has strided rectangles, else 3                                    */
  uint32_t path_mask;      /* which kernels execute the list.
                              1 every unit goes through registers (LDG/STG kernel);
                              3 runs of at least tma_min_row_bytes (any alignment) and rectangles with rows of
                                at least that size whose offsets, row length and pitches are multiples of 16
                                go through the TMA staging kernel (bulk copies via shared memory), the rest
                                through the register kernel;
                              7 as 3, and 16-byte aligned rectangles with rows of 16..2048 bytes are staged
                                with 2-D tensor-map copies (cp.async.bulk.tensor.2d, one command per box of
                                up to 256 rows) instead of one bulk copy per row; their descriptors are
                                re-encoded on the host whenever a buffer address changes;
                              0 default: 7 when at least 4 MiB of payload qualifies for TMA staging, else 1
                                (measured: from there on the staging kernel is the faster one; when all that
                                is left for the register kernel are a few thousand units under small_bytes,
                                the staging kernel's warps copy those too and one kernel is launched)        */
  uint32_t cache_hints;    /* 0 default (= 1); register path: 1 streaming loads and stores, 2 plain accesses;
                              TMA path: 3 evict-first L2 hint on stores, 4 on loads too, else no hint    */
  uint32_t tma_stage_bytes; /* TMA path: bytes per shared-memory stage, multiple of 128; default 32768, or
                               16384 when an eighth or more of the staged payload are shifted runs or
                               rectangles with rows under 2 KiB                                        */
  uint32_t tma_stages;      /* TMA path: stages per CTA, 2..8; default 3 (4 when tensor-map boxes dominate) */
  uint32_t tma_ctas_per_sm; /* TMA path: one-warp CTAs per SM; default 2 (4 in the same case)            */
  uint32_t unroll;          /* register path: 16-byte loads in flight per thread, 4 or 8; default 4    */
  uint32_t worker;          /* register path: 1 a CTA copies a unit together; 2 every warp is a worker of
                               its own (256-thread CTAs); default 2 when this path has at least 128 MiB
                               to move, else 1                                                          */
  uint32_t tma_min_row_bytes; /* TMA path: shortest row (or run) staged through TMA; default 512; multiple of 16 */
  uint32_t allow_replicas;  /* 0 default: two saved entries of one FQN that hold the same element are an
                               error; 1: saved entries with IDENTICAL boxes are replicas (a checkpoint saved
                               without de-duplication): the first in input order is read, the others are
                               ignored; boxes that overlap only partly are still BCP_ERR_OVERLAP        */
  uint32_t tma_wait_ms;     /* TMA path: how long a CTA waits for one stage to fill before it gives up and
                               raises BCP_ERR_DEVICE_TIMEOUT (measured with the device's global timer);
                               default 2000                                                             */
  uint32_t fanout;          /* 0 default (= 1); 1: TMA units that read the same source bytes (replicas of a
                               target shard; needs order 1) are grouped, the source is staged once and
                               written to every member's target (fewer L2 reads; over PCIe, fewer reads
                               at all); 2: every unit is staged on its own (bcp_reshard_host still groups
                               when it works in place)                                                     */
  uint32_t test_stall;      /* test hook, 0 in normal use: 1 makes the first CTA of each staging kernel (copy and
                               conversion) arm its first stage for more bytes than it loads, so that exactly
                               one bounded wait per kernel runs out and the time-out path can be exercised
                               without any fault                                                          */
  uint32_t convert;         /* 0 default: entries of one FQN must agree on itemsize and dtype_tag, bytes are
                               moved unchanged.  BCP_CONVERT_F32_TO_BF16 / BCP_CONVERT_BF16_TO_F32: an FQN
                               whose saved entries have dtype_tag convert_src_tag and whose wanted entries have
                               dtype_tag convert_dst_tag (itemsizes 4 and 2, resp. 2 and 4) is converted
                               element by element while it is resharded; every other FQN is moved unchanged.
                               Entries of a converted FQN must start on a multiple of their item size
                               (BCP_ERR_INVALID otherwise; plain copies may start at any byte).
                               The paper moves bytes only; this serves the hand-over of fp32 master weights
                               to a bf16 evaluation job (and back).                                       */
  uint32_t convert_src_tag; /* see convert */
  uint32_t convert_dst_tag;
  uint32_t src_buf_first;   /* with src_buf_count != 0: matching, the disjointness check and the coverage check run */
  uint32_t src_buf_count;   /* against every saved entry as usual, but the plan keeps only the pieces that are read
                               from source buffers [src_buf_first, src_buf_first + src_buf_count); it writes the
                               target bytes those pieces hold and no others.  Plans for disjoint ranges that
                               together cover all source buffers write every target byte exactly once between
                               them and may run concurrently (the exchange of Sec. 4.1 / 4.2 across GPUs: the
                               pieces read from a rank's own blobs are copied while the segments of the other
                               ranks are still on their way).  0: all source buffers                          */
} bcp_plan_opts;

/*
 * Conversions (bcp_plan_opts.convert).  Values are IEEE-754 binary32 and bfloat16 (the upper
 * 16 bits of a binary32), little endian.
 * F32_TO_BF16 rounds to nearest, ties to even, on the bit pattern: infinities stay, values
 * beyond the largest bfloat16 become infinity, subnormals round like any other value (no
 * flush to zero), and every NaN becomes the quiet NaN 0x7FC0.
 * BF16_TO_F32 appends 16 zero bits (exact for every input, NaN payloads included).
 */
#define BCP_CONVERT_NONE 0u
#define BCP_CONVERT_F32_TO_BF16 1u
#define BCP_CONVERT_BF16_TO_F32 2u

typedef struct bcp_plan_s bcp_plan_t;

/*
 * One unit of the flat work list the planner produces and the kernels execute:
 * rows x row_bytes bytes from src_buf at src_off (rows src_pitch apart) to dst_buf at
 * dst_off (rows dst_pitch apart).  Pitches are 0 when rows == 1.
 */
typedef struct {
  uint64_t src_off;
  uint64_t dst_off;
  uint64_t src_pitch;
  uint64_t dst_pitch;
  uint32_t row_bytes;
  uint32_t rows;
  uint32_t src_buf;
  uint32_t dst_buf;
  uint32_t flags;       /* BCP_TILE_* */
  uint32_t reserved[3];
} bcp_tile;

#define BCP_TILE_GRAN_MASK 0x7u /* log2 of the widest power-of-two access (<= 16 B) that divides
                                   src_off, dst_off, row_bytes and both pitches                  */
#define BCP_TILE_ZERO 0x8u      /* no source: write zero bytes (pack padding)                    */
#define BCP_TILE_SMALL 0x10u    /* executed by one warp                                          */
#define BCP_TILE_TMA 0x20u      /* executed by the TMA staging kernel                            */
#define BCP_TILE_TMA2D 0x40u    /* rows of a rectangle staged with 2-D tensor-map copies: reserved[0] =
                                   rectangle index + 1, reserved[1] = first row inside the rectangle,
                                   reserved[2] = rows per box                                    */
#define BCP_TILE_FOLLOW 0x80u   /* TMA unit with the same source bytes as the unit before it in the list
                                   (a replica of a target shard): the CTA that stages the first unit of
                                   such a group writes every member's target from the one staged copy,
                                   and whoever draws a follower's ticket skips it                 */
#define BCP_TILE_FAN_SHIFT 8    /* bits 8..10 of a group's first unit: how many followers it has (0..7) */
#define BCP_TILE_CVT_SHIFT 11   /* bits 11..12: BCP_CONVERT_* applied by this unit (0: plain copy).  For a
                                   converting unit row_bytes counts TARGET bytes; a source row holds the same
                                   number of elements (twice, resp. half as many bytes)            */
#define BCP_TILE_CVT_MASK (3u << BCP_TILE_CVT_SHIFT)

typedef struct {
  uint64_t n_src_entries;    /* after decomposing flat slices; tensors no wanted entry names are left out */
  uint64_t n_dst_entries;
  uint64_t n_fqns;
  uint64_t n_intersections;  /* non-empty source x target box intersections          */
  uint64_t n_items;          /* after dimension collapse and coalescing               */
  uint64_t n_tiles;          /* CTA-wide work units                                   */
  uint64_t n_small_tiles;    /* warp work units                                       */
  uint64_t n_strided_tiles;  /* work units with rows > 1                              */
  uint64_t n_tma_tiles;      /* work units executed by the TMA staging kernel         */
  uint64_t bytes_copied;     /* payload bytes the list writes = sum of target bytes   */
  uint64_t bytes_src_unique; /* distinct source bytes the list reads                  */
  uint64_t bytes_misaligned; /* payload in units whose access granularity is < 16 B   */
  double plan_ms;            /* host time spent in bcp_plan                           */
  uint64_t n_cvt_tiles;      /* converting work units (bcp_plan_opts.convert)         */
  uint64_t n_kernels;        /* kernels one bcp_reshard of this plan launches (1..4): the staging kernel (which
                                also takes a short rest of unstaged units), the register kernel (a long rest),
                                the staged and the register converting kernel                                 */
} bcp_plan_stats_t;

/* ByteMeta of one tensor inside a packed blob (Sec. 3.2): start offset and length. */
typedef struct {
  uint64_t byte_offset;
  uint64_t byte_length;
} bcp_pack_meta;

/* Library version (major*10000 + minor*100 + patch). Never fails. */
BCP_API int bcp_version(void);

/* Thread-local message of the last failing call on this thread ("" if none). */
BCP_API const char* bcp_last_error(void);

/*
 * Irregular-tensor decomposition (Sec. 3.2, "Decomposing irregular tensors").
 * Elements [flat_begin, flat_end) of the C-order flattening of a dense local tensor of
 * shape lengths[0..ndim) are rewritten as the fewest regular boxes, listed in flat order;
 * each box is a contiguous sub-range of the flattening and together they tile the range.
 * out_off / out_len (host, caller-owned, cap rows of BCP_MAX_NDIM) receive box offsets and
 * lengths RELATIVE to the local tensor; *n receives the box count (at most 2*ndim - 1,
 * 0 for an empty range).  BCP_ERR_CAPACITY if cap is too small (then *n is the needed count).
 */
BCP_API int bcp_decompose(const int64_t* lengths, uint32_t ndim, int64_t flat_begin, int64_t flat_end,
                  int64_t (*out_off)[BCP_MAX_NDIM], int64_t (*out_len)[BCP_MAX_NDIM], size_t cap,
                  size_t* n);

/*
 * Save-side de-duplication with load balancing (Sec. 4.1, "Balancing saving workload").
 * Shard i has shard_bytes[i] bytes and is held by the ranks
 * holders[holder_offsets[i] .. holder_offsets[i+1]) (at least one; rank ids < n_ranks).
 * Shards are taken in input order and each is assigned to the holder whose cumulative
 * assigned bytes are smallest at that moment (worst fit; ties go to the lowest rank id).
 * rank_load[n_ranks] is read as the load every rank starts with (bytes it has to save
 * anyway) and receives the final loads; out_owner[n_shards] receives the owners.
 * Host only; all arrays are host memory, caller-owned.
 */
BCP_API int bcp_dedup_assign(const uint64_t* shard_bytes, const uint64_t* holder_offsets, const uint32_t* holders,
                             size_t n_shards, size_t n_ranks, uint64_t* rank_load, uint32_t* out_owner);

/*
 * Load-time matching and plan construction (Sec. 3.3, Step 2; plan reuse: Sec. 4.1,
 * "Plan and metadata cache").  Host only: no device is touched, so it also runs on a
 * machine without a GPU.
 *
 * src[n_src] are the saved entries, dst[n_dst] the wanted ones; src_buf_bytes[n_src_bufs]
 * and dst_buf_bytes[n_dst_bufs] give each buffer's size for bounds checks.  All arrays are
 * host memory, caller-owned, read only during the call.  For every target entry the
 * planner finds all source entries of the same FQN whose boxes intersect it, checks that
 * they cover it exactly once, and lowers every intersection to work units
 * (bcp_tile).  Source entries of one FQN must be pairwise disjoint (but see
 * bcp_plan_opts.allow_replicas); target entries may overlap one another as boxes (replicas)
 * but not as byte ranges.
 * On success *out_plan owns host (and, after the first bcp_reshard, device) copies of the
 * work list; release it with bcp_plan_destroy.  A plan holds no buffer addresses and can
 * be executed any number of times on any buffers of the planned sizes.
 * Work lists of more than 32k units are built by several host threads (at most 8; the
 * environment variable BCP_PLAN_THREADS, 1..64, overrides the count); the plan does not
 * depend on how many.
 */
BCP_API int bcp_plan(const bcp_shard_meta* src, size_t n_src, const uint64_t* src_buf_bytes,
             size_t n_src_bufs, const bcp_shard_meta* dst, size_t n_dst,
             const uint64_t* dst_buf_bytes, size_t n_dst_bufs, const bcp_plan_opts* opts,
             bcp_plan_t** out_plan);

BCP_API int bcp_plan_stats(const bcp_plan_t* plan, bcp_plan_stats_t* out);

/*
 * Plan cache across processes (Sec. 4.1, "Plan and metadata cache": plans stay constant
 * over a training session, so planning is paid once).  bcp_plan_serialize writes a
 * self-contained, position-independent image of the plan (options, statistics, buffer
 * sizes, work list, checksum) into out[0..cap) and the image size into *n; with cap too
 * small (or out NULL) it writes nothing, stores the needed size and returns
 * BCP_ERR_CAPACITY.  bcp_plan_deserialize rebuilds a plan from an image.  Because a work
 * list drives device copies, the image is verified before use: magic, version, record size,
 * checksum, and every unit against the recorded buffer sizes (in bounds, access width and
 * path flags consistent with its offsets); anything else is BCP_ERR_INVALID.  Images are
 * only meaningful to the library version that wrote them.
 */
BCP_API int bcp_plan_serialize(const bcp_plan_t* plan, void* out, size_t cap, size_t* n);
BCP_API int bcp_plan_deserialize(const void* image, size_t n, bcp_plan_t** out_plan);

/*
 * Host copy of the work list, in execution order (CTA-wide units first, then warp
 * units, then converting units).  Writes min(cap, count) records to out (may be NULL when cap == 0) and the
 * full count to *n.
 */
BCP_API int bcp_plan_tiles(const bcp_plan_t* plan, bcp_tile* out, size_t cap, size_t* n);

/*
 * Which saved entries the plan reads: ascending indices into the `src` array that was given to
 * bcp_plan, one per saved entry that holds at least one element some wanted entry of the plan
 * asks for (the "matching segments" of Sec. 3.3 Step 2, reported per saved shard).  This is what a
 * rank has to obtain before it can run the plan: the cross-GPU exchange (Sec. 4.1, "Eliminating
 * redundant loading"; Sec. 4.2, load pipeline) sends exactly these entries.  Writes min(cap, count)
 * indices to out (may be NULL when cap == 0) and the full count to *n.  Only plans built by
 * bcp_plan record this (BCP_ERR_INVALID for deserialized images).
 */
BCP_API int bcp_plan_used_sources(const bcp_plan_t* plan, uint32_t* out, size_t cap, size_t* n);

/*
 * Execute a plan (Sec. 3.3, Step 5: copy every matched segment into its target shard).
 * src_blobs[n_src_bufs] and dst_bufs[n_dst_bufs] are HOST arrays of DEVICE pointers to
 * buffers at least as large as planned, each 16-byte aligned (BCP_ERR_INVALID otherwise),
 * sources and targets not overlapping; counts must equal the planned ones.  The call uploads the
 * work list on first use, enqueues the pointer tables and the copy kernel on `stream`
 * and returns without waiting; buffers must stay valid until the stream reaches that
 * point.  Executions of one plan share its device-side pointer tables and ticket counters,
 * so they are ordered: on one stream by the stream; when the stream differs from that of the
 * previous execution, the new stream is made to wait (on the device) for what is queued on the
 * previous one (so that stream must still exist then, and when the plan is destroyed).  Calls on
 * one plan from several host threads must not overlap, and inside a stream capture the caller
 * orders the executions.
 * Target bytes not named by any target entry are left untouched.
 * Once a plan has run on a set of buffer addresses, running it again on the same addresses
 * enqueues kernel launches only (no allocation, no copy, no synchronisation), so the call
 * may be recorded by a stream capture and replayed from a CUDA graph.
 */
BCP_API int bcp_reshard(bcp_plan_t* plan, const void* const* src_blobs, size_t n_src_bufs,
                void* const* dst_bufs, size_t n_dst_bufs, void* stream);

/*
 * Same operation with HOST buffers (host pointers to host memory); returns when every target
 * buffer is complete.  Target bytes not named by any target entry come back as zero.
 *   - If every buffer is page-locked memory the device can address (cudaHostAlloc,
 *     cudaHostRegister, torch pin_memory), nothing is staged: the kernels read the sources
 *     and write the targets in place, so data crosses PCIe in both directions at the same
 *     time and each byte crosses once per use.
 *   - Otherwise the source blobs are copied to plan-owned device staging memory, the kernels
 *     run there and the target buffers are copied back; the work is pipelined per target
 *     buffer over three streams (`stream` for the kernels, two plan-owned streams for uploads
 *     and downloads), so that downloads of finished target buffers overlap the uploads still
 *     needed by later ones.
 * Plans restricted to some source buffers (bcp_plan_opts.src_buf_count) are refused: BCP_ERR_INVALID.
 */
BCP_API int bcp_reshard_host(bcp_plan_t* plan, const void* const* src_blobs_host, size_t n_src_bufs,
                     void* const* dst_bufs_host, size_t n_dst_bufs, void* stream);

/*
 * Device status of the plan's executions so far: BCP_OK, or BCP_ERR_DEVICE_TIMEOUT if a
 * bounded wait of the TMA staging kernel gave up (that CTA stopped taking work, so some
 * target bytes of that execution were not written; the plan's counters are reset and it can
 * be executed again).  Synchronises `stream`.
 */
BCP_API int bcp_plan_device_status(bcp_plan_t* plan, void* stream);

/* Waits for the plan's last execution, frees host and device memory. NULL is accepted. */
BCP_API int bcp_plan_destroy(bcp_plan_t* plan);

/*
 * Blob layout for a rank's tensors (ByteMeta table, Sec. 3.2): tensor i of
 * tensor_bytes[i] bytes starts at out_offsets[i], the smallest multiple of `align`
 * (a power of two >= 16) not below the end of tensor i-1; *out_blob_bytes is the end of
 * the last tensor rounded up to `align`.  Host arrays, caller-owned.
 */
BCP_API int bcp_pack_layout(const uint64_t* tensor_bytes, size_t n, uint64_t align, uint64_t* out_offsets,
                    uint64_t* out_blob_bytes);

/*
 * Pack n tensors into one contiguous save blob (the device-side stand-in for the
 * serialisation step of the save pipeline, Sec. 4.2): tensors[i] (device pointer,
 * metas[i].byte_length bytes) is copied to blob + metas[i].byte_offset; every blob byte
 * in [0, blob_bytes) that belongs to no tensor is written as zero.  metas must be sorted
 * by byte_offset and non-overlapping, inside blob_bytes.  tensors and metas are host
 * arrays.  Tensor and blob addresses need no particular alignment (16-byte aligned ones
 * copy fastest).  Asynchronous on `stream`.  Work lists are cached inside the library per
 * (metas, blob_bytes), so repeated packs of the same layout only upload pointers; packs of one
 * layout issued on different streams run one after the other (see bcp_reshard).
 */
BCP_API int bcp_pack(const void* const* tensors, const bcp_pack_meta* metas, size_t n, void* blob,
             uint64_t blob_bytes, void* stream);

/* Inverse of bcp_pack (the deserialisation step of the load pipeline, Sec. 4.2):
 * blob + metas[i].byte_offset -> tensors[i].  Padding is ignored. */
BCP_API int bcp_unpack(const void* blob, uint64_t blob_bytes, const bcp_pack_meta* metas, size_t n,
               void* const* tensors, void* stream);

/* Drops the cached pack / unpack work lists (waits for their last executions). */
BCP_API int bcp_pack_cache_clear(void);

/*
 * Safetensors export (the paper's system exports checkpoints in the Safetensors format for
 * the Hugging Face ecosystem, Sec. 7).  An image is: 8 bytes little-endian header length,
 * the JSON header (every tensor's dtype, shape and [begin, end) offsets into the byte buffer;
 * padded with spaces so that the buffer starts on an 8-byte boundary), then the tensors back
 * to back in the order given.  dtype is one of BOOL U8 I8 F8_E5M2 F8_E4M3 I16 U16 F16 BF16 I32
 * U32 F32 F64 I64 U64; a tensor's byte length is prod(shape) * size of the dtype.
 *
 * bcp_safetensors_layout (host only) writes the first 8 + N bytes of the image to header_out
 * and every tensor's byte range INSIDE THE IMAGE to out_metas (usable as bcp_pack metas);
 * with header_cap too small it still reports *header_bytes, *file_bytes and out_metas and
 * returns BCP_ERR_CAPACITY.
 * bcp_safetensors_export builds the whole image in device memory at `file` (capacity
 * file_cap bytes): the tensors (device pointers, any alignment) are packed by the copy kernels
 * and the header is copied over the front, all on `stream`, asynchronously.  The pageable
 * header is staged by the runtime before the call returns.
 */
typedef struct {
  const char* name;   /* host, NUL-terminated, unique, not "__metadata__" */
  const char* dtype;  /* host, NUL-terminated                                */
  uint32_t ndim;      /* 0..BCP_MAX_NDIM                                     */
  uint32_t reserved;
  int64_t shape[BCP_MAX_NDIM];
} bcp_export_entry;
BCP_API int bcp_safetensors_layout(const bcp_export_entry* entries, size_t n, void* header_out, size_t header_cap,
                                   size_t* header_bytes, bcp_pack_meta* out_metas, uint64_t* file_bytes);
BCP_API int bcp_safetensors_export(const bcp_export_entry* entries, const void* const* tensors, size_t n, void* file,
                                   uint64_t file_cap, uint64_t* file_bytes, void* stream);

/*
 * Asynchronous save / load staging through a pool of pinned host buffers with ping-pong
 * use (Sec. 4.2: the save pipeline copies shards to a pinned memory pool with ping-pong
 * buffering so that only a short step blocks training; loading mirrors it).
 *
 * A stager owns n_slots pairs (device slot, pinned host slot) of slot_bytes each, one side
 * stream and its events; create / destroy allocate and free them on the current device.
 *
 *   save:  bcp_stager_save packs the tensors into a free device slot on `stream` (like
 *          bcp_pack) and queues the download of that slot to its pinned twin on the side
 *          stream; it returns without waiting and reports the slot.  Once `stream` has passed
 *          the pack, the tensors may be modified again: the blocking part of a save is the
 *          pack alone.  bcp_stager_wait blocks until the download is complete and returns the
 *          pinned blob (valid until the slot is released).  With two slots the pack of the next
 *          blob overlaps the download of the previous one.
 *   load:  bcp_stager_acquire hands out a free slot's pinned buffer for the caller to fill
 *          (e.g. from storage); bcp_stager_load queues the upload on the side stream and the
 *          unpack into `tensors` on `stream`, and returns without waiting.
 *   bcp_stager_release returns a slot to the pool (waits for its copy to finish).
 * BCP_ERR_CAPACITY: blob larger than a slot, or no free slot.  One thread at a time per stager.
 */
typedef struct bcp_stager bcp_stager_t;
BCP_API int bcp_stager_create(uint64_t slot_bytes, uint32_t n_slots, bcp_stager_t** out);
BCP_API int bcp_stager_destroy(bcp_stager_t* stager);
BCP_API int bcp_stager_save(bcp_stager_t* stager, const void* const* tensors, const bcp_pack_meta* metas, size_t n,
                            uint64_t blob_bytes, void* stream, uint32_t* out_slot);
BCP_API int bcp_stager_wait(bcp_stager_t* stager, uint32_t slot, void** host_blob);
BCP_API int bcp_stager_acquire(bcp_stager_t* stager, uint32_t* out_slot, void** host_blob);
BCP_API int bcp_stager_load(bcp_stager_t* stager, uint32_t slot, uint64_t blob_bytes, const bcp_pack_meta* metas,
                            size_t n, void* const* tensors, void* stream);
BCP_API int bcp_stager_release(bcp_stager_t* stager, uint32_t slot);

/*
 * Peer mapping of saved blobs, for cross-GPU resharding without an exchange step.  The paper's
 * load pipeline moves the pieces a rank needs from its DP peers in an all-to-all (Sec. 4.1,
 * "Eliminating redundant loading"; Sec. 4.2); with every GPU able to address its peers' memory the
 * same pieces can be read where they lie: a rank plans its own targets against the global saved
 * metadata (a plan may cover any subset of the wanted entries) and hands bcp_reshard the addresses
 * of ALL saved blobs, its own and its peers' mapped ones.  The copy kernels then fetch every tile
 * straight from its owner (plain bulk loads, one destination CTA each; over NVLink when the owner is
 * another GPU) and the transfer overlaps the copy tile by tile; nothing is packed, sent or received.
 *
 *   bcp_ipc_export  fills *out for the device pointer dev_ptr (device current = the one that owns
 *                   it): the CUDA IPC handle of the allocation that contains it, the pointer's offset
 *                   inside that allocation and the bytes from there to the allocation's end.  The
 *                   96 bytes are plain data: send them to the other processes by any means.
 *   bcp_ipc_open    maps the allocation in the calling process (device current = the one that will
 *                   read it; peer access is enabled on demand) and returns the address that
 *                   corresponds to the exported pointer.  An allocation is mapped once per process and
 *                   device however many pointers into it are opened.  A process cannot open its own
 *                   handles: it uses its own pointers.
 *   bcp_ipc_close   gives a pointer from bcp_ipc_open back; the allocation is unmapped with the last one.
 * The owner keeps the memory allocated, and its contents in place, from the export until every
 * reader has closed; ordering between the owner's writes and the readers' kernels is the caller's
 * (a barrier between the processes).  Memory of a virtual-memory pool cannot be exported: BCP_ERR_CUDA.
 */
typedef struct {
  unsigned char handle[64];
  uint64_t offset;
  uint64_t bytes_after;
  int32_t device;     /* device index in the exporting process (informational) */
  int32_t reserved[3];
} bcp_ipc_handle;
BCP_API int bcp_ipc_export(const void* dev_ptr, bcp_ipc_handle* out);
BCP_API int bcp_ipc_open(const bcp_ipc_handle* handle, void** out_ptr);
BCP_API int bcp_ipc_close(void* ptr);

/*
 * bcp_pack for callers that cannot allocate.  (The paper has no counterpart: this entry point
 * exists for the way the library gets embedded, not for the method.)
 *
 * Who needs it: a process whose device memory is already fully handed out to its own pool
 * (a serving engine, a training job sized to the last megabyte), or code that runs where an
 * allocation is not allowed or would synchronise the whole device.  bcp_pack allocates
 * its device-side work list the first time a layout is seen; this call never calls
 * cudaMalloc, cudaFree or any other allocating routine, on the device or on the host.
 * Instead its scratch (control words, pointer table, work list) is a fixed array of about
 * 0.8 MiB in device memory that belongs to the library image: every GPU that loads the library
 * holds it until the process exits, whether or not this call is ever made.
 *
 * Same arguments, result and asynchrony as bcp_pack.  Differences:
 *   - limits: at most BCP_STATIC_MAX_TENSORS tensors and BCP_STATIC_MAX_UNITS work units
 *     (the unit size grows up to 64 MiB to make a blob fit); beyond that the call returns
 *     BCP_ERR_CAPACITY and launches nothing: use bcp_pack.
 *   - the first call on each device looks up the device address of the fixed array, with
 *     that device current; make that first call before any stream capture begins.  A call
 *     whose stream is being captured is refused with BCP_ERR_INVALID: its uploads come from a
 *     host array that every call rewrites.
 *   - all calls share the one array per device.  Each call rewrites what it uses and clears the
 *     control words, so calls that run one after the other on the GPU (same stream, or
 *     otherwise ordered) are safe; two calls whose kernels may overlap on the GPU (different
 *     streams without ordering) race on it and must not be made.  Host-side the call is
 *     serialised by a lock.
 *   - the work list is rebuilt on every call (nothing is cached) and runs on the register
 *     kernel.
 */
#define BCP_STATIC_MAX_TENSORS 4096u
#define BCP_STATIC_MAX_UNITS 12288u
BCP_API int bcp_pack_static(const void* const* tensors, const bcp_pack_meta* metas, size_t n, void* blob,
                            uint64_t blob_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BCP_H_ */
