/*
 * tensorcast.h - C ABI of the descriptor-driven batched tensor mover for NVIDIA B200 (sm_100a).
 *
 * One "plan" is a validated, immutable batch of copy descriptors (source tensor/offset,
 * destination tensor/offset, shape, strides).  Executing a plan is one kernel launch on the
 * caller's stream.  The plan captures geometry only; data pointers are call arguments, so a
 * plan can be re-executed on any buffers of the same geometry and re-execution is idempotent
 * (the paper's call contexts make operations re-entrant, Sec. 3.2 "Plan").
 *
 * Operations and the passages of the paper that define them:
 *   tc_kv_pack             publish(req_id): flush the KV cache of a request's whole context out
 *                          of the engine's paged pool (Table 2 "Instance Operation"; Sec. 3.2;
 *                          Sec. 4.5 steps 3-4).  Also the offload leg to pinned host memory and,
 *                          with a migrate plan, publish fused with hydrate (pool to pool).
 *   tc_kv_unpack           hydrate(req_id, artifacts): load a request's KV cache into the
 *                          destination engine's paged pool (Table 2; Sec. 4.5 step 8).
 *   tc_weights_materialize Artifact.tensor_dict() (materialise), Artifact.view(slice) (one
 *                          tensor-parallel rank's slice, Sec. 6.2) and transform_into(artifact,
 *                          spec, target) (fill a caller-owned target buffer) (Table 2; Sec. 5
 *                          "Tensor Materialization and Transfer").
 *   tc_plan_create/destroy the lifecycle of the plan object itself.
 * The paper defines no memory layout; the layouts below are this library's.
 *
 * Layouts.  E = bytes per element, D = head dim (contiguous everywhere), H = kv heads,
 * B = tokens per block, L = layers, c = 0 for K and 1 for V.
 *   Paged pool, plane (l,c), block b, slot n, head h, element d:
 *     TC_NHD: plane(l,c) + b*block_stride + ((n*H + h)*D + d)*E
 *     TC_HND: plane(l,c) + b*block_stride + ((h*B + n)*D + d)*E
 *     plane(l,c) = bases[l*2 + c]                      when the pool has L*2 table slots
 *                = bases[0] + (l*2 + c)*plane_stride   when it has one slot
 *   Token t of request r lives in block bt[bt_off[r] + t / B], slot t % B.
 *   Packed buffer (always one table slot): requests back to back in request order,
 *     off_0 = 0, off_{r+1} = off_r + L*2*T_r*H*D*E, and inside request r
 *     TC_NHD: off_r + ((((l*2 + c)*T_r + t)*H + h)*D + d)*E
 *     TC_HND: off_r + ((((l*2 + c)*H + h)*T_r + t)*D + d)*E      (request level, no padding)
 *   Only the T_r valid tokens move; the unused slots of a request's last block are neither
 *   read nor written, and no other byte of a destination is ever written.
 *
 * Ownership.  Every data buffer is caller-leased: the library never allocates, frees or
 * retains it and touches it only between the call and the completion of the stream work the
 * call enqueued.  Sources are never written.  The plan object is library-owned: created and
 * destroyed only through this API.  Spec arrays (T, bt_off, bt, index, rules) are read during
 * tc_plan_create only and may be freed afterwards.
 *
 * Memory spaces.  Pointers inside the *tables* passed to the execute calls are DEVICE-
 * addressable addresses: device memory, pinned host memory mapped into the device's
 * address space (cudaHostAlloc / cudaHostRegister under unified addressing), which the kernel
 * then reads or writes directly over the host link (zero copy), or another GPU's memory once
 * peer access is enabled (every CTA then moves its own tile over NVLink with plain loads and
 * stores - misaligned geometry: with per-CTA bulk asynchronous loads into its shared memory;
 * every copy lands in the issuing CTA's own shared memory or registers).  Pageable host memory is not
 * addressable by the device: the execute calls refuse it (TC_ERR_INVALID_ARG) instead of
 * letting a kernel fault.  The tables themselves, the
 * spec and every array it points to are HOST memory.
 *
 * Alignment.  Nothing has to be aligned: base pointers, offsets, strides and row lengths may be
 * any number of bytes.  When every address of a call is a multiple of 16 the kernels move 16-byte
 * vectors register to register.  Otherwise they realign on the fly - aligned 16-byte chunks of
 * the source are staged in shared memory and shifted into aligned 16-byte stores, only the first
 * and last bytes of a row go out in smaller pieces - at 0.9-1.0 of the aligned speed for rows of a
 * few hundred bytes and more.  On that path the SOURCE side is read in whole aligned 16-byte
 * chunks: up to 15 bytes before a row's first byte and after its last one are read (always inside
 * a chunk that holds a byte of the row, hence inside the same page) and ignored; destinations are
 * written byte-exactly.
 *
 * Devices.  A plan belongs to the CUDA device that was current when it was created; execute
 * calls must be made with that device current (TC_ERR_INVALID_ARG otherwise).
 *
 * Synchronisation.  Execute calls are asynchronous on `stream` (a cudaStream_t passed as
 * void*; NULL = the legacy default stream).  Completion is observed through the stream
 * (events, cudaStreamSynchronize): operations are lazy handles that block only when awaited
 * (Sec. 3.2).  The library never synchronises the device.
 *
 * Errors.  Every function returns a tc_status.  All detectable errors are raised on the host
 * before anything is launched; a failed call launches nothing, and a failed tc_plan_create
 * stores NULL in *out.  There is no rollback after a launch (plans have no transactional
 * semantics, Sec. 3.2).  No exception crosses the ABI.  Calls on distinct plans are thread
 * safe; one plan may be executed concurrently on different buffers.
 */
#ifndef TENSORCAST_H_
#define TENSORCAST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define TC_API __attribute__((visibility("default")))
#else
#define TC_API
#endif

typedef enum {
    TC_OK = 0,
    TC_ERR_INVALID_ARG = -1, /* NULL where data is required, bad enum, table length mismatch */
    TC_ERR_SHAPE = -2,       /* non-positive extent, ndim > 4, split dim not divisible by world */
    TC_ERR_BOUNDS = -3,      /* block id >= num_blocks, offset past a slot / blob / packed size */
    TC_ERR_OVERLAP = -4,     /* a destination byte written twice, or read and written in one plan */
    TC_ERR_KIND = -5,        /* execute call does not match the plan's kind */
    TC_ERR_OOM = -6,         /* host or device allocation of plan storage failed */
    TC_ERR_CUDA = -7,        /* a CUDA runtime call failed (no device, launch failure) */
    TC_ERR_DEADLINE = -8,    /* the plan's deadline had already passed at call entry */
    TC_ERR_TOO_LARGE = -9,   /* the request exceeds a fixed capacity of the entry point called */
    TC_ERR_IO = -10          /* reading the blob file failed or hit end of file early */
} tc_status;

typedef enum {
    TC_KV_PACK = 1,    /* paged pool -> packed buffer                    (tc_kv_pack)   */
    TC_KV_UNPACK = 2,  /* packed buffer -> paged pool                    (tc_kv_unpack) */
    TC_KV_MIGRATE = 3, /* src pool -> dst pool, one launch               (tc_kv_pack)   */
    TC_KV_MIXED = 4,   /* offload group src_pool -> dst_pool (tc_kv_pack) plus a reload group
                          dst_pool -> src_pool (tc_kv_unpack) built and checked together   */
    TC_WEIGHTS = 5     /* flat blob -> per-parameter tensors             (tc_weights_materialize) */
} tc_kind;

typedef enum { TC_NHD = 0, TC_HND = 1 } tc_layout;

/* Order of the packed buffer.  Request-major (default): each request is one self-contained
 * contiguous region.  Layer-major: plane (l,c) of ALL requests is contiguous,
 *   plane(l,c) = (l*2 + c) * (sum_q T_q) * Hs*D*E,  request r inside it at (sum_{q<r} T_q) * Hs*D*E,
 * so that a consumer can start on the first layers while later ones are still in flight. */
typedef enum { TC_REQUEST_MAJOR = 0, TC_LAYER_MAJOR = 1 } tc_packed_order;

enum {
    TC_PLAN_HOST_ONLY = 1u, /* validate and lower on the host only: the plan can be inspected
                               (tc_plan_stats, tc_plan_descriptors) but not executed, and no
                               CUDA call is made */
    TC_PLAN_STAGED = 2u,    /* The host side of the plan is PINNED HOST memory and should travel
                               through the copy engines instead of being loaded / stored by the
                               kernel itself (zero copy, the default):
                                 - TC_KV_PACK / TC_KV_UNPACK: the packed buffer;
                                 - TC_KV_MIXED: dst_pool, a page-first host pool in one
                                   allocation (plane_stride = one block of one plane), moved in
                                   full blocks;
                                 - TC_WEIGHTS: the blob, for tensors read in contiguous pieces
                                   (whole tensors, dim-0 slabs).
                               The library cuts the plan into segments whose host bytes are
                               contiguous ranges of at most 64 MiB (a paged pool: runs of 2 MiB
                               pages), copies each segment between host memory and a ring of
                               device staging buffers on an internal stream, and runs the same
                               kernel device to device on the caller's stream, segment by
                               segment, chained by events: the streaming pipeline of pinned
                               buffers and asynchronous streams (Sec. 5) with the scatter /
                               layout transform fused into its device leg.  The copy engines
                               drive the host link with larger transactions than SM loads and
                               stores, so this path is faster (and stays fast when both
                               directions of the link are busy); it costs one launch and one or
                               more copies per segment instead of one launch per call.  The
                               rings (3 x 64 MiB per direction and device) are allocated when
                               the first staged plan is created and kept until the process
                               exits.  Groups that cannot be staged (strided slices of a blob,
                               partial blocks of a paged pool) stay zero copy.  Layer-major
                               packed buffers are cut into runs of whole planes, in layer
                               order.  While they are being enqueued, staged executions in the
                               same direction on the same device wait for one another (the
                               ring is theirs in turn); other devices and the other direction
                               are not held up. */
    TC_PLAN_SAME_POOL = 8u, /* TC_KV_MIGRATE inside ONE pool (compaction / defragmentation): the
                               caller will pass the same table as source and destination.
                               src_pool and dst_pool must describe the same geometry, and no
                               block may be both read and written (TC_ERR_OVERLAP), so that the
                               result does not depend on the order in which tiles run. */
    TC_PLAN_CHECKSUM = 4u,  /* TC_WEIGHTS: the plan can also be run by
                               tc_weights_materialize_checksum, which folds an integrity
                               checksum of every tensor into the same pass as the copy.  Needs
                               16-byte aligned geometry and tensors that start on 4-byte
                               boundaries of the blob (TC_ERR_INVALID_ARG otherwise).  Such
                               plans default to 64 KiB tiles (tuning.tile_bytes overrides). */
    TC_PLAN_OFFLOAD_ZERO_COPY = 32u, /* staged TC_KV_MIXED plans: stage only the reload group
                               (host pages -> copy engine -> staging ring -> kernel); the offload
                               group stores into the host pool straight from the kernel.  Kernel
                               stores to host memory keep their speed while the other direction of
                               the link is busy, and the copy engines then serve one direction only */
    TC_PLAN_TRACE = 64u,    /* record a pair of CUDA events around every execution of the plan, so that
                               tc_plan_stats can report the device time of the last one (the
                               call context's tracing hook, Sec. 3.2).  Two event records per
                               call; executions of one traced plan should not overlap */
    TC_PLAN_DEBUG_BOUNDS = 128u, /* debugging aid (the pool's memory checker tools are not always at hand):
                               the plan also keeps, on the device, the byte extent of every table
                               slot as the spec declares it.  Before every execution a small
                               kernel holds the descriptors AS UPLOADED against those extents; an
                               access outside sets TC_DEVICE_OUT_OF_BOUNDS in the device status
                               word and the copy kernel that follows returns without touching
                               memory (it never traps).  tc_plan_check_device runs the checker
                               alone.  Not for staged or streamed plans */
    TC_PLAN_STREAM = 16u    /* TC_WEIGHTS: the blob is streamed chunk by chunk, from a file
                               (tc_weights_materialize_file) or from pinned host memory
                               (tc_weights_materialize), through the staging ring.  Unlike
                               TC_PLAN_STAGED every tensor is staged: a strided slice travels
                               as the byte range that covers it (whole rows, as a loader
                               reading from storage fetches them) and is cut out on the
                               device.  Chunks start on 4 KiB boundaries of the blob and are at
                               most 64 MiB; a tile whose covering range is larger cannot be
                               streamed (TC_ERR_TOO_LARGE at create). */
};

#define TC_MAX_TABLE_SLOTS 4000 /* src slots + dst slots of one execute call.  The table travels in the
                                   kernel parameters; its size does not change the kernel's speed
                                   (measured: 6.97 TB/s with 1 to 3072 destination slots), only the
                                   host time of the call (one check and one copy per entry). */

/* Geometry of a paged KV pool (the data pointer(s) come at execute time). */
typedef struct {
    int32_t layout;       /* tc_layout inside one block */
    int32_t reserved;     /* 0 */
    int64_t num_blocks;   /* NB: valid block ids are [0, NB) */
    int64_t n_slots;      /* length of the base-pointer table passed at execute: L*2 or 1 */
    int64_t plane_stride; /* n_slots == 1: bytes from plane (l,c) to the next; else ignored */
    int64_t block_stride; /* bytes between consecutive blocks of a plane; 0 = tight B*H*D*E */
    int64_t slot_bytes;   /* byte extent of each table slot, used for bounds checks;
                             0 = the minimum extent that holds NB blocks */
} tc_kv_pool_t;

/* A group of R requests.  Host arrays, read at create only. */
typedef struct {
    int64_t R;             /* number of requests (0 is legal: the group moves nothing) */
    const int64_t *T;      /* [R]   valid tokens of each request (0 is legal) */
    const int64_t *bt_off; /* [R+1] CSR offsets into the block tables; bt_off[r+1]-bt_off[r]
                                    must equal ceil(T[r] / B) */
    const int32_t *bt_src; /* block ids in the source pool (NULL when the source is packed) */
    const int32_t *bt_dst; /* block ids in the destination pool (NULL when the destination
                              is packed).  No id may appear twice in bt_dst. */
} tc_kv_group_t;

typedef struct {
    int64_t L, B, H, D, E;   /* E in {1,2,4,8}; contents are opaque bytes */
    tc_kv_pool_t src_pool;   /* PACK, MIGRATE, MIXED (the device pool) */
    tc_kv_pool_t dst_pool;   /* UNPACK, MIGRATE, MIXED (the host pool) */
    int32_t packed_layout;   /* PACK / UNPACK: tc_layout of the packed buffer */
    int32_t packed_order;    /* PACK / UNPACK: tc_packed_order */
    int64_t packed_bytes;    /* PACK / UNPACK: capacity of the packed buffer, for bounds checks;
                                0 = exactly the required size */
    int64_t head_begin;      /* PACK / UNPACK: the packed buffer holds heads [head_begin, */
    int64_t head_count;      /*   head_begin + head_count) only (a tensor-parallel consumer's view
                                of the request): H becomes Hs = head_count and h becomes
                                h - head_begin in the packed formulas; the other heads of the
                                pool are neither read nor written.  head_count 0 = all H heads */
    tc_kv_group_t group;     /* PACK, UNPACK, MIGRATE; MIXED: the offload group */
    tc_kv_group_t reload;    /* MIXED only: moves dst_pool[bt_src] -> src_pool[bt_dst] */
} tc_kv_spec_t;

/* One record of the blob's binary offset index (64 bytes, little endian when stored). */
typedef struct {
    uint64_t byte_off;   /* start of the tensor in the blob */
    uint64_t nbytes;     /* must equal elem_bytes * prod(shape) */
    uint32_t elem_bytes; /* 1, 2, 4 or 8 */
    uint32_t ndim;       /* 1..4 */
    uint64_t shape[4];   /* row-major, tight; unused trailing dims = 1 */
    uint64_t name_id;    /* opaque: index into the caller's side table of names */
} tc_index_entry_t;

/* Where tensor i goes.  All-default (rules == NULL): whole tensor, tight, into dst slot i. */
typedef struct {
    int32_t split_dim;     /* -1: copy the whole tensor; else rank gets slab
                              [rank*n/world, (rank+1)*n/world) of this dim (n % world == 0) */
    int32_t dst_slot;      /* index into dst_ptrs; -1 = i */
    int64_t dst_off;       /* byte offset inside the slot */
    int64_t dst_stride[4]; /* byte strides of the destination's dims; all 0 = tight row-major
                              strides of the (sliced) shape */
} tc_weight_rule_t;

typedef struct {
    int64_t n_tensors;
    const tc_index_entry_t *index; /* [n_tensors] */
    const tc_weight_rule_t *rules; /* [n_tensors] or NULL */
    int32_t rank, world;           /* tensor-parallel rank and world size (1 = no sharding) */
    int64_t blob_bytes;            /* extent of the blob, for bounds checks */
    int64_t n_dst;                 /* number of destination slots; 0 = n_tensors */
    const int64_t *dst_bytes;      /* [n_dst] extent of each destination slot, or NULL = each
                                      slot is exactly as large as its (sliced) tensor */
} tc_weights_spec_t;

/* Optional knobs; 0 everywhere = the library's defaults. */
typedef struct {
    int32_t tile_bytes;   /* target bytes per tile, the work of one CTA: a power of two in
                             [512, 1 MiB], default 32 KiB (64 KiB for TC_PLAN_CHECKSUM plans).  A
                             tile is a row range of one plane of one descriptor; it may reach
                             1.5 x tile_bytes where that avoids a sliver, and it takes several
                             consecutive planes of a KV block when one plane is at most half
                             of tile_bytes (few KV heads). */
    int32_t ctas_per_sm;  /* > 0: a persistent grid-stride grid of this many CTAs per SM instead
                             of one CTA per tile */
    int32_t max_ctas;     /* > 0: cap on the grid (persistent grid-stride loop).  When a table entry
                             of an execute call is pinned host memory and neither this nor
                             ctas_per_sm is set, the grid is capped at one CTA per SM: few
                             long-lived CTAs serve the host link better than one CTA per tile */
    int32_t tile_order;   /* 0 auto: KV groups run plane-major over descriptors sorted by
                             destination offset (ascending writes in HBM) - unless one side of
                             the call is pinned host memory in which a block's planes lie back to
                             back (a paged host pool): then the planes of one block run
                             consecutively and a page is touched in one go;
                             1: request / descriptor order as given, planes of one block
                             consecutively; 2: plane-major whatever the memory */
    int32_t copy_path;    /* 0 auto: aligned geometry moves register to register (16-byte loads and
                             stores), misaligned geometry through shared memory.  1: always
                             through shared memory - bulk asynchronous copies (cp.async.bulk) bring
                             a tile's rows in, 16-byte stores take them out - whatever the
                             alignment; for comparing the two paths (groups with multi-plane
                             tiles and checksummed executions keep the register path) */
    int32_t reserved;     /* 0 */
} tc_tuning_t;

typedef struct {
    uint32_t struct_size; /* sizeof(tc_plan_spec_t) */
    int32_t kind;         /* tc_kind */
    uint32_t flags;       /* TC_PLAN_* */
    uint32_t reserved;    /* 0 */
    uint64_t trace_id;    /* opaque, echoed in tc_plan_stats (the call context's tracing id) */
    int64_t deadline_ns;  /* absolute CLOCK_MONOTONIC nanoseconds; 0 = none.  A call entered
                             after the deadline returns TC_ERR_DEADLINE and launches nothing */
    tc_tuning_t tuning;
    tc_kv_spec_t kv;           /* kinds 1-4 */
    tc_weights_spec_t weights; /* kind 5 */
} tc_plan_spec_t;

typedef struct tc_plan tc_plan_t;

/*
 * Validate `spec` on the host, lower it to descriptors and tiles, upload them to the current
 * CUDA device (unless TC_PLAN_HOST_ONLY) and return an immutable plan in *out.
 * spec, out: host pointers.  On error *out = NULL and nothing stays allocated.
 * The upload runs on a stream of the library's own and has completed when the call returns, so
 * the plan may be executed on any stream at once.  The call orders itself against NO stream of
 * the caller: it neither waits for work already enqueued (a buffer still being filled on another
 * stream is the caller's to wait for) nor makes later work wait.
 */
TC_API int tc_plan_create(const tc_plan_spec_t *spec, tc_plan_t **out);

/*
 * Run the gather side of `plan` on `stream`:
 *   TC_KV_PACK    src_bases = the pool's table (src_pool.n_slots entries), dst_bases = {packed}
 *   TC_KV_MIGRATE src_bases = source pool table, dst_bases = destination pool table
 *   TC_KV_MIXED   the offload group: src_bases = src_pool table, dst_bases = dst_pool table
 * src_bases / dst_bases: HOST arrays of n_src / n_dst device-addressable pointers; they are
 * read before the call returns.  n_src and n_dst must match the plan (TC_ERR_INVALID_ARG).
 */
TC_API int tc_kv_pack(const tc_plan_t *plan, const void *const *src_bases, size_t n_src,
               void *const *dst_bases, size_t n_dst, void *stream);

/*
 * Run the scatter side of `plan` on `stream`:
 *   TC_KV_UNPACK  src_bases = {packed}, dst_bases = the pool's table (dst_pool.n_slots)
 *   TC_KV_MIXED   the reload group: src_bases = dst_pool table (the host pool it reads),
 *                 dst_bases = src_pool table (the device pool it fills).  The two groups of a
 *                 mixed plan touch disjoint blocks and may run concurrently on two streams.
 * Pool bytes not addressed by the plan keep their contents.
 */
TC_API int tc_kv_unpack(const tc_plan_t *plan, const void *const *src_bases, size_t n_src,
                 void *const *dst_bases, size_t n_dst, void *stream);

/*
 * Scatter tensors out of the flat blob: dst_ptrs[slot] + dst_off <- blob[byte_off ...], whole
 * or one rank's slice, per the plan's rules.  blob: device-addressable pointer (device memory
 * or mapped pinned host memory).  dst_ptrs: HOST array of n_dst device-addressable pointers.
 */
TC_API int tc_weights_materialize(const tc_plan_t *plan, const void *blob, void *const *dst_ptrs,
                           size_t n_dst, void *stream);

/*
 * tc_weights_materialize plus integrity checksums, in one pass over the data (the
 * materialisation pipeline checks integrity before it hands tensors out, Sec. 5).
 * `plan` must have been created with TC_PLAN_CHECKSUM.  checksums: DEVICE pointer to
 * n_tensors uint64 accumulators; the call zeroes them on `stream` and the kernel adds to them.
 * Definition.  Tensor i is read as little-endian 4-byte words x_u at tensor-relative offsets
 * 4u.  With  key(u) = ((u * 0x9E3779B1) << 1 | 1) mod 2^32  (an odd 32-bit weight per position),
 * checksums[i] = sum of x_u * key(u) over the words u of tensor i that this call reads
 * (all of them, or the rank's slice), modulo 2^64: a position-weighted sum, so any change of
 * one word and any exchange of two unequal words changes it.  It depends on positions in the SOURCE
 * tensor, so the checksums of the shards of all ranks add up to the checksum of the whole
 * tensor, and a publisher can store either.  Comparing with the expected values is the
 * caller's step (copy the accumulators back after synchronising the stream).
 */
TC_API int tc_weights_materialize_checksum(const tc_plan_t *plan, const void *blob, void *const *dst_ptrs,
                                           size_t n_dst, uint64_t *checksums, void *stream);

/*
 * Cold path of weight loading: tc_weights_materialize with the blob in a FILE (the
 * storage -> pinned staging buffer -> device memory pipeline of Sec. 5, with the scatter, the
 * rank's slicing and optionally the integrity checksum fused into the device leg).
 * `plan`: a TC_WEIGHTS plan created with TC_PLAN_STREAM.  fd: a file descriptor open for
 * reading (ordinary buffered I/O; the library only calls pread / posix_fadvise on it and never
 * closes it); the blob starts at byte `file_offset` of the file, so a container format's header
 * may precede it.  checksums: NULL, or as for tc_weights_materialize_checksum (the plan then
 * also needs TC_PLAN_CHECKSUM).
 * Reader threads that live for the duration of the call (up to 8) read the plan's chunks, in
 * order, into three 64 MiB pinned host buffers that the library owns (allocated by the first
 * call on a device, kept until tc_trim or exit); as each chunk completes the calling thread
 * hands it to the copy engine and launches the kernel for the chunk's tiles on `stream`.
 * Reading runs up to two chunks ahead of transfer and scatter.
 * The call RETURNS when the last chunk has been read and enqueued, so unlike the other entry
 * points it blocks for about the time the storage reads take; device work completes on
 * `stream` as usual.  Calls on one device are serialised with one another.
 * Errors: everything tc_weights_materialize checks, before the first read; TC_ERR_KIND for a
 * plan without TC_PLAN_STREAM; TC_ERR_IO when a read fails or the file ends early - chunks
 * before the failing one have been enqueued and will still complete, the destination tensors
 * are then partly written (there is no rollback, as for any failure after launch).
 */
TC_API int tc_weights_materialize_file(const tc_plan_t *plan, int fd, int64_t file_offset,
                                       void *const *dst_ptrs, size_t n_dst, uint64_t *checksums,
                                       void *stream);

/*
 * Free the plan's host and device storage.  The caller must first have synchronised every
 * stream that executes it.  NULL is a no-op returning TC_OK.
 */
TC_API int tc_plan_destroy(tc_plan_t *plan);

/*
 * tc_kv_pack without any device allocation.  (The paper has no counterpart: this entry point
 * exists for the library's users, not for one of the paper's operations.)
 *
 * tc_plan_create keeps a plan's descriptors in device memory that it obtains with cudaMalloc.
 * Some callers must not do that: an inference engine that has already handed every free byte
 * of the GPU to its KV pool (a later cudaMalloc fails or eats into that budget), or a
 * scheduler loop that cannot afford the device-wide stall an allocation may cause.  For them
 * this call lowers `spec` (kind TC_KV_PACK, TC_KV_MIGRATE, or the offload group of
 * TC_KV_MIXED) on the host, copies the descriptors into a fixed scratch area that is part of
 * the library image, and launches the same kernel as tc_kv_pack on `stream`, all in one call.
 * It calls no cudaMalloc, cudaFree or other allocating routine; host-side lowering uses
 * ordinary heap memory.  The data buffers are the caller's, exactly as for tc_kv_pack.
 *
 * Capacity: the descriptors and tile list of the call must fit TC_NOALLOC_SCRATCH_BYTES
 * (1 MiB: about 8,000 KV blocks per call); a larger request returns TC_ERR_TOO_LARGE and
 * launches nothing.  Every GPU that loads the library holds that 1 MiB until the process exits.
 *
 * The first call on a device resolves the scratch area's device address for that device (the
 * device must be current, as for every call of this library).  All calls on a device share
 * the one scratch area, and it keeps the
 * previous call's contents: each call overwrites the part it uses and nothing in it needs to
 * start at zero.  Because the area is shared, two calls whose GPU work can overlap - calls on
 * different streams, or from several threads - race on it; issue them on one stream (where the
 * copy of the next call's descriptors is ordered after the previous call's kernel) or
 * synchronise between them.  The descriptor copy comes from pageable host memory, so the call
 * may block until earlier work on `stream` has drained.
 */
#define TC_NOALLOC_SCRATCH_BYTES (1u << 20)
TC_API int tc_kv_pack_noalloc(const tc_plan_spec_t *spec, const void *const *src_bases, size_t n_src,
                              void *const *dst_bases, size_t n_dst, void *stream);

/* ---- off the data path: inspection and diagnostics -------------------------------------- */

typedef struct {
    uint64_t trace_id;
    int32_t kind;
    int32_t executable;            /* 0 for TC_PLAN_HOST_ONLY plans */
    int64_t n_descriptors[2];      /* [0] pack/migrate/offload/weights group, [1] unpack/reload */
    int64_t n_tiles[2];
    int64_t payload_bytes[2];      /* bytes moved by one execution of each group */
    int64_t packed_bytes_required; /* PACK / UNPACK: sum of L*2*T_r*H*D*E */
    int64_t device_bytes;          /* plan storage held on the device */
    int32_t vec_bytes[2];          /* alignment the geometry guarantees, in bytes, up to 16; below 16 - or
                                      with less aligned base pointers - the realigning path runs */
    int32_t launches_per_execute;  /* kernels one execute call launches (1; one per segment for
                                      staged plans) */
    int32_t path[2];               /* 1 direct (zero copy when a buffer is host memory),
                                      3 staged through the copy engines */
    int32_t grid[2];               /* CTAs launched per execution */
    double last_device_us[2];      /* TC_PLAN_TRACE plans: device time of the group's most recent
                                      execution, event to event on the caller's stream; -1 when the
                                      group has not run yet or its last run has not finished (the
                                      query never blocks); 0 for untraced plans */
} tc_plan_stats_t;

/* Fill *out (host pointer) with the plan's figures. */
TC_API int tc_plan_stats(const tc_plan_t *plan, tc_plan_stats_t *out);

/* A lowered descriptor as tests and tools may inspect it: a box of n_outer x rows runs of
 * run_bytes contiguous bytes.  Row k of outer index o starts at
 *   src: slot src_slot + o*src_slot_step, byte src_off + o*src_outer + (k/n0)*src_s1 + (k%n0)*src_s0
 *   dst: likewise.  Slots index the src / dst table of the execute call. */
typedef struct {
    int64_t src_off, dst_off, src_outer, dst_outer, src_s0, src_s1, dst_s0, dst_s1;
    uint32_t src_slot, dst_slot, src_slot_step, dst_slot_step;
    uint32_t run_bytes, n0, rows, n_outer;
    uint32_t rows_per_tile;   /* rows one tile (one CTA pass) moves */
    uint32_t tiles_per_outer; /* tile ids per outer index; parts past the last row are empty */
    uint32_t tile0;           /* global id of tile (outer 0, part 0); tile (o, p) has id
                                 tile0 + (o / planes_per_tile)*tiles_per_outer + p */
    uint32_t planes_per_tile; /* 1, or - small planes, a few KiB each - how many consecutive
                                 outer indices of the descriptor one tile moves */
} tc_descriptor_t;

/* Copy up to `cap` descriptors of `group` (0 or 1) into out (host array); *n_out receives the
 * group's total count. */
TC_API int tc_plan_descriptors(const tc_plan_t *plan, int group, tc_descriptor_t *out, size_t cap,
                        size_t *n_out);

/* One segment (chunk) of a staged or streamed plan: the host bytes [host_off, host_off + bytes)
 * of the blob / packed buffer (a paged host pool: the total of its page runs, host_off = the
 * first run) travel through one staging buffer, and one launch runs
 *   - the tiles [tile0, tile0 + n_tiles) (TC_WEIGHTS plans; n_descs = 0), or
 *   - the window of descriptors [desc0, desc0 + n_descs) x outer indices (planes)
 *     [outer0, outer0 + n_outer) (KV plans; n_tiles = 0)
 * against it, seeing byte host_off of the host side at the start of the staging buffer. */
typedef struct {
    int64_t host_off, bytes;
    uint32_t tile0, n_tiles;
    uint32_t desc0, n_descs, outer0, n_outer;
} tc_segment_t;

/* Copy up to `cap` segments of `group` into out (host array); *n_out receives the count
 * (0 for plans that are not staged). */
TC_API int tc_plan_segments(const tc_plan_t *plan, int group, tc_segment_t *out, size_t cap, size_t *n_out);

/* Give back what the library caches between plans: the pool of device blocks that plan storage
 * is carved from and, if no staged plan exists on the device any more, its staging rings.
 * Synchronises the internal copy streams first.  Safe to call at any time; later calls simply
 * allocate again. */
TC_API int tc_trim(void);

/* Flags a kernel of this library has set on the current device since the last call, then
 * cleared (0 = none).  The execute calls cannot report what happens after the launch; the one
 * condition a kernel can detect and survive is recorded here:
 *   TC_DEVICE_BULK_WAIT_TIMEOUT  a CTA of the realigning path (misaligned geometry or pointers)
 *       waited about a second for its asynchronous bulk copies into shared memory and gave up;
 *       the CTA returned without storing, so the destination of that call is incomplete.  Not
 *       expected to occur; the wait is bounded so that a failure cannot hang the device.
 * flags: host pointer.  The call synchronises the device first (every stream's previously
 * enqueued work, non-blocking streams included) and then copies the word back: it is a
 * diagnostic, off the data path. */
#define TC_DEVICE_BULK_WAIT_TIMEOUT 1u
#define TC_DEVICE_OUT_OF_BOUNDS 2u /* the bounds checker of a TC_PLAN_DEBUG_BOUNDS plan found a descriptor that
                                      reaches outside its table slot; copy kernels of such plans return
                                      without copying while the flag is set (read it to clear it) */
TC_API int tc_device_status(uint32_t *flags);

/* Run only the device-side bounds checker of a TC_PLAN_DEBUG_BOUNDS plan on `stream`: every
 * descriptor of both groups, as it sits in device memory, against the declared extent of its
 * table slots less `shrink` bytes.  shrink = 0 is the real check (a plan that tc_plan_create
 * accepted passes it); a positive shrink pretends every slot is that much smaller and shows the
 * checker firing (tests use it: a plan that uses its slots to the last byte must then raise
 * TC_DEVICE_OUT_OF_BOUNDS).  Nothing is copied.  The outcome is read with tc_device_status. */
TC_API int tc_plan_check_device(const tc_plan_t *plan, int64_t shrink, void *stream);

/* Self-test of that bounded wait: launches one small kernel on `stream` that waits on a barrier
 * nothing will ever arrive at.  The wait gives up after a few milliseconds, the kernel sets
 * TC_DEVICE_BULK_WAIT_TIMEOUT exactly as the copy kernel would and returns normally; the next
 * tc_device_status reports (and clears) the flag.  It shows that a wait which cannot complete ends
 * with a status instead of a hung device. */
TC_API int tc_selftest_wait_timeout(void *stream);

/* Static string naming a status code. */
TC_API const char *tc_strerror(int status);

/* Detail of the calling thread's most recent failure ("" if none); valid until its next call. */
TC_API const char *tc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TENSORCAST_H_ */
