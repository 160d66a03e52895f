/*
 * dte.h - C ABI of the B200 delta-transfer hot path.
 *
 * One pass over a trainer's live AdamW state produces, for every receiver-local
 * inference tensor, the ordered list of BF16 elements that changed in the last
 * optimizer step; a second call scatters such lists into BF16 shard buffers.
 *
 * The operations follow the paper's problem statement:
 *   - Eq. 2 (Section 4.1): the previous fp32 master weight is reconstructed from the
 *     current weight and the AdamW moments by inverting the decoupled AdamW step;
 *   - Eq. 4 (Section 4.2.1): both versions are cast to BF16, their 16-bit patterns are
 *     compared, and changed indices with their *target* values are extracted;
 *   - Eq. 5-6 (Section 4.2.2): each changed index is unravelled, matched against the
 *     precomputed hyper-rectangular overlaps of the transfer plan, and ravelled into
 *     receiver-local coordinates;
 *   - Eq. 7 (Section 4.3): the receiver scatters the values into its live shard.
 *
 * Conventions
 *   - "device pointer" = CUDA global memory of the layout's device; "host pointer" =
 *     ordinary or pinned host memory.  The library never frees or keeps caller memory.
 *   - All tensors are row-major and contiguous.  fp32 inputs should be 16-byte aligned (any
 *     framework allocation is); a call in which some theta / m / v pointer is only 4-byte aligned -
 *     a view into a flat buffer at an odd element - is served with scalar loads throughout, at a
 *     fraction of the speed.
 *   - Every call that takes a stream enqueues on it (void* = cudaStream_t; NULL = the
 *     default stream) and returns without synchronising unless stated otherwise.
 *   - Functions return DTE_OK or an error detected on the host.  Conditions only the
 *     device can detect are reported as DTE_DEV_* bits in dte_delta.counters[2].
 *   - A layout may be used by one extract or apply call at a time (its scratch memory
 *     is per layout).  Different layouts are independent.
 *   - Scratch: the layout owns its device tables, one 8-byte placement record per 9216
 *     scanned elements, and a staging buffer of `capacity` 4-byte words.  The staging buffer is
 *     allocated by the first extract call and re-allocated (with a stream synchronisation) only
 *     when a later call passes a larger capacity.
 *   - What a call enqueues: an extract whose pointer tables equal those of the previous call on
 *     the layout and whose capacity does not exceed an earlier one enqueues kernels only - at
 *     most three for layouts of up to 4096 tiles (37.7 M scanned elements), five beyond - and no
 *     copy or memset: the kernels write every word of `counters` and leave the layout's scratch
 *     ready for the next call.  So dte_extract_delta + dte_apply can be captured into a CUDA
 *     graph after one ordinary call and replayed on new contents of the same buffers.
 *   - There is no CPU fallback: every entry point needs a CUDA device.
 */
#ifndef DTE_H_
#define DTE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DTE_API __attribute__((visibility("default")))
#else
#define DTE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum dte_status {
    DTE_OK = 0,
    DTE_ERR_INVALID_ARG = 1, /* null pointer, bad hyper-parameter, misaligned tensor      */
    DTE_ERR_LAYOUT = 2,      /* the tensor / shard / operation tables are inconsistent    */
    DTE_ERR_CAPACITY = 3,    /* a caller-provided buffer is too small (host-detected)     */
    DTE_ERR_BOUNDS = 4,      /* reserved for host-side bound checks                       */
    DTE_ERR_TIMEOUT = 5,     /* reserved                                                  */
    DTE_ERR_CUDA = 6         /* a CUDA runtime call failed; see dte_last_error()          */
} dte_status;

/* Device-detected conditions, OR-ed into dte_delta.counters[2]. */
#define DTE_DEV_OVERFLOW 1u /* more changed elements than `capacity`; lists not produced   */
#define DTE_DEV_BOUNDS 2u   /* apply met an offset >= numel of its shard, an entry for a NULL
                               shard, or a canonical index outside its tensor; entry skipped */
#define DTE_DEV_TIMEOUT 4u  /* dte_push_wait gave up; no other kernel of this library waits   */
#define DTE_DEV_CORRUPT 8u  /* unpack rejected a chunk (header or checksum); lists have holes */

/* Source tensor p of the canonical training-side space: fp32, row-major.  ndim is 1 or 2;
 * for ndim == 1 shape[1] must be 1.  `group` is the tensor's parameter group (< 65536): the
 * paper's lambda is a per-group weight-decay coefficient and eta_t a per-group learning rate
 * (Section 4.1); dte_extract_delta uses one pair for all groups, dte_extract_delta_groups one
 * pair per group. */
typedef struct dte_tensor_desc {
    uint64_t shape[2];
    uint32_t ndim;
    uint32_t group;
} dte_tensor_desc;

/* Receiver-local destination tensor q, flattened; BF16; numel < 2^32.  One output list
 * per shard descriptor, in descriptor order.  `receiver` is informational. */
typedef struct dte_shard_desc {
    uint64_t numel;
    uint32_t receiver;
    uint32_t reserved;
} dte_shard_desc;

/* One operation o of the transfer plan (Section 4.2.2): the overlap of source tensor
 * `src_tensor` and destination `dst_shard`.  A source coordinate u with
 *     src_origin <= u < src_origin + extent      (component-wise, Eq. 5 and the test after it)
 * maps to the receiver-local flat index (Eq. 6)
 *     j = dst_base + (u0 - src_origin[0] + dst_origin[0]) * dst_ld + (u1 - src_origin[1] + dst_origin[1]).
 * The destination region must be one contiguous flat range: either whole destination rows
 * (dst_origin[1] == 0 and extent[1] == dst_ld) or a single row (extent[0] == 1).
 * Regions of different operations in the same shard must not overlap; slots no operation
 * covers are never emitted and never written. */
typedef struct dte_op_desc {
    uint32_t src_tensor;
    uint32_t dst_shard;
    uint64_t src_origin[2];
    uint64_t extent[2];
    uint64_t dst_base;
    uint64_t dst_ld;
    uint64_t dst_origin[2];
} dte_op_desc;

typedef struct dte_layout dte_layout;

/* Output of extract / input of apply.  All pointers are device pointers owned by the
 * caller.  List k (shard k) occupies entries [list_ptr[k], list_ptr[k+1]) of `offsets`
 * (receiver-local element offsets, strictly ascending within a list) and `values` (BF16
 * bit patterns of theta_t, Eq. 4).  Empty lists keep their slot.
 *   offsets  : capacity x uint32        values : capacity x uint16
 *   list_ptr : (n_shards + 1) x uint64
 *   counters : 4 x uint64 = { total changed, elements scanned, DTE_DEV_* bits, non-finite }
 *              non-finite: scanned elements (a replicated element once per receiver) whose
 *              reconstructed previous value broke - it is NaN (a NaN in theta or a moment, a
 *              negative v, 0/0), or +-Inf although theta is finite (the update overflowed).  The
 *              paper does not say what to do with such values; they are compared like any other
 *              bit pattern, and counted here so that the caller can notice a diverged optimizer
 *              state.  An infinite theta that stays infinite is not counted.
 * If the total exceeds `capacity`, DTE_DEV_OVERFLOW is set, offsets / values hold nothing
 * usable, and list_ptr / counters[0] still hold the exact sizes, so the caller can grow
 * the buffers and call again (Section 3: sizes are learnt in a step of their own, before
 * any payload moves). */
typedef struct dte_delta {
    uint32_t* offsets;
    uint16_t* values;
    uint64_t capacity;
    uint64_t* list_ptr;
    uint64_t* counters;
} dte_delta;

/* Compiles the plan into device tables on `device` (Section 4.2.2: the plan is computed
 * once from shard metadata, before any synchronisation).  Host arrays in, handle out.
 * Allocates the layout's device tables and scratch with cudaMalloc; synchronous.
 * Errors: DTE_ERR_INVALID_ARG (null arrays, ndim, group >= 65536), DTE_ERR_LAYOUT (operation
 * outside its tensor or shard, non-contiguous or overlapping destination regions,
 * numel >= 2^32), DTE_ERR_CUDA. */
DTE_API dte_status dte_layout_create(const dte_tensor_desc* tensors, size_t n_tensors,
                             const dte_shard_desc* shards, size_t n_shards,
                             const dte_op_desc* ops, size_t n_ops, int device, dte_layout** out);

/* Frees the handle and its device memory.  NULL is ignored. */
DTE_API void dte_layout_destroy(dte_layout* layout);

/* Number of output lists (== n_shards). */
DTE_API size_t dte_layout_num_lists(const dte_layout* layout);
/* Number of parameter groups the layout's tensors refer to (largest group index + 1). */
DTE_API size_t dte_layout_num_groups(const dte_layout* layout);
/* Elements one extract call scans (sum of extents; replicated tensors count per copy). */
DTE_API uint64_t dte_layout_num_elements(const dte_layout* layout);
/* Bytes of device workspace dte_extract_delta_host needs (12 bytes per source element,
 * each tensor padded to 256 bytes); UINT64_MAX if the sum does not fit 64 bits. */
DTE_API uint64_t dte_layout_host_workspace_bytes(const dte_layout* layout);

/* The call-uniform fp32 scalars of Eq. 2, derived in double and rounded once:
 * out5 = { 1-beta1^step, 1-beta2^step, 1-lr*wd, lr, eps }.  Host only.
 * Errors (DTE_ERR_INVALID_ARG): step < 1, betas outside [0,1), eps < 0, non-finite
 * inputs, lr*wd >= 1, or a bias correction / decay that rounds to <= 0. */
DTE_API dte_status dte_derive_constants(int64_t step, double lr, double beta1, double beta2, double eps,
                                double wd, float* out5);

/* Eq. 2 + Eq. 4 + Eq. 5-6 in one streaming pass.  theta / m / v: HOST arrays of
 * n_tensors DEVICE pointers (fp32, 16-byte aligned for full speed; entries of tensors no operation
 * reads may be NULL).  `step` is the 1-based index of the optimizer step that produced
 * theta.  Arithmetic: IEEE binary32, every operation rounded to nearest-even on its own,
 * no fused multiply-add across operations, subnormals kept; BF16 by round-to-nearest-even
 * with NaN -> 0x7FC0; +0 and -0 are different patterns.  Deterministic: the same inputs
 * give the same bytes.  Writes every field of `out` described above. */
DTE_API dte_status dte_extract_delta(const dte_layout* layout, const float* const* theta,
                             const float* const* m, const float* const* v, int64_t step,
                             double lr, double beta1, double beta2, double eps, double wd,
                             const dte_delta* out, void* cuda_stream);

/* dte_extract_delta with per-parameter-group learning rate and weight decay (Eq. 2: eta_t and
 * lambda belong to the parameter group of the element).  lr / wd: HOST arrays of n_groups
 * doubles, n_groups >= dte_layout_num_groups(layout); tensor p uses entry tensors[p].group.
 * step, beta1, beta2 and eps are shared.  Everything else as dte_extract_delta. */
DTE_API dte_status dte_extract_delta_groups(const dte_layout* layout, const float* const* theta,
                                            const float* const* m, const float* const* v, int64_t step,
                                            double beta1, double beta2, double eps, const double* lr,
                                            const double* wd, size_t n_groups, const dte_delta* out,
                                            void* cuda_stream);

/* Allocation-free variant of dte_extract_delta.  The paper has no counterpart: this exists
 * for callers that may not allocate device memory at the point where they extract - a
 * trainer whose framework has claimed the whole GPU for its own caching allocator, so that a
 * raw cudaMalloc would fail or fragment it; a process running under a fixed memory budget; a
 * latency-critical loop that cannot afford the implicit synchronisation of cudaMalloc /
 * cudaFree.  dte_extract_delta grows a per-layout staging buffer when a call brings a larger
 * `capacity`; this entry point never does.  Its placement records, block sums, cursor and
 * staging buffer live in one fixed array inside the library's device image (about 8.5 MiB;
 * every GPU that loads the library holds it until the process exits), and it calls no
 * cudaMalloc, cudaFree or other device-allocating routine.
 *   Limits: the layout may have at most DTE_STATIC_MAX_TILES tiles (a tile is the work of one
 * CTA: 9216 consecutive destination slots of one operation, or up to eight shorter runs of one
 * list; a layout of full tiles scans up to 603,979,776 elements, and dte_layout_last_launch
 * reports the tile count of a layout after any extract) and out->capacity at most
 * DTE_STATIC_MAX_CAPACITY entries.  Larger requests return DTE_ERR_CAPACITY with the numbers in
 * dte_last_error(); nothing is enqueued.
 *   The first call on a device looks up the array's address on that device (a host-side
 * query, once per device and process); make that first call before starting a stream capture.
 *   All calls on a device share the array, and it keeps what the last call left.  The call
 * clears the one word that must start at zero and overwrites the rest before reading it, so
 * back-to-back calls on one stream are safe; two calls that can overlap on the GPU (different
 * streams, different layouts or host threads) race on the array and corrupt each other.
 *   Arguments, results and all other error behaviour are those of dte_extract_delta; the
 * caller still provides every input and output buffer. */
#define DTE_STATIC_MAX_TILES 65536u
#define DTE_STATIC_MAX_CAPACITY 2097152u
DTE_API dte_status dte_extract_delta_static(const dte_layout* layout, const float* const* theta,
                                            const float* const* m, const float* const* v, int64_t step,
                                            double lr, double beta1, double beta2, double eps, double wd,
                                            const dte_delta* out, void* cuda_stream);

/* Eq. 7: shard[k][offsets[e]] = values[e] for every entry e of every list k.
 * shard_ptrs: HOST array of n_shards DEVICE pointers (BF16 buffers, numel as declared; a shard
 * whose list is empty may be NULL - a receiver passes only the tensors it holds; an entry that
 * does arrive for a NULL shard is skipped and flagged DTE_DEV_BOUNDS).  Reads list sizes on the device,
 * so it can be enqueued right after extract without a host round trip.  Refuses to write
 * anything (and sets DTE_DEV_OVERFLOW again) if `delta` overflowed its capacity, and nothing
 * if its counters carry DTE_DEV_CORRUPT (lists read from a damaged chunk stream). */
DTE_API dte_status dte_apply(const dte_layout* layout, const dte_delta* delta,
                     uint16_t* const* shard_ptrs, void* cuda_stream);

/* Section 4.4, destination side of the storage-mediated path: the published entries are
 * canonical - list p of `canonical` holds the changed flat indices of SOURCE tensor p (ascending)
 * and their BF16 target values, i.e. Eq. 4's (I, V) per tensor, what an extract over the identity
 * plan of the same tensors produces; list_ptr has n_tensors + 1 entries - and the mapping into
 * the inference layout happens here.  For every entry and every operation of the layout on its
 * tensor, in plan order: u = unravel(i) (Eq. 5), membership src_origin <= u < src_origin + extent,
 * j by Eq. 6, shard[dst_shard][j] = value (Eq. 7).  An operation whose shard pointer is NULL is
 * skipped (the tensor lives on another receiver), so one plan serves every receiver.  Refuses, like
 * dte_apply, a delta that overflowed or carries DTE_DEV_CORRUPT; an index outside its tensor or a
 * j outside its shard is skipped and flagged DTE_DEV_BOUNDS.  The first call on a layout uploads
 * its per-tensor operation tables (cudaMalloc, synchronous; 32 bytes per operation).  Cost is
 * proportional to the operations per source tensor: meant for canonical (HF-shaped) sources.
 * Errors: DTE_ERR_LAYOUT if a tensor the plan reads has >= 2^32 elements. */
DTE_API dte_status dte_apply_canonical(const dte_layout* layout, const dte_delta* canonical,
                                       uint16_t* const* shard_ptrs, void* cuda_stream);

/* Section 4.3, round 1 of the two-round transfer: the entry count c_o = |I_o| of every
 * operation of the plan, in plan order, zero-length operations included (both peers keep
 * the position of an empty operation, so the schedule stays aligned).  `counts`: DEVICE array
 * of dte_layout_num_ops(layout) uint64.  Entries of operation o are those of list dst_shard(o)
 * whose offset lies in the operation's destination range, a contiguous run of that list.  Like
 * dte_apply it may be enqueued right after the extract: if `delta` turns out incomplete (its
 * counters carry DTE_DEV_OVERFLOW or DTE_DEV_CORRUPT, or its total exceeds its capacity) every
 * count is written as zero, DTE_DEV_OVERFLOW is set and no entry is read. */
DTE_API dte_status dte_op_counts(const dte_layout* layout, const dte_delta* delta, uint64_t* counts,
                                 void* cuda_stream);
/* Number of operations the layout was created with. */
DTE_API size_t dte_layout_num_ops(const dte_layout* layout);

/* ---- Same-cluster transfer fused into the extract's tail (Section 4.3) ----------------------------
 * Section 4.3 moves the update in two rounds: first the entry count of every planned operation,
 * zeros included, then indices and values in the same order; a receiver applies an update only
 * once all of it has arrived.  With NVLink peer access the sender can store straight into the
 * receivers' memory, so both rounds collapse into the kernel that already moves every changed
 * entry from the staging buffer to its ordered position: dte_extract_delta_push makes that kernel
 * store each entry a second time, into the landing buffers of the receiver that owns the entry's
 * list, and a closing kernel delivers, per receiver, the list boundaries, the per-operation counts
 * (plan order, zeros included) and - after a system-scope fence, last of all - a status block
 * whose epoch word tells the receiver that everything before it is complete.
 *
 * A receiver is the value of dte_shard_desc.receiver; the shards of one receiver must be
 * consecutive in shard order (then its entries are one contiguous slice of the output).  All
 * pointers of a target are DEVICE pointers this GPU can store to: its own memory, or a peer's
 * mapped by CUDA peer access or IPC.  Only plain stores go to them.
 *   offsets / values : `capacity` entries; receive the receiver's slice, lists in shard order
 *   list_ptr  : (n_shards + 1) x uint64, boundaries RELATIVE to the slice; lists of other
 *               receivers come out empty, so {offsets, values, capacity, list_ptr, counters} is a
 *               dte_delta that dte_apply takes with the full layout and NULL for foreign shards
 *   op_counts : dte_layout_receiver_num_ops(layout, r) x uint64: c_o of the operations whose
 *               shard belongs to receiver r, in plan order, zeros included
 *   status    : 4 x uint64 = { entries of the slice, epoch, DTE_DEV_* bits, operations }.  The
 *               epoch word is written last (release at system scope).  DTE_DEV_OVERFLOW: the slice
 *               exceeds `capacity`, or the sender's own delta overflowed; list_ptr and the entry
 *               total are exact, the entries are not usable (and if it was the sender's delta
 *               that overflowed, the per-operation counts are all zero). */
typedef struct dte_push_target {
    uint32_t* offsets;
    uint16_t* values;
    uint64_t capacity;
    uint64_t* list_ptr;
    uint64_t* op_counts;
    uint64_t* status;
} dte_push_target;

/* Number of receivers (largest dte_shard_desc.receiver + 1; 0 without shards) and the number of
 * operations whose shard belongs to `receiver`. */
DTE_API size_t dte_layout_num_receivers(const dte_layout* layout);
DTE_API size_t dte_layout_receiver_num_ops(const dte_layout* layout, uint32_t receiver);

/* dte_extract_delta that also delivers every receiver's share (see above).  `out` is filled
 * exactly as by dte_extract_delta (the sender keeps its lists: the storage path or a retry may
 * need them).  targets: HOST array of n_receivers >= dte_layout_num_receivers(layout) entries; a
 * receiver without shards is skipped, a target whose `status` is NULL as well (nothing is
 * delivered to it).  `epoch` is the value the receivers wait for: use one the status word cannot
 * hold already, e.g. the policy version.  The first call on a layout uploads its receiver tables
 * (cudaMalloc, synchronous).  Errors: DTE_ERR_LAYOUT if some receiver's shards are not
 * consecutive; DTE_ERR_INVALID_ARG for null buffers of a used target; else as dte_extract_delta. */
DTE_API dte_status dte_extract_delta_push(const dte_layout* layout, const float* const* theta,
                                          const float* const* m, const float* const* v, int64_t step,
                                          double lr, double beta1, double beta2, double eps, double wd,
                                          const dte_delta* out, const dte_push_target* targets,
                                          size_t n_receivers, uint64_t epoch, void* cuda_stream);

/* Receiver side: enqueues a one-thread kernel that waits until status[1] == epoch (acquire at
 * system scope), for at most timeout_ms milliseconds, and then fills `counters` (DEVICE, 4 x
 * uint64) = { status[0], 0, status[2], 0 } so that a dte_apply enqueued behind it on the same
 * stream sees a complete dte_delta.  If the time runs out, DTE_DEV_TIMEOUT is set in counters[2]
 * together with DTE_DEV_OVERFLOW (so that dte_apply writes nothing) and the kernel returns; the
 * context stays usable.  The wait holds one thread of one SM; enqueue it only when the sender's
 * push is known to be on its way (on one GPU: after it, on the same stream), never in front of
 * work it depends on.  timeout_ms is capped at 10000. */
DTE_API dte_status dte_push_wait(const uint64_t* status, uint64_t epoch, uint32_t timeout_ms,
                                 uint64_t* counters, int device, void* cuda_stream);

/* ---- Chunk codec of the storage-mediated path (Section 4.4) ---------------------------------
 * Between clusters the changes travel through object storage (Section 4.4): what changed is
 * written out in chunks, four bytes of index and two bytes of BF16 value per element, next to a
 * manifest that says where each chunk lies, how long it is and what it must hash to; the
 * destination checks the chunks before it applies them.
 * The paper prints no byte layout; this library's is:
 *   stream  : chunks back to back, each on a 16-byte boundary, lists in order, entries of a
 *             list in ascending order, at most `chunk_entries` entries of ONE list per chunk,
 *             no chunk for an empty list.
 *   chunk   : 32-byte header + payload.  Header = eight little-endian uint32: DTE_CHUNK_MAGIC,
 *             format, list, first_entry (rank of the chunk's first entry within its list),
 *             count, payload_bytes, checksum, 0.
 *   payload : DTE_CHUNK_PLAIN - count x int32 index, count x BF16 value, zeros to a multiple
 *             of 16 bytes.  DTE_CHUNK_BYTE_PLANES - six planes of P = count rounded up to a
 *             multiple of 16 bytes: byte 0, 1, 2, 3 of every index, byte 0, 1 of every value,
 *             each zero-padded; the same entries transposed so that a byte-oriented compressor
 *             (the paper uses Zstandard, a host library outside this path) finds the slowly
 *             varying bytes together.  DTE_CHUNK_DELTA_PLANES - as the byte planes, but the index
 *             planes hold the gaps g_0 = index_0, g_i = index_i - index_{i-1} within the chunk
 *             (lists ascend, so the upper gap planes are almost all zero); the reader restores
 *             the indices by a running sum modulo 2^32.  Smallest under a compressor.
 *   checksum: Adler-32 (RFC 1950) of header bytes [0, 24) followed by the payload.
 *   directory (the manifest's locations): one dte_chunk_ref per chunk and a final entry
 *             {total bytes, 0xFFFFFFFF, 0}.
 * Lists are whatever the layout's shards are: with an identity plan (every source tensor its
 * own destination) they are the canonical (index, value) pairs of Eq. 4 that this path ships. */
#define DTE_CHUNK_MAGIC 0x43455444u /* "DTEC" */
#define DTE_CHUNK_HEADER_BYTES 32u
#define DTE_CHUNK_PLAIN 0u
#define DTE_CHUNK_BYTE_PLANES 1u
#define DTE_CHUNK_DELTA_PLANES 2u
#define DTE_CHUNK_MAX_ENTRIES 1048576u

typedef struct dte_chunk_ref {
    uint64_t byte_offset; /* of the chunk's header in the stream; multiple of 16 */
    uint32_t list;
    uint32_t first_entry;
} dte_chunk_ref;

/* Upper bounds for sizing: chunks (the directory needs one entry more) and stream bytes for a
 * delta of at most `entries` entries in `n_lists` lists.  Host only; 0 if chunk_entries is 0. */
DTE_API uint64_t dte_chunk_count_bound(size_t n_lists, uint64_t entries, uint32_t chunk_entries);
DTE_API uint64_t dte_chunk_bytes_bound(size_t n_lists, uint64_t entries, uint32_t chunk_entries,
                                       uint32_t format);

/* Serialises a complete extract result.  All buffers are DEVICE memory owned by the caller:
 *   stream    : stream_capacity bytes, 16-byte aligned
 *   directory : directory_capacity + 1 entries
 *   info      : 4 x uint64 = { chunks, stream bytes, DTE_DEV_* bits, entries }
 * chunk_entries: a multiple of 8 in [8, DTE_CHUNK_MAX_ENTRIES]; format: DTE_CHUNK_*.
 * Sizes are found on the device (no host round trip after extract).  If the delta overflowed,
 * or the chunks do not fit the directory or the stream, DTE_DEV_OVERFLOW is set in info[2] and
 * nothing is serialised; in the second case info[0] and info[1] hold the exact requirement.
 * Deterministic: the same lists give the same bytes.  Errors: DTE_ERR_INVALID_ARG, DTE_ERR_CUDA. */
DTE_API dte_status dte_pack_chunks(const dte_layout* layout, const dte_delta* delta, uint32_t chunk_entries,
                                   uint32_t format, void* stream, uint64_t stream_capacity,
                                   dte_chunk_ref* directory, uint64_t directory_capacity, uint64_t* info,
                                   void* cuda_stream);

/* Reads a stream back into lists.  stream / directory: DEVICE memory (stream 16-byte aligned;
 * n_chunks + 1 directory entries, as published).  out->list_ptr is an INPUT here: the list
 * boundaries from the manifest ((num_lists + 1) x uint64, device); out->offsets / values receive
 * the entries; out->counters = { entries written, chunks accepted, DTE_DEV_* bits, chunks
 * rejected }.  A chunk is rejected - none of its entries written, DTE_DEV_CORRUPT set - when the
 * directory places it outside the stream or off a 16-byte boundary, when its header disagrees
 * with the directory, the lists or its own size, or when its checksum does not match; the
 * checksum is verified before the first entry of the chunk is written.  dte_apply refuses a
 * delta whose counters carry DTE_DEV_CORRUPT.  If list_ptr's total exceeds out->capacity every
 * chunk is rejected and DTE_DEV_OVERFLOW is set as well. */
DTE_API dte_status dte_unpack_chunks(const dte_layout* layout, const void* stream, uint64_t stream_bytes,
                                     const dte_chunk_ref* directory, uint64_t n_chunks,
                                     const dte_delta* out, void* cuda_stream);

/* End-to-end variant for optimizer state that lives in HOST memory (pinned for full
 * copy speed).  Copies theta / m / v (HOST arrays of n_tensors HOST pointers) into
 * `workspace` (device, >= dte_layout_host_workspace_bytes), runs the same extract into
 * `out` (device buffers, as above), then copies counters, list_ptr and the filled part
 * of offsets / values to the given host buffers (offsets_h / values_h hold `capacity`
 * entries; either may be NULL to skip that copy).  SYNCHRONISES the stream before
 * returning.  Returns DTE_ERR_CAPACITY if the delta overflowed. */
DTE_API dte_status dte_extract_delta_host(const dte_layout* layout, const float* const* theta_h,
                                  const float* const* m_h, const float* const* v_h, int64_t step,
                                  double lr, double beta1, double beta2, double eps, double wd,
                                  void* workspace, uint64_t workspace_bytes, const dte_delta* out,
                                  uint32_t* offsets_h, uint16_t* values_h, uint64_t* list_ptr_h,
                                  uint64_t* counters_h, void* cuda_stream);

/* Static strings. */
DTE_API const char* dte_status_string(dte_status s);
/* Message of the calling thread's most recent failed call ("" if none). */
DTE_API const char* dte_last_error(void);

/* Launch statistics of the most recent extract on this layout (host bookkeeping):
 * out3 = { tiles, CTAs launched, kernels launched by the call }. */
DTE_API void dte_layout_last_launch(const dte_layout* layout, uint64_t* out3);

#ifdef __cplusplus
}
#endif
#endif /* DTE_H_ */
