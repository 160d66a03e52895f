// Internal structures shared by the layout compiler and the kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "dte.h"

namespace dte {

// ---- tiling ---------------------------------------------------------------
// The destination space (lists in shard order, ascending offset inside a list) is cut into
// tiles, the work of one CTA each, numbered in output order: the output position of a tile
// is the exclusive prefix sum of the changed counts of all tiles before it.
//   regular tile: kTile consecutive receiver-local slots of ONE operation, one descriptor;
//       warp w takes slots [w * kWarpTile, (w+1) * kWarpTile).  The descriptor address
//       depends on blockIdx only, so everything decoded from it lives in uniform registers.
//   packed tile: runs shorter than a tile (ragged ends, small tensors, one-row operations)
//       are cut into pieces of <= kWarpTile slots; kSub consecutive pieces of one list -
//       possibly from different operations and source tensors - share a CTA, each warp with
//       a descriptor of its own (unused slots have length 0).  Handled by a second launch.
// A tile never spans two lists.
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
// Measured on B200 (8 Qwen3-8B layers, 1.5 % changed): 3 items x 3 chunks at 4 CTAs/SM (64
// registers, 36 KB of queue) streams 6.4 TB/s; 4 x 2 at 3 CTAs/SM 6.0; 2 x 4 at 5 CTAs/SM 6.1;
// any shape whose queues push shared memory past ~150 KB/SM loses the L1 and drops below 4.6.
constexpr int kItems = 3;                              // float4 loads per thread, array and chunk
constexpr int kChunk = 32 * 4 * kItems;                // elements a warp loads at once: 384
constexpr int kChunksPerWarpTile = 3;
constexpr int kWarpTile = kChunk * kChunksPerWarpTile; // 1152
constexpr int kSub = 8;                                // warp-tiles per tile
constexpr int kTile = kSub * kWarpTile;                // 9216 elements
static_assert(kTile < 16384, "a tile's changed count must fit kRecCountBits");
constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr int kMaxDevices = 64;                        // device ordinals with per-device host state

constexpr uint32_t kLenMask = 0xFFFFu;
constexpr uint32_t kFlagScalar = 1u << 18;             // not 16-byte alignable: scalar loads
constexpr uint32_t kFlagStrided = 1u << 19;            // crosses source rows (see SegRec)

struct __align__(32) TileDesc {
    uint64_t src_off;    // element offset in the source tensor of the run's row start
    uint32_t tensor;     // source tensor index
    uint32_t dst_off;    // receiver-local offset of the run's first element
    uint32_t len_flags;  // low 16 bits: elements (0: padding); high bits: kFlag*
    uint32_t tile;       // index of the tile (placement record) this descriptor belongs to
    uint32_t seg;        // SegRec index when strided
    uint32_t col0;       // strided: column (within the operation's extent) of the first element
};
static_assert(sizeof(TileDesc) == 32, "TileDesc must be one 32-byte sector");

// A strided operation reads `w` elements from each source row of stride `s`.
// For a tile element with c = col0 + e:  row = c / w = umulhi(c, magic), col = c - row*w,
// source element = src_off + row*s + col.  magic = ceil(2^32 / w), verified on the host
// for every c a tile can produce.
struct SegRec {
    uint32_t w, s, magic, pad;
};

// ---- placement ------------------------------------------------------------------
// The streaming kernel appends each tile's changed entries, in order, to a staging buffer
// at a position taken from an atomic cursor (tiles land in arrival order), and records
// (position << kRecCountBits | count) per tile.  A scan over the records then gives every
// tile its final, ordered output position and a gather moves the entries there.  Nothing in the path waits on another CTA.
constexpr int kRecCountBits = 14;                      // count <= kTile
constexpr uint64_t kRecCountMask = (1ull << kRecCountBits) - 1;
constexpr int kRecsPerBlock = 64;                      // records one gather CTA handles
constexpr int kSmallBlocks = 64;                       // layouts up to this many gather blocks: one gather launch
// A staged entry is one 32-bit word: (warp * kWarpTile + element index in the warp-tile) in the low
// 16 bits, the BF16 value in the high 16.  The gather turns it into (offset, value) with the tile's
// destination base: rec_base[r] = dst_off of a regular tile, or kRecBasePacked | index of a packed
// tile, whose eight pieces have a dst_off each.  (Writing full offsets and values into two staging
// arrays cost a third more write traffic in the middle of the read stream.)
constexpr uint64_t kRecBasePacked = 1ull << 63;

struct Consts {
    float bc1, bc2, decay, lr, eps;
};

// Constants of the conservative "cannot have changed" screen (see dte_extract.cu).
struct Screen {
    float ka, kb, kc, kappa, tiny;
};

// Per-parameter-group constants (exact path + screen), read with three 16-byte loads.
struct __align__(16) GroupConsts {
    Consts c;
    Screen s;
    float pad[2];
};
static_assert(sizeof(GroupConsts) == 48, "GroupConsts is read as three uint4");

struct GatherParams {
    const uint64_t* rec;
    uint64_t* block_sum;             // n_blocks; reduce writes sums, scan turns them into bases
    uint32_t n_rec, n_blocks;
    const uint32_t* list_first_rec;  // n_lists: first record of each list (n_rec if none follows)
    uint32_t n_lists;
    uint64_t scanned;
    const uint32_t* stage;           // staged words (see ExtractParams)
    const uint64_t* rec_base;        // n_rec: destination base of each tile (see kRecBasePacked)
    const TileDesc* packed;          // packed descriptors, kSub per packed tile
    uint32_t* offsets;
    uint16_t* values;
    uint64_t capacity;
    uint64_t* list_ptr;
    uint64_t* counters;
    unsigned long long* cursor;      // staging cursor and non-finite count: left at zero for the next call
    // delivery to the receivers (dte_extract_delta_push); n_recv == 0: none
    uint32_t n_recv;
    const uint32_t* recv_first_list; // n_recv: first list of each receiver (then n_recv: one past its last)
    uint64_t* recv_base;             // n_recv: output position where each receiver's slice starts
    const uint16_t* rec_recv;        // n_rec: receiver of each tile's list
    const dte_push_target* targets;  // n_recv, device copy
};

struct ExtractParams {
    const TileDesc* tiles;       // regular tiles: one descriptor each
    const TileDesc* packed;      // packed tiles: kSub descriptors each
    uint32_t n_regular, n_packed;
    const SegRec* segs;
    const float* const* theta;   // device table, n_tensors
    const float* const* m;
    const float* const* v;
    unsigned long long* cursor;  // [0] entries appended to the staging buffer, [1] non-finite elements seen; both rest at zero
    uint64_t* rec;               // n_tiles placement records (written in full)
    uint32_t* stage;             // staging buffer, stage_capacity words: tile-relative index | value << 16
    uint64_t stage_capacity;
    Consts c;                    // single-group calls: constants in the kernel parameters
    Screen s;
    uint32_t force_flags;           // OR-ed into every tile's flags: kFlagScalar when a source pointer of the call is not 16-byte aligned
    const uint32_t* tensor_group;   // per-group calls: group of each source tensor ...
    const GroupConsts* groups;      // ... and the constants of each group (NULL otherwise)
};


struct ApplyParams {
    const uint32_t* offsets;
    const uint16_t* values;
    uint64_t capacity;
    const uint64_t* list_ptr;
    uint64_t* counters;
    uint16_t* const* shards;     // device table, n_lists
    const uint64_t* shard_numel; // device table, n_lists
    uint32_t n_lists;
};

// One operation as the destination-side mapping needs it (Eq. 5-6 per received canonical entry):
// membership a <= u < a + e, then j = dst0 + (u0 - a0) * ld + (u1 - a1).  Sorted by source tensor,
// plan order within a tensor.
struct __align__(16) SrcOp {
    uint32_t a0, a1, e0, e1;
    uint32_t dst0;       // flat receiver index of the region's first element (< 2^32)
    uint32_t shard;
    uint64_t ld;
};
static_assert(sizeof(SrcOp) == 32, "SrcOp is read as two uint4");

struct CanonParams {
    const uint32_t* indices;       // canonical flat indices, list p = source tensor p
    const uint16_t* values;
    uint64_t capacity;
    const uint64_t* list_ptr;      // n_tensors + 1
    uint64_t* counters;
    uint16_t* const* shards;       // device table, n_shards (NULL: another receiver's)
    const uint64_t* shard_numel;
    uint32_t n_tensors;
    const SrcOp* ops;
    const uint32_t* op_ptr;        // n_tensors + 1
    const uint32_t* tensor_cols;   // n_tensors: n_s[1]
    const uint32_t* tensor_numel;  // n_tensors
};

// Destination range of one operation, in plan order (for the per-operation counts).
struct OpRange {
    uint32_t list;
    uint32_t pad;
    uint64_t begin, end;   // receiver-local flat range [begin, end); begin == end for empty overlaps
};

// Closing kernel of dte_extract_delta_push: per-operation counts, list boundaries and the status
// block of every receiver.
struct PushFinishParams {
    const OpRange* ranges;
    uint32_t n_ops;
    const uint32_t* op_recv;          // n_ops: receiver of the operation's shard
    const uint32_t* op_slot;          // n_ops: position among that receiver's operations (plan order)
    const uint32_t* offsets;          // the sender's own lists
    const uint64_t* list_ptr;
    const uint64_t* counters;
    uint64_t capacity;
    uint32_t n_lists;
    uint32_t n_recv;
    const uint32_t* recv_first_list;  // 2 n_recv: first list, then one past the last list
    const uint32_t* recv_num_ops;     // n_recv
    const dte_push_target* targets;   // n_recv, device copy
    uint64_t epoch;
    unsigned int* ticket;             // rests at zero
};

// Chunk codec (storage-mediated path).
struct PackParams {
    const uint32_t* offsets;
    const uint16_t* values;
    const uint64_t* list_ptr;
    const uint64_t* counters;   // of the delta: an overflowed delta is not packed
    uint64_t capacity;          // of the delta
    uint32_t n_lists, chunk_entries, format;
    uint8_t* stream;
    uint64_t stream_capacity;
    dte_chunk_ref* dir;
    uint64_t dir_capacity;      // chunks the directory can hold (it has one more entry)
    uint64_t* info;
};

struct UnpackParams {
    const uint8_t* stream;
    uint64_t stream_bytes;
    const dte_chunk_ref* dir;
    uint64_t n_chunks;
    uint32_t n_lists;
    const uint64_t* list_ptr;
    uint32_t* offsets;
    uint16_t* values;
    uint64_t capacity;
    uint64_t* counters;   // {entries written, chunks accepted, DTE_DEV_* bits, chunks rejected}
};

#ifdef __CUDACC__
// Totals of one extract, once the number of changed entries is known: every counter word is
// written (no memset of the caller's counters is needed), and lists after which no tile follows
// end - and start - at the total.  Called by `n_threads` threads of one CTA with tid = 0 .. n_threads-1.
__device__ __forceinline__ void gather_finish_totals(const GatherParams& p, uint64_t total, uint32_t tid,
                                                     uint32_t n_threads, bool with_recv_base) {
    if (tid == 0) {
        p.counters[0] = total;
        p.counters[1] = p.scanned;
        p.counters[2] = total > p.capacity ? (uint64_t)DTE_DEV_OVERFLOW : 0ull;
        p.counters[3] = __ldcg(p.cursor + 1);      // non-finite elements the extract counted (atomics: L2)
        p.cursor[1] = 0ull;                         // ready for the next call
        p.list_ptr[p.n_lists] = total;
    }
    for (uint32_t k = tid; k < p.n_lists; k += n_threads)
        if (p.list_first_rec[k] >= p.n_rec) p.list_ptr[k] = total;
    // where each receiver's slice starts: the output position of the first tile of its first list
    // (block bases are final and visible to this CTA by now)
    for (uint32_t r = tid; with_recv_base && r < p.n_recv; r += n_threads) {
        const uint32_t fl = p.recv_first_list[r];
        const uint32_t fr = fl < p.n_lists ? p.list_first_rec[fl] : p.n_rec;
        uint64_t pos = total;
        if (fr < p.n_rec) {
            const uint32_t b = fr / kRecsPerBlock;
            pos = __ldcg(p.block_sum + b);
            for (uint32_t j = b * kRecsPerBlock; j < fr; ++j) pos += __ldcg(p.rec + j) & kRecCountMask;
        }
        p.recv_base[r] = pos;
    }
}
#endif

void set_error(const std::string& msg);
dte_status cuda_fail(cudaError_t e, const char* what);

#define DTE_CUDA(call)                                             \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return dte::cuda_fail(e__, #call); \
    } while (0)

dte_status launch_extract(const ExtractParams& p, bool div_bc1, bool div_decay, cudaStream_t st);
dte_status launch_gather(const GatherParams& p, bool small, cudaStream_t st);
dte_status launch_apply(const ApplyParams& p, int device, cudaStream_t st);
dte_status launch_apply_canonical(const CanonParams& p, int device, cudaStream_t st);
dte_status launch_pack_chunks(const PackParams& p, int device, cudaStream_t st);
dte_status launch_unpack_chunks(const UnpackParams& p, int device, cudaStream_t st);
dte_status launch_push_finish(const PushFinishParams& p, cudaStream_t st);
dte_status launch_push_wait(const uint64_t* status, uint64_t epoch, uint32_t timeout_ms, uint64_t* counters,
                            cudaStream_t st);
dte_status launch_op_counts(const OpRange* ranges, uint32_t n_ops, const dte_delta& d, uint32_t n_lists,
                            uint64_t* counts, cudaStream_t st);

}  // namespace dte

struct dte_layout {
    int device = 0;
    uint32_t n_tensors = 0, n_lists = 0, n_tiles = 0, n_segs = 0;
    uint64_t scanned = 0;
    std::vector<uint64_t> tensor_numel;
    std::vector<uint8_t> tensor_used;
    std::vector<uint64_t> shard_numel;
    std::vector<uint8_t> list_has_tiles;
    // device memory owned by the layout
    dte::TileDesc* d_tiles = nullptr;      // n_regular descriptors
    dte::TileDesc* d_packed = nullptr;     // n_packed * kSub descriptors
    uint32_t n_regular = 0, n_packed = 0;  // n_tiles = n_regular + n_packed
    dte::SegRec* d_segs = nullptr;
    uint64_t* d_rec = nullptr;             // n_tiles placement records
    uint64_t* d_block_sum = nullptr;       // one word per gather block
    uint64_t* d_cursor = nullptr;          // staging cursor, non-finite count, ticket of the push's closing kernel: all rest at zero
    bool scratch_clean = false;            // the last call was enqueued completely, so they are at zero
    uint32_t* d_stage = nullptr;           // staging buffer, grown on demand to the caller's capacity
    uint64_t* d_rec_base = nullptr;        // n_tiles: destination base per placement record
    uint64_t stage_capacity = 0;
    const float** d_ptrs = nullptr;        // 3 * n_tensors source pointers
    uint16_t** d_shards = nullptr;         // n_lists
    uint64_t* d_shard_numel = nullptr;     // n_lists
    uint32_t* d_list_first_rec = nullptr;  // n_lists
    uint32_t* d_tensor_group = nullptr;    // n_tensors
    dte::GroupConsts* d_groups = nullptr;  // n_groups
    uint32_t n_groups = 1;
    dte::OpRange* d_op_ranges = nullptr;   // n_ops, plan order
    uint32_t n_ops = 0;
    // destination-side mapping tables: built at create on the host, uploaded by the first call
    // that needs them (dte_apply_canonical)
    std::vector<dte::SrcOp> h_src_ops;
    std::vector<uint32_t> h_src_op_ptr, h_tensor_cols, h_tensor_numel32;
    bool canonical_ok = true;              // every tensor an operation reads has numel < 2^32
    dte::SrcOp* d_src_ops = nullptr;
    uint32_t* d_src_op_ptr = nullptr;
    uint32_t* d_tensor_cols = nullptr;
    uint32_t* d_tensor_numel32 = nullptr;
    // receivers (dte_extract_delta_push): host tables from create, device copies on first use
    uint32_t n_receivers = 0;
    bool recv_contiguous = true;           // every receiver's shards are consecutive in shard order
    std::vector<uint32_t> h_recv_first_list, h_recv_num_ops, h_op_recv, h_op_slot;
    std::vector<uint16_t> h_rec_recv;
    uint32_t* d_recv_first_list = nullptr;
    uint32_t* d_recv_num_ops = nullptr;
    uint32_t* d_op_recv = nullptr;
    uint32_t* d_op_slot = nullptr;
    uint16_t* d_rec_recv = nullptr;
    uint64_t* d_recv_base = nullptr;
    dte_push_target* d_targets = nullptr;
    std::vector<dte_push_target> h_targets;
    bool targets_valid = false;
    // host mirrors of the pointer tables last uploaded
    std::vector<const float*> h_ptrs;
    std::vector<uint16_t*> h_shards;
    bool ptrs_valid = false, shards_valid = false;
    bool scalar_loads = false;             // the current call's source pointers are not all 16-byte aligned
    uint64_t last_launch[3] = {0, 0, 0};
};
