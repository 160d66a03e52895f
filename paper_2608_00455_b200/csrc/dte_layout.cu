// Host side: error plumbing, constant derivation, and the layout compiler that turns the
// transfer plan (Section 4.2.2) into a destination-ordered tile table.
#include <algorithm>
#include <cmath>
#include <cstring>

#include "dte_internal.cuh"

namespace dte {

static thread_local std::string g_last_error;

void set_error(const std::string& msg) { g_last_error = msg; }

dte_status cuda_fail(cudaError_t e, const char* what) {
    set_error(std::string(what) + ": " + cudaGetErrorString(e));
    return DTE_ERR_CUDA;
}

static dte_status fail(dte_status s, const std::string& msg) {
    set_error(msg);
    return s;
}

struct Piece {                 // one operation seen from its destination list
    uint64_t dst_start, len;   // flat destination range
    uint64_t src_start;        // element offset of (a_s0, a_s1) in the source tensor
    uint64_t w, s, rows;       // strided view; contiguous pieces have rows == 1, w == len
    uint32_t tensor;
    size_t op;
};

}  // namespace dte

using namespace dte;

extern "C" const char* dte_status_string(dte_status s) {
    switch (s) {
        case DTE_OK: return "ok";
        case DTE_ERR_INVALID_ARG: return "invalid argument";
        case DTE_ERR_LAYOUT: return "inconsistent layout";
        case DTE_ERR_CAPACITY: return "buffer too small";
        case DTE_ERR_BOUNDS: return "index out of bounds";
        case DTE_ERR_TIMEOUT: return "timed out";
        case DTE_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

extern "C" const char* dte_last_error(void) { return g_last_error.c_str(); }

extern "C" dte_status dte_derive_constants(int64_t step, double lr, double beta1, double beta2,
                                           double eps, double wd, float* out5) {
    if (!out5) return fail(DTE_ERR_INVALID_ARG, "out5 is null");
    if (step < 1) return fail(DTE_ERR_INVALID_ARG, "step must be >= 1 (1-based optimizer step)");
    if (!std::isfinite(lr) || !std::isfinite(beta1) || !std::isfinite(beta2) ||
        !std::isfinite(eps) || !std::isfinite(wd))
        return fail(DTE_ERR_INVALID_ARG, "non-finite hyper-parameter");
    if (beta1 < 0.0 || beta1 >= 1.0 || beta2 < 0.0 || beta2 >= 1.0)
        return fail(DTE_ERR_INVALID_ARG, "betas must lie in [0, 1)");
    if (eps < 0.0) return fail(DTE_ERR_INVALID_ARG, "eps must be >= 0");
    if (lr * wd >= 1.0) return fail(DTE_ERR_INVALID_ARG, "lr * wd must be < 1");
    const double t = (double)step;
    const float bc1 = (float)(1.0 - std::pow(beta1, t));
    const float bc2 = (float)(1.0 - std::pow(beta2, t));
    const float decay = (float)(1.0 - lr * wd);
    if (!(bc1 > 0.f) || !(bc2 > 0.f) || !(decay > 0.f))
        return fail(DTE_ERR_INVALID_ARG, "bias correction or decay factor rounds to <= 0");
    out5[0] = bc1;
    out5[1] = bc2;
    out5[2] = decay;
    out5[3] = (float)lr;
    out5[4] = (float)eps;
    return DTE_OK;
}

extern "C" void dte_layout_destroy(dte_layout* L) {
    if (!L) return;
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(L->device);
    cudaFree(L->d_tiles);
    cudaFree(L->d_packed);
    cudaFree(L->d_segs);
    cudaFree(L->d_rec);
    cudaFree(L->d_block_sum);
    cudaFree(L->d_cursor);
    cudaFree(L->d_stage);
    cudaFree(L->d_rec_base);
    cudaFree((void*)L->d_ptrs);
    cudaFree((void*)L->d_shards);
    cudaFree(L->d_shard_numel);
    cudaFree(L->d_list_first_rec);
    cudaFree(L->d_tensor_group);
    cudaFree(L->d_op_ranges);
    cudaFree(L->d_groups);
    cudaFree(L->d_src_ops);
    cudaFree(L->d_src_op_ptr);
    cudaFree(L->d_tensor_cols);
    cudaFree(L->d_tensor_numel32);
    cudaFree(L->d_recv_first_list);
    cudaFree(L->d_recv_num_ops);
    cudaFree(L->d_op_recv);
    cudaFree(L->d_op_slot);
    cudaFree(L->d_rec_recv);
    cudaFree(L->d_recv_base);
    cudaFree(L->d_targets);
    if (prev >= 0) cudaSetDevice(prev);
    delete L;
}

extern "C" size_t dte_layout_num_lists(const dte_layout* L) { return L ? L->n_lists : 0; }
extern "C" uint64_t dte_layout_num_elements(const dte_layout* L) { return L ? L->scanned : 0; }
extern "C" size_t dte_layout_num_ops(const dte_layout* L) { return L ? L->n_ops : 0; }
extern "C" size_t dte_layout_num_groups(const dte_layout* L) { return L ? L->n_groups : 0; }
extern "C" size_t dte_layout_num_receivers(const dte_layout* L) { return L ? L->n_receivers : 0; }
extern "C" size_t dte_layout_receiver_num_ops(const dte_layout* L, uint32_t receiver) {
    return (L && receiver < L->h_recv_num_ops.size()) ? L->h_recv_num_ops[receiver] : 0;
}

extern "C" uint64_t dte_layout_host_workspace_bytes(const dte_layout* L) {
    if (!L) return 0;
    uint64_t b = 0;
    for (size_t p = 0; p < L->tensor_numel.size(); ++p)
        if (L->tensor_used[p]) {
            if (L->tensor_numel[p] > (uint64_t(1) << 56) || b > (uint64_t(1) << 62)) return UINT64_MAX;   // no such host
            b += 3 * ((L->tensor_numel[p] * 4 + 255) / 256 * 256);
        }
    return b;
}

extern "C" void dte_layout_last_launch(const dte_layout* L, uint64_t* out3) {
    for (int i = 0; i < 3; ++i) out3[i] = L ? L->last_launch[i] : 0;
}

template <class T>
static dte_status upload(T** dst, const std::vector<T>& src, size_t min_elems = 1) {
    size_t n = std::max(src.size(), min_elems);
    DTE_CUDA(cudaMalloc((void**)dst, n * sizeof(T)));
    if (!src.empty())
        DTE_CUDA(cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice));
    return DTE_OK;
}

extern "C" dte_status dte_layout_create(const dte_tensor_desc* tensors, size_t n_tensors,
                                        const dte_shard_desc* shards, size_t n_shards,
                                        const dte_op_desc* ops, size_t n_ops, int device,
                                        dte_layout** out) {
    if (!out) return fail(DTE_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    if ((n_tensors && !tensors) || (n_shards && !shards) || (n_ops && !ops))
        return fail(DTE_ERR_INVALID_ARG, "null descriptor array");
    if (n_tensors >= kNone || n_shards >= kNone || n_ops >= kNone)
        return fail(DTE_ERR_LAYOUT, "too many tensors or shards");

    std::vector<uint64_t> numel(n_tensors);
    for (size_t p = 0; p < n_tensors; ++p) {
        const dte_tensor_desc& t = tensors[p];
        if (t.ndim != 1 && t.ndim != 2) return fail(DTE_ERR_INVALID_ARG, "tensor ndim must be 1 or 2");
        if (t.ndim == 1 && t.shape[1] != 1) return fail(DTE_ERR_INVALID_ARG, "1-D tensor needs shape[1] == 1");
        if (t.group >= 65536) return fail(DTE_ERR_INVALID_ARG, "parameter group index must be < 65536");
        if (t.shape[1] != 0 && t.shape[0] > (uint64_t(1) << 62) / t.shape[1])
            return fail(DTE_ERR_LAYOUT, "tensor too large");
        numel[p] = t.shape[0] * t.shape[1];
    }
    for (size_t k = 0; k < n_shards; ++k)
        if (shards[k].numel >= (uint64_t(1) << 32))
            return fail(DTE_ERR_LAYOUT, "shard numel must be < 2^32 (offsets are uint32)");

    // --- operations -> destination pieces, grouped by list -------------------
    std::vector<std::vector<Piece>> by_list(n_shards);
    std::vector<OpRange> op_ranges(n_ops);
    std::vector<uint8_t> used(n_tensors, 0);
    for (size_t o = 0; o < n_ops; ++o) {
        const dte_op_desc& op = ops[o];
        const std::string tag = "operation " + std::to_string(o) + ": ";
        if (op.src_tensor >= n_tensors || op.dst_shard >= n_shards)
            return fail(DTE_ERR_LAYOUT, tag + "unknown tensor or shard");
        const uint64_t n0 = tensors[op.src_tensor].shape[0], n1 = tensors[op.src_tensor].shape[1];
        const uint64_t e0 = op.extent[0], e1 = op.extent[1];
        op_ranges[o] = OpRange{op.dst_shard, 0, 0, 0};
        if (e0 == 0 || e1 == 0) continue;  // empty overlap: legal, contributes nothing
        if (op.src_origin[0] > n0 || e0 > n0 - op.src_origin[0] || op.src_origin[1] > n1 ||
            e1 > n1 - op.src_origin[1])
            return fail(DTE_ERR_LAYOUT, tag + "overlap leaves the source tensor");
        const bool whole_rows = (op.dst_origin[1] == 0 && e1 == op.dst_ld);
        const bool one_row = (e0 == 1 && op.dst_origin[1] <= op.dst_ld && e1 <= op.dst_ld - op.dst_origin[1]);
        if (!whole_rows && !one_row)
            return fail(DTE_ERR_LAYOUT, tag + "destination region is not a contiguous flat range");
        const uint64_t numel_q = shards[op.dst_shard].numel;
        // all terms < 2^32 after these checks, so the products below cannot overflow
        if (op.dst_base > numel_q || op.dst_ld > numel_q + 1 || op.dst_origin[0] > numel_q)
            return fail(DTE_ERR_LAYOUT, tag + "destination region leaves the shard");
        Piece pc;
        pc.dst_start = op.dst_base + op.dst_origin[0] * op.dst_ld + op.dst_origin[1];
        pc.len = e0 * e1;
        if (pc.dst_start > numel_q || pc.len > numel_q - pc.dst_start)
            return fail(DTE_ERR_LAYOUT, tag + "destination region leaves the shard");
        op_ranges[o].begin = pc.dst_start;
        op_ranges[o].end = pc.dst_start + pc.len;
        pc.src_start = op.src_origin[0] * n1 + op.src_origin[1];
        pc.tensor = op.src_tensor;
        pc.op = o;
        if (e1 == n1 || e0 == 1) {          // source run is contiguous too
            pc.w = pc.len; pc.s = pc.len; pc.rows = 1;
        } else {
            if (n1 >= (uint64_t(1) << 32)) return fail(DTE_ERR_LAYOUT, tag + "strided source row too long");
            pc.w = e1; pc.s = n1; pc.rows = e0;
        }
        used[op.src_tensor] = 1;
        by_list[op.dst_shard].push_back(pc);
    }

    std::vector<TileDesc> tiles, packed;            // regular: one per tile; packed: kSub per tile
    uint32_t n_rec = 0;                             // tiles so far, in output order
    std::vector<uint32_t> rec_list;                 // list of each tile
    std::vector<uint32_t> list_first_tile(n_shards + 1, 0);
    std::vector<SegRec> segs;
    std::vector<uint8_t> has_tiles(n_shards, 0);
    uint64_t scanned = 0;
    for (size_t k = 0; k < n_shards; ++k) {
        auto& P = by_list[k];
        std::sort(P.begin(), P.end(), [](const Piece& a, const Piece& b) { return a.dst_start < b.dst_start; });
        for (size_t i = 1; i < P.size(); ++i)
            if (P[i].dst_start < P[i - 1].dst_start + P[i - 1].len)
                return fail(DTE_ERR_LAYOUT, "operations " + std::to_string(P[i - 1].op) + " and " +
                                                std::to_string(P[i].op) + " overlap in shard " + std::to_string(k));
        bool first = true;
        std::vector<TileDesc> pending;      // pieces (<= kWarpTile slots) waiting to share a CTA
        auto note_tile = [&](uint32_t tile) {
            if (first) list_first_tile[k] = tile;
            first = false;
        };
        auto flush_pending = [&]() {
            if (pending.empty()) return;
            const uint32_t tile = n_rec++;
            rec_list.push_back((uint32_t)k);
            note_tile(tile);
            TileDesc empty;
            std::memset(&empty, 0, sizeof empty);
            pending.resize(kSub, empty);
            for (TileDesc& q : pending) q.tile = tile;
            packed.insert(packed.end(), pending.begin(), pending.end());
            pending.clear();
        };
        for (const Piece& pc : P) {
            scanned += pc.len;
            // a run of <= kTile slots of this piece: a regular tile if full, else warp-level pieces
            auto push = [&](uint64_t src_off, uint64_t dst_off, uint64_t len, uint32_t flags,
                            uint32_t seg, uint32_t col0) {
                TileDesc t;
                t.src_off = src_off;
                t.tensor = pc.tensor;
                t.dst_off = (uint32_t)dst_off;
                t.len_flags = (uint32_t)len | flags;
                t.seg = seg;
                t.col0 = col0;
                if (len == (uint64_t)kTile) {
                    flush_pending();
                    t.tile = n_rec++;
                    rec_list.push_back((uint32_t)k);
                    note_tile(t.tile);
                    tiles.push_back(t);
                    return;
                }
                for (uint64_t c = 0; c < len; c += kWarpTile) {
                    TileDesc q = t;
                    const uint64_t n = std::min<uint64_t>(kWarpTile, len - c);
                    q.dst_off = (uint32_t)(dst_off + c);
                    q.len_flags = (uint32_t)n | flags;
                    if (flags & kFlagStrided) {
                        const uint64_t cc = col0 + c;
                        q.src_off = src_off + (cc / pc.w) * pc.s;
                        q.col0 = (uint32_t)(cc % pc.w);
                    } else {
                        q.src_off = src_off + c;
                    }
                    pending.push_back(q);
                    if (pending.size() == (size_t)kSub) flush_pending();
                }
            };
            if (pc.rows == 1) {
                const bool vec = (pc.src_start % 4 == 0);
                for (uint64_t s = 0; s < pc.len; s += kTile) {
                    const uint64_t len = std::min<uint64_t>(kTile, pc.len - s);
                    push(pc.src_start + s, pc.dst_start + s, len,
                         (vec && len % 4 == 0) ? 0u : kFlagScalar, kNone, 0);
                }
            } else if (pc.w >= 4ull * kTile) {
                // long rows: cut tiles at row ends, each tile is a contiguous source run
                for (uint64_t r = 0; r < pc.rows; ++r)
                    for (uint64_t c0 = 0; c0 < pc.w; c0 += kTile) {
                        const uint64_t len = std::min<uint64_t>(kTile, pc.w - c0);
                        const uint64_t so = pc.src_start + r * pc.s + c0;
                        push(so, pc.dst_start + r * pc.w + c0, len,
                             (so % 4 == 0 && len % 4 == 0) ? 0u : kFlagScalar, kNone, 0);
                    }
            } else {
                SegRec sr;
                sr.w = (uint32_t)pc.w;
                sr.s = (uint32_t)pc.s;
                sr.magic = pc.w >= 2 ? (uint32_t)(((uint64_t(1) << 32) + pc.w - 1) / pc.w) : 0u;
                sr.pad = 0;
                for (uint64_t c = 0; sr.w >= 2 && c < pc.w + kTile; ++c)
                    if ((uint32_t)((c * sr.magic) >> 32) != (uint32_t)(c / pc.w))
                        return fail(DTE_ERR_LAYOUT, "internal: row divisor check failed");
                const uint32_t seg = (uint32_t)segs.size();
                segs.push_back(sr);
                const bool vec = (pc.w % 4 == 0 && pc.s % 4 == 0 && pc.src_start % 4 == 0);
                const uint64_t n = pc.rows * pc.w;
                for (uint64_t s = 0; s < n; s += kTile) {
                    const uint64_t len = std::min<uint64_t>(kTile, n - s);
                    const uint64_t row0 = s / pc.w, col0 = s % pc.w;
                    push(pc.src_start + row0 * pc.s, pc.dst_start + s, len,
                         kFlagStrided | ((vec && len % 4 == 0) ? 0u : kFlagScalar), seg, (uint32_t)col0);
                }
            }
        }
        flush_pending();
        has_tiles[k] = !first;
    }
    const size_t n_ctas = n_rec;
    if (tiles.size() + packed.size() >= kNone) return fail(DTE_ERR_LAYOUT, "too many tiles");

    int prev = -1;
    DTE_CUDA(cudaGetDevice(&prev));
    DTE_CUDA(cudaSetDevice(device));
    dte_layout* L = new dte_layout();
    L->device = device;
    L->n_tensors = (uint32_t)n_tensors;
    L->n_lists = (uint32_t)n_shards;
    L->n_tiles = (uint32_t)n_ctas;
    L->n_regular = (uint32_t)tiles.size();
    L->n_packed = (uint32_t)(packed.size() / kSub);
    L->n_segs = (uint32_t)segs.size();
    L->scanned = scanned;
    L->tensor_numel = numel;
    L->tensor_used = used;
    L->shard_numel.resize(n_shards);
    for (size_t k = 0; k < n_shards; ++k) L->shard_numel[k] = shards[k].numel;
    L->list_has_tiles = has_tiles;
    // first placement record of each list; lists without tiles start where the next list
    // with tiles starts (n_rec if none follows)
    std::vector<uint32_t> first_rec(n_shards, 0);
    list_first_tile[n_shards] = (uint32_t)n_ctas;
    for (size_t k = n_shards; k-- > 0;) {
        if (!has_tiles[k]) list_first_tile[k] = list_first_tile[k + 1];
        first_rec[k] = list_first_tile[k];
    }
    dte_status st = DTE_OK;
    auto guard = [&](dte_status s) { if (st == DTE_OK) st = s; };
    {   // destination base of every placement record, for the gather
        std::vector<uint64_t> rec_base(n_ctas, 0);
        for (const TileDesc& t : tiles) rec_base[t.tile] = t.dst_off;
        for (size_t i = 0; i < packed.size(); i += kSub) rec_base[packed[i].tile] = kRecBasePacked | (uint64_t)(i / kSub);
        guard(upload(&L->d_rec_base, rec_base));
    }
    guard(upload(&L->d_tiles, tiles));
    guard(upload(&L->d_packed, packed));
    guard(upload(&L->d_segs, segs));
    guard(upload(&L->d_shard_numel, L->shard_numel));
    guard(upload(&L->d_list_first_rec, first_rec));
    guard(upload(&L->d_op_ranges, op_ranges));
    L->n_ops = (uint32_t)n_ops;
    {   // destination-side mapping tables (host only until first used)
        L->h_src_op_ptr.assign(n_tensors + 1, 0);
        L->h_tensor_cols.resize(n_tensors);
        L->h_tensor_numel32.resize(n_tensors);
        for (size_t p = 0; p < n_tensors; ++p) {
            const bool fits = numel[p] < (uint64_t(1) << 32);
            if (used[p] && !fits) L->canonical_ok = false;
            L->h_tensor_cols[p] = fits ? (uint32_t)tensors[p].shape[1] : 0u;
            L->h_tensor_numel32[p] = fits ? (uint32_t)numel[p] : 0u;
        }
        for (size_t o = 0; o < n_ops; ++o)
            if (ops[o].extent[0] && ops[o].extent[1]) L->h_src_op_ptr[ops[o].src_tensor + 1] += 1;
        for (size_t p = 0; p < n_tensors; ++p) L->h_src_op_ptr[p + 1] += L->h_src_op_ptr[p];
        L->h_src_ops.resize(L->h_src_op_ptr[n_tensors]);
        std::vector<uint32_t> at(L->h_src_op_ptr.begin(), L->h_src_op_ptr.end() - 1);
        if (L->canonical_ok)
            for (size_t o = 0; o < n_ops; ++o) {
                const dte_op_desc& op = ops[o];
                if (!op.extent[0] || !op.extent[1]) continue;
                SrcOp so;
                so.a0 = (uint32_t)op.src_origin[0]; so.a1 = (uint32_t)op.src_origin[1];
                so.e0 = (uint32_t)op.extent[0]; so.e1 = (uint32_t)op.extent[1];
                so.dst0 = (uint32_t)op_ranges[o].begin;
                so.shard = op.dst_shard;
                so.ld = op.dst_ld;
                L->h_src_ops[at[op.src_tensor]++] = so;
            }
    }
    {   // receivers: who owns which list, tile and operation (used by dte_extract_delta_push only)
        uint64_t max_recv = 0;       // 64 bits: a receiver id of 2^32 - 1 must not wrap to a count of zero
        for (size_t k = 0; k < n_shards; ++k) max_recv = std::max<uint64_t>(max_recv, (uint64_t)shards[k].receiver + 1);
        if (n_shards && max_recv <= 65535) {
            const uint32_t n_recv = (uint32_t)max_recv;
            L->n_receivers = n_recv;
            // [0, n_recv): first list of each receiver; [n_recv, 2 n_recv): one past its last list
            // (both 0 for a receiver without shards: an empty slice)
            L->h_recv_first_list.assign(2 * (size_t)n_recv, 0u);
            std::vector<uint32_t> count(n_recv, 0);
            for (size_t k = n_shards; k-- > 0;) L->h_recv_first_list[shards[k].receiver] = (uint32_t)k;
            for (size_t k = 0; k < n_shards; ++k) {
                L->h_recv_first_list[n_recv + shards[k].receiver] = (uint32_t)k + 1;
                count[shards[k].receiver] += 1;
            }
            // the slice of a receiver is contiguous in the output iff its shards are consecutive
            for (uint32_t r = 0; r < n_recv; ++r)
                if (count[r] && L->h_recv_first_list[n_recv + r] - L->h_recv_first_list[r] != count[r])
                    L->recv_contiguous = false;
            L->h_recv_num_ops.assign(n_recv, 0);
            L->h_op_recv.resize(n_ops);
            L->h_op_slot.resize(n_ops);
            for (size_t o = 0; o < n_ops; ++o) {
                const uint32_t r = shards[ops[o].dst_shard].receiver;
                L->h_op_recv[o] = r;
                L->h_op_slot[o] = L->h_recv_num_ops[r]++;
            }
            L->h_rec_recv.resize(rec_list.size());
            for (size_t t = 0; t < rec_list.size(); ++t) L->h_rec_recv[t] = (uint16_t)shards[rec_list[t]].receiver;
        } else {
            L->recv_contiguous = false;
        }
    }
    {
        std::vector<uint32_t> grp(n_tensors);
        for (size_t p = 0; p < n_tensors; ++p) {
            grp[p] = tensors[p].group;
            L->n_groups = std::max(L->n_groups, tensors[p].group + 1);
        }
        guard(upload(&L->d_tensor_group, grp));
    }
    if (st == DTE_OK) {
        const size_t n_records = n_ctas;
        const size_t n_blocks = (n_records + kRecsPerBlock - 1) / kRecsPerBlock;
        cudaError_t e = cudaMalloc((void**)&L->d_rec, std::max<size_t>(1, n_records) * sizeof(uint64_t));
        if (e == cudaSuccess) e = cudaMalloc((void**)&L->d_block_sum, std::max<size_t>(1, n_blocks) * sizeof(uint64_t));
        // staging cursor, count of non-finite elements, push ticket, spare: all rest at zero
        if (e == cudaSuccess) e = cudaMalloc((void**)&L->d_cursor, 4 * sizeof(uint64_t));
        if (e == cudaSuccess) e = cudaMemset(L->d_cursor, 0, 4 * sizeof(uint64_t));
        if (e == cudaSuccess) L->scratch_clean = true;
        if (e == cudaSuccess) e = cudaMalloc((void**)&L->d_groups, L->n_groups * sizeof(GroupConsts));
        if (e == cudaSuccess) e = cudaMalloc((void**)&L->d_ptrs, std::max<size_t>(1, 3 * n_tensors) * sizeof(void*));
        if (e == cudaSuccess) e = cudaMalloc((void**)&L->d_shards, std::max<size_t>(1, n_shards) * sizeof(void*));
        if (e != cudaSuccess) st = cuda_fail(e, "cudaMalloc(layout scratch)");
    }
    if (prev >= 0) cudaSetDevice(prev);
    if (st != DTE_OK) {
        std::string keep = g_last_error;
        dte_layout_destroy(L);
        set_error(keep);
        return st;
    }
    *out = L;
    return DTE_OK;
}
