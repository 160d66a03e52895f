// C entry points that enqueue the kernels: the extract variants, dte_apply, dte_op_counts,
// the chunk codec and the host-buffer variant dte_extract_delta_host.
#include <atomic>
#include <cmath>
#include <cstring>
#include <limits>

#include "dte_internal.cuh"

using namespace dte;

namespace {

dte_status fail(dte_status s, const char* msg) {
    set_error(msg);
    return s;
}

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        cudaGetDevice(&prev);
        if (prev != dev) cudaSetDevice(dev); else prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

dte_status check_delta(const dte_delta* d) {
    if (!d) return fail(DTE_ERR_INVALID_ARG, "delta is null");
    if (!d->list_ptr || !d->counters) return fail(DTE_ERR_INVALID_ARG, "delta.list_ptr / counters is null");
    if (d->capacity && (!d->offsets || !d->values))
        return fail(DTE_ERR_INVALID_ARG, "delta.offsets / values is null with capacity > 0");
    return DTE_OK;
}

// Upload the per-call source pointer table unless it equals the one already on the device.
dte_status sync_source_table(dte_layout* L, const float* const* theta, const float* const* m,
                             const float* const* v, cudaStream_t st) {
    const size_t n = L->n_tensors;
    std::vector<const float*> tab(3 * n);
    bool unaligned = false;
    for (size_t p = 0; p < n; ++p) {
        tab[p] = theta[p]; tab[n + p] = m[p]; tab[2 * n + p] = v[p];
        if (!L->tensor_used[p]) continue;
        if (!theta[p] || !m[p] || !v[p]) return fail(DTE_ERR_INVALID_ARG, "null theta / m / v pointer for a tensor the plan reads");
        const uintptr_t bits = (uintptr_t)theta[p] | (uintptr_t)m[p] | (uintptr_t)v[p];
        if (bits & 3u) return fail(DTE_ERR_INVALID_ARG, "theta / m / v must be 4-byte aligned");
        // A tensor that is only 4-byte aligned (a view into a flat buffer at an odd element)
        // cannot be read with 128-bit loads: the whole call then takes the scalar-load path.
        if (bits & 15u) unaligned = true;
    }
    L->scalar_loads = unaligned;
    if (L->ptrs_valid && tab == L->h_ptrs) return DTE_OK;
    L->ptrs_valid = false;
    // pageable source: the runtime stages the bytes before returning, so `tab` may die
    if (n) DTE_CUDA(cudaMemcpyAsync((void*)L->d_ptrs, tab.data(), tab.size() * sizeof(void*), cudaMemcpyHostToDevice, st));
    L->h_ptrs.swap(tab);
    L->ptrs_valid = true;
    return DTE_OK;
}

// Constants of the kernel's conservative screen (see dte_extract.cu), each rounded up:
//   ka    >= 1 / bc1
//   kb    >= sqrt(bc2) * (1 + 2^-10)
//   kc    >= 1 / eps                      (+inf when eps == 0)
//   kappa >= (|1/decay - 1| + 2^-24) * (1 + 2^-7) * (1 + 2^-10)
//   tiny  >= 2^-133 * kappa + 2^-148    (the absolute part of the decay bound, for subnormal ranges)
float round_up(double x) {
    if (!(x == x)) return std::numeric_limits<float>::infinity();
    float f = (float)x;
    if ((double)f < x) f = std::nextafter(f, std::numeric_limits<float>::infinity());
    return f;
}

Screen make_screen(const Consts& c) {
    const double infl = 1.0 + 1.0 / 1024.0;
    Screen s;
    s.ka = round_up(1.0 / (double)c.bc1);
    s.kb = round_up(std::sqrt((double)c.bc2) * infl);
    s.kc = c.eps > 0.f ? round_up(1.0 / (double)c.eps) : std::numeric_limits<float>::infinity();
    s.kappa = round_up((std::fabs(1.0 / (double)c.decay - 1.0) + std::ldexp(1.0, -24)) * (1.0 + 1.0 / 128.0) * infl);
    s.tiny = round_up(std::ldexp((double)s.kappa, -133) + std::ldexp(1.0, -148));
    return s;
}

// Where one extract call keeps its placement records, block sums, staging cursor and staged
// entries: the layout's own buffers, or the fixed array of the allocation-free entry point.
struct Scratch {
    uint64_t* cursor;       // two words: the staging cursor, the count of non-finite elements
    uint64_t* rec;
    uint64_t* block_sum;
    uint32_t* stage;
    bool clear_first;       // the two words are not known to be zero: clear them in the stream
};

// Enqueues the kernels of one extract: both extract launches (packed and regular tiles), then
// what puts the staged entries in order - one launch for layouts of at most kSmallBlocks gather
// blocks (every block scans the records itself), else reduce, scan and move.  `groups`:
// per-parameter-group constants (NULL: `c` applies to every tensor).  The scan writes every word
// of out->counters, and it leaves the cursor at zero, the only scratch word that must start
// there (records and block sums are rewritten in full, staged entries are read only where this
// call wrote them): an ordinary call enqueues kernels and nothing else.
dte_status enqueue_kernels(dte_layout* L, const Consts& c, const std::vector<GroupConsts>* groups,
                           const Scratch& sc, const dte_delta* out, cudaStream_t st, bool push = false) {
    if (L->n_tiles == 0) {
        DTE_CUDA(cudaMemsetAsync(out->counters, 0, 4 * sizeof(uint64_t), st));
        DTE_CUDA(cudaMemsetAsync(out->list_ptr, 0, (L->n_lists + 1) * sizeof(uint64_t), st));
        L->last_launch[0] = 0; L->last_launch[1] = 0; L->last_launch[2] = 0;
        return DTE_OK;
    }
    if (sc.clear_first) DTE_CUDA(cudaMemsetAsync(sc.cursor, 0, 2 * sizeof(uint64_t), st));
    GatherParams g;
    g.rec = sc.rec;
    g.block_sum = sc.block_sum;
    g.n_rec = L->n_tiles;
    g.n_blocks = (L->n_tiles + kRecsPerBlock - 1) / kRecsPerBlock;
    g.list_first_rec = L->d_list_first_rec;
    g.n_lists = L->n_lists;
    g.scanned = L->scanned;
    g.stage = sc.stage;
    g.rec_base = L->d_rec_base;
    g.packed = L->d_packed;
    g.offsets = out->offsets;
    g.values = out->values;
    g.capacity = out->capacity;
    g.list_ptr = out->list_ptr;
    g.counters = out->counters;
    g.cursor = reinterpret_cast<unsigned long long*>(sc.cursor);
    g.n_recv = push ? L->n_receivers : 0;
    g.recv_first_list = L->d_recv_first_list;
    g.recv_base = L->d_recv_base;
    g.rec_recv = L->d_rec_recv;
    g.targets = L->d_targets;
    const bool small = g.n_blocks <= (uint32_t)kSmallBlocks;
    ExtractParams p;
    p.segs = L->d_segs;
    p.theta = L->d_ptrs;
    p.m = L->d_ptrs + L->n_tensors;
    p.v = L->d_ptrs + 2 * (size_t)L->n_tensors;
    p.cursor = reinterpret_cast<unsigned long long*>(sc.cursor);
    p.rec = sc.rec;
    p.stage = sc.stage;
    p.stage_capacity = out->capacity;
    p.c = c;
    p.s = make_screen(c);
    p.tensor_group = nullptr;
    p.groups = nullptr;
    p.force_flags = L->scalar_loads ? kFlagScalar : 0u;
    bool div_bc1 = c.bc1 != 1.0f, div_decay = c.decay != 1.0f;
    if (groups) {
        // pageable source: staged by the runtime before the call returns
        DTE_CUDA(cudaMemcpyAsync(L->d_groups, groups->data(), groups->size() * sizeof(GroupConsts),
                                 cudaMemcpyHostToDevice, st));
        p.tensor_group = L->d_tensor_group;
        p.groups = L->d_groups;
        div_bc1 = div_decay = false;
        for (const GroupConsts& gc : *groups) {
            div_bc1 |= gc.c.bc1 != 1.0f;
            div_decay |= gc.c.decay != 1.0f;
        }
    }
    // one CTA per tile, packed tiles (short runs sharing a CTA; few) and full tiles: they share
    // nothing but the staging cursor (atomic) and write different placement records
    p.tiles = L->d_tiles;
    p.packed = L->d_packed;
    p.n_regular = L->n_regular;
    p.n_packed = L->n_packed;
    dte_status s = launch_extract(p, div_bc1, div_decay, st);
    if (s != DTE_OK) return s;
    s = launch_gather(g, small, st);
    if (s != DTE_OK) return s;
    L->last_launch[0] = L->n_tiles;
    L->last_launch[1] = L->n_tiles;                         // one CTA per tile
    L->last_launch[2] = (small ? 1 : 3) + (L->n_regular ? 1 : 0) + (L->n_packed ? 1 : 0);
    return DTE_OK;
}

// The ordinary entry points keep their scratch in the layout.  The staging buffer mirrors the
// caller's capacity; it is (re)allocated only when a call brings a larger capacity than any
// before it.
dte_status enqueue_extract(dte_layout* L, const Consts& c, const dte_delta* out, cudaStream_t st,
                           const std::vector<GroupConsts>* groups = nullptr, bool push = false) {
    if (L->n_tiles && out->capacity > L->stage_capacity) {
        DTE_CUDA(cudaStreamSynchronize(st));
        cudaFree(L->d_stage);
        L->d_stage = nullptr;
        L->stage_capacity = 0;
        DTE_CUDA(cudaMalloc((void**)&L->d_stage, out->capacity * sizeof(uint32_t)));
        L->stage_capacity = out->capacity;
    }
    // The kernels leave the cursor at zero.  If an earlier call stopped half-way (a launch failed),
    // it may not be: clear it in the stream this once.
    const Scratch sc{L->d_cursor, L->d_rec, L->d_block_sum, L->d_stage, !L->scratch_clean};
    L->scratch_clean = false;
    const dte_status s = enqueue_kernels(L, c, groups, sc, out, st, push);
    L->scratch_clean = (s == DTE_OK);
    return s;
}

}  // namespace

extern "C" dte_status dte_extract_delta(const dte_layout* layout, const float* const* theta,
                                        const float* const* m, const float* const* v, int64_t step,
                                        double lr, double beta1, double beta2, double eps, double wd,
                                        const dte_delta* out, void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    if (layout->n_tensors && (!theta || !m || !v)) return fail(DTE_ERR_INVALID_ARG, "null pointer table");
    dte_status s = check_delta(out);
    if (s != DTE_OK) return s;
    float c5[5];
    s = dte_derive_constants(step, lr, beta1, beta2, eps, wd, c5);
    if (s != DTE_OK) return s;
    dte_layout* L = const_cast<dte_layout*>(layout);  // scratch and pointer-table cache
    DeviceGuard g(L->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    s = sync_source_table(L, theta, m, v, st);
    if (s != DTE_OK) return s;
    const Consts c{c5[0], c5[1], c5[2], c5[3], c5[4]};
    return enqueue_extract(L, c, out, st);
}

extern "C" dte_status dte_extract_delta_groups(const dte_layout* layout, const float* const* theta,
                                               const float* const* m, const float* const* v,
                                               int64_t step, double beta1, double beta2, double eps,
                                               const double* lr, const double* wd, size_t n_groups,
                                               const dte_delta* out, void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    if (layout->n_tensors && (!theta || !m || !v)) return fail(DTE_ERR_INVALID_ARG, "null pointer table");
    if (!lr || !wd) return fail(DTE_ERR_INVALID_ARG, "lr / wd array is null");
    if (n_groups < layout->n_groups) return fail(DTE_ERR_INVALID_ARG, "fewer hyper-parameter groups than the layout's tensors use");
    dte_status s = check_delta(out);
    if (s != DTE_OK) return s;
    std::vector<GroupConsts> groups(layout->n_groups);
    for (size_t gi = 0; gi < groups.size(); ++gi) {
        float c5[5];
        s = dte_derive_constants(step, lr[gi], beta1, beta2, eps, wd[gi], c5);
        if (s != DTE_OK) return s;
        groups[gi].c = Consts{c5[0], c5[1], c5[2], c5[3], c5[4]};
        groups[gi].s = make_screen(groups[gi].c);
        for (float& x : groups[gi].pad) x = 0.f;
    }
    dte_layout* L = const_cast<dte_layout*>(layout);
    DeviceGuard g(L->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    s = sync_source_table(L, theta, m, v, st);
    if (s != DTE_OK) return s;
    return enqueue_extract(L, groups[0].c, out, st, &groups);
}

// ---- extract + delivery to the receivers (Section 4.3) -----------------------------------------
namespace {
template <class T>
dte_status upload_once(T** dst, const std::vector<T>& src) {
    if (*dst) return DTE_OK;
    T* ptr = nullptr;
    DTE_CUDA(cudaMalloc((void**)&ptr, std::max<size_t>(1, src.size()) * sizeof(T)));
    if (!src.empty()) {
        const cudaError_t e = cudaMemcpy(ptr, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { cudaFree(ptr); return cuda_fail(e, "upload of the receiver tables"); }
    }
    *dst = ptr;
    return DTE_OK;
}
}  // namespace

extern "C" dte_status dte_extract_delta_push(const dte_layout* layout, const float* const* theta,
                                             const float* const* m, const float* const* v, int64_t step,
                                             double lr, double beta1, double beta2, double eps, double wd,
                                             const dte_delta* out, const dte_push_target* targets,
                                             size_t n_receivers, uint64_t epoch, void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    if (layout->n_tensors && (!theta || !m || !v)) return fail(DTE_ERR_INVALID_ARG, "null pointer table");
    dte_status s = check_delta(out);
    if (s != DTE_OK) return s;
    dte_layout* L = const_cast<dte_layout*>(layout);
    if (L->n_receivers == 0) return fail(DTE_ERR_LAYOUT, "the layout has no receivers (no shards, or receiver ids above 65534)");
    if (!L->recv_contiguous)
        return fail(DTE_ERR_LAYOUT, "the shards of some receiver are not consecutive in shard order: its entries are not one slice");
    if (!targets || n_receivers < L->n_receivers) return fail(DTE_ERR_INVALID_ARG, "fewer targets than receivers");
    std::vector<dte_push_target> tab(targets, targets + L->n_receivers);
    for (uint32_t r = 0; r < L->n_receivers; ++r) {
        dte_push_target& t = tab[r];
        const bool has_shards = L->h_recv_first_list[L->n_receivers + r] > L->h_recv_first_list[r];
        if (!has_shards || !t.status) { t = dte_push_target{}; continue; }     // nothing is delivered to it
        if (!t.list_ptr || (t.capacity && (!t.offsets || !t.values)) || (L->h_recv_num_ops[r] && !t.op_counts))
            return fail(DTE_ERR_INVALID_ARG, "a push target with a status block lacks list_ptr, entry or count buffers");
    }
    float c5[5];
    s = dte_derive_constants(step, lr, beta1, beta2, eps, wd, c5);
    if (s != DTE_OK) return s;
    DeviceGuard g(L->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // first use: receiver tables to the device
    s = upload_once(&L->d_recv_first_list, L->h_recv_first_list);
    if (s == DTE_OK) s = upload_once(&L->d_recv_num_ops, L->h_recv_num_ops);
    if (s == DTE_OK) s = upload_once(&L->d_op_recv, L->h_op_recv);
    if (s == DTE_OK) s = upload_once(&L->d_op_slot, L->h_op_slot);
    if (s == DTE_OK) s = upload_once(&L->d_rec_recv, L->h_rec_recv);
    if (s == DTE_OK && !L->d_recv_base) DTE_CUDA(cudaMalloc((void**)&L->d_recv_base, L->n_receivers * sizeof(uint64_t)));
    if (s == DTE_OK && !L->d_targets) DTE_CUDA(cudaMalloc((void**)&L->d_targets, L->n_receivers * sizeof(dte_push_target)));
    if (s != DTE_OK) return s;
    const bool same = L->targets_valid && L->h_targets.size() == tab.size() &&
                      std::memcmp(L->h_targets.data(), tab.data(), tab.size() * sizeof(dte_push_target)) == 0;
    if (!same) {
        L->targets_valid = false;
        // pageable source: staged by the runtime before the call returns
        DTE_CUDA(cudaMemcpyAsync(L->d_targets, tab.data(), tab.size() * sizeof(dte_push_target), cudaMemcpyHostToDevice, st));
        L->h_targets.swap(tab);
        L->targets_valid = true;
    }
    s = sync_source_table(L, theta, m, v, st);
    if (s != DTE_OK) return s;
    const Consts c{c5[0], c5[1], c5[2], c5[3], c5[4]};
    s = enqueue_extract(L, c, out, st, nullptr, true);
    if (s != DTE_OK) return s;
    PushFinishParams f;
    f.ranges = L->d_op_ranges;
    f.n_ops = L->n_ops;
    f.op_recv = L->d_op_recv;
    f.op_slot = L->d_op_slot;
    f.offsets = out->offsets;
    f.list_ptr = out->list_ptr;
    f.counters = out->counters;
    f.capacity = out->capacity;
    f.n_lists = L->n_lists;
    f.n_recv = L->n_receivers;
    f.recv_first_list = L->d_recv_first_list;
    f.recv_num_ops = L->d_recv_num_ops;
    f.targets = L->d_targets;
    f.epoch = epoch;
    f.ticket = reinterpret_cast<unsigned int*>(L->d_cursor + 2);
    s = launch_push_finish(f, st);
    if (s == DTE_OK) L->last_launch[2] += 1;
    return s;
}

extern "C" dte_status dte_push_wait(const uint64_t* status, uint64_t epoch, uint32_t timeout_ms,
                                    uint64_t* counters, int device, void* cuda_stream) {
    if (!status || !counters) return fail(DTE_ERR_INVALID_ARG, "status / counters is null");
    if (((uintptr_t)status | (uintptr_t)counters) & 7u) return fail(DTE_ERR_INVALID_ARG, "status / counters must be 8-byte aligned");
    DeviceGuard g(device);
    return launch_push_wait(status, epoch, timeout_ms, counters, (cudaStream_t)cuda_stream);
}

namespace {
// Upload the shard pointer table unless it equals the one already on the device.
dte_status sync_shard_table(dte_layout* L, uint16_t* const* shard_ptrs, cudaStream_t st) {
    const size_t n = L->n_lists;
    std::vector<uint16_t*> tab(shard_ptrs, shard_ptrs + n);
    for (size_t k = 0; k < n; ++k)
        if ((uintptr_t)tab[k] & 1u) return fail(DTE_ERR_INVALID_ARG, "shard pointers must be 2-byte aligned");
    if (L->shards_valid && tab == L->h_shards) return DTE_OK;
    L->shards_valid = false;
    DTE_CUDA(cudaMemcpyAsync((void*)L->d_shards, tab.data(), n * sizeof(void*), cudaMemcpyHostToDevice, st));
    L->h_shards.swap(tab);
    L->shards_valid = true;
    return DTE_OK;
}
}  // namespace

extern "C" dte_status dte_apply(const dte_layout* layout, const dte_delta* delta,
                                uint16_t* const* shard_ptrs, void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    dte_status s = check_delta(delta);
    if (s != DTE_OK) return s;
    if (layout->n_lists && !shard_ptrs) return fail(DTE_ERR_INVALID_ARG, "shard pointer table is null");
    dte_layout* L = const_cast<dte_layout*>(layout);
    DeviceGuard g(L->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (L->n_lists == 0) return DTE_OK;
    s = sync_shard_table(L, shard_ptrs, st);
    if (s != DTE_OK) return s;
    ApplyParams p;
    p.offsets = delta->offsets;
    p.values = delta->values;
    p.capacity = delta->capacity;
    p.list_ptr = delta->list_ptr;
    p.counters = delta->counters;
    p.shards = L->d_shards;
    p.shard_numel = L->d_shard_numel;
    p.n_lists = L->n_lists;
    return launch_apply(p, L->device, st);
}

extern "C" dte_status dte_apply_canonical(const dte_layout* layout, const dte_delta* canonical,
                                          uint16_t* const* shard_ptrs, void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    dte_status s = check_delta(canonical);
    if (s != DTE_OK) return s;
    if (layout->n_lists && !shard_ptrs) return fail(DTE_ERR_INVALID_ARG, "shard pointer table is null");
    dte_layout* L = const_cast<dte_layout*>(layout);
    if (!L->canonical_ok)
        return fail(DTE_ERR_LAYOUT, "a source tensor the plan reads has 2^32 or more elements: no uint32 canonical index");
    DeviceGuard g(L->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (L->n_tensors == 0 || L->n_lists == 0) return DTE_OK;
    if (!L->d_src_ops) {      // first use: the per-source-tensor operation tables go to the device
        const size_t n_ops = std::max<size_t>(L->h_src_ops.size(), 1), nt = L->n_tensors;
        DTE_CUDA(cudaMalloc((void**)&L->d_src_op_ptr, (nt + 1) * sizeof(uint32_t)));
        DTE_CUDA(cudaMalloc((void**)&L->d_tensor_cols, nt * sizeof(uint32_t)));
        DTE_CUDA(cudaMalloc((void**)&L->d_tensor_numel32, nt * sizeof(uint32_t)));
        SrcOp* ops = nullptr;
        DTE_CUDA(cudaMalloc((void**)&ops, n_ops * sizeof(SrcOp)));
        cudaError_t e = cudaMemcpy(ops, L->h_src_ops.data(), L->h_src_ops.size() * sizeof(SrcOp), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(L->d_src_op_ptr, L->h_src_op_ptr.data(), (nt + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(L->d_tensor_cols, L->h_tensor_cols.data(), nt * sizeof(uint32_t), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(L->d_tensor_numel32, L->h_tensor_numel32.data(), nt * sizeof(uint32_t), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            cudaFree(ops);
            return cuda_fail(e, "upload of the destination-side mapping tables");
        }
        L->d_src_ops = ops;
    }
    s = sync_shard_table(L, shard_ptrs, st);
    if (s != DTE_OK) return s;
    CanonParams p;
    p.indices = canonical->offsets;
    p.values = canonical->values;
    p.capacity = canonical->capacity;
    p.list_ptr = canonical->list_ptr;
    p.counters = canonical->counters;
    p.shards = L->d_shards;
    p.shard_numel = L->d_shard_numel;
    p.n_tensors = L->n_tensors;
    p.ops = L->d_src_ops;
    p.op_ptr = L->d_src_op_ptr;
    p.tensor_cols = L->d_tensor_cols;
    p.tensor_numel = L->d_tensor_numel32;
    return launch_apply_canonical(p, L->device, st);
}

extern "C" dte_status dte_op_counts(const dte_layout* layout, const dte_delta* delta, uint64_t* counts,
                                    void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    dte_status s = check_delta(delta);
    if (s != DTE_OK) return s;
    if (layout->n_ops && !counts) return fail(DTE_ERR_INVALID_ARG, "counts is null");
    DeviceGuard g(layout->device);
    return launch_op_counts(layout->d_op_ranges, layout->n_ops, *delta, layout->n_lists, counts,
                            (cudaStream_t)cuda_stream);
}

// ---- chunk codec -------------------------------------------------------------------------
extern "C" uint64_t dte_chunk_count_bound(size_t n_lists, uint64_t entries, uint32_t chunk_entries) {
    return chunk_entries ? entries / chunk_entries + n_lists : 0;
}

extern "C" uint64_t dte_chunk_bytes_bound(size_t n_lists, uint64_t entries, uint32_t chunk_entries,
                                          uint32_t format) {
    // per chunk: the header and at most 15 (plain) or 6 * 15 (byte planes) bytes of padding
    const uint64_t pad = format == DTE_CHUNK_PLAIN ? 15 : 90;
    return 6 * entries + dte_chunk_count_bound(n_lists, entries, chunk_entries) * (DTE_CHUNK_HEADER_BYTES + pad);
}

extern "C" dte_status dte_pack_chunks(const dte_layout* layout, const dte_delta* delta, uint32_t chunk_entries,
                                      uint32_t format, void* stream, uint64_t stream_capacity,
                                      dte_chunk_ref* directory, uint64_t directory_capacity,
                                      uint64_t* info, void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    dte_status s = check_delta(delta);
    if (s != DTE_OK) return s;
    if (chunk_entries < 8 || chunk_entries % 8 != 0 || chunk_entries > DTE_CHUNK_MAX_ENTRIES)
        return fail(DTE_ERR_INVALID_ARG, "chunk_entries must be a multiple of 8 in [8, DTE_CHUNK_MAX_ENTRIES]");
    if (format > DTE_CHUNK_DELTA_PLANES) return fail(DTE_ERR_INVALID_ARG, "unknown chunk format");
    if (!directory || !info) return fail(DTE_ERR_INVALID_ARG, "directory / info is null");
    if (stream_capacity && !stream) return fail(DTE_ERR_INVALID_ARG, "stream is null with capacity > 0");
    if ((uintptr_t)stream & 15u) return fail(DTE_ERR_INVALID_ARG, "stream must be 16-byte aligned");
    DeviceGuard g(layout->device);
    PackParams p;
    p.offsets = delta->offsets;
    p.values = delta->values;
    p.list_ptr = delta->list_ptr;
    p.counters = delta->counters;
    p.capacity = delta->capacity;
    p.n_lists = layout->n_lists;
    p.chunk_entries = chunk_entries;
    p.format = format;
    p.stream = (uint8_t*)stream;
    p.stream_capacity = stream_capacity;
    p.dir = directory;
    p.dir_capacity = directory_capacity;
    p.info = info;
    return launch_pack_chunks(p, layout->device, (cudaStream_t)cuda_stream);
}

extern "C" dte_status dte_unpack_chunks(const dte_layout* layout, const void* stream, uint64_t stream_bytes,
                                        const dte_chunk_ref* directory, uint64_t n_chunks,
                                        const dte_delta* out, void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    dte_status s = check_delta(out);
    if (s != DTE_OK) return s;
    if (!directory) return fail(DTE_ERR_INVALID_ARG, "directory is null");
    if (stream_bytes && !stream) return fail(DTE_ERR_INVALID_ARG, "stream is null with bytes > 0");
    if ((uintptr_t)stream & 15u) return fail(DTE_ERR_INVALID_ARG, "stream must be 16-byte aligned");
    DeviceGuard g(layout->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    DTE_CUDA(cudaMemsetAsync(out->counters, 0, 4 * sizeof(uint64_t), st));
    UnpackParams p;
    p.stream = (const uint8_t*)stream;
    p.stream_bytes = stream_bytes;
    p.dir = directory;
    p.n_chunks = n_chunks;
    p.n_lists = layout->n_lists;
    p.list_ptr = out->list_ptr;
    p.offsets = out->offsets;
    p.values = out->values;
    p.capacity = out->capacity;
    p.counters = out->counters;
    return launch_unpack_chunks(p, layout->device, st);
}

extern "C" dte_status dte_extract_delta_host(const dte_layout* layout, const float* const* theta_h,
                                             const float* const* m_h, const float* const* v_h,
                                             int64_t step, double lr, double beta1, double beta2,
                                             double eps, double wd, void* workspace,
                                             uint64_t workspace_bytes, const dte_delta* out,
                                             uint32_t* offsets_h, uint16_t* values_h,
                                             uint64_t* list_ptr_h, uint64_t* counters_h,
                                             void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    if (layout->n_tensors && (!theta_h || !m_h || !v_h)) return fail(DTE_ERR_INVALID_ARG, "null pointer table");
    if (!list_ptr_h || !counters_h) return fail(DTE_ERR_INVALID_ARG, "list_ptr_h / counters_h is null");
    dte_status s = check_delta(out);
    if (s != DTE_OK) return s;
    float c5[5];
    s = dte_derive_constants(step, lr, beta1, beta2, eps, wd, c5);
    if (s != DTE_OK) return s;
    dte_layout* L = const_cast<dte_layout*>(layout);
    if (workspace_bytes < dte_layout_host_workspace_bytes(L)) return fail(DTE_ERR_CAPACITY, "workspace too small");
    if (!workspace && workspace_bytes) return fail(DTE_ERR_INVALID_ARG, "workspace is null");
    if ((uintptr_t)workspace & 255u) return fail(DTE_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    DeviceGuard g(L->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t n = L->n_tensors;
    std::vector<const float*> th(n, nullptr), mm(n, nullptr), vv(n, nullptr);
    char* w = (char*)workspace;
    for (size_t p = 0; p < n; ++p) {
        if (!L->tensor_used[p]) continue;
        if (!theta_h[p] || !m_h[p] || !v_h[p]) return fail(DTE_ERR_INVALID_ARG, "null host tensor pointer");
        const size_t bytes = L->tensor_numel[p] * 4, pad = (bytes + 255) / 256 * 256;
        const float* const src[3] = {theta_h[p], m_h[p], v_h[p]};
        const float** dst[3] = {&th[p], &mm[p], &vv[p]};
        for (int a = 0; a < 3; ++a) {
            DTE_CUDA(cudaMemcpyAsync(w, src[a], bytes, cudaMemcpyHostToDevice, st));
            *dst[a] = (const float*)w;
            w += pad;
        }
    }
    s = sync_source_table(L, th.data(), mm.data(), vv.data(), st);
    if (s != DTE_OK) return s;
    const Consts c{c5[0], c5[1], c5[2], c5[3], c5[4]};
    s = enqueue_extract(L, c, out, st);
    if (s != DTE_OK) return s;
    DTE_CUDA(cudaMemcpyAsync(counters_h, out->counters, 4 * sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
    DTE_CUDA(cudaMemcpyAsync(list_ptr_h, out->list_ptr, (L->n_lists + 1) * sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
    DTE_CUDA(cudaStreamSynchronize(st));
    const uint64_t total = counters_h[0];
    if (total > out->capacity || (counters_h[2] & DTE_DEV_OVERFLOW))
        return fail(DTE_ERR_CAPACITY, "delta buffers too small; counters[0] holds the required capacity");
    if (total && offsets_h) DTE_CUDA(cudaMemcpyAsync(offsets_h, out->offsets, total * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    if (total && values_h) DTE_CUDA(cudaMemcpyAsync(values_h, out->values, total * sizeof(uint16_t), cudaMemcpyDeviceToHost, st));
    DTE_CUDA(cudaStreamSynchronize(st));
    return DTE_OK;
}

// ---- allocation-free extract --------------------------------------------------------------
//
// Same computation as dte_extract_delta, for callers that must not allocate device memory
// while they run.  Everything the ordinary call keeps in per-layout scratch that it may
// have to (re)allocate - the placement records, the gather's block sums, the staging cursor
// and the staging buffer - lives here in one fixed array in the library's device image.
// Each GPU that loads the library carries the array until the process exits.

namespace {

constexpr uint64_t kStaticMaxTiles = DTE_STATIC_MAX_TILES;
constexpr uint64_t kStaticMaxCapacity = DTE_STATIC_MAX_CAPACITY;
constexpr uint64_t kStaticCursorOff = 0;                                       // 256 bytes reserved
constexpr uint64_t kStaticRecOff = 256;
constexpr uint64_t kStaticBlockSumOff = kStaticRecOff + kStaticMaxTiles * 8;
constexpr uint64_t kStaticStageOff =
    kStaticBlockSumOff + ((kStaticMaxTiles + kRecsPerBlock - 1) / kRecsPerBlock) * 8;
constexpr uint64_t kStaticScratchBytes = (kStaticStageOff + kStaticMaxCapacity * 4 + 255) / 256 * 256;
static_assert(kStaticBlockSumOff % 8 == 0 && kStaticStageOff % 8 == 0, "sub-buffers must keep their natural alignment");

// In host code this name is only a handle for the runtime's symbol table, never a device
// address: the address each device gave the array comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// One slot per device ordinal; atomic because two host threads may make their first call on a
// device at the same time (both then ask the runtime and store the same address).
std::atomic<unsigned char*> g_static_addr[kMaxDevices];

// First use on a device (that device current): ask the runtime where the array lives there.
dte_status static_scratch_address(int device, unsigned char** out) {
    if (device < 0 || device >= kMaxDevices) return fail(DTE_ERR_INVALID_ARG, "device ordinal out of range");
    unsigned char* addr = g_static_addr[device].load(std::memory_order_acquire);
    if (!addr) {
        void* ptr = nullptr;
        DTE_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return fail(DTE_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        addr = static_cast<unsigned char*>(ptr);
        g_static_addr[device].store(addr, std::memory_order_release);
    }
    *out = addr;
    return DTE_OK;
}

}  // namespace

extern "C" dte_status dte_extract_delta_static(const dte_layout* layout, const float* const* theta,
                                               const float* const* m, const float* const* v,
                                               int64_t step, double lr, double beta1, double beta2,
                                               double eps, double wd, const dte_delta* out,
                                               void* cuda_stream) {
    if (!layout) return fail(DTE_ERR_INVALID_ARG, "layout is null");
    if (layout->n_tensors && (!theta || !m || !v)) return fail(DTE_ERR_INVALID_ARG, "null pointer table");
    dte_status s = check_delta(out);
    if (s != DTE_OK) return s;
    if (layout->n_tiles > kStaticMaxTiles) {
        set_error("dte_extract_delta_static: the layout has " + std::to_string(layout->n_tiles) +
                  " tiles, the fixed scratch holds " + std::to_string(kStaticMaxTiles) +
                  "; use dte_extract_delta");
        return DTE_ERR_CAPACITY;
    }
    if (out->capacity > kStaticMaxCapacity) {
        set_error("dte_extract_delta_static: capacity " + std::to_string(out->capacity) +
                  " exceeds the fixed staging buffer of " + std::to_string(kStaticMaxCapacity) +
                  " entries; use dte_extract_delta");
        return DTE_ERR_CAPACITY;
    }
    float c5[5];
    s = dte_derive_constants(step, lr, beta1, beta2, eps, wd, c5);
    if (s != DTE_OK) return s;
    dte_layout* L = const_cast<dte_layout*>(layout);
    DeviceGuard g(L->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    unsigned char* base = nullptr;
    s = static_scratch_address(L->device, &base);
    if (s != DTE_OK) return s;
    s = sync_source_table(L, theta, m, v, st);
    if (s != DTE_OK) return s;
    // the array keeps whatever the previous call left - possibly a call on another layout, or one
    // that was cut short - so the two words that must start at zero (the staging cursor and the
    // count of non-finite elements) are cleared in the stream every time; every other part is
    // written before it is read
    const Consts c{c5[0], c5[1], c5[2], c5[3], c5[4]};
    const Scratch sc{reinterpret_cast<uint64_t*>(base + kStaticCursorOff),
                     reinterpret_cast<uint64_t*>(base + kStaticRecOff),
                     reinterpret_cast<uint64_t*>(base + kStaticBlockSumOff),
                     reinterpret_cast<uint32_t*>(base + kStaticStageOff), true};
    return enqueue_kernels(L, c, nullptr, sc, out, st);
}
