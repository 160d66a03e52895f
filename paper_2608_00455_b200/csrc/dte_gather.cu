// Ordered placement of the staged entries ("count, then write"): a scan over the
// per-tile placement records gives every tile its position in the concatenated,
// list-ordered output (lists in shard order, ascending offsets within a list), and a gather
// moves its entries from the staging buffer to that position.  Three small launches (one for small
// layouts, whose blocks each scan all records themselves);
// the data they touch are the records (8 bytes per 9216 scanned elements) and the changed
// entries themselves.  No kernel waits on another CTA.
#include <algorithm>

#include "dte_internal.cuh"

namespace dte {

constexpr int kGatherThreads = 256;
constexpr int kRecsPerWarp = kRecsPerBlock / (kGatherThreads / 32);   // 8

// ---- 1. per-block sums of the counts ----------------------------------------------------
__global__ void __launch_bounds__(kGatherThreads) gather_reduce_kernel(const GatherParams p) {
    __shared__ uint32_t s_warp[kGatherThreads / 32];
    const uint32_t base = blockIdx.x * kRecsPerBlock;
    uint32_t sum = 0;
    for (uint32_t j = threadIdx.x; j < (uint32_t)kRecsPerBlock; j += kGatherThreads) {
        const uint32_t r = base + j;
        if (r < p.n_rec) sum += (uint32_t)(p.rec[r] & kRecCountMask);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint64_t tot = 0;
        for (int w = 0; w < kGatherThreads / 32; ++w) tot += s_warp[w];
        p.block_sum[blockIdx.x] = tot;
    }
}

// ---- 2. exclusive scan of the block sums (one CTA), totals, trailing empty lists ------------
constexpr int kScanThreads = 1024;

__global__ void __launch_bounds__(kScanThreads) gather_scan_kernel(const GatherParams p) {
    __shared__ uint64_t s_warp[kScanThreads / 32];
    __shared__ uint64_t s_carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (uint32_t b0 = 0; b0 < p.n_blocks; b0 += kScanThreads) {
        const uint32_t b = b0 + threadIdx.x;
        const uint64_t x = b < p.n_blocks ? p.block_sum[b] : 0ull;
        uint64_t incl = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint64_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const uint64_t w = s_warp[lane];
            uint64_t wi = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint64_t up = __shfl_up_sync(0xFFFFFFFFu, wi, d);
                if (lane >= d) wi += up;
            }
            s_warp[lane] = wi - w;   // exclusive over warps
        }
        __syncthreads();
        const uint64_t carry = s_carry;
        const uint64_t excl = carry + s_warp[warp] + (incl - x);
        if (b < p.n_blocks) p.block_sum[b] = excl;
        __syncthreads();
        if (threadIdx.x == kScanThreads - 1) s_carry = excl + x;
        __syncthreads();
    }
    gather_finish_totals(p, s_carry, threadIdx.x, kScanThreads, true);
    if (threadIdx.x == 0) *p.cursor = 0ull;     // every tile has reserved its room: ready for the next call
}

// ---- 3. per block: local scan, list starts, gather ---------------------------------------------
// PUSH: every entry is also stored into the landing buffers of the receiver that owns its list
// (dte_extract_delta_push): plain stores to memory that may be a peer GPU's.
// SMALL (at most kSmallBlocks blocks, i.e. 4096 tiles): the only gather launch of the call.  Every
// block scans ALL placement records itself (32 KB from L2 at most, cheaper than two more launches
// in front of a 30 microsecond stream), so it knows its output base, the total and where each
// receiver's slice starts without help; the last block also writes the totals and puts the
// staging cursor back to zero.
constexpr int kSmallRecs = kSmallBlocks * kRecsPerBlock;     // 4096
constexpr int kSmallPerThread = kSmallRecs / kGatherThreads; // 16

template <bool PUSH, bool SMALL>
__global__ void __launch_bounds__(kGatherThreads, 3) gather_move_kernel(const GatherParams p) {
    // A small layout's gather is launched so that it may be set up while the last extract tiles
    // still run (programmatic dependent launch): nothing the extract wrote may be read before
    // this.  Returns at once in an ordinary launch.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __shared__ uint32_t s_all[SMALL ? kSmallRecs + 1 : 1];      // exclusive prefix of the counts of all records
    // the block's own records (threads 0 .. kRecsPerBlock-1 own one each): asked for first, so that
    // a small layout's scan of all records below does not stand between the request and its use
    uint64_t own_rec = 0;
    if (threadIdx.x < kRecsPerBlock && blockIdx.x * kRecsPerBlock + threadIdx.x < p.n_rec)
        own_rec = __ldcg(p.rec + blockIdx.x * kRecsPerBlock + threadIdx.x);
    if (SMALL) {
        __shared__ uint32_t s_thread_sum[kGatherThreads / 32];
        uint32_t c[kSmallPerThread];
        const uint32_t r0 = threadIdx.x * kSmallPerThread;
#pragma unroll
        for (int i = 0; i < kSmallPerThread; ++i)                 // independent loads; the records come from other SMs: L2
            c[i] = r0 + i < p.n_rec ? (uint32_t)(__ldcg(p.rec + r0 + i) & kRecCountMask) : 0u;
        uint32_t mine = 0;
#pragma unroll
        for (int i = 0; i < kSmallPerThread; ++i) mine += c[i];
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if ((threadIdx.x & 31) >= d) incl += up;
        }
        if ((threadIdx.x & 31) == 31) s_thread_sum[threadIdx.x >> 5] = incl;
        __syncthreads();
        uint32_t run = incl - mine;
        for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) run += s_thread_sum[w];
#pragma unroll
        for (int i = 0; i < kSmallPerThread; ++i) {
            s_all[r0 + i] = run;
            run += c[i];
        }
        if (threadIdx.x == kGatherThreads - 1) s_all[kSmallRecs] = run;
        __syncthreads();
    }
    __shared__ uint32_t s_prefix[kRecsPerBlock + 1];   // exclusive prefix of counts within the block
    __shared__ uint64_t s_pos[kRecsPerBlock];          // staging position of each record
    __shared__ uint32_t s_warp[kGatherThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t base_rec = blockIdx.x * kRecsPerBlock;
    const uint32_t n_here = min((uint32_t)kRecsPerBlock, p.n_rec - base_rec);

    // threads 0 .. kRecsPerBlock-1 (the first two warps) own one record each
    static_assert(kRecsPerBlock == 64, "two warps scan the block's records");
    uint32_t cnt = 0;
    if (tid < kRecsPerBlock) {
        cnt = (uint32_t)(own_rec & kRecCountMask);
        s_pos[tid] = own_rec >> kRecCountBits;
    }
    uint32_t incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += up;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (tid < kRecsPerBlock) {
        const uint32_t wbase = warp ? s_warp[0] : 0u;
        s_prefix[tid] = wbase + incl - cnt;
        if (tid == kRecsPerBlock - 1) s_prefix[kRecsPerBlock] = wbase + incl;
    }
    __syncthreads();
    const uint32_t block_total = s_prefix[kRecsPerBlock];
    const uint64_t out_base = SMALL ? (uint64_t)s_all[base_rec] : p.block_sum[blockIdx.x];
    const uint64_t total = SMALL ? (uint64_t)s_all[kSmallRecs] : p.counters[0];
    if (SMALL && blockIdx.x == gridDim.x - 1) {
        gather_finish_totals(p, total, threadIdx.x, kGatherThreads, false);
        if (threadIdx.x == 0) *p.cursor = 0ull;     // every tile has reserved its room: ready for the next call
    }

    // list starts that fall into this block (list_first_rec is non-decreasing)
    {
        uint32_t lo = 0, hi = p.n_lists;   // first k with list_first_rec[k] >= base_rec
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (p.list_first_rec[mid] < base_rec) lo = mid + 1; else hi = mid;
        }
        for (uint32_t k = lo + tid; k < p.n_lists; k += kGatherThreads) {
            const uint32_t fr = p.list_first_rec[k];
            if (fr >= base_rec + n_here) break;
            p.list_ptr[k] = out_base + s_prefix[fr - base_rec];
        }
    }

    // the staged entries are complete only if everything fitted
    if (total > p.capacity) return;
    // warp w moves records 8w .. 8w+7; the eight copies are interleaved, two rounds at a time, so
    // that sixteen independent loads per lane are in flight (the kernel is bound by memory
    // latency: a block holds only 64 records, and a one-layer workload has a few hundred blocks).
    // Output positions are kept as 32-bit distances from the block's base to spare registers.
    (void)block_total;
    uint32_t cnt8[kRecsPerWarp], base8[kRecsPerWarp], first8[kRecsPerWarp];
    const uint32_t* src8[kRecsPerWarp];
    uint32_t* const out_off = p.offsets + out_base;
    uint16_t* const out_val = p.values + out_base;
    // PUSH: the same run in the receiver's buffers, cut where the receiver's capacity ends; kept in
    // shared memory (one set per record, written by the record's thread) to spare registers
    __shared__ uint32_t* s_roff[PUSH ? kRecsPerBlock : 1];
    __shared__ uint16_t* s_rval[PUSH ? kRecsPerBlock : 1];
    __shared__ uint32_t s_rcnt[PUSH ? kRecsPerBlock : 1];
    if (PUSH) {
        if (tid < kRecsPerBlock) {
            uint32_t n = 0;
            uint32_t* ro = nullptr;
            uint16_t* rv = nullptr;
            const uint32_t c = s_prefix[tid + 1] - s_prefix[tid];
            if (c) {
                const uint32_t recv = p.rec_recv[base_rec + tid];
                const dte_push_target t = p.targets[recv];
                // where the receiver's slice starts: the output position of the first tile of its first list
                const uint64_t slice0 = SMALL ? (uint64_t)s_all[p.list_first_rec[p.recv_first_list[recv]]]
                                              : p.recv_base[recv];
                const uint64_t at = out_base + s_prefix[tid] - slice0;          // position in the receiver's slice
                if (t.status && at < t.capacity) {
                    n = (uint32_t)min((uint64_t)c, t.capacity - at);
                    ro = t.offsets + at;
                    rv = t.values + at;
                }
            }
            s_rcnt[tid] = n; s_roff[tid] = ro; s_rval[tid] = rv;
        }
        __syncthreads();
    }
    uint32_t longest = 0, packed_recs = 0;
#pragma unroll
    for (int r = 0; r < kRecsPerWarp; ++r) {
        const uint32_t j = warp * kRecsPerWarp + r;
        first8[r] = s_prefix[j];
        cnt8[r] = s_prefix[j + 1] - first8[r];
        src8[r] = p.stage + s_pos[j];
        const uint64_t b = cnt8[r] ? p.rec_base[base_rec + j] : 0ull;
        base8[r] = (uint32_t)b;
        if (b & kRecBasePacked) packed_recs |= 1u << r;
        longest = max(longest, cnt8[r]);
    }
    for (uint32_t q0 = lane; q0 < longest; q0 += 64) {
        uint32_t w[2][kRecsPerWarp];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int r = 0; r < kRecsPerWarp; ++r)
                if (q0 + 32 * h < cnt8[r]) w[h][r] = src8[r][q0 + 32 * h];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int r = 0; r < kRecsPerWarp; ++r) {
                const uint32_t q = q0 + 32 * h;
                if (q < cnt8[r]) {
                    // a regular tile is one destination run: base + (warp * kWarpTile + index); the
                    // offsets of packed tiles are put right below
                    const uint32_t off = base8[r] + (w[h][r] & 0xFFFFu);
                    out_off[first8[r] + q] = off;
                    out_val[first8[r] + q] = (uint16_t)(w[h][r] >> 16);
                    if (PUSH && q < s_rcnt[warp * kRecsPerWarp + r]) {
                        s_roff[warp * kRecsPerWarp + r][q] = off;
                        s_rval[warp * kRecsPerWarp + r][q] = (uint16_t)(w[h][r] >> 16);
                    }
                }
            }
    }
    // packed tiles (few): every piece has a destination base of its own
    if (packed_recs) {
#pragma unroll
        for (int r = 0; r < kRecsPerWarp; ++r) {
            if (!(packed_recs & (1u << r))) continue;
            const TileDesc* d = p.packed + (size_t)base8[r] * kSub;
            for (uint32_t q = lane; q < cnt8[r]; q += 32) {
                const uint32_t idx = src8[r][q] & 0xFFFFu;
                const uint32_t piece = idx / kWarpTile;
                const uint32_t off = __ldg(&d[piece].dst_off) + (idx - piece * kWarpTile);
                out_off[first8[r] + q] = off;
                if (PUSH && q < s_rcnt[warp * kRecsPerWarp + r]) s_roff[warp * kRecsPerWarp + r][q] = off;
            }
        }
    }
    // the receivers' memory may be another GPU's: this thread's stores must have arrived there
    // before anything later in the stream (the status block) tells the receiver so
    if (PUSH) __threadfence_system();
}

// ---- 4. closing kernel of a push: counts, boundaries and the status block of every receiver -----
__device__ __forceinline__ uint64_t lower_bound_offset(const uint32_t* offsets, uint64_t lo, uint64_t hi, uint64_t key) {
    while (lo < hi) {          // first entry in [lo, hi) with offset >= key
        const uint64_t mid = (lo + hi) >> 1;
        if ((uint64_t)offsets[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

constexpr int kFinishThreads = 256;

__global__ void __launch_bounds__(kFinishThreads) push_finish_kernel(const PushFinishParams p) {
    __shared__ uint32_t s_last;
    const uint64_t bits = p.counters[2];
    const uint64_t total = p.list_ptr[p.n_lists];
    const bool incomplete = total > p.capacity || (bits & (DTE_DEV_OVERFLOW | DTE_DEV_CORRUPT));
    const uint32_t tid = blockIdx.x * kFinishThreads + threadIdx.x, n_thr = gridDim.x * kFinishThreads;
    // c_o of every operation, into its receiver's count array at the operation's plan position
    for (uint32_t o = tid; o < p.n_ops; o += n_thr) {
        const dte_push_target t = p.targets[p.op_recv[o]];
        if (!t.status) continue;
        uint64_t c = 0;
        if (!incomplete) {
            const OpRange r = p.ranges[o];
            const uint64_t a = p.list_ptr[r.list], b = p.list_ptr[r.list + 1];
            c = lower_bound_offset(p.offsets, a, b, r.end) - lower_bound_offset(p.offsets, a, b, r.begin);
        }
        t.op_counts[p.op_slot[o]] = c;
    }
    // list boundaries relative to the receiver's slice (lists of other receivers: empty)
    const uint32_t per = p.n_lists + 1;
    for (uint64_t i = tid; i < (uint64_t)p.n_recv * per; i += n_thr) {
        const uint32_t r = (uint32_t)(i / per), k = (uint32_t)(i - (uint64_t)r * per);
        const dte_push_target t = p.targets[r];
        if (!t.status) continue;
        const uint64_t lo = p.list_ptr[p.recv_first_list[r]], hi = p.list_ptr[p.recv_first_list[p.n_recv + r]];
        t.list_ptr[k] = min(max(p.list_ptr[k], lo), hi) - lo;
    }
    // the block that finishes last publishes: everything above must have arrived first
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(p.ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence_system();
    for (uint32_t r = threadIdx.x; r < p.n_recv; r += kFinishThreads) {
        const dte_push_target t = p.targets[r];
        if (!t.status) continue;
        const uint64_t n = p.list_ptr[p.recv_first_list[p.n_recv + r]] - p.list_ptr[p.recv_first_list[r]];
        t.status[0] = n;
        t.status[2] = (bits & ~(uint64_t)DTE_DEV_OVERFLOW) | ((incomplete || n > t.capacity) ? DTE_DEV_OVERFLOW : 0u);
        t.status[3] = p.recv_num_ops[r];
        __threadfence_system();
        asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(t.status + 1), "l"(p.epoch) : "memory");
    }
    if (threadIdx.x == 0) *p.ticket = 0u;
}

dte_status launch_push_finish(const PushFinishParams& p, cudaStream_t st) {
    const uint64_t work = std::max<uint64_t>(p.n_ops, (uint64_t)p.n_recv * (p.n_lists + 1));
    const int blocks = (int)std::min<uint64_t>(std::max<uint64_t>(1, (work + kFinishThreads - 1) / kFinishThreads), 1024);
    push_finish_kernel<<<blocks, kFinishThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

// ---- receiver side: wait (bounded) for the status block of an epoch -----------------------------
__global__ void push_wait_kernel(const uint64_t* status, uint64_t epoch, uint64_t timeout_ns, uint64_t max_polls,
                                 uint64_t* counters) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    unsigned long long t0, now;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    bool arrived = false;
    for (uint64_t i = 0; i < max_polls; ++i) {       // two limits: the clock, and a poll count should the clock stall
        unsigned long long v;
        asm volatile("ld.acquire.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(status + 1) : "memory");
        if (v == epoch) { arrived = true; break; }
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (now - t0 > timeout_ns) break;
        __nanosleep(500);
    }
    if (arrived) {
        unsigned long long n, b;
        asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(n) : "l"(status) : "memory");
        asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(b) : "l"(status + 2) : "memory");
        counters[0] = n; counters[1] = 0; counters[2] = b; counters[3] = 0;
    } else {
        counters[0] = 0; counters[1] = 0; counters[3] = 0;
        counters[2] = DTE_DEV_TIMEOUT | DTE_DEV_OVERFLOW;     // nothing usable: apply must not write
    }
}

dte_status launch_push_wait(const uint64_t* status, uint64_t epoch, uint32_t timeout_ms, uint64_t* counters,
                            cudaStream_t st) {
    const uint64_t ms = std::min<uint32_t>(timeout_ms, 10000u);
    // the poll count is the second limit, for a clock that does not advance: generous enough (a
    // poll is a system-scope load and a sleep, never under 50 ns) not to cut the time limit short
    push_wait_kernel<<<1, 32, 0, st>>>(status, epoch, ms * 1000000ull, ms * 20000ull + 1000, counters);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

// small: one launch (every block scans the records itself), set up under the extract's tail.
dte_status launch_gather(const GatherParams& p, bool small, cudaStream_t st) {
    if (small) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(p.n_blocks);
        cfg.blockDim = dim3(kGatherThreads);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (p.n_recv) DTE_CUDA(cudaLaunchKernelEx(&cfg, gather_move_kernel<true, true>, p));
        else DTE_CUDA(cudaLaunchKernelEx(&cfg, gather_move_kernel<false, true>, p));
        return DTE_OK;
    }
    gather_reduce_kernel<<<p.n_blocks, kGatherThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    gather_scan_kernel<<<1, kScanThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    if (p.n_recv) gather_move_kernel<true, false><<<p.n_blocks, kGatherThreads, 0, st>>>(p);
    else gather_move_kernel<false, false><<<p.n_blocks, kGatherThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
