// Ordered placement of the staged entries ("count, then write"): a scan over the
// per-tile placement records gives every tile its position in the concatenated,
// list-ordered output (lists in shard order, ascending offsets within a list), and a gather
// moves its entries from the staging buffer to that position.  Three small launches; the
// data they touch are the records (8 bytes per 9216 scanned elements) and the changed
// entries themselves.  No kernel waits on another CTA.
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
    const uint64_t total = s_carry;
    if (threadIdx.x == 0) {
        p.counters[0] = total;
        p.counters[1] = p.scanned;
        p.list_ptr[p.n_lists] = total;
        if (total > p.capacity) atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_OVERFLOW);
    }
    // lists after which no tile follows end (and start) at the total
    for (uint32_t k = threadIdx.x; k < p.n_lists; k += kScanThreads)
        if (p.list_first_rec[k] >= p.n_rec) p.list_ptr[k] = total;
}

// ---- 3. per block: local scan, list starts, gather ---------------------------------------------
__global__ void __launch_bounds__(kGatherThreads, 3) gather_move_kernel(const GatherParams p) {
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
        uint64_t r = 0;
        if ((uint32_t)tid < n_here) r = p.rec[base_rec + tid];
        cnt = (uint32_t)(r & kRecCountMask);
        s_pos[tid] = r >> kRecCountBits;
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
    const uint64_t out_base = p.block_sum[blockIdx.x];

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
    const uint64_t total = p.counters[0];
    if (total > p.capacity) return;
    // warp w moves records 8w .. 8w+7; the eight copies are interleaved so that eight
    // independent loads per lane are in flight (a record holds ~125 entries: few rounds)
    (void)block_total;
    uint32_t cnt8[kRecsPerWarp], base8[kRecsPerWarp];
    const uint32_t* src8[kRecsPerWarp];
    uint32_t* off8[kRecsPerWarp];
    uint16_t* val8[kRecsPerWarp];
    uint32_t longest = 0, packed_recs = 0;
#pragma unroll
    for (int r = 0; r < kRecsPerWarp; ++r) {
        const uint32_t j = warp * kRecsPerWarp + r;
        const uint32_t first = s_prefix[j];
        cnt8[r] = s_prefix[j + 1] - first;
        src8[r] = p.stage + s_pos[j];
        off8[r] = p.offsets + (out_base + first);
        val8[r] = p.values + (out_base + first);
        const uint64_t b = cnt8[r] ? p.rec_base[base_rec + j] : 0ull;
        base8[r] = (uint32_t)b;
        if (b & kRecBasePacked) packed_recs |= 1u << r;
        longest = max(longest, cnt8[r]);
    }
    for (uint32_t q = lane; q < longest; q += 32) {
        uint32_t w[kRecsPerWarp];
#pragma unroll
        for (int r = 0; r < kRecsPerWarp; ++r)
            if (q < cnt8[r]) w[r] = src8[r][q];
#pragma unroll
        for (int r = 0; r < kRecsPerWarp; ++r)
            if (q < cnt8[r]) {
                // a regular tile is one destination run: base + (warp * kWarpTile + index); the
                // offsets of packed tiles are put right below
                off8[r][q] = base8[r] + (w[r] & 0xFFFFu);
                val8[r][q] = (uint16_t)(w[r] >> 16);
            }
    }
    // packed tiles (few): every piece has a destination base of its own
    if (packed_recs == 0) return;
#pragma unroll
    for (int r = 0; r < kRecsPerWarp; ++r) {
        if (!(packed_recs & (1u << r))) continue;
        const TileDesc* d = p.packed + (size_t)base8[r] * kSub;
        for (uint32_t q = lane; q < cnt8[r]; q += 32) {
            const uint32_t idx = src8[r][q] & 0xFFFFu;
            const uint32_t piece = idx / kWarpTile;
            off8[r][q] = __ldg(&d[piece].dst_off) + (idx - piece * kWarpTile);
        }
    }
}

dte_status launch_gather(const GatherParams& p, cudaStream_t st) {
    gather_reduce_kernel<<<p.n_blocks, kGatherThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    gather_scan_kernel<<<1, kScanThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    gather_move_kernel<<<p.n_blocks, kGatherThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
