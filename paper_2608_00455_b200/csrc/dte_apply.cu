// Direct sparse apply (Eq. 7): shard[k][offsets[e]] = values[e] for every entry of every
// list.  Entry counts are read on the device (list_ptr), so the launch needs no host
// round trip after extract.
#include <algorithm>

#include "dte_internal.cuh"

namespace dte {

constexpr int kApplyThreads = 256;
constexpr int kApplyPerThread = 8;                      // entries in flight per thread
constexpr int kApplyChunk = kApplyThreads * kApplyPerThread;
constexpr int kApplySmemLists = 4096;  // list_ptr entries cached in shared memory

__global__ void __launch_bounds__(kApplyThreads) apply_kernel(const ApplyParams p) {
    __shared__ uint64_t s_ptr[kApplySmemLists + 1];
    const uint32_t L = p.n_lists;
    const bool cached = L <= (uint32_t)kApplySmemLists;
    if (cached)
        for (uint32_t k = threadIdx.x; k <= L; k += blockDim.x) s_ptr[k] = p.list_ptr[k];
    __syncthreads();
    const uint64_t* lp = cached ? s_ptr : p.list_ptr;
    const uint64_t total = lp[L];
    const uint64_t dev_bits = p.counters[2];
    if (total > p.capacity || (dev_bits & (DTE_DEV_OVERFLOW | DTE_DEV_CORRUPT))) {
        // the lists are incomplete: writing part of a version would leave the shard in a
        // state that is neither the old nor the new one
        if (blockIdx.x == 0 && threadIdx.x == 0 && !(dev_bits & DTE_DEV_CORRUPT))
            atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_OVERFLOW);
        return;
    }
    bool bad = false;
    for (uint64_t base = (uint64_t)blockIdx.x * kApplyChunk; base < total; base += (uint64_t)gridDim.x * kApplyChunk) {
        // all loads of the chunk first: 16 independent requests per thread
        uint32_t off[kApplyPerThread];
        uint16_t val[kApplyPerThread];
#pragma unroll
        for (int j = 0; j < kApplyPerThread; ++j) {
            const uint64_t e = base + (uint64_t)j * kApplyThreads + threadIdx.x;
            if (e < total) {
                off[j] = __ldcs(p.offsets + e);
                val[j] = __ldcs(p.values + e);
            }
        }
        // list of the thread's first entry: largest k with lp[k] <= e (lists may be empty);
        // the later entries of the thread only ever move forward from there
        uint32_t k = 0;
        {
            const uint64_t e = base + threadIdx.x;
            uint32_t lo = 0, hi = L;
            while (hi - lo > 1) {
                const uint32_t mid = (lo + hi) >> 1;
                if (lp[mid] <= e) lo = mid; else hi = mid;
            }
            k = lo;
        }
#pragma unroll
        for (int j = 0; j < kApplyPerThread; ++j) {
            const uint64_t e = base + (uint64_t)j * kApplyThreads + threadIdx.x;
            if (e < total) {
                while (e >= lp[k + 1]) ++k;          // e < total = lp[L] keeps k < L
                uint16_t* dst = reinterpret_cast<uint16_t*>(__ldg(reinterpret_cast<const unsigned long long*>(p.shards + k)));
                if (dst && (uint64_t)off[j] < __ldg(p.shard_numel + k)) dst[off[j]] = val[j];
                else bad = true;          // outside the shard, or an entry for a shard the caller did not give
            }
        }
    }
    if (bad) atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_BOUNDS);
}

dte_status launch_apply(const ApplyParams& p, int device, cudaStream_t st) {
    int sms = 0;
    DTE_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    // 6 CTAs per SM is what the 32 KB list_ptr cache allows; measured on B200: 3, 6 and 12 CTAs
    // per SM and .cs / .cg / .wt store hints all give the same ~39 G entries/s - isolated
    // 2-byte writes are bound by the memory system's sector read-modify-write rate.  Touching
    // the sector first (a load: 8 G/s; an L2 prefetch one chunk ahead: 31 G/s) only hurts.
    apply_kernel<<<sms * 6, kApplyThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

// ---- destination-side mapping of canonical entries (Section 4.4) -------------------------------
// The storage-mediated path ships canonical (index, value) pairs and maps them to the inference
// layout on the destination.  Per entry: unravel (Eq. 5), test the operations of its source tensor
// for membership, ravel (Eq. 6) and store (Eq. 7) - the paper's own source-major form, which is the
// right one here because only the changed entries exist on this side.
__global__ void __launch_bounds__(kApplyThreads) apply_canonical_kernel(const CanonParams p) {
    __shared__ uint64_t s_ptr[kApplySmemLists + 1];
    const uint32_t L = p.n_tensors;
    const bool cached = L <= (uint32_t)kApplySmemLists;
    if (cached)
        for (uint32_t k = threadIdx.x; k <= L; k += blockDim.x) s_ptr[k] = p.list_ptr[k];
    __syncthreads();
    const uint64_t* lp = cached ? s_ptr : p.list_ptr;
    const uint64_t total = lp[L];
    const uint64_t dev_bits = p.counters[2];
    if (total > p.capacity || (dev_bits & (DTE_DEV_OVERFLOW | DTE_DEV_CORRUPT))) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && !(dev_bits & DTE_DEV_CORRUPT))
            atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_OVERFLOW);
        return;
    }
    bool bad = false;
    for (uint64_t base = (uint64_t)blockIdx.x * kApplyChunk; base < total; base += (uint64_t)gridDim.x * kApplyChunk) {
        uint32_t idx[kApplyPerThread];
        uint16_t val[kApplyPerThread];
#pragma unroll
        for (int j = 0; j < kApplyPerThread; ++j) {
            const uint64_t e = base + (uint64_t)j * kApplyThreads + threadIdx.x;
            if (e < total) {
                idx[j] = __ldcs(p.indices + e);
                val[j] = __ldcs(p.values + e);
            }
        }
        uint32_t k = 0;
        {
            const uint64_t e = base + threadIdx.x;
            uint32_t lo = 0, hi = L;
            while (hi - lo > 1) {
                const uint32_t mid = (lo + hi) >> 1;
                if (lp[mid] <= e) lo = mid; else hi = mid;
            }
            k = lo;
        }
#pragma unroll
        for (int j = 0; j < kApplyPerThread; ++j) {
            const uint64_t e = base + (uint64_t)j * kApplyThreads + threadIdx.x;
            if (e >= total) continue;
            while (e >= lp[k + 1]) ++k;
            const uint32_t i = idx[j];
            if (i >= __ldg(p.tensor_numel + k)) { bad = true; continue; }
            const uint32_t n1 = __ldg(p.tensor_cols + k);
            const uint32_t u0 = i / n1, u1 = i - u0 * n1;                     // Eq. 5
            const uint32_t o_end = __ldg(p.op_ptr + k + 1);
            for (uint32_t o = __ldg(p.op_ptr + k); o < o_end; ++o) {
                const uint4* q = reinterpret_cast<const uint4*>(p.ops + o);
                const uint4 w0 = __ldg(q);
                const uint32_t r0 = u0 - w0.x, r1 = u1 - w0.y;                 // wraps when below the origin
                if (r0 >= w0.z || r1 >= w0.w) continue;                         // a_s <= u < a_s + e
                const uint4 w1 = __ldg(q + 1);
                const uint32_t shard = w1.y;
                uint16_t* dst = reinterpret_cast<uint16_t*>(__ldg(reinterpret_cast<const unsigned long long*>(p.shards + shard)));
                if (!dst) continue;                                             // another receiver's tensor
                const uint64_t ld = (uint64_t)w1.z | ((uint64_t)w1.w << 32);
                const uint64_t jj = (uint64_t)w1.x + (uint64_t)r0 * ld + r1;   // Eq. 6
                if (jj < __ldg(p.shard_numel + shard)) dst[jj] = val[j];       // Eq. 7
                else bad = true;
            }
        }
    }
    if (bad) atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_BOUNDS);
}

dte_status launch_apply_canonical(const CanonParams& p, int device, cudaStream_t st) {
    int sms = 0;
    DTE_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    apply_canonical_kernel<<<sms * 6, kApplyThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

// ---- per-operation counts (Section 4.3, round 1) ---------------------------------------------
// c_o = number of entries of the operation's list whose offset lies in the operation's
// destination range: two binary searches in the (ascending) list.  An incomplete delta (its
// extract overflowed, or it was read from a damaged chunk stream) has list boundaries beyond the
// entry arrays: it gets zero counts and the overflow bit, and no entry is read.
__global__ void op_counts_kernel(const OpRange* __restrict__ ranges, uint32_t n_ops,
                                 const uint32_t* __restrict__ offsets, const uint64_t* __restrict__ list_ptr,
                                 uint32_t n_lists, uint64_t capacity, uint64_t* counters,
                                 uint64_t* __restrict__ counts) {
    const uint64_t dev_bits = counters[2];
    if (list_ptr[n_lists] > capacity || (dev_bits & (DTE_DEV_OVERFLOW | DTE_DEV_CORRUPT))) {
        for (uint32_t o = blockIdx.x * blockDim.x + threadIdx.x; o < n_ops; o += gridDim.x * blockDim.x) counts[o] = 0;
        if (blockIdx.x == 0 && threadIdx.x == 0 && !(dev_bits & DTE_DEV_CORRUPT))
            atomicOr((unsigned long long*)(counters + 2), (unsigned long long)DTE_DEV_OVERFLOW);
        return;
    }
    for (uint32_t o = blockIdx.x * blockDim.x + threadIdx.x; o < n_ops; o += gridDim.x * blockDim.x) {
        const OpRange r = ranges[o];
        const uint64_t a = list_ptr[r.list], b = list_ptr[r.list + 1];
        uint64_t pos[2];
        const uint64_t key[2] = {r.begin, r.end};
#pragma unroll
        for (int i = 0; i < 2; ++i) {          // first entry with offset >= key
            uint64_t lo = a, hi = b;
            while (lo < hi) {
                const uint64_t mid = (lo + hi) >> 1;
                if ((uint64_t)offsets[mid] < key[i]) lo = mid + 1; else hi = mid;
            }
            pos[i] = lo;
        }
        counts[o] = pos[1] - pos[0];
    }
}

dte_status launch_op_counts(const OpRange* ranges, uint32_t n_ops, const dte_delta& d, uint32_t n_lists,
                            uint64_t* counts, cudaStream_t st) {
    if (n_ops == 0) return DTE_OK;
    const int threads = 128, blocks = (int)std::min<uint32_t>((n_ops + threads - 1) / threads, 4096u);
    op_counts_kernel<<<blocks, threads, 0, st>>>(ranges, n_ops, d.offsets, d.list_ptr, n_lists, d.capacity,
                                                 d.counters, counts);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
