// Direct sparse apply (Eq. 7): shard[k][offsets[e]] = values[e] for every entry of every
// list.  Entry counts are read on the device (list_ptr), so the launch needs no host
// round trip after extract.
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
    if (total > p.capacity || (p.counters[2] & DTE_DEV_OVERFLOW)) {
        // the lists are incomplete: writing part of a version would leave the shard in a
        // state that is neither the old nor the new one
        if (blockIdx.x == 0 && threadIdx.x == 0)
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
                if ((uint64_t)off[j] < __ldg(p.shard_numel + k)) {
                    uint16_t* dst = reinterpret_cast<uint16_t*>(__ldg(reinterpret_cast<const unsigned long long*>(p.shards + k)));
                    dst[off[j]] = val[j];
                } else {
                    bad = true;
                }
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
    // 2-byte writes are bound by the memory system's sector read-modify-write rate
    apply_kernel<<<sms * 6, kApplyThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
