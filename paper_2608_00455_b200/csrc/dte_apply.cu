// Direct sparse apply (Eq. 7): shard[k][offsets[e]] = values[e] for every entry of every
// list.  Entry counts are read on the device (list_ptr), so the launch needs no host
// round trip after extract.
#include "dte_internal.cuh"

namespace dte {

constexpr int kApplyThreads = 256;
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
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
        // largest k with lp[k] <= e (lists may be empty, so take the upper bound)
        uint32_t lo = 0, hi = L;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (lp[mid] <= e) lo = mid; else hi = mid;
        }
        const uint32_t off = __ldcs(p.offsets + e);
        const uint16_t val = __ldcs(p.values + e);
        if ((uint64_t)off < p.shard_numel[lo]) p.shards[lo][off] = val;
        else bad = true;
    }
    if (bad) atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_BOUNDS);
}

dte_status launch_apply(const ApplyParams& p, int device, cudaStream_t st) {
    int sms = 0;
    DTE_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    apply_kernel<<<sms * 8, kApplyThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
