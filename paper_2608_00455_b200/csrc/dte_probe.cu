// Measurement aid: a read-only streaming pass over caller memory, the practical ceiling for a
// kernel whose traffic is all reads (the extract reads 12 bytes per element and writes almost
// nothing, while a copy - the usual bandwidth yardstick - is half writes).
#include "dte_internal.cuh"

namespace dte {

constexpr int kProbeThreads = 256;
constexpr int kProbeLoads = 8;    // independent 16-byte loads per thread and step

__global__ void __launch_bounds__(kProbeThreads) read_probe_kernel(const uint4* __restrict__ src, uint64_t n_vec,
                                                                   unsigned long long* out) {
    const uint64_t stride = (uint64_t)gridDim.x * kProbeThreads;
    uint64_t i = (uint64_t)blockIdx.x * kProbeThreads + threadIdx.x;
    uint32_t acc = 0;
    for (; i + (kProbeLoads - 1) * stride < n_vec; i += kProbeLoads * stride) {
        uint4 w[kProbeLoads];
#pragma unroll
        for (int j = 0; j < kProbeLoads; ++j) w[j] = __ldg(src + i + j * stride);
#pragma unroll
        for (int j = 0; j < kProbeLoads; ++j) acc ^= w[j].x ^ w[j].y ^ w[j].z ^ w[j].w;
    }
    for (; i < n_vec; i += stride) {
        const uint4 w = __ldg(src + i);
        acc ^= w.x ^ w.y ^ w.z ^ w.w;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc ^= __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    if ((threadIdx.x & 31) == 0 && acc) atomicXor(out, (unsigned long long)acc);
}

dte_status launch_read_probe(const void* src, uint64_t bytes, uint64_t* out, int device, cudaStream_t st) {
    int sms = 0;
    DTE_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    read_probe_kernel<<<sms * 8, kProbeThreads, 0, st>>>((const uint4*)src, bytes / 16, (unsigned long long*)out);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
