// Measurement probes (libdte_probes.so).  NOT part of the product library: nothing here is a
// step of the delta-transfer path and libdte.so neither links nor loads this file.  The
// benchmark uses the probes to put the path's kernels next to what the memory system itself
// can do for the same access pattern:
//   - a read-only streaming pass (the extract reads 12 bytes per element and writes almost
//     nothing, while a copy - the usual bandwidth yardstick - is half writes);
//   - isolated small accesses at ascending, widely spaced offsets (the apply kernel writes one
//     2-byte value into, on average, every fourth 32-byte sector of the receiver's tensors).
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int kThreads = 256;
constexpr int kLoads = 8;     // independent accesses per thread and step

__global__ void __launch_bounds__(kThreads) read_kernel(const uint4* __restrict__ src, uint64_t n_vec,
                                                        unsigned long long* out) {
    const uint64_t stride = (uint64_t)gridDim.x * kThreads;
    uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    uint32_t acc = 0;
    for (; i + (kLoads - 1) * stride < n_vec; i += kLoads * stride) {
        uint4 w[kLoads];
#pragma unroll
        for (int j = 0; j < kLoads; ++j) w[j] = __ldg(src + i + j * stride);
#pragma unroll
        for (int j = 0; j < kLoads; ++j) acc ^= w[j].x ^ w[j].y ^ w[j].z ^ w[j].w;
    }
    for (; i < n_vec; i += stride) {
        const uint4 w = __ldg(src + i);
        acc ^= w.x ^ w.y ^ w.z ^ w.w;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc ^= __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    if ((threadIdx.x & 31) == 0 && acc) atomicXor(out, (unsigned long long)acc);
}

// offsets[i] = i * stride + hash(i) % jitter  (ascending when jitter <= stride)
__global__ void offsets_kernel(uint32_t* off, uint64_t n, uint32_t stride, uint32_t jitter) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t h = (uint32_t)i * 2654435761u;
    h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
    off[i] = (uint32_t)(i * stride + (jitter ? h % jitter : 0u));
}

// MODE 0: 2-byte store; 1: 4-byte store of the aligned word; 2: store of the whole 32-byte
// sector (no read); 3: load the sector, store the sector; 4: load half the sector only.
template <int MODE>
__global__ void __launch_bounds__(kThreads) sparse_kernel(const uint32_t* __restrict__ off, uint64_t n,
                                                          uint16_t* dst, uint32_t* sink) {
    uint32_t acc = 0;
    for (uint64_t base = (uint64_t)blockIdx.x * kThreads * kLoads; base < n;
         base += (uint64_t)gridDim.x * kThreads * kLoads) {
        uint32_t o[kLoads];
        uint4 a[kLoads], b[kLoads];
#pragma unroll
        for (int j = 0; j < kLoads; ++j) {
            const uint64_t e = base + (uint64_t)j * kThreads + threadIdx.x;
            o[j] = e < n ? __ldcs(off + e) : 0u;
        }
        if (MODE == 3 || MODE == 4) {
#pragma unroll
            for (int j = 0; j < kLoads; ++j) {
                const uint64_t e = base + (uint64_t)j * kThreads + threadIdx.x;
                if (e < n) {
                    const uint4* p = reinterpret_cast<const uint4*>(dst + (o[j] & ~15u));
                    a[j] = __ldcg(p);
                    if (MODE == 3) b[j] = __ldcg(p + 1);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kLoads; ++j) {
            const uint64_t e = base + (uint64_t)j * kThreads + threadIdx.x;
            if (e >= n) continue;
            if (MODE == 0) dst[o[j]] = (uint16_t)e;
            if (MODE == 1) reinterpret_cast<uint32_t*>(dst)[o[j] >> 1] = (uint32_t)e;
            if (MODE == 2) {
                uint4* p = reinterpret_cast<uint4*>(dst + (o[j] & ~15u));
                const uint4 w = make_uint4((uint32_t)e, 1u, 2u, 3u);
                p[0] = w; p[1] = w;
            }
            if (MODE == 3) {
                uint4* p = reinterpret_cast<uint4*>(dst + (o[j] & ~15u));
                a[j].x ^= (uint32_t)e;
                p[0] = a[j]; p[1] = b[j];
            }
            if (MODE == 4) acc ^= a[j].x ^ a[j].w;
        }
    }
    if (MODE == 4 && acc == 0x12345678u) *sink = acc;
}

int sm_count(int device) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) sms = 1;
    return sms;
}

}  // namespace

#define PROBE_API extern "C" __attribute__((visibility("default")))

// One read-only streaming pass over `bytes` bytes of device memory at `src` (16-byte aligned; a
// trailing bytes % 16 is ignored), XOR-folded into *xor_out (device, 8 bytes, not cleared).
// Returns the cudaError_t of the launch.
PROBE_API int dte_probe_read_bandwidth(const void* src, uint64_t bytes, uint64_t* xor_out, int device,
                                       void* cuda_stream) {
    if (!src || !xor_out || ((uintptr_t)src & 15u)) return (int)cudaErrorInvalidValue;
    read_kernel<<<sm_count(device) * 8, kThreads, 0, (cudaStream_t)cuda_stream>>>(
        (const uint4*)src, bytes / 16, (unsigned long long*)xor_out);
    return (int)cudaGetLastError();
}

// offsets[i] = i * stride + (hash(i) mod jitter), i < n: the ascending, isolated element offsets
// of a sparse list of density 1 / stride.  `offsets`: device, n x uint32.
PROBE_API int dte_probe_make_offsets(uint32_t* offsets, uint64_t n, uint32_t stride, uint32_t jitter,
                                     void* cuda_stream) {
    if (!offsets || (n && (n - 1) * (uint64_t)stride + jitter >= (1ull << 32))) return (int)cudaErrorInvalidValue;
    if (n) offsets_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)cuda_stream>>>(offsets, n, stride, jitter);
    return (int)cudaGetLastError();
}

// One access per offset into `dst` (device, uint16 elements, 32-byte aligned, covering the
// largest offset rounded up to a sector).  mode 0: 2-byte store; 1: 4-byte store; 2: 32-byte
// sector store; 3: sector load + sector store; 4: sector load only (`sink`: device, 4 bytes).
PROBE_API int dte_probe_sparse_access(int mode, const uint32_t* offsets, uint64_t n, uint16_t* dst, uint32_t* sink,
                                      int ctas_per_sm, int device, void* cuda_stream) {
    if (!offsets || !dst || !sink || ctas_per_sm < 1 || ((uintptr_t)dst & 31u)) return (int)cudaErrorInvalidValue;
    const int grid = sm_count(device) * ctas_per_sm;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    switch (mode) {
        case 0: sparse_kernel<0><<<grid, kThreads, 0, st>>>(offsets, n, dst, sink); break;
        case 1: sparse_kernel<1><<<grid, kThreads, 0, st>>>(offsets, n, dst, sink); break;
        case 2: sparse_kernel<2><<<grid, kThreads, 0, st>>>(offsets, n, dst, sink); break;
        case 3: sparse_kernel<3><<<grid, kThreads, 0, st>>>(offsets, n, dst, sink); break;
        case 4: sparse_kernel<4><<<grid, kThreads, 0, st>>>(offsets, n, dst, sink); break;
        default: return (int)cudaErrorInvalidValue;
    }
    return (int)cudaGetLastError();
}
