// The fused streaming extract kernel: AdamW inversion (Eq. 2), BF16 cast and bit compare
// (Eq. 4), ordered stream compaction, and receiver-local remap (Eq. 5-6, evaluated
// destination-major through the tile table) in a single pass over theta / m / v.
//
// Build flags that matter for bit-exactness: -fmad=false -ftz=false -prec-div=true
// -prec-sqrt=true.  The arithmetic below additionally spells every operation as a
// round-to-nearest intrinsic so that no flag can silently change it.
#include "dte_internal.cuh"

namespace dte {

// ---- arithmetic -----------------------------------------------------------------

// Eq. 2, one fp32 operation at a time.  DIV_BC1 / DIV_DECAY are false when the divisor is
// exactly 1.0f (x / 1 == x for every x, NaN included as far as the BF16 cast can tell).
template <bool DIV_BC1, bool DIV_DECAY>
__device__ __forceinline__ float invert_adamw(float theta, float m, float v, const Consts& c) {
    const float mhat = DIV_BC1 ? __fdiv_rn(m, c.bc1) : m;
    const float vhat = __fdiv_rn(v, c.bc2);
    const float den = __fadd_rn(__fsqrt_rn(vhat), c.eps);
    const float u = __fdiv_rn(mhat, den);
    const float num = __fadd_rn(theta, __fmul_rn(c.lr, u));
    return DIV_DECAY ? __fdiv_rn(num, c.decay) : num;
}

// BF16 round-to-nearest-even on the bit pattern; any NaN becomes 0x7FC0.
__device__ __forceinline__ uint32_t bf16_rne_bits(float x) {
    const uint32_t u = __float_as_uint(x);
    const uint32_t r = (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
    return ((u & 0x7FFFFFFFu) > 0x7F800000u) ? 0x7FC0u : r;
}

__device__ __forceinline__ const float* ldg_ptr(const float* const* slot) {
    return reinterpret_cast<const float*>(__ldg(reinterpret_cast<const unsigned long long*>(slot)));
}

// ---- look-back words ---------------------------------------------------------------

__device__ __forceinline__ uint64_t ld_status(const uint64_t* p) {
    uint64_t w;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(w) : "l"(p) : "memory");
    return w;
}
__device__ __forceinline__ void st_status(uint64_t* p, uint64_t w) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(w) : "memory");
}

constexpr int kMaxPolls = 1 << 20;  // bounded wait: ~0.1-1 s of back-off before giving up

// Exclusive prefix of tile `t`, computed by warp 0.  Returns false on error / timeout.
// Tiles take their index from an atomic ticket, so every predecessor is owned by a CTA
// that is already running (or done) and waits only on its own predecessors: progress
// does not depend on how CTAs are scheduled.
__device__ __forceinline__ bool look_back(uint64_t* status, uint32_t t, uint32_t aggregate,
                                          int lane, uint64_t* excl_out) {
    if (t == 0) {
        if (lane == 0) st_status(status, (kStatePrefix << kStateShift) | aggregate);
        *excl_out = 0;
        return true;
    }
    if (lane == 0) st_status(status + t, (kStateAggregate << kStateShift) | aggregate);
    uint64_t excl = 0;
    int64_t pos = (int64_t)t - 1;
    int polls = 0;
    bool ok = true;
    while (true) {
        const int64_t idx = pos - lane;
        uint64_t w = (idx >= 0) ? ld_status(status + idx) : (kStatePrefix << kStateShift);
        const uint32_t state = (uint32_t)(w >> kStateShift);
        const uint32_t m_prefix = __ballot_sync(0xFFFFFFFFu, state == kStatePrefix);
        const uint32_t m_invalid = __ballot_sync(0xFFFFFFFFu, state == kStateInvalid);
        const uint32_t m_error = __ballot_sync(0xFFFFFFFFu, state == kStateError);
        const int first_prefix = m_prefix ? (__ffs(m_prefix) - 1) : 32;
        const uint32_t needed = first_prefix < 32 ? (0xFFFFFFFFu >> (31 - first_prefix)) : 0xFFFFFFFFu;
        if (m_error & needed) { ok = false; break; }
        if (m_invalid & needed) {
            if (++polls > kMaxPolls) { ok = false; break; }
            __nanosleep(polls < 64 ? 32 : 256);
            continue;
        }
        uint64_t val = ((needed >> lane) & 1u) ? (w & kValueMask) : 0ull;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) val += __shfl_xor_sync(0xFFFFFFFFu, val, d);
        excl += val;
        if (first_prefix < 32) break;
        pos -= 32;
    }
    if (lane == 0)
        st_status(status + t, ok ? ((kStatePrefix << kStateShift) | (excl + aggregate))
                                 : (kStateError << kStateShift));
    *excl_out = excl;
    return ok;
}

// ---- the kernel --------------------------------------------------------------------

struct __align__(16) Smem {
    uint32_t warp_total[kWarps];
    uint64_t tile_excl;
    uint32_t ticket;
    uint32_t ok;
};

template <bool DIV_BC1, bool DIV_DECAY>
__global__ void __launch_bounds__(kThreads, 4) extract_kernel(const ExtractParams p) {
    __shared__ Smem sm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Consts c = p.c;

    while (true) {
        if (tid == 0) sm.ticket = atomicAdd(p.ticket, 1u);
        __syncthreads();
        const uint32_t t = sm.ticket;
        if (t >= p.n_tiles) break;

        // all threads read the same 32-byte descriptor (one sector, broadcast)
        const uint4* td = reinterpret_cast<const uint4*>(p.tiles + t);
        const uint4 d0 = __ldg(td), d1 = __ldg(td + 1);
        const uint64_t src_off = (uint64_t)d0.x | ((uint64_t)d0.y << 32);
        const uint32_t tensor = d0.z, dst_off = d0.w, len_flags = d1.x, list = d1.y;
        const uint32_t len = len_flags & kLenMask;
        const float* __restrict__ th = ldg_ptr(p.theta + tensor);
        const float* __restrict__ mm = ldg_ptr(p.m + tensor);
        const float* __restrict__ vv = ldg_ptr(p.v + tensor);

        uint32_t mask[kItems];   // bit j: element 4*lane + j of the item changed
        uint32_t val[kItems][2]; // BF16(theta) of the item's 4 elements, packed 2 x 16
        const uint32_t e_warp = warp * kWarpSpan;

        if (!(len_flags & (kFlagScalar | kFlagStrided))) {
            // ---- contiguous, 16-byte aligned: three 128-bit loads per item --------------
            float4 a[kItems], b[kItems], g[kItems];
#pragma unroll
            for (int i = 0; i < kItems; ++i) {
                const uint32_t e = e_warp + i * 128 + lane * 4;
                if (e < len) {
                    a[i] = __ldcs(reinterpret_cast<const float4*>(th + src_off + e));
                    b[i] = __ldcs(reinterpret_cast<const float4*>(mm + src_off + e));
                    g[i] = __ldcs(reinterpret_cast<const float4*>(vv + src_off + e));
                }
            }
#pragma unroll
            for (int i = 0; i < kItems; ++i) {
                const uint32_t e = e_warp + i * 128 + lane * 4;
                mask[i] = 0; val[i][0] = 0; val[i][1] = 0;
                if (e < len) {
                    const float tt[4] = {a[i].x, a[i].y, a[i].z, a[i].w};
                    const float m4[4] = {b[i].x, b[i].y, b[i].z, b[i].w};
                    const float v4[4] = {g[i].x, g[i].y, g[i].z, g[i].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float prev = invert_adamw<DIV_BC1, DIV_DECAY>(tt[j], m4[j], v4[j], c);
                        const uint32_t bt = bf16_rne_bits(tt[j]), bp = bf16_rne_bits(prev);
                        mask[i] |= (bt != bp ? 1u : 0u) << j;
                        val[i][j >> 1] |= bt << ((j & 1) * 16);
                    }
                }
            }
        } else {
            // ---- generic path: scalar loads, optional row stride --------------------------
            uint32_t w = 0, s = 0, magic = 0, col0 = 0;
            const bool strided = len_flags & kFlagStrided;
            if (strided) {
                const uint4 sr = __ldg(reinterpret_cast<const uint4*>(p.segs + d1.z));
                w = sr.x; s = sr.y; magic = sr.z; col0 = d1.w;
            }
#pragma unroll
            for (int i = 0; i < kItems; ++i) {
                mask[i] = 0; val[i][0] = 0; val[i][1] = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t e = e_warp + i * 128 + lane * 4 + j;
                    if (e < len) {
                        uint64_t so = src_off + e;
                        if (strided) {
                            const uint32_t cc = col0 + e;
                            const uint32_t row = (w == 1) ? cc : __umulhi(cc, magic);
                            so = src_off + (uint64_t)row * s + (cc - row * w);
                        }
                        const float tj = __ldcs(th + so), mj = __ldcs(mm + so), vj = __ldcs(vv + so);
                        const float prev = invert_adamw<DIV_BC1, DIV_DECAY>(tj, mj, vj, c);
                        const uint32_t bt = bf16_rne_bits(tj), bp = bf16_rne_bits(prev);
                        mask[i] |= (bt != bp ? 1u : 0u) << j;
                        val[i][j >> 1] |= bt << ((j & 1) * 16);
                    }
                }
            }
        }

        // ---- ordered ranks: warp scan of per-item counts packed 4 x 8 bits ------------------
        uint32_t cnt = 0;
#pragma unroll
        for (int i = 0; i < kItems; ++i) cnt |= __popc(mask[i]) << (8 * i);
        uint32_t incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += up;
        }
        const uint32_t excl = incl - cnt;                       // per item: changed in lanes below
        const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);  // per item: changed in this warp
        uint32_t item_base[kItems];
        uint32_t run = 0;
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            item_base[i] = run + ((excl >> (8 * i)) & 0xFFu);
            run += (tot >> (8 * i)) & 0xFFu;
        }
        if (lane == 0) sm.warp_total[warp] = run;
        __syncthreads();

        uint32_t warp_base = 0, tile_total = 0;
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) {
            const uint32_t x = sm.warp_total[w2];
            if (w2 < warp) warp_base += x;
            tile_total += x;
        }
        if (warp == 0) {
            uint64_t ex;
            const bool ok = look_back(p.status, t, tile_total, lane, &ex);
            if (lane == 0) { sm.tile_excl = ex; sm.ok = ok ? 1u : 0u; }
        }
        __syncthreads();
        const uint64_t tile_excl = sm.tile_excl;
        const bool ok = sm.ok != 0;
        if (!ok) {
            if (tid == 0) atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_TIMEOUT);
        } else {
            // ---- ordered writes --------------------------------------------------------
            bool dropped = false;
#pragma unroll
            for (int i = 0; i < kItems; ++i) {
                uint32_t mk = mask[i];
                uint64_t pos = tile_excl + warp_base + item_base[i];
                while (mk) {
                    const int j = __ffs(mk) - 1;
                    mk &= mk - 1;
                    if (pos < p.capacity) {
                        p.offsets[pos] = dst_off + e_warp + i * 128 + lane * 4 + j;
                        p.values[pos] = (uint16_t)(val[i][j >> 1] >> ((j & 1) * 16));
                    } else {
                        dropped = true;
                    }
                    ++pos;
                }
            }
            if (dropped) atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_OVERFLOW);
            if (tid == 0) {
                if (len_flags & kFlagFirstOfList) p.list_ptr[list] = tile_excl;
                if (len_flags & kFlagLastTile) {
                    p.list_ptr[p.n_lists] = tile_excl + tile_total;
                    p.counters[0] = tile_excl + tile_total;
                    p.counters[1] = p.scanned;
                }
            }
        }
        // sm.ticket / sm.tile_excl are rewritten only after the next __syncthreads pair
    }
}

// Lists without any tile (empty shard, or no operation targets it) start where the next
// list with tiles starts.  Only launched for layouts that have such lists.
__global__ void fill_empty_lists_kernel(uint64_t* list_ptr, const uint32_t* next_with_tiles,
                                        uint32_t n_lists) {
    for (uint32_t k = blockIdx.x * blockDim.x + threadIdx.x; k < n_lists; k += gridDim.x * blockDim.x) {
        const uint32_t nx = next_with_tiles[k];
        if (nx != k) list_ptr[k] = list_ptr[nx];
    }
}

template <bool A, bool B>
static dte_status launch_t(const ExtractParams& p, int n_ctas, cudaStream_t st) {
    extract_kernel<A, B><<<n_ctas, kThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

dte_status launch_extract(const ExtractParams& p, int n_ctas, cudaStream_t st) {
    const bool a = p.c.bc1 != 1.0f, b = p.c.decay != 1.0f;
    if (a && b) return launch_t<true, true>(p, n_ctas, st);
    if (a) return launch_t<true, false>(p, n_ctas, st);
    if (b) return launch_t<false, true>(p, n_ctas, st);
    return launch_t<false, false>(p, n_ctas, st);
}

dte_status extract_max_ctas(int device, int* n_ctas) {
    int sms = 0, per_sm = 0;
    DTE_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    DTE_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, extract_kernel<true, true>, kThreads, 0));
    if (per_sm < 1) per_sm = 1;
    *n_ctas = sms * per_sm;
    return DTE_OK;
}

dte_status launch_fill_empty_lists(uint64_t* list_ptr, const uint32_t* next_with_tiles,
                                   uint32_t n_lists, cudaStream_t st) {
    fill_empty_lists_kernel<<<1, 256, 0, st>>>(list_ptr, next_with_tiles, n_lists);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
