// Chunk codec of the storage-mediated path (Section 4.4): the ordered (index, value) lists
// are serialised into self-describing chunks - int32 index + BF16 value per entry, as the
// paper's data-volume discussion states - with a checksum per chunk for the manifest, and
// read back (checksum verified before anything is written) on the destination.
//
//   plan   (1 CTA):   chunk count and byte offset of every list by a scan over list_ptr; one
//                     directory entry per chunk; totals and the overflow decision.
//   pack   (1 CTA per chunk, grid-stride): copy / transpose the entries, Adler-32 on the fly.
//   unpack (1 CTA per chunk, grid-stride): validate, checksum pass, then decode pass (the
//                     second read of a chunk comes from L2).
// Adler-32 in parallel: with N bytes b_0..b_{N-1}, s1 = 1 + sum b_q and s2 = N + sum (N-q) b_q
// (both mod 65521), so every thread adds weighted bytes independently; sums are kept in 64 bits
// and reduced once per chunk.  No kernel waits on another CTA.
#include "dte_internal.cuh"

namespace dte {

constexpr int kChunkThreads = 256;
constexpr int kPlanThreads = 1024;
constexpr uint32_t kHeaderBytes = DTE_CHUNK_HEADER_BYTES;
constexpr uint32_t kSummedHeaderBytes = 24;   // header bytes covered by the checksum
constexpr uint32_t kAdlerMod = 65521u;

__host__ __device__ inline uint64_t round16(uint64_t x) { return (x + 15) & ~15ull; }

__host__ __device__ inline uint64_t payload_bytes(uint64_t count, uint32_t format) {
    return format == DTE_CHUNK_PLAIN ? round16(6 * count) : 6 * round16(count);
}

struct Sums {
    uint64_t s1, s2;
};

// Adds the four bytes of a little-endian word whose byte 0 has weight `wt` (bytes 1..3: wt-1 ..):
// two byte-wise dot products give the plain and the position-weighted byte sums.
__device__ __forceinline__ void add_word(Sums& a, uint32_t w, uint32_t wt) {
    const uint32_t sum = __dp4a(w, 0x01010101u, 0u);       // b0 + b1 + b2 + b3
    const uint32_t skew = __dp4a(w, 0x03020100u, 0u);      // b1 + 2 b2 + 3 b3
    a.s1 += sum;
    a.s2 += (uint64_t)wt * sum - skew;
}

__device__ __forceinline__ void add_half(Sums& a, uint32_t h, uint32_t wt) {
    const uint32_t sum = __dp4a(h, 0x00000101u, 0u);
    a.s1 += sum;
    a.s2 += (uint64_t)wt * sum - (h >> 8);
}

// Sum over the CTA; every thread gets the result.  s_red: 2 * warps words of shared memory.
__device__ Sums block_sum(Sums a, uint64_t* s_red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        a.s1 += __shfl_xor_sync(0xFFFFFFFFu, a.s1, d);
        a.s2 += __shfl_xor_sync(0xFFFFFFFFu, a.s2, d);
    }
    __syncthreads();   // s_red may still be read from the previous chunk
    if (lane == 0) {
        s_red[2 * warp] = a.s1;
        s_red[2 * warp + 1] = a.s2;
    }
    __syncthreads();
    Sums t{0, 0};
    for (int w = 0; w < warps; ++w) {
        t.s1 += s_red[2 * w];
        t.s2 += s_red[2 * w + 1];
    }
    return t;
}

// Checksum of a chunk from the payload's sums: adds the covered header words, then reduces.
__device__ uint32_t finish_checksum(Sums pay, const uint32_t* head6, uint32_t pb) {
    const uint32_t N = kSummedHeaderBytes + pb;
#pragma unroll
    for (int j = 0; j < 6; ++j) add_word(pay, head6[j], N - 4 * j);
    const uint32_t s1 = (uint32_t)((1 + pay.s1) % kAdlerMod);
    const uint32_t s2 = (uint32_t)((N + pay.s2) % kAdlerMod);
    return (s2 << 16) | s1;
}

// ---- plan ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPlanThreads) chunk_plan_kernel(const PackParams p) {
    __shared__ uint64_t s_warp[2 * (kPlanThreads / 32)];
    __shared__ uint64_t s_carry[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t total = p.list_ptr[p.n_lists];
    if (total > p.capacity || (p.counters[2] & DTE_DEV_OVERFLOW)) {
        if (threadIdx.x == 0) {
            p.info[0] = 0; p.info[1] = 0; p.info[2] = DTE_DEV_OVERFLOW; p.info[3] = 0;
        }
        return;
    }
    if (threadIdx.x == 0) s_carry[0] = s_carry[1] = 0;
    __syncthreads();
    const uint64_t C = p.chunk_entries;
    const uint64_t full_bytes = kHeaderBytes + payload_bytes(C, p.format);
    for (uint32_t l0 = 0; l0 < p.n_lists; l0 += kPlanThreads) {
        const uint32_t l = l0 + threadIdx.x;
        uint64_t n = 0;
        if (l < p.n_lists) n = p.list_ptr[l + 1] - p.list_ptr[l];
        const uint64_t nfull = n / C, tail = n % C;
        const uint64_t x0 = nfull + (tail ? 1 : 0);
        const uint64_t x1 = nfull * full_bytes + (tail ? kHeaderBytes + payload_bytes(tail, p.format) : 0);
        uint64_t i0 = x0, i1 = x1;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint64_t u0 = __shfl_up_sync(0xFFFFFFFFu, i0, d), u1 = __shfl_up_sync(0xFFFFFFFFu, i1, d);
            if (lane >= d) { i0 += u0; i1 += u1; }
        }
        if (lane == 31) { s_warp[2 * warp] = i0; s_warp[2 * warp + 1] = i1; }
        __syncthreads();
        if (warp == 0) {
            const uint64_t w0 = s_warp[2 * lane], w1 = s_warp[2 * lane + 1];
            uint64_t j0 = w0, j1 = w1;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint64_t u0 = __shfl_up_sync(0xFFFFFFFFu, j0, d), u1 = __shfl_up_sync(0xFFFFFFFFu, j1, d);
                if (lane >= d) { j0 += u0; j1 += u1; }
            }
            s_warp[2 * lane] = j0 - w0;
            s_warp[2 * lane + 1] = j1 - w1;
        }
        __syncthreads();
        const uint64_t first_chunk = s_carry[0] + s_warp[2 * warp] + (i0 - x0);
        const uint64_t first_byte = s_carry[1] + s_warp[2 * warp + 1] + (i1 - x1);
        for (uint64_t k = 0; k < x0; ++k) {
            const uint64_t c = first_chunk + k;
            if (c < p.dir_capacity) {
                dte_chunk_ref r;
                r.byte_offset = first_byte + k * full_bytes;
                r.list = l;
                r.first_entry = (uint32_t)(k * C);
                p.dir[c] = r;
            }
        }
        __syncthreads();
        if (threadIdx.x == kPlanThreads - 1) {
            s_carry[0] = first_chunk + x0;
            s_carry[1] = first_byte + x1;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const uint64_t n_chunks = s_carry[0], bytes = s_carry[1];
        const bool fits = n_chunks <= p.dir_capacity && bytes <= p.stream_capacity;
        if (fits) {
            dte_chunk_ref r;
            r.byte_offset = bytes;
            r.list = 0xFFFFFFFFu;
            r.first_entry = 0;
            p.dir[n_chunks] = r;
        }
        p.info[0] = n_chunks;
        p.info[1] = bytes;
        p.info[2] = fits ? 0 : DTE_DEV_OVERFLOW;
        p.info[3] = total;
    }
}

// ---- pack ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kChunkThreads) chunk_pack_kernel(const PackParams p) {
    __shared__ uint64_t s_red[2 * (kChunkThreads / 32)];
    if (p.info[2] & DTE_DEV_OVERFLOW) return;
    const uint64_t n_chunks = p.info[0];
    const uint32_t tid = threadIdx.x;
    for (uint64_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const dte_chunk_ref ref = p.dir[c];
        const uint64_t lbeg = p.list_ptr[ref.list], lend = p.list_ptr[ref.list + 1];
        const uint32_t count = (uint32_t)min((uint64_t)p.chunk_entries, lend - lbeg - ref.first_entry);
        const uint32_t pb = (uint32_t)payload_bytes(count, p.format);
        const uint32_t* src_o = p.offsets + lbeg + ref.first_entry;
        const uint16_t* src_v = p.values + lbeg + ref.first_entry;
        uint8_t* head = p.stream + ref.byte_offset;
        uint8_t* pay = head + kHeaderBytes;
        Sums acc{0, 0};
        if (p.format == DTE_CHUNK_PLAIN) {
            uint32_t* out_o = reinterpret_cast<uint32_t*>(pay);
            uint16_t* out_v = reinterpret_cast<uint16_t*>(pay + 4ull * count);
            // four coalesced entries per thread in flight
            for (uint32_t i0 = tid; i0 < count; i0 += 4 * kChunkThreads) {
                uint32_t o[4], v[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t i = i0 + e * kChunkThreads;
                    if (i < count) {
                        o[e] = src_o[i];
                        v[e] = src_v[i];
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t i = i0 + e * kChunkThreads;
                    if (i < count) {
                        out_o[i] = o[e];
                        out_v[i] = (uint16_t)v[e];
                        add_word(acc, o[e], pb - 4 * i);
                        add_half(acc, v[e], pb - (4 * count + 2 * i));
                    }
                }
            }
            for (uint32_t q = 6 * count + tid; q < pb; q += kChunkThreads) pay[q] = 0;
        } else {
            // four entries per thread and step: one 32-bit word of each of the six planes
            const uint32_t P = (uint32_t)round16(count);
            for (uint32_t i = 4 * tid; i < P; i += 4 * kChunkThreads) {
                uint32_t o[4], v[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool in = i + e < count;
                    o[e] = in ? src_o[i + e] : 0u;
                    v[e] = in ? (uint32_t)src_v[i + e] : 0u;
                }
                if (p.format == DTE_CHUNK_DELTA_PLANES) {   // gaps to the previous entry of the chunk
                    const uint32_t before = (i > 0 && i < count) ? src_o[i - 1] : 0u;
#pragma unroll
                    for (int e = 3; e > 0; --e)
                        if (i + e < count) o[e] -= o[e - 1];
                    o[0] -= before;
                }
                const uint32_t lo01 = __byte_perm(o[0], o[1], 0x5140), lo23 = __byte_perm(o[2], o[3], 0x5140);
                const uint32_t hi01 = __byte_perm(o[0], o[1], 0x7362), hi23 = __byte_perm(o[2], o[3], 0x7362);
                const uint32_t v01 = v[0] | (v[1] << 16), v23 = v[2] | (v[3] << 16);
                uint32_t plane[6];
                plane[0] = __byte_perm(lo01, lo23, 0x5410);
                plane[1] = __byte_perm(lo01, lo23, 0x7632);
                plane[2] = __byte_perm(hi01, hi23, 0x5410);
                plane[3] = __byte_perm(hi01, hi23, 0x7632);
                plane[4] = __byte_perm(v01, v23, 0x6420);
                plane[5] = __byte_perm(v01, v23, 0x7531);
#pragma unroll
                for (int b = 0; b < 6; ++b) {
                    const uint32_t q = b * P + i;
                    *reinterpret_cast<uint32_t*>(pay + q) = plane[b];
                    add_word(acc, plane[b], pb - q);
                }
            }
        }
        const Sums tot = block_sum(acc, s_red);
        if (tid == 0) {
            uint32_t h[8] = {DTE_CHUNK_MAGIC, p.format, ref.list, ref.first_entry, count, pb, 0u, 0u};
            h[6] = finish_checksum(tot, h, pb);
            uint4* hp = reinterpret_cast<uint4*>(head);
            hp[0] = make_uint4(h[0], h[1], h[2], h[3]);
            hp[1] = make_uint4(h[4], h[5], h[6], h[7]);
        }
    }
}

// ---- unpack ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kChunkThreads) chunk_unpack_kernel(const UnpackParams p) {
    __shared__ uint64_t s_red[2 * (kChunkThreads / 32)];
    __shared__ uint32_t s_scan[kChunkThreads / 32];
    __shared__ __align__(16) uint32_t s_o[4 * kChunkThreads];   // one decode step of the plane layouts
    __shared__ __align__(16) uint16_t s_v[4 * kChunkThreads];
    const uint32_t tid = threadIdx.x;
    const uint64_t total = p.list_ptr[p.n_lists];
    uint64_t accepted = 0, rejected = 0, written = 0;   // meaningful in thread 0
    for (uint64_t c = blockIdx.x; c < p.n_chunks; c += gridDim.x) {
        // every thread evaluates the same (uniform) checks; nothing is read before the
        // directory has placed the chunk inside the stream on a 16-byte boundary
        const dte_chunk_ref ref = p.dir[c];
        const uint64_t begin = ref.byte_offset, end = p.dir[c + 1].byte_offset;
        bool ok = total <= p.capacity && (begin & 15) == 0 && end >= begin &&
                  end - begin >= kHeaderBytes && end <= p.stream_bytes;
        uint32_t h[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (ok) {
            const uint4* hp = reinterpret_cast<const uint4*>(p.stream + begin);
            const uint4 a = hp[0], b = hp[1];
            h[0] = a.x; h[1] = a.y; h[2] = a.z; h[3] = a.w;
            h[4] = b.x; h[5] = b.y; h[6] = b.z; h[7] = b.w;
        }
        const uint32_t format = h[1], list = h[2], first = h[3], count = h[4], pb = h[5];
        ok = ok && h[0] == DTE_CHUNK_MAGIC && format <= DTE_CHUNK_DELTA_PLANES && list < p.n_lists &&
             count > 0 && list == ref.list && first == ref.first_entry;
        uint64_t lbeg = 0;
        if (ok) {
            lbeg = p.list_ptr[list];
            const uint64_t lend = p.list_ptr[list + 1];
            // the list boundaries come from a manifest too: they must nest inside the buffers
            ok = lbeg <= lend && lend <= total && (uint64_t)first + count <= lend - lbeg &&
                 (uint64_t)pb == payload_bytes(count, format) && end - begin == kHeaderBytes + (uint64_t)pb;
        }
        const uint8_t* pay = p.stream + begin + kHeaderBytes;
        if (ok) {   // pass 1: checksum of what is about to be decoded
            Sums acc{0, 0};
            for (uint32_t q0 = 16 * tid; q0 < pb; q0 += 4 * 16 * kChunkThreads) {
                uint4 w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t q = q0 + e * 16 * kChunkThreads;
                    w[e] = q < pb ? *reinterpret_cast<const uint4*>(pay + q) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t q = q0 + e * 16 * kChunkThreads;
                    if (q < pb) {
                        add_word(acc, w[e].x, pb - q);
                        add_word(acc, w[e].y, pb - q - 4);
                        add_word(acc, w[e].z, pb - q - 8);
                        add_word(acc, w[e].w, pb - q - 12);
                    }
                }
            }
            const Sums tot = block_sum(acc, s_red);
            ok = finish_checksum(tot, h, pb) == h[6];
        }
        if (!ok) {
            rejected += 1;
            continue;
        }
        accepted += 1;
        written += count;
        uint32_t* out_o = p.offsets + lbeg + first;
        uint16_t* out_v = p.values + lbeg + first;
        if (format == DTE_CHUNK_PLAIN) {
            const uint32_t* in_o = reinterpret_cast<const uint32_t*>(pay);
            const uint16_t* in_v = reinterpret_cast<const uint16_t*>(pay + 4ull * count);
            for (uint32_t i0 = tid; i0 < count; i0 += 4 * kChunkThreads) {
                uint32_t o[4];
                uint16_t v[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t i = i0 + e * kChunkThreads;
                    if (i < count) {
                        o[e] = in_o[i];
                        v[e] = in_v[i];
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t i = i0 + e * kChunkThreads;
                    if (i < count) {
                        out_o[i] = o[e];
                        out_v[i] = v[e];
                    }
                }
            }
        } else {
            const uint32_t P = (uint32_t)round16(count);
            const bool gaps = format == DTE_CHUNK_DELTA_PLANES;
            uint32_t carry = 0;                       // gaps: sum of all gaps before this step's entries
            // uniform trip count: every thread takes part in the scan of every step
            for (uint32_t i0 = 0; i0 < count; i0 += 4 * kChunkThreads) {
                const uint32_t i = i0 + 4 * tid;
                uint32_t plane[6] = {0, 0, 0, 0, 0, 0};
                if (i < count) {
#pragma unroll
                    for (int b = 0; b < 6; ++b) plane[b] = *reinterpret_cast<const uint32_t*>(pay + b * P + i);
                }
                const uint32_t lo01 = __byte_perm(plane[0], plane[1], 0x5140);   // e0: b0 b1, e1: b0 b1
                const uint32_t lo23 = __byte_perm(plane[0], plane[1], 0x7362);
                const uint32_t hi01 = __byte_perm(plane[2], plane[3], 0x5140);
                const uint32_t hi23 = __byte_perm(plane[2], plane[3], 0x7362);
                uint32_t o[4], v[4];
                o[0] = __byte_perm(lo01, hi01, 0x5410);
                o[1] = __byte_perm(lo01, hi01, 0x7632);
                o[2] = __byte_perm(lo23, hi23, 0x5410);
                o[3] = __byte_perm(lo23, hi23, 0x7632);
                const uint32_t v01 = __byte_perm(plane[4], plane[5], 0x5140);
                const uint32_t v23 = __byte_perm(plane[4], plane[5], 0x7362);
                v[0] = v01 & 0xFFFF; v[1] = v01 >> 16; v[2] = v23 & 0xFFFF; v[3] = v23 >> 16;
                if (gaps) {   // index = running sum of the gaps (mod 2^32): thread, warp, CTA, carry
#pragma unroll
                    for (int e = 1; e < 4; ++e)
                        if (i + e < count) o[e] += o[e - 1]; else o[e] = o[e - 1];
                    const int lane = tid & 31, warp = tid >> 5;
                    uint32_t incl = o[3];
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                        if (lane >= d) incl += up;
                    }
                    __syncthreads();                  // s_scan may still be read from the previous step
                    if (lane == 31) s_scan[warp] = incl;
                    __syncthreads();
                    uint32_t before = carry + incl - o[3], step_total = 0;
#pragma unroll
                    for (int w = 0; w < kChunkThreads / 32; ++w) {
                        const uint32_t t = s_scan[w];
                        if (w < warp) before += t;
                        step_total += t;
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) o[e] += before;
                    carry += step_total;
                }
                // through shared memory, so that the global stores are consecutive across lanes
                __syncthreads();                      // the previous step's entries have been written out
                *reinterpret_cast<uint4*>(s_o + 4 * tid) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint2*>(s_v + 4 * tid) = make_uint2(v[0] | (v[1] << 16), v[2] | (v[3] << 16));
                __syncthreads();
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t r = e * kChunkThreads + tid;
                    if (i0 + r < count) {
                        out_o[i0 + r] = s_o[r];
                        out_v[i0 + r] = s_v[r];
                    }
                }
            }
        }
    }
    if (tid == 0) {
        if (written) atomicAdd((unsigned long long*)(p.counters + 0), (unsigned long long)written);
        if (accepted) atomicAdd((unsigned long long*)(p.counters + 1), (unsigned long long)accepted);
        if (rejected) {
            atomicAdd((unsigned long long*)(p.counters + 3), (unsigned long long)rejected);
            atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_CORRUPT);
        }
        if (blockIdx.x == 0 && total > p.capacity)
            atomicOr((unsigned long long*)(p.counters + 2), (unsigned long long)DTE_DEV_OVERFLOW);
    }
}

static dte_status chunk_grid(int device, uint64_t chunks, int* out) {
    int sms = 0;
    DTE_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    const uint64_t want = (uint64_t)sms * 8;   // 8 CTAs of 256 threads per SM
    *out = (int)(chunks < want ? (chunks ? chunks : 1) : want);
    return DTE_OK;
}

dte_status launch_pack_chunks(const PackParams& p, int device, cudaStream_t st) {
    int grid = 1;
    dte_status rc = chunk_grid(device, p.dir_capacity, &grid);
    if (rc != DTE_OK) return rc;
    chunk_plan_kernel<<<1, kPlanThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    chunk_pack_kernel<<<grid, kChunkThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

dte_status launch_unpack_chunks(const UnpackParams& p, int device, cudaStream_t st) {
    int grid = 1;
    dte_status rc = chunk_grid(device, p.n_chunks, &grid);
    if (rc != DTE_OK) return rc;
    chunk_unpack_kernel<<<grid, kChunkThreads, 0, st>>>(p);
    DTE_CUDA(cudaGetLastError());
    return DTE_OK;
}

}  // namespace dte
