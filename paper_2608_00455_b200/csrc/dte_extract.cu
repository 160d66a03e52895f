// The fused streaming extract kernel: AdamW inversion (Eq. 2), BF16 cast and bit compare
// (Eq. 4), ordered stream compaction, and receiver-local remap (Eq. 5-6, evaluated
// destination-major through the tile table) in a single pass over theta / m / v.
//
// Structure.  One CTA per tile, one warp per warp-tile, no block-wide barrier until the
// very end.  A warp streams its warp-tile's theta / m / v through registers with 128-bit
// loads and classifies each element with a cheap conservative screen ("the BF16 pattern
// cannot have changed").  Elements the screen cannot clear (a few per cent) are queued in
// shared memory in element order and then evaluated densely, 32 at a time, with the exact
// IEEE arithmetic; the changed ones are compacted in place.  The CTA then reserves room
// for all its entries in a staging buffer with ONE atomic add, the warps write their
// (offset, value) pairs there with coalesced stores, in tile order, and the CTA records
// (position, count) for its tile.  No CTA waits on another; the ordered placement happens
// in the gather kernels (dte_gather.cu), which touch only the placement records and the
// changed entries.
//
// Build flags that matter for bit-exactness: -fmad=false -ftz=false -prec-div=true
// -prec-sqrt=true.  The exact path additionally spells every operation as a
// round-to-nearest intrinsic so that no flag can silently change it.
#include <atomic>

#include "dte_internal.cuh"

namespace dte {

constexpr int kMinCtasPerSm = 4;

// ---- exact arithmetic ------------------------------------------------------------

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

// ---- the screen --------------------------------------------------------------------
//
// Most elements cannot have changed, and the screen proves it for them without the divisions and
// the square root of Eq. 2.  It brackets the reconstruction between two fp32 numbers q and p and
// casts both: if they have the same BF16 pattern, so has everything between them.  Every step
// leans on one fact: round-to-nearest is monotone (real x <= y  =>  RN(x) <= RN(y), overflow and
// underflow included), so a bound pushed through the SAME rounded operation stays a bound, with
// no margin for rounding errors.
//     exact                      bound (operands non-negative)
//     mhat = RN(m / bc1)         A = RN(|m| * ka),        ka >= 1/bc1          => A >= |mhat|
//     den  = RN(RN(sqrt(RN(v/bc2))) + eps)
//                                W = min(|rsqrt(v)| * kb, kc),  kb >= sqrt(bc2)(1+2^-10),
//                                    kc >= 1/eps                               => W >= 1/den
//     u    = RN(mhat / den)      U = RN(A * W)                                 => U >= |u|
//     s    = RN(lr * u)          S = RN(U * |lr|)                              => S >= |s|
// (2^-10 in kb covers the 2^-22 error of the hardware rsqrt and the roundings of v/bc2, of the
// root and of the product; rsqrt.ftz turns a subnormal v into +Inf, so W = kc there, and
// den >= eps always.)  The step s has the sign of lr * m, because den >= +0 or NaN.  With that
// sign on S (it comes by itself when m and lr enter the products signed: rounding is symmetric),
// theta + s lies between theta and theta + S, hence
//     num = RN(theta + s)  lies between  theta  and  far = RN(theta + S)       (by value).
// Without a division by decay the reconstruction is num: q = theta, p = far.
// With it, recon = RN(num / decay) differs from num by at most
//     |num| |1/decay - 1|  +  2^-24 |num| / decay  (rounding; 2^-150 if the quotient is subnormal).
// If q and p (below) cast to the same BF16 pattern then theta and far, which lie between them,
// are in one BF16 rounding cell, so |num| <= |theta| (1 + 2^-7) where BF16 is normal and
// |num| <= |theta| + 2^-133 (a subnormal cell's width) where it is not.  With
//     kappa >= (|1/decay - 1| + 2^-24)(1 + 2^-7)(1 + 2^-10),   tiny >= 2^-133 kappa + 2^-148,
//     D = RN(|theta| kappa + tiny)   (one fma; its own rounding is inside the 2^-10 and the 2^-148)
// recon lies within D of num, so between the reals theta - D and theta + S + D (signs as for S), and,
// being an fp32 number, between their roundings
//     q = RN(theta - D),   p = RN(far + D).
// Equal values may still differ in pattern as +0 and -0; a reconstruction of -0 needs theta = -0
// and a step of -0, and then q or p is -0 or negative too.  Elements whose reconstruction is
// infinite or NaN must reach the exact path (it counts them): then p or q is infinite or NaN
// (monotonicity again; NaN arises only from NaN or infinite operands, which make S, far or D
// NaN or infinite), so a non-finite p or q never passes.  Everything else that is odd - negative
// v (W = -Inf or NaN), v = 0 with eps = 0, overflowing intermediates - makes S infinite or NaN and
// ends the same way.
__device__ __forceinline__ float min_nan(float x, float y) {
    float r;
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(x), "f"(y));
    return r;
}
__device__ __forceinline__ float rsqrt_ftz(float x) {
    float r;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
// Two BF16 casts (round to nearest even, subnormals kept, any NaN -> 0x7FFF) in one instruction.
// Only equality of the two halves is used, and never when either is NaN or infinite; the values
// that are emitted come from bf16_rne_bits.
__device__ __forceinline__ uint32_t bf16x2_rn(float hi, float lo) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <bool DIV_BC1, bool DIV_DECAY>
__device__ __forceinline__ bool surely_unchanged(float theta, float m, float v, const Screen& s, float lr) {
    // m and lr go in with their signs: rounding is symmetric, so the product is S with the sign of
    // lr * m, the step's (W >= +0; a negative v makes it -Inf or NaN, and the product infinite or NaN)
    const float ms = DIV_BC1 ? __fmul_rn(m, s.ka) : m;
    const float w = min_nan(__fmul_rn(rsqrt_ftz(v), s.kb), s.kc);      // -Inf for v = -0 or a negative subnormal
    const float sb = __fmul_rn(__fmul_rn(ms, w), lr);
    const float far = __fadd_rn(theta, sb);
    if (DIV_DECAY) {
        const float d = __uint_as_float(__float_as_uint(__fmaf_rn(fabsf(theta), s.kappa, s.tiny)) |
                                        (__float_as_uint(sb) & 0x80000000u));      // D, signed like S
        const uint32_t r = bf16x2_rn(__fadd_rn(far, d), __fsub_rn(theta, d));
        // halves equal, and (one test for both then) neither infinite nor NaN
        return r == __byte_perm(r, 0, 0x1032) && (r << 1) < 0xFF000000u;
    }
    const uint32_t r = bf16x2_rn(far, theta);
    // far is at least as extreme as theta: finite far, finite both (ordered compare: NaN fails)
    return r == __byte_perm(r, 0, 0x1032) && fabsf(far) < __int_as_float(0x7F800000);
}

__device__ __forceinline__ const float* ldg_ptr(const float* const* slot) {
    return reinterpret_cast<const float*>(__ldg(reinterpret_cast<const unsigned long long*>(slot)));
}
// ---- the kernel --------------------------------------------------------------------

// Row geometry of a strided (column-split) warp-tile; lives in shared memory, one per warp,
// because it is needed only when addresses are formed and registers are scarce.
struct StridedGeom {
    uint32_t w, s, magic;  // row width / source row stride / divisor (SegRec)
};

// Decoded descriptor of one warp-tile.  th / mm / vv already point at the warp-tile's first
// element (contiguous) or at the first column of its first source row (strided).
struct WarpTile {
    const float* th;
    const float* mm;
    const float* vv;
    const StridedGeom* geom;
    uint32_t col0;         // strided: column of warp-tile element 0 within the operation's extent
    uint32_t len;          // elements of this warp-tile (0 for the unused tail of a short tile)
    uint32_t dst0;         // receiver-local offset of element 0 of this warp-tile
    uint32_t len_flags;

    // source element offset (relative to th / mm / vv) of warp-tile element e
    __device__ __forceinline__ uint64_t src(uint32_t e) const {
        if (!(len_flags & kFlagStrided)) return e;
        const uint32_t w = geom->w, cc = col0 + e;
        const uint32_t row = (w == 1) ? cc : __umulhi(cc, geom->magic);
        return (uint64_t)row * geom->s + (cc - row * w);
    }
};

// Returns the source tensor index (needed once, for the parameter group); `tile` receives the
// index of the placement record.  PACKED: every warp has a descriptor of its own; otherwise
// the CTA shares one (its address depends on blockIdx only: uniform registers) and warp w
// takes the w-th kWarpTile slots of it.
template <bool PACKED>
__device__ __forceinline__ uint32_t decode(const ExtractParams& p, uint32_t index, int lane, int warp,
                                           StridedGeom* geom, WarpTile& wt, uint32_t& tile) {
    const uint4* td = reinterpret_cast<const uint4*>(PACKED ? p.packed + ((size_t)index * kSub + warp)
                                                            : p.tiles + index);
    const uint4 d0 = __ldg(td), d1 = __ldg(td + 1);
    const uint32_t e0 = PACKED ? 0u : (uint32_t)warp * kWarpTile;
    const uint32_t run_len = d1.x & kLenMask;
    tile = d1.y;
    wt.len_flags = d1.x | p.force_flags;
    wt.len = run_len > e0 ? min(run_len - e0, (uint32_t)kWarpTile) : 0u;
    wt.dst0 = d0.w + e0;
    wt.geom = geom;
    wt.col0 = 0;
    uint64_t off = ((uint64_t)d0.x | ((uint64_t)d0.y << 32));
    if (d1.x & kFlagStrided) {
        if (lane == 0) {
            const uint4 sr = __ldg(reinterpret_cast<const uint4*>(p.segs + d1.z));
            geom->w = sr.x; geom->s = sr.y; geom->magic = sr.z;
        }
        __syncwarp();
        wt.col0 = d1.w + e0;
    } else {
        off += e0;
    }
    wt.th = ldg_ptr(p.theta + d0.z) + off;
    wt.mm = ldg_ptr(p.m + d0.z) + off;
    wt.vv = ldg_ptr(p.v + d0.z) + off;
    return d0.z;
}

// One chunk (kChunk elements from warp-tile element cb) of theta / m / v into registers.
__device__ __forceinline__ void load_chunk(const WarpTile& wt, uint32_t cb, int lane,
                                           float4 (&a)[kItems], float4 (&b)[kItems], float4 (&g)[kItems]) {
    if (!(wt.len_flags & kFlagScalar)) {
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            const uint32_t e = cb + i * 128 + lane * 4;
            if (e < wt.len) {
                const uint64_t so = wt.src(e);
                // default caching on purpose: evict-first hints (ld.cs / ld.lu) push the lines out
                // of L2 before the exact path re-reads its few elements (measured: -25 %)
                a[i] = __ldg(reinterpret_cast<const float4*>(wt.th + so));
                b[i] = __ldg(reinterpret_cast<const float4*>(wt.mm + so));
                g[i] = __ldg(reinterpret_cast<const float4*>(wt.vv + so));
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            float ta[4], tb[4], tg[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t e = cb + i * 128 + lane * 4 + j;
                ta[j] = tb[j] = tg[j] = 0.f;
                if (e < wt.len) {
                    const uint64_t so = wt.src(e);
                    ta[j] = __ldg(wt.th + so); tb[j] = __ldg(wt.mm + so); tg[j] = __ldg(wt.vv + so);
                }
            }
            a[i] = make_float4(ta[0], ta[1], ta[2], ta[3]);
            b[i] = make_float4(tb[0], tb[1], tb[2], tb[3]);
            g[i] = make_float4(tg[0], tg[1], tg[2], tg[3]);
        }
    }
}

// Phase A of one warp-tile: stream theta / m / v chunk by chunk, screen every element, and
// append the indices of the undecided ones to the warp's queue in element order.  Returns the
// queue length.
template <bool DIV_BC1, bool DIV_DECAY, bool FAST>
__device__ __forceinline__ uint32_t phase_a(const WarpTile& cur, int lane, uint32_t* queue, const Screen& sc,
                                            float lr) {
    float4 a[kItems], b[kItems], g[kItems];
    uint32_t qn = 0;
#pragma unroll 1
    for (uint32_t cb = 0; cb < (FAST ? (uint32_t)kWarpTile : cur.len); cb += kChunk) {
        // chunk_fast: the whole chunk is inside the warp-tile and contiguous in the source (for a
        // column-split operation: inside one source row), so its loads need no bounds checks and
        // one address computation (warp-uniform decision)
        bool chunk_fast = FAST;
        uint64_t chunk_off = cb;
        if (!FAST && !(cur.len_flags & kFlagScalar) && cb + kChunk <= cur.len) {
            if (cur.len_flags & kFlagStrided) {
                const uint32_t w = cur.geom->w, cc = cur.col0 + cb;
                const uint32_t row = (w == 1) ? cc : __umulhi(cc, cur.geom->magic);
                const uint32_t col = cc - row * w;
                chunk_fast = col + kChunk <= w;
                chunk_off = (uint64_t)row * cur.geom->s + col;
            } else {
                chunk_fast = true;
            }
        }
        if (chunk_fast) {
            const float4* pt = reinterpret_cast<const float4*>(cur.th + chunk_off) + lane;
            const float4* pm = reinterpret_cast<const float4*>(cur.mm + chunk_off) + lane;
            const float4* pv = reinterpret_cast<const float4*>(cur.vv + chunk_off) + lane;
#pragma unroll
            for (int i = 0; i < kItems; ++i) {
                a[i] = __ldg(pt + i * 32);
                b[i] = __ldg(pm + i * 32);
                g[i] = __ldg(pv + i * 32);
            }
        } else {
            load_chunk(cur, cb, lane, a, b, g);
        }
        uint32_t amb[kItems];
        uint32_t cnt = 0;
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            const uint32_t e = cb + i * 128 + lane * 4;
            amb[i] = 0;
            if (chunk_fast || e < cur.len) {
                const float tt[4] = {a[i].x, a[i].y, a[i].z, a[i].w};
                const float m4[4] = {b[i].x, b[i].y, b[i].z, b[i].w};
                const float v4[4] = {g[i].x, g[i].y, g[i].z, g[i].w};
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (!surely_unchanged<DIV_BC1, DIV_DECAY>(tt[j], m4[j], v4[j], sc, lr)) amb[i] |= 1u << j;
                if (!FAST && (cur.len_flags & kFlagScalar))           // ragged tail of a scalar tile
                    amb[i] &= (1u << min(cur.len - e, 4u)) - 1u;
            }
            cnt |= __popc(amb[i]) << (8 * i);
        }
        // ordered slots: warp scan of the per-item counts, packed 8 bits each (each <= 128)
        uint32_t incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += up;
        }
        const uint32_t excl = incl - cnt;
        const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
        uint32_t run = qn;
#pragma unroll
        for (int i = 0; i < kItems; ++i) {
            uint32_t pos = run + ((excl >> (8 * i)) & 0xFFu);
            uint32_t mk = amb[i];
            while (mk) {
                const int j = __ffs(mk) - 1;
                mk &= mk - 1;
                queue[pos++] = cb + i * 128 + lane * 4 + j;
            }
            run += (tot >> (8 * i)) & 0xFFu;
        }
        qn = run;
    }
    return qn;
}

constexpr uint32_t kDescAhead = 4 * 148;   // CTAs resident at once: 4 per SM (registers and shared memory) on 148 SMs

// One tile: `index` counts within the tiles of its kind.  GROUPS: the constants come from the
// tile's parameter group instead of the kernel parameters.  EARLY: give the dependent-launch
// signal at once instead of after the stream (see the kernels below).
template <bool DIV_BC1, bool DIV_DECAY, bool GROUPS, bool PACKED, bool EARLY>
__device__ __forceinline__ void extract_tile(const ExtractParams& p, uint32_t index, uint32_t* s_queue,
                                             uint32_t* s_count, unsigned long long& s_pos, StridedGeom* s_geom) {
    if (EARLY) asm volatile("griddepcontrol.launch_dependents;");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* queue = s_queue + warp * kWarpTile;
    Consts c = p.c;
    Screen sc = p.s;
    const uint32_t lanemask_lt = (1u << lane) - 1u;
    static_assert(kSub == kWarps, "one warp per warp-tile");

    WarpTile cur;
    uint32_t tile;
    // A hint for the CTA that will take this one's place about one wave from now: its descriptor
    // is the first link of its start-up chain (descriptor, source pointers, first chunk) and the
    // only one that would otherwise come from DRAM.  Measured: 0.3 % of the step on the large
    // workloads, 1 % on a single matrix.
    if (!PACKED && threadIdx.x == 0 && index + kDescAhead < p.n_regular)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p.tiles + index + kDescAhead));
    {
        const uint32_t tensor = decode<PACKED>(p, index, lane, warp, &s_geom[warp], cur, tile);
        if (GROUPS) {   // one 48-byte record per parameter group
            const uint4* gp = reinterpret_cast<const uint4*>(p.groups + __ldg(p.tensor_group + tensor));
            const uint4 g0 = __ldg(gp), g1 = __ldg(gp + 1), g2 = __ldg(gp + 2);
            c.bc1 = __uint_as_float(g0.x); c.bc2 = __uint_as_float(g0.y); c.decay = __uint_as_float(g0.z);
            c.lr = __uint_as_float(g0.w); c.eps = __uint_as_float(g1.x);
            sc.ka = __uint_as_float(g1.y); sc.kb = __uint_as_float(g1.z); sc.kc = __uint_as_float(g1.w);
            sc.kappa = __uint_as_float(g2.x); sc.tiny = __uint_as_float(g2.y);
        }

        const float lr = c.lr;

        // ---- phase A: stream, screen, queue the undecided elements in element order ---------
        // FAST: a full, contiguous, 16-byte-aligned warp-tile (nearly all of them): no bounds
        // checks and no per-item address arithmetic (pointer + immediate).
        uint32_t qn = 0;
        if (cur.len == (uint32_t)kWarpTile && !(cur.len_flags & (kFlagScalar | kFlagStrided)))
            qn = phase_a<DIV_BC1, DIV_DECAY, true>(cur, lane, queue, sc, lr);
        else
            qn = phase_a<DIV_BC1, DIV_DECAY, false>(cur, lane, queue, sc, lr);
        __syncwarp();
        if (!EARLY) asm volatile("griddepcontrol.launch_dependents;");

        // ---- phase B: exact evaluation of the queue, 32 entries per round; the changed
        //      entries are compacted to the front of the queue as (index | value << 16) -----
        uint32_t n_changed = 0;
        uint32_t n_odd = 0;     // this lane's elements whose reconstruction is NaN, or Inf from a finite theta
        // the loads of round r + 1 are issued before round r is evaluated (their latency is an
        // L2 hit, several hundred ns, and rounds are otherwise serial)
        uint32_t e_cur = 0;
        float tj = 0.f, mj = 0.f, vj = 0.f;
        if ((uint32_t)lane < qn) {
            e_cur = queue[lane];
            const uint64_t so = cur.src(e_cur);
            tj = __ldg(cur.th + so); mj = __ldg(cur.mm + so); vj = __ldg(cur.vv + so);
        }
#pragma unroll 1
        for (uint32_t q0 = 0; q0 < qn; q0 += 32) {
            const uint32_t q = q0 + lane, qnext = q + 32;
            uint32_t e_nxt = 0;
            float tn = 0.f, mn = 0.f, vn = 0.f;
            if (qnext < qn) {
                e_nxt = queue[qnext];
                const uint64_t so = cur.src(e_nxt);
                tn = __ldg(cur.th + so); mn = __ldg(cur.mm + so); vn = __ldg(cur.vv + so);
            }
            bool changed = false;
            uint32_t entry = 0;
            if (q < qn) {
                const float prev = invert_adamw<DIV_BC1, DIV_DECAY>(tj, mj, vj, c);
                const uint32_t bt = bf16_rne_bits(tj), bp = bf16_rne_bits(prev);
                changed = bt != bp;
                entry = e_cur | (bt << 16);
                // reconstructions that broke: NaN, or an overflow from a finite theta (every such
                // element reaches this path: the screen's ordered compares fail on NaN and on an
                // infinite bound; an infinite theta that stays infinite may pass it and is not counted)
                n_odd += (prev != prev) | (isinf(prev) & (fabsf(tj) <= 3.402823466e38f));
            }
            // the ballot also orders this round's (and the next round's) queue reads before the
            // writes below, which land at or before slot q0 + 31
            const uint32_t msk = __ballot_sync(0xFFFFFFFFu, changed);
            if (changed) queue[n_changed + __popc(msk & lanemask_lt)] = entry;
            n_changed += __popc(msk);
            e_cur = e_nxt; tj = tn; mj = mn; vj = vn;
        }
        __syncwarp();
        if (__any_sync(0xFFFFFFFFu, n_odd != 0)) {      // rare: one atomic per warp-tile that saw any
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) n_odd += __shfl_xor_sync(0xFFFFFFFFu, n_odd, d);
            if (lane == 0) atomicAdd(p.cursor + 1, (unsigned long long)n_odd);
        }

        // ---- phase C: one reservation per CTA, coalesced writes in tile order, the record -----
        if (lane == 0) s_count[warp] = n_changed;
        __syncthreads();
        // exclusive prefix and total of the eight warp counts: lanes 0..7 of every warp scan them
        uint32_t incl = lane < kWarps ? s_count[lane] : 0u;
#pragma unroll
        for (int d = 1; d < kWarps; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += up;
        }
        const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, kWarps - 1);
        const uint32_t before = __shfl_sync(0xFFFFFFFFu, incl, warp) - n_changed;
        if (threadIdx.x == 0) {
            unsigned long long pos0 = 0;
            if (total) pos0 = atomicAdd(p.cursor, (unsigned long long)total);
            s_pos = pos0;
            p.rec[tile] = ((uint64_t)pos0 << kRecCountBits) | total;
        }
        __syncthreads();
        const unsigned long long pos = s_pos + before;
        const uint32_t rel = (uint32_t)warp * kWarpTile;        // tile-relative index: < kTile < 2^16, no carry
        for (uint32_t q = lane; q < n_changed; q += 32)
            if (pos + q < p.stage_capacity)               // beyond it the call overflows anyway
                p.stage[pos + q] = queue[q] + rel;
    }
}

// Shared memory of a CTA: per warp the queue of element indices awaiting exact evaluation, later
// (index | value << 16) - dynamic, kWarps * kWarpTile words, may exceed the 48 KB static limit.
#define DTE_EXTRACT_SHARED                              \
    extern __shared__ __align__(16) uint32_t s_queue[]; \
    __shared__ uint32_t s_count[kWarps];                \
    __shared__ unsigned long long s_pos;                \
    __shared__ StridedGeom s_geom[kWarps]

// One launch per kind of tile.  The packed-tile launch (few CTAs, each a serial chain of short
// runs) goes first and lets the regular-tile launch start at once (programmatic dependent
// launch): the two share nothing but the atomic staging cursor.  The regular-tile launch keeps
// its descriptor address a function of blockIdx alone (uniform registers; one kernel with a
// branch for both kinds of tile ran the regular tiles 15 % slower).  It gives its own signal
// after the stream, so that the gather of a small layout, launched the same way, is set up while
// the last tiles finish and does not sit on the SMs before.
template <bool DIV_BC1, bool DIV_DECAY, bool GROUPS, bool PACKED>
__global__ void __launch_bounds__(kThreads, kMinCtasPerSm) extract_kernel(const ExtractParams p) {
    DTE_EXTRACT_SHARED;
    extract_tile<DIV_BC1, DIV_DECAY, GROUPS, PACKED, PACKED>(p, blockIdx.x, s_queue, s_count, s_pos, s_geom);
    // The launch of the regular tiles may have begun before the launch of the packed tiles ended.
    // What follows in the stream (the gather) is ordered after THIS grid only, so this grid must
    // not complete before the one it overlapped: wait for it here, where nothing is left to do.
    // A no-op for a launch that did not overlap anything.
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

constexpr size_t kQueueBytes = (size_t)kWarps * kWarpTile * sizeof(uint32_t);

// Per device, once: allow more than 48 KB of dynamic shared memory.  Host threads may race here
// (two layouts on two threads); setting the attribute twice is harmless, so an atomic flag per
// device and kernel is enough.
template <class K>
static dte_status allow_queue_memory(K kernel, std::atomic<bool>* configured) {
    int dev = 0;
    DTE_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices || !configured[dev].load(std::memory_order_acquire)) {
        DTE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kQueueBytes));
        if (dev >= 0 && dev < kMaxDevices) configured[dev].store(true, std::memory_order_release);
    }
    return DTE_OK;
}

static dte_status launch_on(const void* kernel, const ExtractParams& p, uint32_t grid, bool overlap, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kQueueBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;      // may begin before the previous kernel in the stream has finished
    void* args[] = {const_cast<ExtractParams*>(&p)};
    DTE_CUDA(cudaLaunchKernelExC(&cfg, kernel, args));
    return DTE_OK;
}

// One call's extract launches: the packed tiles first, the regular tiles overlapping them.
template <bool A, bool B, bool G>
static dte_status launch_t(const ExtractParams& p, cudaStream_t st) {
    static std::atomic<bool> cfg_packed[kMaxDevices], cfg_regular[kMaxDevices];
    if (p.n_packed) {
        dte_status s = allow_queue_memory(extract_kernel<A, B, G, true>, cfg_packed);
        if (s == DTE_OK) s = launch_on((const void*)extract_kernel<A, B, G, true>, p, p.n_packed, false, st);
        if (s != DTE_OK) return s;
    }
    if (p.n_regular) {
        dte_status s = allow_queue_memory(extract_kernel<A, B, G, false>, cfg_regular);
        if (s == DTE_OK) s = launch_on((const void*)extract_kernel<A, B, G, false>, p, p.n_regular, p.n_packed != 0, st);
        if (s != DTE_OK) return s;
    }
    return DTE_OK;
}

// div_bc1 / div_decay: whether any group in the call has a divisor different from 1.0f.
dte_status launch_extract(const ExtractParams& p, bool div_bc1, bool div_decay, cudaStream_t st) {
    if (p.n_packed + p.n_regular == 0) return DTE_OK;
    const bool a = div_bc1, b = div_decay;
    if (p.groups) {
        if (a && b) return launch_t<true, true, true>(p, st);
        if (a) return launch_t<true, false, true>(p, st);
        if (b) return launch_t<false, true, true>(p, st);
        return launch_t<false, false, true>(p, st);
    }
    if (a && b) return launch_t<true, true, false>(p, st);
    if (a) return launch_t<true, false, false>(p, st);
    if (b) return launch_t<false, true, false>(p, st);
    return launch_t<false, false, false>(p, st);
}

}  // namespace dte
