// Batch-1 dual-trit-plane GEMV for sm_100a on packed format 2:  y = alpha1 (.) (T1 x) + alpha2 (.) (T2 x).
//
// Why this shape.  On sm_100 a mask (LOP3), a packed fp16 FMA and an integer dot product all issue at 64
// lanes/clk/SM, so a decode that spends one mask and one FMA per two trits is issue bound well below the HBM
// rate.  Format 2 puts the four codes of one input column (two rows x two planes) in one byte; one mask with
// 0x03030303 << 2f then yields, for field f, four byte-sized codes q * 4^f of four consecutive columns, which
// feed integer dot products (dp4a) directly: one mask per four trits, and the power 4^f is a constant of
// the accumulator that the scale epilogue divides out.
//
//   * Activations become 16-bit block fixed point: per 64-column lane block, X_j = round(x_j * 2^s) with
//     2^s chosen so the block maximum lies in [2^14, 2^15); X_j = 256 * hi_j + lo_j (hi signed, lo unsigned
//     byte).  fp16 values within 2^-5 of the block maximum are represented exactly; smaller ones are rounded
//     to 2^-16 of the maximum.  All sums over a lane block are exact int32.
//   * sum_j t_j X_j = sum_j q_j X_j - sum_j X_j (q = t + 1): the low accumulators start at minus the block sum.
//   * A CTA owns a contiguous range of row pairs.  Warp w is bound to the 2048-column slice (w mod S), takes a
//     contiguous share of the CTA's row pairs and keeps the slice's X (32 registers per lane) while it stays
//     there; lanes own 64 consecutive columns, so a lane's four accumulator pairs (2 rows x 2 planes) see one
//     scale group half and get the group's scales (the method's only multiplies) in an fp32 epilogue.
//   * The slice units of consecutive row pairs (2048 code bytes + 128 scale bytes each) are contiguous in HBM.
//     Each warp streams its run of units through a private shared-memory ring: one bulk copy (cp.async.bulk,
//     no multicast) per RU units, issued by lane 0 and completed on an mbarrier, several copies in flight.
//     Issuing a copy and waiting for it cost about 40 instructions, which is why a copy brings several units.
//     Bulk copies cost no load/store-unit time.
//     Every wait on an mbarrier is bounded: if one gives up the warp writes NaN rows, records an error in a
//     device status word (ptqtp_kernel_status) and still runs to the end.
//   * Rows are reduced over the lanes by shuffles, over the slices through shared memory in a fixed order
//     (deterministic), rounded once to fp16.
//   * Two CTAs per SM whenever the activations leave room: the head and the tail of one CTA (fetching x, the
//     final reduction) overlap the streaming of the other, also across consecutive launches.
//   * Speculative execution under programmatic dependent launch.  x and y belong to the stream's order, the
//     packed planes do not.  Earlier work of the stream may still be running when this kernel starts; most
//     calls of a decoder read an x that was finished long before.  The kernel therefore reads x at once,
//     computes everything into shared memory, then waits for the earlier work, reads x again and compares it
//     bit by bit with its first read (kept in shared memory).  Only then y is written; if a single bit of x
//     differed, the whole computation is repeated from the second read.  Results never depend on the timing.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

// Device-side status of the GEMV kernels: set when a bounded wait for a bulk copy gave up.
__device__ int g_gemv2_status = 0;

namespace {

constexpr int kMaxWarps2 = 16;
constexpr int kMaxThreads2 = kMaxWarps2 * 32;
constexpr int kSpinLimit = 1 << 22;             // polls of an mbarrier before a wait gives up
constexpr int kSpinLimitAfterFailure = 1 << 8;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
// (the mbarriers and ring slots are addressed by their 32-bit shared-memory addresses)
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bulk copy global -> this CTA's shared memory, completion counted in bytes on an mbarrier (no multicast).
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// d = c + sum_b u8(a.b) * s8(x.b)   and   d = c + sum_b u8(a.b) * u8(x.b)
__device__ __forceinline__ int dot_us(uint32_t a, uint32_t x, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(x), "r"(c));
    return d;
}
__device__ __forceinline__ int dot_uu(uint32_t a, uint32_t x, int c) {
    int d;
    asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(x), "r"(c));
    return d;
}

// Convert 16 activations (two uint4 of fp16: columns base .. base + 15) to block fixed point and store them.
//   xhi, xlo : [K/64 blocks][16 words]  bytes of hi_j / lo_j in column order, 16-byte chunks permuted (see below)
//   meta     : [K/64 blocks] (2^-s as float bits, sum_j X_j)
// Four adjacent threads share a 64-column block (16 columns each); the whole warp must call this.
__device__ __noinline__ void convert_x16(uint4 ra, uint4 rb, int base, bool valid, uint32_t* xhi, uint32_t* xlo, int2* meta) {
    const uint32_t rw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
    // block maximum of |x| on the fp16 bit patterns (ordered like the values once the sign is cleared)
    uint32_t m2 = 0u;
#pragma unroll
    for (int e = 0; e < 8; ++e) m2 = __vmaxu2(m2, rw[e] & 0x7fff7fffu);
    uint32_t mxb = max(m2 & 0xffffu, m2 >> 16);
    mxb = max(mxb, __shfl_xor_sync(0xffffffffu, mxb, 1));
    mxb = max(mxb, __shfl_xor_sync(0xffffffffu, mxb, 2));
    // exponent of the block maximum, in [-24, 15] for finite inputs; subnormal fp16 (exponent field 0) are
    // integers times 2^-24
    int s = 0;
    if (mxb != 0u) {
        const int ef = (int)(mxb >> 10);
        const int ex = ef ? ef - 15 : (31 - __clz((int)mxb)) - 24;
        s = 14 - ex;
    }
    const float scale = __uint_as_float((uint32_t)(127 + s) << 23);
    // x * 2^s is exact and below 2^15 in magnitude; adding 1.5 * 2^23 rounds it to the nearest integer (ties to
    // even) and leaves that integer, as a 16-bit two's complement number, in the low 16 bits of the float
    uint32_t B[16];
    uint32_t sum = 0u;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&rw[e]));
        B[2 * e] = __float_as_uint(fmaf(v.x, scale, 12582912.f));
        B[2 * e + 1] = __float_as_uint(fmaf(v.y, scale, 12582912.f));
        sum += B[2 * e] + B[2 * e + 1];
    }
    int isum = (int)(sum - 16u * 0x4B400000u);          // sum of the integers themselves
    isum += __shfl_xor_sync(0xffffffffu, isum, 1);
    isum += __shfl_xor_sync(0xffffffffu, isum, 2);
    uint32_t hw[4], lw[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        // byte 0 (lo) and byte 1 (hi) of four consecutive X gathered into one word each
        const uint32_t lo01 = __byte_perm(B[4 * w], B[4 * w + 1], 0x0040), lo23 = __byte_perm(B[4 * w + 2], B[4 * w + 3], 0x0040);
        const uint32_t hi01 = __byte_perm(B[4 * w], B[4 * w + 1], 0x0051), hi23 = __byte_perm(B[4 * w + 2], B[4 * w + 3], 0x0051);
        lw[w] = __byte_perm(lo01, lo23, 0x5410);
        hw[w] = __byte_perm(hi01, hi23, 0x5410);
    }
    if (valid) {
        // the four 16-byte chunks of a block are stored permuted (chunk v at v ^ swz) so that the lanes of a warp,
        // which each read a whole block with 128-bit loads, do not collide on shared-memory banks
        const int blk = base >> 6, v = (base >> 4) & 3;
        const int pos = blk * 16 + ((v ^ ((blk >> 1) & 3)) << 2);
        *reinterpret_cast<uint4*>(xhi + pos) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        *reinterpret_cast<uint4*>(xlo + pos) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
        if (v == 0) meta[blk] = make_int2((int)((uint32_t)(127 - s) << 23), isum);
    }
}

// Shared memory: x as two byte planes and block records, the first read of x (fp16 as read, only when executing
// speculatively), the per-slice partial sums, one mbarrier per ring slot, then the ring (one slice unit, kUnit2
// bytes, RU of them per slot; D slots per warp).
struct Smem2 {
    size_t raw_off, partial_off, bar_off, ring_off, total;
};
__host__ __device__ inline Smem2 smem_layout2(int k, int slices, int rows_cap, int warps, int depth, int ru, int speculate) {
    Smem2 m;
    m.raw_off = ((size_t)(k / kLane2) * 136 + 15) / 16 * 16;
    m.partial_off = m.raw_off + (speculate ? (size_t)2 * k : 0);
    m.bar_off = (m.partial_off + (size_t)rows_cap * slices * 4 + 7) / 8 * 8;
    m.ring_off = (m.bar_off + (size_t)warps * depth * 8 + 15) / 16 * 16;
    m.total = m.ring_off + (size_t)warps * depth * ru * kUnit2;
    return m;
}

template <int D, int RU>
__global__ void __launch_bounds__(kMaxThreads2, 1)
gemv2_kernel(Layout2 L, const unsigned char* __restrict__ packed, const __half* __restrict__ x,
             __half* __restrict__ y, int rows_cap, int rp_base, int rp_rem, int speculate, int gated) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int nblk = L.k / kLane2;
    uint32_t* xhi = reinterpret_cast<uint32_t*>(smem);
    uint32_t* xlo = xhi + nblk * 16;
    int2* meta = reinterpret_cast<int2*>(xlo + nblk * 16);
    const int warps = blockDim.x >> 5;
    const Smem2 sm = smem_layout2(L.k, L.slices, rows_cap, warps, D, RU, speculate);
    uint4* first_read = reinterpret_cast<uint4*>(smem + sm.raw_off);        // x as read before the dependency wait
    float* partial = reinterpret_cast<float*>(smem + sm.partial_off);       // [rows_cap][slices]
    // (the shuffle tells the compiler that the warp index is the same in all lanes: what derives from it can live
    // in uniform registers, which the bulk-copy instruction wants)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bar_off) + warp * D;
    constexpr int kSlot = RU * kUnit2;                 // a ring slot holds the RU units of one copy
    unsigned char* ring = smem + sm.ring_off + (size_t)warp * D * kSlot;

    // Let the next kernel on the stream start while this one runs.
    asm volatile("griddepcontrol.launch_dependents;");

    // this CTA's row pairs, and this warp's share of their slice units
    // balanced partition computed on the host: the first rp_rem CTAs take rp_base + 1 row pairs, the rest rp_base
    const int rp0 = (int)blockIdx.x * rp_base + min((int)blockIdx.x, rp_rem);
    const int rp1 = rp0 + rp_base + ((int)blockIdx.x < rp_rem ? 1 : 0);
    const int S = L.slices;
    const int Wc = min(S, warps);                       // slice lanes among the warps
    const int m = warps / Wc;                           // warps sharing a slice lane
    const int sl_lane = warp % Wc, wi = warp / Wc;
    const bool idle = wi >= m;
    const int n_sl = idle ? 0 : (S - sl_lane + Wc - 1) / Wc;
    // the m warps of a slice lane split the CTA's row pairs into contiguous runs (balanced +-1)
    const int n_cta = rp1 - rp0;
    const int rpw = rp0 + (idle ? 0 : wi * (n_cta / m) + min(wi, n_cta % m));
    const int n_rp = idle ? 0 : n_cta / m + (wi < n_cta % m ? 1 : 0);
    const unsigned char* codes = packed + L.codes_off;
    const int nchunks = L.k >> 3, nchunks16 = L.k >> 4, cthreads = blockDim.x;

    if (lane == 0) {
#pragma unroll
        for (int d = 0; d < D; ++d) mbar_init(bars + d, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    // producer (lane 0): slice pass pt, units left in it, source and unit size of the next copy, ring slot
    const uint32_t bars_a = smem_u32(bars), ring_a = smem_u32(ring);
    int pt = 0, pleft = 0, pslot = 0;
    uint32_t pbytes = 0;
    const unsigned char* psrc = codes;
    auto issue = [&]() {
        if (pt < n_sl) {
            const int nun = min(RU, pleft);
            const uint32_t bytes = (uint32_t)nun * pbytes;
            if (lane == 0) {
                mbar_expect_tx(bars_a + 8 * pslot, bytes);
                bulk_copy_g2s(ring_a + pslot * kSlot, psrc, bytes, bars_a + 8 * pslot);
            }
            psrc += bytes;
            pleft -= nun;
            if (pleft == 0) {
                ++pt;
                pleft = n_rp;
                psrc = codes + unit_offset(L, rpw, min(sl_lane + pt * Wc, S - 1));
                pbytes = (sl_lane + pt * Wc) == S - 1 ? (uint32_t)L.last_unit : (uint32_t)kUnit2;
            }
        }
        pslot = pslot + 1 == D ? 0 : pslot + 1;
    };

    int cslot = 0;
    uint32_t phase = 0;                                 // parity of the ring pass being consumed
    bool failed = false, waited = false;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // Pass 0 is speculative when allowed: x is read before earlier work of the stream is known to be complete.
        const bool spec = speculate && attempt == 0;
        if (!spec && !waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = true;
        }
        pt = n_rp > 0 ? 0 : n_sl;
        pleft = n_rp;
        psrc = codes + unit_offset(L, rpw, min(sl_lane, S - 1));
        pbytes = sl_lane == S - 1 ? (uint32_t)L.last_unit : (uint32_t)kUnit2;
        // x -> block fixed point in shared memory, two 16-column chunks per thread in flight.  Reads go to L2
        // (ld.global.cg), the point of coherence, never through L1.  The first reads are issued before the ring
        // is filled (behind the fill they would wait for all of it); the packed planes do not depend on earlier
        // work of the stream, so the fill never waits for that work.
        bool filled = false;
        for (int cb = (int)threadIdx.x; (cb & ~31) < nchunks16; cb += 2 * cthreads) {
            uint4 r[4];
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                const int c = cb + p * cthreads;
                r[2 * p] = r[2 * p + 1] = make_uint4(0u, 0u, 0u, 0u);
                if (c < nchunks16) {
                    r[2 * p] = __ldcg(reinterpret_cast<const uint4*>(x) + 2 * c);
                    r[2 * p + 1] = __ldcg(reinterpret_cast<const uint4*>(x) + 2 * c + 1);
                }
            }
            if (!filled) {
                filled = true;
#pragma unroll
                for (int d = 0; d < D; ++d) issue();
            }
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                const int c = cb + p * cthreads;
                if ((c & ~31) < nchunks16) {
                    if (spec && c < nchunks16) { first_read[2 * c] = r[2 * p]; first_read[2 * c + 1] = r[2 * p + 1]; }
                    convert_x16(r[2 * p], r[2 * p + 1], c << 4, c < nchunks16, xhi, xlo, meta);
                }
            }
        }
        if (!filled) {                                  // a warp with no part of x to convert
#pragma unroll
            for (int d = 0; d < D; ++d) issue();
        }
        __syncthreads();

        for (int t = 0; t < n_sl; ++t) {
            const int sl = sl_lane + t * Wc;
            const int active = sl == S - 1 ? L.last_active : 32;
            const bool live = lane < active;
            // this lane's X block for the slice stays in registers
            uint32_t xh[16], xl[16];
            const int blk = sl * 32 + (live ? lane : 0);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int pos = blk * 16 + ((v ^ ((blk >> 1) & 3)) << 2);
                const uint4 a = *reinterpret_cast<const uint4*>(xhi + pos);
                const uint4 b = *reinterpret_cast<const uint4*>(xlo + pos);
                xh[4 * v] = a.x; xh[4 * v + 1] = a.y; xh[4 * v + 2] = a.z; xh[4 * v + 3] = a.w;
                xl[4 * v] = b.x; xl[4 * v + 1] = b.y; xl[4 * v + 2] = b.z; xl[4 * v + 3] = b.w;
            }
            const int2 mt = meta[blk];
            const float c0 = live ? __int_as_float(mt.x) : 0.f, c1 = 0.0625f * c0;
            // sum_j t_j X_j = sum_j q_j X_j - sum_j X_j: the low accumulators start at minus 4^f times the block sum;
            // the unmasked word stands for all four fields at once and starts at minus (1 + 4 + 16 + 64) times it
            const int n0 = -mt.y, n1 = -(mt.y << 2), n2 = -(mt.y << 4), n3 = -(mt.y * 85);
            float* ppart = partial + (size_t)(2 * (rpw - rp0) + (lane >> 4)) * S + sl;
            const int ubytes = sl == S - 1 ? L.last_unit : kUnit2;
            // a slot holds the unit as it lies in memory: atom (i, l) at 16 (i A + l), the scale quads after the atoms
            const int ln = live ? lane : 0;
            const int atom_stride = active * 16;
            const int scale_off = active * 64 + (ln >> 1) * 8 - ln * 16;
            for (int j0 = 0; j0 < n_rp; j0 += RU) {
                // wait (bounded) for the copy in slot cslot; it has normally arrived long ago
                if (!mbar_try_wait(bars_a + 8 * cslot, phase)) {
                    const int limit = failed ? kSpinLimitAfterFailure : kSpinLimit;
                    int spins = 0;
                    while (!mbar_try_wait(bars_a + 8 * cslot, phase)) {
                        if (++spins >= limit) { failed = true; break; }
                    }
                }
                const int nun = min(RU, n_rp - j0);
                const unsigned char* buf = ring + cslot * kSlot + ln * 16;
                auto unit_body = [&](const unsigned char* ub, float* pp) {
                // Fields 0..2 are masked out of each code word; the unmasked word gives the sum of all four fields
                // (a byte is q0 + 4 q1 + 16 q2 + 64 q3 <= 170), so field 3 is "all" minus the other three.
                int ah[4] = {0, 0, 0, 0};
                int al[4] = {n0, n1, n2, n3};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 cw = *reinterpret_cast<const uint4*>(ub + i * atom_stride);
                    const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
                    for (int ww = 0; ww < 4; ++ww) {
#pragma unroll
                        for (int f = 0; f < 3; ++f) {
                            const uint32_t mk = w[ww] & (0x03030303u << (2 * f));
                            ah[f] = dot_us(mk, xh[4 * i + ww], ah[f]);
                            al[f] = dot_uu(mk, xl[4 * i + ww], al[f]);
                        }
                        ah[3] = dot_us(w[ww], xh[4 * i + ww], ah[3]);
                        al[3] = dot_uu(w[ww], xl[4 * i + ww], al[3]);
                    }
                }
                const uint2 sc = *reinterpret_cast<const uint2*>(ub + scale_off);
                const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&sc.x));   // alpha1, alpha2 of row 0
                const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&sc.y));   // ... of row 1
                // Q0..Q2 = 4^f * sum_j t_j X_j of fields 0..2; the unmasked word minus those three is field 3's
                const int Q0 = (ah[0] << 8) + al[0], Q1 = (ah[1] << 8) + al[1], Q2 = (ah[2] << 8) + al[2];
                const int Q3 = (ah[3] << 8) + al[3] - Q0 - Q1 - Q2;
                // lanes past the slice's columns redo lane 0 and contribute zero
                // (their block scale c0 is zero and the unit they read is real data, so their products are zero)
                float y0 = c0 * fmaf(0.25f, s0.y * (float)Q1, s0.x * (float)Q0);
                float y1 = c1 * fmaf(0.25f, s1.y * (float)Q3, s1.x * (float)Q2);
                // lanes 0-15 reduce row 0, lanes 16-31 row 1
                const float send = (lane & 16) ? y0 : y1;
                float v = ((lane & 16) ? y1 : y0) + __shfl_xor_sync(0xffffffffu, send, 16);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if ((lane & 15) == 0) *pp = failed ? __int_as_float(0x7fc00000) : v;
                };
                if (RU == 2 && nun == 2) {
                    // both units in one basic block: the second unit's loads and dot products fill the latencies of
                    // the first unit's epilogue and reduction
                    unit_body(buf, ppart);
                    unit_body(buf + ubytes, ppart + 2 * S);
                    ppart += 4 * S;
                } else {
#pragma unroll 1
                    for (int u = 0; u < nun; ++u, buf += ubytes, ppart += 2 * S) unit_body(buf, ppart);
                }
                // every lane has consumed the slot: lane 0 may refill it
                __syncwarp();
                issue();
                if (++cslot == D) { cslot = 0; phase ^= 1u; }
            }
        }
        if (!spec) break;
        // Earlier work of the stream is complete after this wait: if x still reads as it did, the pass stands.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
        int stale = 0;
#pragma unroll 4
        for (int c = (int)threadIdx.x; c < nchunks; c += cthreads) {
            const uint4 now = __ldcg(reinterpret_cast<const uint4*>(x) + c);
            const uint4 was = first_read[c];
            stale |= (now.x != was.x) | (now.y != was.y) | (now.z != was.z) | (now.w != was.w);
        }
        if (!__syncthreads_or(stale)) break;
    }
    if (failed && lane == 0) atomicExch(&g_gemv2_status, (int)PTQTP_ERR_CUDA);
    __syncthreads();
    if (gated) {
        // gated pair epilogue: a row pair is (gate row, up row) and gives one output silu(gate) * up, computed
        // from the unrounded fp32 sums
        for (int r = threadIdx.x; r < rp1 - rp0; r += blockDim.x) {
            float g = 0.f, u = 0.f;
            for (int s = 0; s < S; ++s) {
                g += partial[(size_t)(2 * r) * S + s];
                u += partial[(size_t)(2 * r + 1) * S + s];
            }
            y[rp0 + r] = __float2half_rn(g / (1.f + expf(-g)) * u);
        }
        return;
    }
    const int rows = 2 * (rp1 - rp0);
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        const int row = 2 * rp0 + r;
        float t = 0.f;
        for (int s = 0; s < S; ++s) t += partial[(size_t)r * S + s];
        if (row < L.n) y[row] = __float2half_rn(t);
    }
}

size_t smem_bytes(const Layout2& L, int rows_cap, int warps, int depth, int ru, int speculate) {
    return smem_layout2(L.k, L.slices, rows_cap, warps, depth, ru, speculate).total;
}

template <int D, int RU>
ptqtp_status launch_d(const Layout2& L, const void* packed, const uint16_t* x, uint16_t* y, int grid, int warps,
                      int rows_cap, size_t smem, int speculate, int gated, cudaStream_t st) {
    auto kern = gemv2_kernel<D, RU>;
    const ptqtp_status cs = configure_once<gemv2_kernel<D, RU>>();
    if (cs != PTQTP_OK) return cs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_enabled() && !consume_pack(st) ? 1 : 0;   // plain right after a pack on this stream
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, L, static_cast<const unsigned char*>(packed),
                                       reinterpret_cast<const __half*>(x), reinterpret_cast<__half*>(y), rows_cap,
                                       L.nrp / grid, L.nrp % grid, speculate, gated);
    if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

}  // namespace

// Address of the status word on the current device, for the other kernels that report through it.
ptqtp_status gemv_status_word(int** out) {
    static thread_local int* cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PTQTP_ERR_CUDA;
    if (!cache[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_gemv2_status);
        if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
        cache[dev] = static_cast<int*>(p);
    }
    *out = cache[dev];
    return PTQTP_OK;
}

ptqtp_status copy_gemv2_status(int32_t* status_host, cudaStream_t st) {
    cudaError_t e = cudaMemcpyFromSymbolAsync(status_host, g_gemv2_status, sizeof(int), 0, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

// gated: y[i] = silu(row 2i) * row 2i+1 instead of the rows themselves (N even).
// warps: per CTA, 0 = the default below, -1 = as many as fit (for a call that is known to run alone).
// ctas_per_sm: CTAs of this launch per SM (0 = one).  units: slice units per bulk copy (1, 2 or 4; 0 = 2).
// The defaults keep a CTA small (4 to 8 warps, two ring slots of two units per warp) so that the CTAs of several
// consecutive launches are resident on an SM at once: under programmatic dependent launch with speculative
// execution the head of one launch (fetching x) and the tail of another (verifying x, reducing) then overlap the
// streaming of a third.  Measured on the LLaMA-3-8B shapes, 4 warps beat 8 and 16.
ptqtp_status launch_gemv2(const Layout2& L, const void* packed, const uint16_t* x, uint16_t* y, int warps,
                          int ctas_per_sm, int depth, int units, cudaStream_t st, bool gated) {
    const int S = L.slices;
    const int speculate = speculation_enabled() ? 1 : 0;
    if (ctas_per_sm < 0 || ctas_per_sm > 4) return PTQTP_ERR_CONFIG;
    if (warps < -1 || warps > kMaxWarps2) return PTQTP_ERR_CONFIG;
    if (units != 0 && units != 1 && units != 2 && units != 4) return PTQTP_ERR_CONFIG;
    const int per_sm = ctas_per_sm ? ctas_per_sm : 1;
    const int max_warps = kMaxWarps2 / per_sm;
    const size_t budget = (size_t)(228 / per_sm - 1) * 1024;          // 228 KB per SM, 1 KB of it reserved per CTA
    const int grid = min(per_sm * sm_count(), L.nrp);
    if (warps == 0 && !overlap_enabled()) warps = -1;   // plain launches never share an SM
    if (warps == -1) {
        // the caller knows that the call runs alone (copies on both sides of it): one CTA takes the whole SM
        warps = S >= max_warps ? max_warps : S * (max_warps / S);
    } else if (warps == 0) {
        // a multiple of the slice count (every slice lane gets as many warps): at least 4, at least 8 when a CTA
        // streams many units, and all 16 when that is what it takes to give every slice a warp
        const long units_per_cta = (long)((L.nrp + grid - 1) / grid) * S;
        const int target = units_per_cta >= 160 ? 8 : 4;  // (a long launch with 4 warps holds up the short ones behind it)
        warps = S >= max_warps ? max_warps : S * ((target + S - 1) / S);
        if (warps > max_warps) warps = S * (max_warps / S);
    }
    if (warps < 1 || warps > max_warps) return PTQTP_ERR_CONFIG;
    const int rows_cap = 2 * ((L.nrp + grid - 1) / grid);
    if (depth == 0) depth = 2;
    int spec = speculate;
    if (units == 0) {
        // two units per copy; for long K one, and then without the second copy of x that speculative execution keeps
        // (two only while three such CTAs still fit on an SM: sharing the SM with the neighbouring launches is
        // worth more than cheaper copies)
        units = smem_bytes(L, rows_cap, warps, depth, 2, spec) <= min(budget, (size_t)75 * 1024) ? 2 : 1;
        if (smem_bytes(L, rows_cap, warps, depth, units, spec) > budget) spec = 0;
    }
    const size_t smem = smem_bytes(L, rows_cap, warps, depth, units, spec);
    if (smem > budget) return depth > 2 || warps > 1 || units > 1 || ctas_per_sm == 2 ? PTQTP_ERR_CONFIG : PTQTP_ERR_SHAPE;
#define PTQTP_LAUNCH_D(DD)                                                                                            \
    case DD:                                                                                                          \
        return units == 1 ? launch_d<DD, 1>(L, packed, x, y, grid, warps, rows_cap, smem, spec, gated ? 1 : 0, st)                   \
             : units == 2 ? launch_d<DD, 2>(L, packed, x, y, grid, warps, rows_cap, smem, spec, gated ? 1 : 0, st)                   \
                          : launch_d<DD, 4>(L, packed, x, y, grid, warps, rows_cap, smem, spec, gated ? 1 : 0, st);
    switch (depth) {
        PTQTP_LAUNCH_D(2)
        PTQTP_LAUNCH_D(3)
        PTQTP_LAUNCH_D(4)
        PTQTP_LAUNCH_D(6)
        PTQTP_LAUNCH_D(8)
    }
#undef PTQTP_LAUNCH_D
    return PTQTP_ERR_CONFIG;
}

}  // namespace ptqtp
