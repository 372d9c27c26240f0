// Dual-trit-plane layer for 2 to 4 activation rows on packed format 3 (the batch-1 layout):
//     Y[m] = alpha1 (.) (T1 X[m]) + alpha2 (.) (T2 X[m]),   m < M, 2 <= M <= 4.
//
// Same tiles, same three-masks-per-code-word decode and the same exact int32 arithmetic as the batch-1 kernel
// (gemv4.cu); what changes is the meaning of the 8 MMA columns.  A k-step's 32 k-slots are 8 columns of each of the
// tile's four scale groups, so an MMA whose B fragment held x in all of them would add up four groups that have
// different scales.  The batch-1 kernel uses the columns for the four groups.  Here the columns are
//   MB = 2:  (group pair member, batch row, high | low byte): per k-step and code-row chain one MMA for groups 0, 1
//            (B non-zero in k-slots 0..15 only) and one for groups 2, 3 (k-slots 16..31 only);
//   MB = 4:  (batch row, high | low byte): one MMA per group, B non-zero only in that group's eight k-slots.
// The tensor pipe does 2 or 4 times the work of batch 1 for 2 or 4 rows (64 or 128 MMAs per tile: 128 or 256
// SM-cycles against 187 cycles of HBM time per tile), the masks, shared-memory loads and the stream of tiles are
// those of one row.  A lane ends a tile with the complete sums of (row pair g, batch row, one or all groups); the
// scale epilogue is per lane and fp32 as in the batch-1 kernel.
//
// Everything else -- x by one bulk copy requested before the tiles, conversion per warp and superblock, the ring of
// bulk copies with bounded waits, programmatic dependent launch with speculative execution -- is as in gemv4.cu.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kMaxWarps5 = 16;
constexpr int kMaxThreads5 = kMaxWarps5 * 32;
constexpr int kSpinAfterFailure5 = 1 << 8;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
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
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Shared memory: X as read (fp16, MB rows of K), one staging area per warp (per batch row the superblock in
// B-fragment order, 1024 bytes, and its four group records), the per-superblock partial sums [MB][rows_cap][S], the
// output rows [MB][rows_cap] (fp16), the mbarriers (one per ring slot, then one for X), then the ring.
constexpr int kStageRow5 = 1024 + 32;
struct Smem5 {
    size_t stage_off, partial_off, yout_off, bar_off, ring_off, total;
};
__host__ __device__ inline Smem5 smem_layout5(int k, int mb, int sbs, int rows_cap, int warps, int depth) {
    Smem5 m;
    m.stage_off = (size_t)mb * 2 * k;
    m.partial_off = m.stage_off + (size_t)warps * mb * kStageRow5;
    m.yout_off = m.partial_off + (size_t)mb * rows_cap * sbs * 4;
    m.bar_off = (m.yout_off + (size_t)mb * rows_cap * 2 + 7) / 8 * 8;
    m.ring_off = (m.bar_off + (size_t)(warps * depth + 1) * 8 + 127) / 128 * 128;
    m.total = m.ring_off + (size_t)warps * depth * kTile3;
    return m;
}

// Convert the 512 activations of a superblock to block fixed point, 16 columns per lane (two uint4 of fp16:
// columns 16 lane .. 16 lane + 15 of the superblock; zeros past K), into the warp's staging area.  Eight adjacent
// lanes share a 128-column group.
__device__ __noinline__ void convert5_x16(uint4 ra, uint4 rb, int lane, unsigned char* stage) {
    const uint32_t rw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
    // group maximum of |x| on the fp16 bit patterns (ordered like the values once the sign is cleared)
    uint32_t m2 = 0u;
#pragma unroll
    for (int e = 0; e < 8; ++e) m2 = __vmaxu2(m2, rw[e] & 0x7fff7fffu);
    uint32_t mxb = max(m2 & 0xffffu, m2 >> 16);
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) mxb = max(mxb, __shfl_xor_sync(0xffffffffu, mxb, o));
    // exponent of the maximum, in [-24, 15] for finite inputs; subnormal fp16 are integers times 2^-24
    int s = 0;
    if (mxb != 0u) {
        const int ef = (int)(mxb >> 10);
        const int ex = ef ? ef - 15 : (31 - __clz((int)mxb)) - 24;
        s = 13 - ex;                                   // group maximum in [2^13, 2^14): high byte within [-64, 64]
    }
    const float scale = __uint_as_float((uint32_t)(127 + s) << 23);
    // x * 2^s is exact and below 2^14 in magnitude; adding 1.5 * 2^23 rounds it to the nearest integer (ties to
    // even) and leaves that integer X, as a 16-bit two's complement number, in the low 16 bits of the float.
    // X = 256 hi + lo with both bytes signed: lo is byte 0 of X, hi is byte 1 of X + 128.
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
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) isum += __shfl_xor_sync(0xffffffffu, isum, o);
    uint32_t hw[4], lw[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        const uint32_t h0 = B[4 * w] + 0x80u, h1 = B[4 * w + 1] + 0x80u, h2 = B[4 * w + 2] + 0x80u, h3 = B[4 * w + 3] + 0x80u;
        lw[w] = __byte_perm(__byte_perm(B[4 * w], B[4 * w + 1], 0x0040), __byte_perm(B[4 * w + 2], B[4 * w + 3], 0x0040), 0x5410);
        hw[w] = __byte_perm(__byte_perm(h0, h1, 0x0051), __byte_perm(h2, h3, 0x0051), 0x5410);
    }
    // the lane's 16 columns are k-steps i0 (even) and i0 + 1 of group j, both halves: words (i0, i0 + 1) of a slot
    // are adjacent, so each (byte, half) pair of words goes out as one 8-byte store
    const int j = lane >> 3, i0 = (lane & 7) << 1;
    unsigned char* base = stage + (i0 >> 2) * 256 + j * 64 + (i0 & 3) * 4;
    *reinterpret_cast<uint2*>(base) = make_uint2(hw[0], hw[2]);            // high byte, columns 0-3 of each k-step
    *reinterpret_cast<uint2*>(base + 16) = make_uint2(hw[1], hw[3]);       // high byte, columns 4-7
    *reinterpret_cast<uint2*>(base + 32) = make_uint2(lw[0], lw[2]);       // low byte, columns 0-3
    *reinterpret_cast<uint2*>(base + 48) = make_uint2(lw[1], lw[3]);       // low byte, columns 4-7
    if ((lane & 7) == 0) reinterpret_cast<int2*>(stage + 1024)[j] = make_int2((int)((uint32_t)(127 - s) << 23), isum);
}

template <int D, int MB>
__global__ void __launch_bounds__(kMaxThreads5, 1)
gemv5_kernel(Layout3 L, const unsigned char* __restrict__ packed, const __half* __restrict__ X, __half* __restrict__ Y,
             int m, int rows_cap, int rb_base, int rb_rem, int speculate, int overlap, int spin_limit,
             int* __restrict__ status_word) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int S = L.sbs;
    const int warps = blockDim.x >> 5;
    const Smem5 sm = smem_layout5(L.k, MB, S, rows_cap, warps, D);
    uint4* raw = reinterpret_cast<uint4*>(smem);                             // X as read: [MB][K] fp16
    float* partial = reinterpret_cast<float*>(smem + sm.partial_off);       // [MB][rows_cap][S]
    __half* yout = reinterpret_cast<__half*>(smem + sm.yout_off);            // [MB][rows_cap]
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    unsigned char* stage = smem + sm.stage_off + (size_t)warp * MB * kStageRow5;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bar_off) + warp * D;
    uint64_t* xbar = reinterpret_cast<uint64_t*>(smem + sm.bar_off) + warps * D;
    unsigned char* ring = smem + sm.ring_off + (size_t)warp * D * kTile3;

    // Let the next kernel on the stream start while this one runs.
    asm volatile("griddepcontrol.launch_dependents;");

    // this CTA's row blocks (balanced partition from the host) and this warp's share of their tiles
    const int rb0 = (int)blockIdx.x * rb_base + min((int)blockIdx.x, rb_rem);
    const int n_cta = rb_base + ((int)blockIdx.x < rb_rem ? 1 : 0);
    const int Wc = min(S, warps);                       // superblock lanes among the warps
    const int mw = warps / Wc;                          // warps sharing a superblock lane
    const int sl_lane = warp % Wc, wi = warp / Wc;
    const bool idle = wi >= mw;
    const int n_sl = idle ? 0 : (S - sl_lane + Wc - 1) / Wc;
    const int rbw = rb0 + (idle ? 0 : wi * (n_cta / mw) + min(wi, n_cta % mw));
    const int n_rb = idle ? 0 : n_cta / mw + (wi < n_cta % mw ? 1 : 0);
    const unsigned char* codes = packed + L.codes_off;
    const int row_chunks = L.k >> 3;                    // 16-byte chunks per row of X
    const int nchunks = m * row_chunks, cthreads = blockDim.x;
    const uint32_t xbytes = (uint32_t)m * (uint32_t)L.k * 2u;

    if (lane == 0) {
#pragma unroll
        for (int d = 0; d < D; ++d) mbar_init(bars + d, 1);
        if (warp == 0) mbar_init(xbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // batch rows that do not exist (m < MB) read as zeros
    for (int c = nchunks + (int)threadIdx.x; c < MB * row_chunks; c += cthreads) raw[c] = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();

    // producer (lane 0): superblock pass pt, tiles left in it, source of the next copy, ring slot
    const uint32_t bars_a = smem_u32(bars), ring_a = smem_u32(ring), xbar_a = smem_u32(xbar);
    int pt = 0, pleft = 0, pslot = 0;
    const unsigned char* psrc = codes;
    auto issue = [&]() {
        if (pt < n_sl) {
            if (lane == 0) {
                mbar_expect_tx(bars_a + 8 * pslot, kTile3);
                bulk_copy_g2s(ring_a + pslot * kTile3, psrc, kTile3, bars_a + 8 * pslot);
            }
            psrc += kTile3;
            if (--pleft == 0) {
                ++pt;
                pleft = n_rb;
                psrc = codes + tile_offset3(L, rbw, min(sl_lane + pt * Wc, S - 1));
            }
        }
        pslot = pslot + 1 == D ? 0 : pslot + 1;
    };

    // lane constants.  MB = 2: MMA column g = (group pair member g/4, batch row (g/2)%2, byte g%2); the lane holds x
    // where its k-slots' group is that member: t/2 == g/4.  MB = 4: column g = (batch row g/2, byte g%2); the lane's
    // k-slots belong to groups t/2 (slots 0..15) and 2 + t/2 (slots 16..31).
    const int xrow = MB == 2 ? (g >> 1) & 1 : g >> 1;                   // batch row of this lane's MMA column
    const int xgrp = MB == 2 ? g >> 2 : t >> 1;                         // group (0 | 1) of its low k-slots; high: 2 + xgrp
    const bool x_active = MB == 4 || (t >> 1) == (g >> 2);
    const unsigned char* xs_lo = stage + xrow * kStageRow5 + ((xgrp * 4 + (g & 1) * 2 + (t & 1)) * 16);
    const unsigned char* xs_hi = xs_lo + 2 * 64;                        // group 2 + xgrp
    const bool u0 = (t >> 1) == 0;
    constexpr uint32_t kM0 = 0x03030303u, kM1 = 0x0c0c0c0cu, kM2 = 0x30303030u;

    int cslot = 0;
    uint32_t phase = 0;                                 // parity of the ring pass being consumed
    bool failed = false, waited = false;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // Pass 0 is speculative when allowed: X is read before earlier work of the stream is known to be complete.
        const bool spec = speculate && attempt == 0;
        pt = n_rb > 0 ? 0 : n_sl;
        pleft = n_rb;
        psrc = codes + tile_offset3(L, rbw, min(sl_lane, S - 1));
        const bool fill_first = !spec && !waited && overlap;
        if (fill_first) {
#pragma unroll
            for (int d = 0; d < D; ++d) issue();
        }
        if (!spec && !waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = true;
        }
        if (threadIdx.x == 0) {                         // X by one bulk copy, requested before any tile
            mbar_expect_tx(xbar_a, xbytes);
            bulk_copy_g2s(smem_u32(raw), X, xbytes, xbar_a);
        }
        __syncthreads();
        if (!fill_first) {
#pragma unroll
            for (int d = 0; d < D; ++d) issue();
        }
        if (!mbar_try_wait(xbar_a, (uint32_t)attempt)) {
            const int limit = failed ? kSpinAfterFailure5 : spin_limit;
            int spins = 0;
            while (!mbar_try_wait(xbar_a, (uint32_t)attempt)) {
                if (++spins >= limit) { failed = true; break; }
            }
        }

        for (int ts = 0; ts < n_sl; ++ts) {
            const int sb = sl_lane + ts * Wc;
            // the superblock's activations of every batch row -> block fixed point in the warp's staging area, then
            // this lane's words: lowv feeds k-slots 0..15 (group xgrp), highv k-slots 16..31 (group 2 + xgrp)
            uint32_t lowv[16], highv[16];
            __syncwarp();                               // the previous superblock's staging area has been read by all lanes
#pragma unroll
            for (int b = 0; b < MB; ++b) {
                uint4 ra = make_uint4(0u, 0u, 0u, 0u), rb = ra;
                if (sb * kSuper3 + 16 * lane < L.k) {
                    ra = raw[b * row_chunks + sb * 64 + 2 * lane];
                    rb = raw[b * row_chunks + sb * 64 + 2 * lane + 1];
                }
                convert5_x16(ra, rb, lane, stage + b * kStageRow5);
            }
            __syncwarp();
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint4 lo4 = make_uint4(0u, 0u, 0u, 0u), hi4 = make_uint4(0u, 0u, 0u, 0u);
                if (x_active) {
                    lo4 = *reinterpret_cast<const uint4*>(xs_lo + q * 256);
                    hi4 = *reinterpret_cast<const uint4*>(xs_hi + q * 256);
                }
                lowv[4 * q] = lo4.x; lowv[4 * q + 1] = lo4.y; lowv[4 * q + 2] = lo4.z; lowv[4 * q + 3] = lo4.w;
                highv[4 * q] = hi4.x; highv[4 * q + 1] = hi4.y; highv[4 * q + 2] = hi4.z; highv[4 * q + 3] = hi4.w;
            }
            // The epilogue of lane (g, t).  MB = 2: batch row t % 2, groups t / 2 and 2 + t / 2.  MB = 4: batch row t,
            // all four groups.  Group records of that batch row: (2^-s as float bits, sum of the group's integers).
            const int erow = MB == 2 ? t & 1 : t;
            const int2* meta = reinterpret_cast<const int2*>(stage + erow * kStageRow5 + 1024);
            int2 mt[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) mt[j] = meta[j];
            float* ppart = partial + ((size_t)erow * rows_cap + 16 * (rbw - rb0) + 2 * g) * S + sb;
            for (int j0 = 0; j0 < n_rb; ++j0) {
                // wait (bounded) for the copy in slot cslot; it has normally arrived long ago
                if (!mbar_try_wait(bars_a + 8 * cslot, phase)) {
                    const int limit = failed ? kSpinAfterFailure5 : spin_limit;
                    int spins = 0;
                    while (!mbar_try_wait(bars_a + 8 * cslot, phase)) {
                        if (++spins >= limit) { failed = true; break; }
                    }
                }
                const unsigned char* tb = ring + cslot * kTile3 + lane * 16;
                const unsigned char* quads = tb + kTileCodes3 - lane * 16 + g * 32;      // the four scale quads of row pair g
                float y0 = 0.f, y1 = 0.f;
                // one group's sums -> fp32 with its scales: Q_f = 4^f sum_j t_j X_j (column 2t high, 2t + 1 low byte)
                auto finish = [&](const int (&ca)[4], const int (&cb)[4], int grp, const int2 rec) {
                    const uint2 sc = *reinterpret_cast<const uint2*>(quads + grp * 8);
                    const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&sc.x));
                    const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&sc.y));
                    const int Q0 = (ca[0] << 8) + ca[1], Q1 = (ca[2] << 8) + ca[3], Q2 = (cb[0] << 8) + cb[1];
                    const int Q3 = (cb[2] << 8) + cb[3] - Q0 - Q1 - Q2;
                    const float cx = __int_as_float(rec.x);
                    y0 = fmaf(cx, fmaf(0.25f, s0.y * (float)Q1, s0.x * (float)Q0), y0);
                    y1 = fmaf(0.0625f * cx, fmaf(0.25f, s1.y * (float)Q3, s1.x * (float)Q2), y1);
                };
                if constexpr (MB == 2) {
                    const int gl = t >> 1, gh = 2 + (t >> 1);
                    const int2 ml = gl ? mt[1] : mt[0], mh = gl ? mt[3] : mt[2];     // (selected, not indexed: registers)
                    int cal[4] = {0, -ml.y, 0, -(ml.y << 2)}, cbl[4] = {0, -(ml.y << 4), 0, -(ml.y * 85)};
                    int cah[4] = {0, -mh.y, 0, -(mh.y << 2)}, cbh[4] = {0, -(mh.y << 4), 0, -(mh.y * 85)};
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 w = *reinterpret_cast<const uint4*>(tb + c * 512);
                        const uint32_t wd[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                        for (int s = 0; s < 2; ++s) {
                            const uint32_t w1 = wd[2 * s], w2 = wd[2 * s + 1];
                            const int i = 2 * c + s;
                            mma_u8s8(cal, w1 & kM0, w1 & kM1, w2 & kM0, w2 & kM1, lowv[i], 0u);
                            mma_u8s8(cah, w1 & kM0, w1 & kM1, w2 & kM0, w2 & kM1, 0u, highv[i]);
                            mma_u8s8(cbl, w1 & kM2, w1, w2 & kM2, w2, lowv[i], 0u);
                            mma_u8s8(cbh, w1 & kM2, w1, w2 & kM2, w2, 0u, highv[i]);
                        }
                    }
                    finish(cal, cbl, gl, ml);
                    finish(cah, cbh, gh, mh);
                    // lanes t and t ^ 2 hold the other groups of the same batch row
                    y0 += __shfl_xor_sync(0xffffffffu, y0, 2);
                    y1 += __shfl_xor_sync(0xffffffffu, y1, 2);
                    if (t < 2) {
                        ppart[0] = failed ? __int_as_float(0x7fc00000) : y0;
                        ppart[S] = failed ? __int_as_float(0x7fc00000) : y1;
                    }
                } else {
                    int ca[4][4], cb[4][4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        ca[j][0] = 0; ca[j][1] = -mt[j].y; ca[j][2] = 0; ca[j][3] = -(mt[j].y << 2);
                        cb[j][0] = 0; cb[j][1] = -(mt[j].y << 4); cb[j][2] = 0; cb[j][3] = -(mt[j].y * 85);
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 w = *reinterpret_cast<const uint4*>(tb + c * 512);
                        const uint32_t wd[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                        for (int s = 0; s < 2; ++s) {
                            const uint32_t w1 = wd[2 * s], w2 = wd[2 * s + 1];
                            const int i = 2 * c + s;
                            // the lane's words count only in the MMA of their own group
                            const uint32_t l0 = u0 ? lowv[i] : 0u, l1 = u0 ? 0u : lowv[i];
                            const uint32_t h0 = u0 ? highv[i] : 0u, h1 = u0 ? 0u : highv[i];
                            const uint32_t a0 = w1 & kM0, a1 = w1 & kM1, a2 = w2 & kM0, a3 = w2 & kM1;
                            const uint32_t e0 = w1 & kM2, e2 = w2 & kM2;
                            mma_u8s8(ca[0], a0, a1, a2, a3, l0, 0u);
                            mma_u8s8(ca[1], a0, a1, a2, a3, l1, 0u);
                            mma_u8s8(ca[2], a0, a1, a2, a3, 0u, h0);
                            mma_u8s8(ca[3], a0, a1, a2, a3, 0u, h1);
                            mma_u8s8(cb[0], e0, w1, e2, w2, l0, 0u);
                            mma_u8s8(cb[1], e0, w1, e2, w2, l1, 0u);
                            mma_u8s8(cb[2], e0, w1, e2, w2, 0u, h0);
                            mma_u8s8(cb[3], e0, w1, e2, w2, 0u, h1);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) finish(ca[j], cb[j], j, mt[j]);
                    ppart[0] = failed ? __int_as_float(0x7fc00000) : y0;
                    ppart[S] = failed ? __int_as_float(0x7fc00000) : y1;
                }
                ppart += 16 * S;
                // every lane has consumed the slot: lane 0 may refill it
                __syncwarp();
                issue();
                if (++cslot == D) { cslot = 0; phase ^= 1u; }
            }
        }
        // all partial sums are in shared memory: final sums in a fixed order, one rounding to fp16, before the wait
        __syncthreads();
        for (int idx = threadIdx.x; idx < m * 16 * n_cta; idx += cthreads) {
            const int b = idx / (16 * n_cta), r = idx - b * 16 * n_cta;
            const float* pp = partial + ((size_t)b * rows_cap + r) * S;
            float acc = 0.f;
            for (int s = 0; s < S; ++s) acc += pp[s];
            yout[b * rows_cap + r] = __float2half_rn(acc);
        }
        if (!spec) break;
        // Earlier work of the stream is complete after this wait: if X still reads as it did, the pass stands.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
        int stale = 0;
        constexpr int kVB = 8;
        for (int c0 = (int)threadIdx.x; c0 < nchunks; c0 += kVB * cthreads) {
            uint4 now[kVB];
#pragma unroll
            for (int p = 0; p < kVB; ++p) {
                const int c = c0 + p * cthreads;
                now[p] = make_uint4(0u, 0u, 0u, 0u);
                if (c < nchunks) now[p] = __ldcg(reinterpret_cast<const uint4*>(X) + c);
            }
#pragma unroll
            for (int p = 0; p < kVB; ++p) {
                const int c = c0 + p * cthreads;
                if (c < nchunks) {
                    const uint4 was = raw[c];
                    stale |= (now[p].x != was.x) | (now[p].y != was.y) | (now[p].z != was.z) | (now[p].w != was.w);
                }
            }
        }
        if (!__syncthreads_or(stale)) break;
    }
    if (failed) {
        if (lane == 0) atomicExch(status_word, (int)PTQTP_ERR_CUDA);
        // a copy whose wait gave up may still be in flight: give it time to land before the CTA's memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    __syncthreads();
    const int rows = min(16 * n_cta, L.n - 16 * rb0);
    for (int idx = threadIdx.x; idx < m * rows; idx += cthreads) {
        const int b = idx / rows, r = idx - b * rows;
        Y[(size_t)b * L.n + 16 * rb0 + r] = yout[b * rows_cap + r];
    }
}

template <int D, int MB>
ptqtp_status launch_d5(const Layout3& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int grid, int warps,
                       int rows_cap, size_t smem, cudaStream_t st) {
    ptqtp_status s = configure_once<gemv5_kernel<D, MB>>();
    if (s != PTQTP_OK) return s;
    int* status_word = nullptr;                           // shared with the other GEMV kernels (ptqtp_kernel_status)
    if (gemv_status_word(&status_word) != PTQTP_OK) return PTQTP_ERR_CUDA;
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv5_kernel<D, MB>, L, static_cast<const unsigned char*>(packed),
                                       reinterpret_cast<const __half*>(X), reinterpret_cast<__half*>(Y), m, rows_cap,
                                       L.nrb / grid, L.nrb % grid, speculation_enabled() ? 1 : 0, overlap_enabled() ? 1 : 0,
                                       wait_poll_limit(), status_word);
    if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

}  // namespace

// 2 <= m <= 4.  PTQTP_ERR_SHAPE when m rows of x leave no room in shared memory for a two-slot ring with one warp.
// warps: per CTA (0 = library choice); depth: copies in flight per warp (2 or 3; 0 = 2).
ptqtp_status launch_gemv5(const Layout3& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int warps, int depth,
                          cudaStream_t st) {
    if (m < 2 || m > 4) return PTQTP_ERR_SHAPE;
    if (warps < 0 || warps > kMaxWarps5 || (depth != 0 && depth != 2 && depth != 3)) return PTQTP_ERR_CONFIG;
    const int S = L.sbs, mb = m <= 2 ? 2 : 4;
    const size_t budget = (size_t)227 * 1024;
    const int grid = min(sm_count(), L.nrb);
    const int rb_cap = (L.nrb + grid - 1) / grid;
    const int rows_cap = 16 * rb_cap;
    if (depth == 0) depth = 2;
    const bool auto_warps = warps == 0;
    if (auto_warps) {
        const int target = !overlap_enabled() ? 16 : (long)rb_cap * S >= 40 ? 8 : 4;
        warps = min(kMaxWarps5, S >= target ? target : S * (target / S));
        while (warps > 1 && smem_layout5(L.k, mb, S, rows_cap, warps, depth).total > budget) warps = warps > 4 ? warps - 4 : warps - 1;
    }
    const size_t smem = smem_layout5(L.k, mb, S, rows_cap, warps, depth).total;
    if (smem > budget) return auto_warps ? PTQTP_ERR_SHAPE : PTQTP_ERR_CONFIG;
    if (mb == 2) return depth == 2 ? launch_d5<2, 2>(L, packed, m, X, Y, grid, warps, rows_cap, smem, st)
                                   : launch_d5<3, 2>(L, packed, m, X, Y, grid, warps, rows_cap, smem, st);
    return depth == 2 ? launch_d5<2, 4>(L, packed, m, X, Y, grid, warps, rows_cap, smem, st)
                      : launch_d5<3, 4>(L, packed, m, X, Y, grid, warps, rows_cap, smem, st);
}

}  // namespace ptqtp
