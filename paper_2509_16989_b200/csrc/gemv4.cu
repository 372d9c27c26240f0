// Batch-1 dual-trit-plane GEMV for sm_100a on packed format 3:  y = alpha1 (.) (T1 x) + alpha2 (.) (T2 x).
//
// Why this shape.  The CUDA-core kernel (gemv2.cu: one mask + two integer dot products per four trits) needs
// 287 warp instructions per 2176 packed bytes and is bound by instruction issue and the dp4a pipe at about 85 %
// of the HBM rate.  Here the packed bytes are laid out at pack time in the operand order of the int8 warp MMA
// (mma.sync.m16n8k32, u8 x s8 -> s32), so that decoding is three masks per code word and nothing else:
//
//   * A tile is 8 row pairs x 512 columns (four 128-column scale groups), 4096 code bytes + 32 scale quads.  A
//     code byte holds the four codes of one column of a row pair (row 0 plane 1, row 0 plane 2, row 1 plane 1,
//     row 1 plane 2 at bits 0-1, 2-3, 4-5, 6-7; code = trit + 1).  Lane (g, t) owns row pair g: one 128-bit
//     shared-memory load gives it the two code words of two k-steps; word & (0x03030303 << 2f) is the u8
//     operand q * 4^f of field f for four columns, and the unmasked word is the operand of "all four fields at
//     once" (q0 + 4 q1 + 16 q2 + 64 q3 <= 170), from which field 3 follows by subtraction.  Per k-step two MMAs:
//     rows (field 0 | field 1) and (field 2 | all) of the eight row pairs.
//   * The 32 k-slots of a k-step are 8 columns of each of the tile's four scale groups, and the 8 MMA columns
//     are (group, high byte | low byte of x): the B fragment holds x only where the k-slot's group equals the
//     column's group and zero elsewhere.  After the 16 k-steps of a tile lane (g, t) therefore holds the
//     complete integer sums of row pair g over group t for all four fields: every lane has epilogue work
//     (32 of 32 lanes, against 8 of 32 when the MMA columns are batch rows), and no sum crosses lanes before
//     the group scales have been applied.
//   * Activations are 15-bit block fixed point per 128-column group, X = 256 hi + lo with both bytes signed;
//     sum_j t_j X_j = sum_j q_j X_j - sum_j X_j (q = t + 1): the low accumulators start at -4^f sum_j X_j.  All
//     sums are exact int32; the group scales (the method's only multiplies) are applied in fp32.
//   * x reaches the CTA as it is (fp16) by one bulk copy, i.e. one round trip to L2 whatever K is.  A warp
//     converts the 512 columns of a superblock when it turns to that superblock (16 columns per lane, through a
//     1 KB staging area of its own), so there is no CTA-wide conversion phase, no barrier before the first MMA,
//     and shared memory holds x once (2 K bytes) however long x is.
//   * A warp is bound to a superblock (512 columns), keeps its B fragments in 32 registers and walks down the
//     CTA's row blocks; the tiles of one superblock for consecutive row blocks are contiguous in HBM and stream
//     through a private shared-memory ring by bulk copies (cp.async.bulk, no multicast) completed on mbarriers.
//     Every wait is bounded: if one gives up the warp writes NaN rows, records an error in the device status
//     word (ptqtp_kernel_status) and still runs to the end.
//   * Rows are reduced over the four lanes of a row pair by shuffles, over the superblocks through shared
//     memory in a fixed order (deterministic), rounded once to fp16.
//   * Programmatic dependent launch and speculative execution as in gemv2.cu: x is read at once, everything is
//     computed into shared memory, then the kernel waits for earlier work of the stream, reads x again and
//     compares bit by bit; y is written only then, and the pass is repeated if x had changed.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kMaxWarps4 = 16;
constexpr int kMaxThreads4 = kMaxWarps4 * 32;
// launch bound that sets the register budget (65536 / 576 -> 112 per thread): four 4-warp CTAs, or an 8-warp CTA and
// two 4-warp CTAs, of consecutive launches fit into an SM's register file
constexpr int kRegBound4 = 512;
constexpr int kSpinAfterFailure4 = 1 << 8;

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

// Shared memory: x as read (fp16, 2 K bytes), one staging area per warp (the superblock the warp is on, in
// B-fragment order, 1024 bytes, then its four group records: 2^-s as float bits, sum of the group's integers, then
// the warp's share of every job: first row block, row blocks, first row among the CTA's rows), the
// per-superblock partial sums, the output rows (fp16), the mbarriers (one per ring slot, then one for x), then
// the ring (RU tiles per slot, D slots per warp).
//
// Staging area: for q = 0..3, slot = 4 j + 2 hl + th (group j of the superblock, hl = 0 high | 1 low byte, th =
// which half of a k-step's 8 columns), 16 bytes at 256 q + 16 slot: the words of k-steps 4q .. 4q+3, word i
// holding the bytes of columns 128 j + 8 i + 4 th + 0..3.  The lane with g = 2 j + hl and t = 2 (j % 2) + th
// reads its 16 words with four 128-bit loads; the other lanes hold zeros.
constexpr int kStage4 = 1024 + 32 + 64;            // B-fragment words, four group records, the warp's job table
struct Smem4 {
    size_t stage_off, partial_off, yout_off, jobs_off, bar_off, ring_off, total;
};
__host__ __device__ inline Smem4 smem_layout4(int k, int sbs, int rows_cap, int warps, int depth, int ru) {
    Smem4 m;
    m.stage_off = (size_t)2 * k;
    m.partial_off = m.stage_off + (size_t)warps * kStage4;
    m.yout_off = m.partial_off + (size_t)rows_cap * sbs * 4;
    m.jobs_off = (m.yout_off + (size_t)rows_cap * 2 + 15) / 16 * 16;      // the CTA's share of every job
    m.bar_off = m.jobs_off + kMaxJobs4 * 16;
    m.ring_off = (m.bar_off + (size_t)(warps * depth + 1) * 8 + 127) / 128 * 128;
    m.total = m.ring_off + (size_t)warps * depth * ru * kTile3;
    return m;
}

// Convert the 512 activations of a superblock to block fixed point, 16 columns per lane (two uint4 of fp16:
// columns 16 lane .. 16 lane + 15 of the superblock; zeros past K), into the warp's staging area.  Eight adjacent
// lanes share a 128-column group.
__device__ __noinline__ void convert4_x16(uint4 ra, uint4 rb, int lane, unsigned char* stage) {
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

// This CTA's and this warp's share of job j: the CTA's row blocks [rb0, rb0 + n_cta) (balanced partition of the
// job over the grid, the CTAs that take one block more starting at CTA rb_off[j]), of which the warp streams
// [rbw, rbw + n_rb) (the m warps of a superblock lane split them into contiguous runs, balanced +-1).
struct Share4 {
    int rb0, n_cta, rbw, n_rb;
};
__device__ __forceinline__ Share4 share_of(const Jobs4& J, int j, int wi, int m, bool idle) {
    int idx = (int)blockIdx.x - J.rb_off[j];
    if (idx < 0) idx += (int)gridDim.x;
    Share4 s;
    s.rb0 = idx * J.rb_base[j] + min(idx, J.rb_rem[j]);
    s.n_cta = J.rb_base[j] + (idx < J.rb_rem[j] ? 1 : 0);
    s.rbw = s.rb0 + (idle ? 0 : wi * (s.n_cta / m) + min(wi, s.n_cta % m));
    s.n_rb = idle ? 0 : s.n_cta / m + (wi < s.n_cta % m ? 1 : 0);
    return s;
}

// One launch serves up to kMaxJobs4 matrices ("jobs") that share x: a warp, once on a superblock, streams its
// tiles of job 0, then of job 1, ...; x is fetched, converted and verified once for all of them.
// kMulti = false is the same kernel for a single matrix with the job loops folded away.
template <int D, int RU, bool kMulti>
__global__ void __launch_bounds__(kRegBound4, 1)
gemv4_kernel(const __grid_constant__ Jobs4 J, const __half* __restrict__ x, int rows_cap, int speculate, int overlap,
             int gated, int spin_limit, int inject, int* __restrict__ status_word) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int S = J.sbs;
    const int warps = blockDim.x >> 5;
    const Smem4 sm = smem_layout4(J.k, S, rows_cap, warps, D, RU);
    uint4* raw = reinterpret_cast<uint4*>(smem);                             // x as read (fp16)
    float* partial = reinterpret_cast<float*>(smem + sm.partial_off);       // [rows_cap][S]
    __half* yout = reinterpret_cast<__half*>(smem + sm.yout_off);            // [rows_cap]: the rows as they will be stored
    // (the shuffle tells the compiler that the warp index is the same in all lanes)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    unsigned char* stage = smem + sm.stage_off + (size_t)warp * kStage4;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bar_off) + warp * D;
    uint64_t* xbar = reinterpret_cast<uint64_t*>(smem + sm.bar_off) + warps * D;
    constexpr int kSlot = RU * kTile3;                 // a ring slot holds the RU tiles of one copy
    unsigned char* ring = smem + sm.ring_off + (size_t)warp * D * kSlot;

    // Let the next kernel on the stream start while this one runs.
    asm volatile("griddepcontrol.launch_dependents;");

    const int Wc = min(S, warps);                       // superblock lanes among the warps
    const int m = warps / Wc;                           // warps sharing a superblock lane
    const int sl_lane = warp % Wc, wi = warp / Wc;
    const bool idle = wi >= m;
    const int n_sl = idle ? 0 : (S - sl_lane + Wc - 1) / Wc;
    const int nchunks = J.k >> 3, cthreads = blockDim.x;
    const uint32_t xbytes = (uint32_t)J.k * 2u;
    const int njobs = kMulti ? J.count : 1;
    // The shares are worked out once, by lane j for job j: the warp's into its staging area (first row block, row
    // blocks, first row among the CTA's rows), the CTA's into a table of its own (first row block, row blocks,
    // first row); rows_total = rows of all jobs in this CTA (16 per row block).
    int4* wtab = reinterpret_cast<int4*>(stage + 1024 + 32);
    int4* ctab = reinterpret_cast<int4*>(smem + sm.jobs_off);
    int rows_total = 0;
    {
        const Share4 mine = share_of(J, min(lane, njobs - 1), wi, m, idle);
        int before = 0;
        for (int j = 0; j < njobs; ++j) {
            int idx = (int)blockIdx.x - J.rb_off[j];
            if (idx < 0) idx += (int)gridDim.x;
            const int rows = 16 * (J.rb_base[j] + (idx < J.rb_rem[j] ? 1 : 0));
            if (j < lane) before += rows;
            rows_total += rows;
        }
        if (lane < njobs) {
            wtab[lane] = make_int4(mine.rbw, mine.n_rb, before + 16 * (mine.rbw - mine.rb0), 0);
            if (warp == 0) ctab[lane] = make_int4(mine.rb0, mine.n_cta, before, 0);
        }
    }

    if (lane == 0) {
#pragma unroll
        for (int d = 0; d < D; ++d) mbar_init(bars + d, 1);
        if (warp == 0) mbar_init(xbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    // producer (lane 0): superblock pass pt and job pj of the segment being requested, tiles left in it, source of
    // the next copy, ring slot
    const uint32_t bars_a = smem_u32(bars), ring_a = smem_u32(ring), xbar_a = smem_u32(xbar);
    int pt = 0, pj = 0, pleft = 0, pslot = 0;
    // test hook: the first copy of warp 0 of CTA 0 announces more bytes than it brings, so its wait runs out
    uint32_t surplus = (inject && blockIdx.x == 0 && warp == 0) ? 16u : 0u;
    const unsigned char* psrc = nullptr;
    auto seek = [&]() {                                 // from (pt, pj) on, the next segment that has tiles
        while (pt < n_sl) {
            if (pj < njobs) {
                const int4 sh = wtab[pj];
                if (sh.y > 0) {
                    pleft = sh.y;
                    psrc = J.codes[pj] + ((size_t)(sl_lane + pt * Wc) * J.nrb[pj] + sh.x) * kTile3;
                    return;
                }
                ++pj;
            } else {
                pj = 0;
                ++pt;
            }
        }
        pleft = 0;
    };
    auto issue = [&]() {
        if (pt < n_sl) {
            const int nun = min(RU, pleft);
            const uint32_t bytes = (uint32_t)nun * kTile3;
            if (lane == 0) {
                mbar_expect_tx(bars_a + 8 * pslot, bytes + surplus);
                bulk_copy_g2s(ring_a + pslot * kSlot, psrc, bytes, bars_a + 8 * pslot);
            }
            surplus = 0u;
            psrc += bytes;
            pleft -= nun;
            if (pleft == 0) {
                ++pj;
                seek();
            }
        }
        pslot = pslot + 1 == D ? 0 : pslot + 1;
    };

    // lane constants: which words of x this lane holds (see the staging area), the code-field masks
    const int xj = g >> 1;                                               // group of this lane's MMA column
    const bool x_active = (t >> 1) == (xj & 1);
    const bool x_low = xj < 2;                                           // its k-slots are 0..15 (b0) or 16..31 (b1)
    const int x_slot = (xj * 4 + (g & 1) * 2 + (t & 1)) * 16;
    constexpr uint32_t kM0 = 0x03030303u, kM1 = 0x0c0c0c0cu, kM2 = 0x30303030u;

    int cslot = 0;
    uint32_t phase = 0;                                 // parity of the ring pass being consumed
    bool failed = false, waited = false;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // Pass 0 is speculative when allowed: x is read before earlier work of the stream is known to be complete.
        const bool spec = speculate && attempt == 0;
        // x as it is, by one bulk copy (through L2, the point of coherence): one round trip whatever K is.  It is
        // requested before the ring is filled (copies complete in the order they were requested: behind a full
        // ring x would arrive microseconds later), except under a dependent launch without speculative execution,
        // where the planes, which do not depend on earlier work of the stream, are requested before the wait.
        pt = 0;
        pj = 0;
        seek();
        const bool fill_first = !spec && !waited && overlap;
        if (fill_first) {
#pragma unroll
            for (int d = 0; d < D; ++d) issue();
        }
        if (!spec && !waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = true;
        }
        if (threadIdx.x == 0) {
            mbar_expect_tx(xbar_a, xbytes);
            bulk_copy_g2s(smem_u32(raw), x, xbytes, xbar_a);
        }
        __syncthreads();                                // the mbarrier of x is initialised and armed before anyone polls it
        if (!fill_first) {                              // (and x has been requested before any tile)
#pragma unroll
            for (int d = 0; d < D; ++d) issue();
        }
        if (!mbar_try_wait(xbar_a, (uint32_t)attempt)) {
            const int limit = failed ? kSpinAfterFailure4 : spin_limit;
            int spins = 0;
            while (!mbar_try_wait(xbar_a, (uint32_t)attempt)) {
                if (++spins >= limit) { failed = true; break; }
            }
        }

        for (int ts = 0; ts < n_sl; ++ts) {
            const int sb = sl_lane + ts * Wc;
            // the superblock's activations: fp16 -> block fixed point in the warp's staging area (zeros past K), then
            // this lane's part of the B fragments to registers: b0 feeds k-slots 0..15, b1 16..31
            uint32_t b0[16], b1[16];
            {
                uint4 ra = make_uint4(0u, 0u, 0u, 0u), rb = ra;
                if (sb * kSuper3 + 16 * lane < J.k) {
                    ra = raw[sb * 64 + 2 * lane];
                    rb = raw[sb * 64 + 2 * lane + 1];
                }
                __syncwarp();                           // the previous superblock's staging area has been read by all lanes
                convert4_x16(ra, rb, lane, stage);
                __syncwarp();
                const unsigned char* xs = stage + x_slot;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 lo4 = make_uint4(0u, 0u, 0u, 0u), hi4 = make_uint4(0u, 0u, 0u, 0u);
                    if (x_active && x_low) lo4 = *reinterpret_cast<const uint4*>(xs + q * 256);
                    if (x_active && !x_low) hi4 = *reinterpret_cast<const uint4*>(xs + q * 256);
                    b0[4 * q] = lo4.x; b0[4 * q + 1] = lo4.y; b0[4 * q + 2] = lo4.z; b0[4 * q + 3] = lo4.w;
                    b1[4 * q] = hi4.x; b1[4 * q + 1] = hi4.y; b1[4 * q + 2] = hi4.z; b1[4 * q + 3] = hi4.w;
                }
            }
            // the epilogue of lane (g, t) is for group t of the superblock
            const int2 mt = reinterpret_cast<const int2*>(stage + 1024)[t];
            const float cx0 = __int_as_float(mt.x), cx1 = 0.0625f * cx0;
            const int n0 = -mt.y, n1 = -(mt.y << 2), n2 = -(mt.y << 4), n3 = -(mt.y * 85);
            for (int jb = 0; jb < njobs; ++jb) {
            const int4 sh = wtab[jb];                   // (first row block, row blocks, first row among the CTA's rows)
            float* ppart = partial + (size_t)(sh.z + 2 * g + (t & 1)) * S + sb;
            for (int j0 = 0; j0 < sh.y; j0 += RU) {
                // wait (bounded) for the copy in slot cslot; it has normally arrived long ago
                if (!mbar_try_wait(bars_a + 8 * cslot, phase)) {
                    const int limit = failed ? kSpinAfterFailure4 : spin_limit;
                    int spins = 0;
                    while (!mbar_try_wait(bars_a + 8 * cslot, phase)) {
                        if (++spins >= limit) { failed = true; break; }
                    }
                }
                const int nun = min(RU, sh.y - j0);
                const unsigned char* buf = ring + cslot * kSlot + lane * 16;
                auto tile_body = [&](const unsigned char* tb, float* pp) {
                    // chains A: rows (field 0 | field 1), B: rows (field 2 | all fields); even and odd k-steps apart
                    int ca0[4] = {0, n0, 0, n1}, cb0[4] = {0, n2, 0, n3};
                    int ca1[4] = {0, 0, 0, 0}, cb1[4] = {0, 0, 0, 0};
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 w = *reinterpret_cast<const uint4*>(tb + c * 512);
                        mma_u8s8(ca0, w.x & kM0, w.x & kM1, w.y & kM0, w.y & kM1, b0[2 * c], b1[2 * c]);
                        mma_u8s8(cb0, w.x & kM2, w.x, w.y & kM2, w.y, b0[2 * c], b1[2 * c]);
                        mma_u8s8(ca1, w.z & kM0, w.z & kM1, w.w & kM0, w.w & kM1, b0[2 * c + 1], b1[2 * c + 1]);
                        mma_u8s8(cb1, w.z & kM2, w.z, w.w & kM2, w.w, b0[2 * c + 1], b1[2 * c + 1]);
                    }
                    const uint2 sc = *reinterpret_cast<const uint2*>(tb + kTileCodes3 - lane * 8);   // quad of (row pair g, group t)
                    const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&sc.x));   // alpha1, alpha2 of row 0
                    const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&sc.y));   // ... of row 1
                    // Q_f = 4^f * sum_j t_j X_j over the group (column 2t is the high, 2t + 1 the low byte of x)
                    const int Q0 = ((ca0[0] + ca1[0]) << 8) + ca0[1] + ca1[1];
                    const int Q1 = ((ca0[2] + ca1[2]) << 8) + ca0[3] + ca1[3];
                    const int Q2 = ((cb0[0] + cb1[0]) << 8) + cb0[1] + cb1[1];
                    const int Q3 = ((cb0[2] + cb1[2]) << 8) + cb0[3] + cb1[3] - Q0 - Q1 - Q2;
                    const float y0 = cx0 * fmaf(0.25f, s0.y * (float)Q1, s0.x * (float)Q0);
                    const float y1 = cx1 * fmaf(0.25f, s1.y * (float)Q3, s1.x * (float)Q2);
                    // the four lanes of a row pair: even t end up with row 0, odd t with row 1
                    const float send = (t & 1) ? y0 : y1;
                    float v = ((t & 1) ? y1 : y0) + __shfl_xor_sync(0xffffffffu, send, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    if (t < 2) *pp = failed ? __int_as_float(0x7fc00000) : v;
                };
#pragma unroll 1
                for (int u = 0; u < nun; ++u, buf += kTile3, ppart += 16 * S) tile_body(buf, ppart);
                // every lane has consumed the slot: lane 0 may refill it
                __syncwarp();
                issue();
                if (++cslot == D) { cslot = 0; phase ^= 1u; }
            }
            }
        }
        // All partial sums of this pass are in shared memory: sum them over the superblocks in a fixed order and
        // round once to fp16 now, so that after the dependency wait only the verification of x and the store remain.
        __syncthreads();
        if (gated == 1) {
            // gated pair epilogue: a row pair is (gate row, up row) and gives one output silu(gate) * up, computed
            // from the unrounded fp32 sums
            for (int r = threadIdx.x; r < rows_total / 2; r += cthreads) {
                float gt = 0.f, up = 0.f;
                for (int s = 0; s < S; ++s) {
                    gt += partial[(size_t)(2 * r) * S + s];
                    up += partial[(size_t)(2 * r + 1) * S + s];
                }
                yout[r] = __float2half_rn(gt / (1.f + expf(-gt)) * up);
            }
        } else if (gated == 2) {
            // the same with the gate rows in job 0 and the up rows in job 1 (equal shapes, equal partitions)
            const int half_rows = rows_total / 2;
            for (int r = threadIdx.x; r < half_rows; r += cthreads) {
                float gt = 0.f, up = 0.f;
                for (int s = 0; s < S; ++s) {
                    gt += partial[(size_t)r * S + s];
                    up += partial[(size_t)(half_rows + r) * S + s];
                }
                yout[r] = __float2half_rn(gt / (1.f + expf(-gt)) * up);
            }
        } else {
            for (int r = threadIdx.x; r < rows_total; r += cthreads) {
                float acc = 0.f;
                for (int s = 0; s < S; ++s) acc += partial[(size_t)r * S + s];
                yout[r] = __float2half_rn(acc);
            }
        }
        if (!spec) break;
        // Earlier work of the stream is complete after this wait: if x still reads as it did, the pass stands.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
        int stale = 0;
        constexpr int kVB = 8;                          // reads of x in flight per thread: one round trip to L2 for up to 64 K / threads columns
        for (int c0 = (int)threadIdx.x; c0 < nchunks; c0 += kVB * cthreads) {
            uint4 now[kVB];
#pragma unroll
            for (int p = 0; p < kVB; ++p) {
                const int c = c0 + p * cthreads;
                now[p] = make_uint4(0u, 0u, 0u, 0u);
                if (c < nchunks) now[p] = __ldcg(reinterpret_cast<const uint4*>(x) + c);
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
    if (gated == 2) {
        const int4 sh = ctab[0];                        // (first row block, row blocks, first row)
        const int rows = min(16 * sh.y, J.n[0] - 16 * sh.x);
        for (int r = threadIdx.x; r < rows; r += cthreads) J.y[0][16 * sh.x + r] = yout[r];
        return;
    }
    for (int j = 0; j < njobs; ++j) {
        const int4 sh = ctab[j];
        if (gated == 1) {
            const int npairs = min(8 * sh.y, J.nrp[j] - 8 * sh.x);
            for (int r = threadIdx.x; r < npairs; r += cthreads) J.y[j][8 * sh.x + r] = yout[sh.z / 2 + r];
        } else {
            const int rows = min(16 * sh.y, J.n[j] - 16 * sh.x);
            for (int r = threadIdx.x; r < rows; r += cthreads) J.y[j][16 * sh.x + r] = yout[sh.z + r];
        }
    }
}

template <int D, int RU, bool kMulti>
ptqtp_status launch_d4(const Jobs4& J, const uint16_t* x, int grid, int warps, int rows_cap, size_t smem, int speculate,
                       int gated, cudaStream_t st) {
    ptqtp_status s = configure_once<gemv4_kernel<D, RU, kMulti>>();
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv4_kernel<D, RU, kMulti>, J, reinterpret_cast<const __half*>(x), rows_cap, speculate,
                                       overlap_enabled() ? 1 : 0, gated, wait_poll_limit(),
                                       take_injected_wait_failure() ? 1 : 0, status_word);
    if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

}  // namespace

// jobs: the matrices of the launch (codes, y, n, nrp, nrb, count, k, sbs filled in by the caller; the partition
// fields are set here).  gated: 0 = the rows themselves; 1 = y[i] = silu(row 2i) * row 2i+1 within every job (N
// even); 2 = y0[i] = silu(row i of job 0) * row i of job 1 (two jobs of equal shape).
// warps: per CTA, 0 = the default below, -1 = as many as fit (for a call that is known to run alone).
// ctas_per_sm: CTAs of this launch per SM (0 = one).  units: tiles per bulk copy (1 or 2; 0 = library choice).
// depth: copies in flight per warp (2, 3, 4, 6; 0 = library choice).
ptqtp_status launch_gemv4_jobs(Jobs4& J, const uint16_t* x, int warps, int ctas_per_sm, int depth, int units,
                               cudaStream_t st, int gated) {
    const int S = J.sbs;
    if (ctas_per_sm < 0 || ctas_per_sm > 4) return PTQTP_ERR_CONFIG;
    if (warps < -1 || warps > kMaxWarps4) return PTQTP_ERR_CONFIG;
    if (units != 0 && units != 1 && units != 2) return PTQTP_ERR_CONFIG;
    if (depth != 0 && depth != 2 && depth != 3 && depth != 4 && depth != 6) return PTQTP_ERR_CONFIG;
    const int per_sm = ctas_per_sm ? ctas_per_sm : 1;
    const int max_warps = kMaxWarps4 / per_sm;
    const size_t budget = (size_t)(228 / per_sm - 1) * 1024;          // 228 KB per SM, 1 KB of it reserved per CTA
    int total_rb = 0;
    for (int j = 0; j < J.count; ++j) total_rb += J.nrb[j];
    const int grid = min(per_sm * sm_count(), total_rb);
    // every job is spread over the whole grid; the CTAs that take one row block more start, job after job, where
    // the previous job's stopped, so that the sums differ by one block at most (a gated pair of two jobs keeps
    // equal partitions: both rows of an output must be in the same CTA)
    int rb_cap = 0, off = 0;
    for (int j = 0; j < J.count; ++j) {
        J.rb_base[j] = J.nrb[j] / grid;
        J.rb_rem[j] = J.nrb[j] % grid;
        J.rb_off[j] = gated == 2 ? 0 : off;
        off = (off + J.rb_rem[j]) % grid;
        rb_cap += J.rb_base[j] + (J.rb_rem[j] ? 1 : 0);
    }
    const int rows_cap = 16 * rb_cap;
    const bool alone = warps == -1 || (warps == 0 && !overlap_enabled());   // plain launches never share an SM
    if (warps <= 0) {
        if (alone) {
            // one CTA has the SM to itself: as many warps as have tiles to stream
            warps = S >= max_warps ? max_warps : S * min(max_warps / S, max(1, rb_cap));
        } else {
            // small CTAs, so that the CTAs of consecutive launches are resident on an SM together
            const int target = (long)rb_cap * S >= 40 ? 8 : 4;   // (measured in the mixed sequence of a decoder layer, not in a chain of one shape)
            warps = min(max_warps, S >= target ? target : S * (target / S));
        }
    }
    if (warps < 1 || warps > max_warps) return PTQTP_ERR_CONFIG;
    const int spec = speculation_enabled() ? 1 : 0;
    const bool auto_units = units == 0, auto_depth = depth == 0;
    if (auto_depth) depth = alone ? 4 : 2;
    if (auto_units) units = 1;
    if (auto_depth)
        while (depth > 2 && smem_layout4(J.k, S, rows_cap, warps, depth, units).total > budget) --depth;
    if (depth == 5) depth = 4;
    const size_t smem = smem_layout4(J.k, S, rows_cap, warps, depth, units).total;
    if (smem > budget) return !auto_depth || !auto_units || ctas_per_sm > 1 || warps > 1 ? PTQTP_ERR_CONFIG : PTQTP_ERR_SHAPE;
#define PTQTP_LAUNCH_D4(DD)                                                                        \
    case DD:                                                                                       \
        if (J.count > 1)                                                                                  \
            return units == 1 ? launch_d4<DD, 1, true>(J, x, grid, warps, rows_cap, smem, spec, gated, st)   \
                              : launch_d4<DD, 2, true>(J, x, grid, warps, rows_cap, smem, spec, gated, st);  \
        return units == 1 ? launch_d4<DD, 1, false>(J, x, grid, warps, rows_cap, smem, spec, gated, st)      \
                          : launch_d4<DD, 2, false>(J, x, grid, warps, rows_cap, smem, spec, gated, st);
    switch (depth) {
        PTQTP_LAUNCH_D4(2)
        PTQTP_LAUNCH_D4(3)
        PTQTP_LAUNCH_D4(4)
        PTQTP_LAUNCH_D4(6)
    }
#undef PTQTP_LAUNCH_D4
    return PTQTP_ERR_CONFIG;
}

void add_job4(Jobs4& J, const Layout3& L, const void* packed, uint16_t* y) {
    const int j = J.count++;
    J.codes[j] = static_cast<const unsigned char*>(packed) + L.codes_off;
    J.y[j] = reinterpret_cast<__half*>(y);
    J.n[j] = L.n;
    J.nrp[j] = L.nrp;
    J.nrb[j] = L.nrb;
    J.k = L.k;
    J.sbs = L.sbs;
}

ptqtp_status launch_gemv4(const Layout3& L, const void* packed, const uint16_t* x, uint16_t* y, int warps,
                          int ctas_per_sm, int depth, int units, cudaStream_t st, bool gated) {
    Jobs4 J = {};
    add_job4(J, L, packed, y);
    return launch_gemv4_jobs(J, x, warps, ctas_per_sm, depth, units, st, gated ? 1 : 0);
}

}  // namespace ptqtp
