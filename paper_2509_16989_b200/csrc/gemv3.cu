// Dual-trit-plane layer for 1 to 4 activation rows on packed format 2, contraction on the int8 tensor-core path:
//     Y[m] = alpha1 (.) (T1 X[m]) + alpha2 (.) (T2 X[m]),   m < M <= 4.
//
// Why tensor cores for a matrix-vector product.  The CUDA-core kernel (gemv2.cu) spends 3 masks + 8 integer dot
// products per 16 trits and is bound by instruction issue and the dp4a pipe (64 lanes/clk/SM on sm_100), not by
// HBM.  One mma.sync.m16n8k32 (u8 x s8 -> s32) contracts 16 code rows with 32 columns for 8 activation columns
// in a single issue slot: with the 8 columns holding the (high byte, low byte) of up to four batch rows, a slice
// unit costs about 160 warp instructions instead of 300, and the stream of packed planes from HBM becomes the
// bound.  The arithmetic is the same exact integer arithmetic as in the CUDA-core kernel.
//
//   * MMA rows = 4 code fields x 4 consecutive row pairs (a "quad", 8 output rows).  A code byte holds the four
//     codes of one input column (row 0 plane 1, row 0 plane 2, row 1 plane 1, row 1 plane 2 at bits 0-1, 2-3, 4-5,
//     6-7); lane (g, t) masks field g/4 (MMA row g) and field 2 + g/4 (MMA row g + 8) out of the code word of row
//     pair g%4.  The masked bytes q * 4^f are the u8 operand as they stand; 4^-f goes into the scale epilogue.
//   * ldmatrix distributes the 16-byte atoms (16 columns of one row pair) of four row pairs over the lanes in
//     exactly the A-fragment order: one ldmatrix.x4 feeds two MMAs (64 columns of four row pairs).
//   * Activations are 15-bit block fixed point per 128-column scale group, X = 256 hi + lo with both bytes
//     signed; MMA column 2b is hi and 2b + 1 is lo of batch row b.  A warp is bound to one quarter (512 columns)
//     of a 2048-column slice and keeps that quarter's B fragments in 32 registers for as long as it stays there.
//   * sum_j t_j X_j = sum_j q_j X_j - sum_j X_j (q = t + 1): the low accumulator starts at -4^f sum_j X_j.
//   * Four MMAs finish a 128-column scale group; its int32 sums get the fp32 epilogue (group scales, 4^-f, block
//     scale of x): the method's only multiplies besides the integer products by 0, 1, 2.  Two scale groups are
//     contracted side by side so that every warp has two independent MMA chains in flight.
//   * Four warps (a team: the quarters of a slice) share a ring of stages; a stage holds the four slice units of
//     a quad, each brought by one bulk copy (cp.async.bulk, no multicast) that completes on the stage's "full"
//     mbarrier; every warp of the team arrives on its "empty" mbarrier when done.  Issuing a bulk copy holds
//     the issuing warp for a few hundred cycles, so the four copies of a stage are spread over the four warps
//     of the team (warp i brings the unit of row pair i), one stage behind the one being consumed.  A team works
//     through a contiguous range of the CTA's (slice, quad) list, so all teams carry the same load for any K.
//     Every mbarrier wait is bounded; if one gives up, the warp writes NaN, records an error in a device status
//     word (ptqtp_kernel_status) and still runs to the end.
//   * Two CTAs per SM (two teams each) whenever the activations leave room: the head and the tail of one CTA
//     (fetching x, the final reduction) overlap the streaming of the other, also across consecutive launches.
//   * Speculative execution under programmatic dependent launch.  x and y belong to the stream's order, the
//     packed planes do not.  Earlier work of the stream may still be running when this kernel starts; most
//     calls of a decoder read an x that was finished long before.  The kernel therefore reads x at once,
//     computes everything into shared memory, then waits for the earlier work, reads x again and compares it
//     bit by bit with its first read (kept in shared memory).  Only then y is written; if a single bit of x
//     differed, the whole computation is repeated from the second read.  Results never depend on the timing.
//   * Rows are reduced over the two plane lanes by one shuffle, over the slice quarters through shared memory in
//     a fixed order (deterministic), rounded once to fp16.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kNB = 8;                          // 64-column lane blocks per warp (a quarter slice)
constexpr int kTeamWarps = 32 / kNB;            // warps sharing a stage
constexpr int kMaxTeams = 4;                    // teams per CTA: 2 (two CTAs per SM) or 4 (one)
constexpr int kMaxThreads3 = kMaxTeams * kTeamWarps * 32;
constexpr int kUnitStride3 = kUnit2 + 16;       // units of a stage 16 bytes apart modulo 128: conflict-free ldmatrix
constexpr int kStage3 = 4 * kUnitStride3;
constexpr int kGroupCols = 128;
constexpr int kPlanePad = 64;                   // byte planes of x (K + 64) apart: conflict-free fragment loads
constexpr int kMaxBatch3 = 4;
constexpr int kSpin3 = 1 << 22;                 // polls of an mbarrier before a wait gives up
constexpr int kSpinAfterFailure3 = 1 << 8;

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(bar)) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(s32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// returns false when the wait gave up
__device__ __forceinline__ bool bar_wait_bounded(uint64_t* bar, uint32_t parity, bool already_failed) {
    if (bar_try_wait(bar, parity)) return true;         // what is waited for has normally happened long ago
    const int limit = already_failed ? kSpinAfterFailure3 : kSpin3;
    int spins = 0;
    while (!bar_try_wait(bar, parity)) {
        if (++spins >= limit) return false;
    }
    return true;
}
// Bulk copy global -> this CTA's shared memory, completion counted in bytes on an mbarrier (no multicast).
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(s32(dst_smem)), "l"(src), "r"(bytes), "r"(s32(bar)) : "memory");
}
__device__ __forceinline__ void ldmatrix4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Shared memory: the byte planes of x ([batch row][hi, lo][K + 64]), the group records ([batch row][K/128]:
// 2^-s as float bits, sum_j X_j), the first read of x (fp16 as read, only when executing speculatively), the
// partial sums ([batch row][rows_cap][slices * kTeamWarps]), the mbarriers (per team: depth "full", depth
// "empty"), the ring (per team: depth stages).
// Inside a byte plane the 64 bytes of a lane block are permuted, column 16 r + 4 t + e at 16 t + 4 r + e: the
// four words lane t feeds to the two MMAs of the block (k slots 4t.. and 16 + 4t.. of each) are contiguous.
struct Smem3 {
    size_t meta_off, raw_off, partial_off, bar_off, ring_off, total;
};
__host__ __device__ inline Smem3 smem_layout3(int k, int m, int slices, int rows_cap, int teams, int depth, int speculate) {
    Smem3 s;
    s.meta_off = (size_t)2 * m * (k + kPlanePad);
    s.raw_off = (s.meta_off + (size_t)m * (k / kGroupCols) * 8 + 15) / 16 * 16;
    s.partial_off = s.raw_off + (speculate ? (size_t)2 * m * k : 0);
    s.bar_off = (s.partial_off + (size_t)m * rows_cap * kTeamWarps * slices * 4 + 7) / 8 * 8;
    s.ring_off = (s.bar_off + (size_t)teams * depth * 16 + 15) / 16 * 16;
    s.total = s.ring_off + (size_t)teams * depth * kStage3;
    return s;
}

// Convert 16 activations (two uint4 of fp16, columns col..col+15 of batch row mi) to block fixed point and store
// them.  Eight adjacent threads share a 128-column group; the whole warp must call this.
__device__ __noinline__ void convert3_x16(uint4 ra, uint4 rb, int mi, int col, bool valid, int k, unsigned char* xs, int2* meta) {
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
    if (valid) {
        // columns col + 4 t .. col + 4 t + 3 are word r = (col % 64) / 16 of lane t of their 64-column block
        const int c0 = col & 63;
        unsigned char* hi = xs + (size_t)(2 * mi) * (k + kPlanePad) + (col - c0) + (c0 >> 4) * 4;
        unsigned char* lo = hi + k + kPlanePad;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            *reinterpret_cast<uint32_t*>(hi + 16 * w) = hw[w];
            *reinterpret_cast<uint32_t*>(lo + 16 * w) = lw[w];
        }
        if (((col >> 4) & 7) == 0) meta[mi * (k / kGroupCols) + (col >> 7)] = make_int2((int)((uint32_t)(127 - s) << 23), isum);
    }
}

__global__ void __launch_bounds__(kMaxThreads3, 1)
gemv3_kernel(Layout2 L, const unsigned char* __restrict__ packed, const __half* __restrict__ X,
             __half* __restrict__ Y, int m, int rows_cap, int q_base, int q_rem, int teams, int depth, int speculate,
             int* __restrict__ status_word) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int S = L.slices, ngroups = L.k / kGroupCols, PS = L.k + kPlanePad;
    const Smem3 sm = smem_layout3(L.k, m, S, rows_cap, teams, depth, speculate);
    unsigned char* xs = smem;
    int2* meta = reinterpret_cast<int2*>(smem + sm.meta_off);
    uint4* first_read = reinterpret_cast<uint4*>(smem + sm.raw_off);        // x as read before the dependency wait
    float* partial = reinterpret_cast<float*>(smem + sm.partial_off);       // [m][rows_cap][S kTeamWarps]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bar_off);        // per team: depth "full", depth "empty"
    unsigned char* rings = smem + sm.ring_off;
    // (the shuffle tells the compiler that the warp index is the same in all lanes)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int cthreads = teams * kTeamWarps * 32;
    const int team = warp / kTeamWarps, hq = warp % kTeamWarps, g = lane >> 2, t = lane & 3;
    uint64_t* full = bars + team * 2 * depth;
    uint64_t* empty = full + depth;
    unsigned char* ring = rings + (size_t)team * depth * kStage3;

    // Let the next kernel on the stream start while this one runs.
    asm volatile("griddepcontrol.launch_dependents;");

    // this CTA's quads (balanced partition from the host); team tm takes tasks [tm T / teams, (tm + 1) T / teams)
    // of the (slice, quad) list
    const int q0 = (int)blockIdx.x * q_base + min((int)blockIdx.x, q_rem);
    const int nq = q_base + ((int)blockIdx.x < q_rem ? 1 : 0);
    const int T = nq * S;
    const int t0 = team * T / teams, ntask = (team + 1) * T / teams - t0;
    const int nchunks = m * (L.k >> 3), chunks16_per_row = L.k >> 4, nchunks16 = m * chunks16_per_row;
    const unsigned char* codes = packed + L.codes_off;

    if ((int)threadIdx.x < teams * depth) {
        bar_init(bars + (threadIdx.x / depth) * 2 * depth + threadIdx.x % depth, kTeamWarps);
        bar_init(bars + (threadIdx.x / depth) * 2 * depth + depth + threadIdx.x % depth, kTeamWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    bool failed = false;
    // Copy side of this warp: it brings the unit of row pair hq of every task of its team.  State: tasks given
    // out so far in this pass, their slice and quad, the ring stage and how often the ring has been filled.
    int pn = 0, ps = 0, pq = 0, pstage = 0, pround = 0;
    auto produce = [&]() {
        if (pn < ntask) {
            const int q = q0 + pq;
            if (lane == 0) {
                // a stage is refilled only after all warps of the team have released its previous contents
                if (pround > 0 && !bar_wait_bounded(empty + pstage, (uint32_t)(pround - 1) & 1u, failed)) {
                    failed = true;
                }
                if (4 * q + hq < L.nrp) {
                    const uint32_t bytes = ps == S - 1 ? (uint32_t)L.last_unit : (uint32_t)kUnit2;
                    bar_expect_tx(full + pstage, bytes);
                    bulk_g2s(ring + pstage * kStage3 + hq * kUnitStride3,
                             codes + unit_offset(L, 4 * q + hq, ps), bytes, full + pstage);
                } else {
                    bar_arrive(full + pstage);          // a row pair past the end of the matrix: nothing to bring
                }
            }
            failed = __any_sync(0xffffffffu, failed);
            if (++pq == nq) { pq = 0; ++ps; }
            if (++pstage == depth) { pstage = 0; ++pround; }
        }
        ++pn;
    };

    // lane constants: code fields of this lane's two MMA rows, selector of its two scales in a scale quad
    const int f0 = g >> 2;                                              // MMA row g: field f0; row g + 8: field 2 + f0
    const uint32_t mask0 = 0x03030303u << (2 * f0), mask1 = mask0 << 4;
    const uint32_t alpha_sel = f0 ? 0x7632u : 0x5410u;
    const float field_scale = f0 ? 0.25f : 1.f;                        // 4^-f0; row g + 8 gets another 1/16 at the end
    const bool batch_lane = t < m;                                      // this lane's accumulator columns are batch row t

    int stage = 0;
    uint32_t parity = 0;
    bool waited = false;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // Pass 0 is speculative when allowed: x is read before earlier work of the stream is known to be complete.
        const bool spec = speculate && attempt == 0;
        if (!spec && !waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = true;
        }
        // The packed planes do not depend on earlier work of the stream: two stages are requested first, the
        // rest of the ring while the first reads of x are in flight.
        pn = 0;
        ps = t0 / nq;
        pq = t0 - ps * nq;
        produce();
        produce();
        // x -> block fixed point in shared memory, two 16-column chunks per thread in flight.  Reads go to L2
        // (ld.global.cg), the point of coherence, never through L1.
        for (int cb = (int)threadIdx.x; (cb & ~31) < nchunks16; cb += 2 * cthreads) {
            uint4 r[4];
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                const int c = cb + p * cthreads;
                r[2 * p] = r[2 * p + 1] = make_uint4(0u, 0u, 0u, 0u);
                if (c < nchunks16) {
                    r[2 * p] = __ldcg(reinterpret_cast<const uint4*>(X) + 2 * c);
                    r[2 * p + 1] = __ldcg(reinterpret_cast<const uint4*>(X) + 2 * c + 1);
                }
            }
            if (cb == (int)threadIdx.x)
                for (int d = 2; d < depth; ++d) produce();
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                const int c = cb + p * cthreads;
                if ((c & ~31) < nchunks16) {
                    if (spec && c < nchunks16) { first_read[2 * c] = r[2 * p]; first_read[2 * c + 1] = r[2 * p + 1]; }
                    const int mi = c / chunks16_per_row;
                    convert3_x16(r[2 * p], r[2 * p + 1], mi, (c - mi * chunks16_per_row) << 4, c < nchunks16, L.k, xs, meta);
                }
            }
        }
        __syncthreads();

        uint32_t b[kNB][4];                 // B fragments of the warp's slice quarter: [lane block][MMA 0: k-lo, k-hi, MMA 1: ...]
        float xscale[kNB / 2];              // per scale group: 2^-s of batch row t times 4^-f0
        int negsum[kNB / 2];                // per scale group: -4^f0 sum_j X_j of batch row t
        int cur_slice = -1, nb = 0, A = 32;
        int cs = t0 / nq, cq = t0 - cs * nq;
        for (int i = 0; i < ntask; ++i) {
            if (cs != cur_slice) {
                // entering a slice: this warp's quarter of its activations goes to registers (zeros past the end
                // of a short last slice and for batch rows that do not exist)
                cur_slice = cs;
                A = cs == S - 1 ? L.last_active : 32;
                nb = max(0, min(kNB, A - kNB * hq));                    // lane blocks of this quarter (even)
                const unsigned char* xrow = xs + (size_t)g * PS + (cs * 32 + kNB * hq) * 64 + 16 * t;   // plane g%2 of batch row g/2
                const bool have = (g >> 1) < m;
#pragma unroll
                for (int bb = 0; bb < kNB; ++bb) {
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (have && bb < nb) v = *reinterpret_cast<const uint4*>(xrow + 64 * bb);
                    b[bb][0] = v.x; b[bb][1] = v.y; b[bb][2] = v.z; b[bb][3] = v.w;
                }
                const int g0 = cs * 16 + hq * (kNB / 2);
#pragma unroll
                for (int j = 0; j < kNB / 2; ++j) {
                    int2 mt = make_int2(0, 0);
                    if (batch_lane && 2 * j < nb) mt = meta[t * ngroups + g0 + j];
                    xscale[j] = __int_as_float(mt.x) * field_scale;
                    negsum[j] = -(mt.y << (2 * f0));
                }
            }
            if (i >= 1) produce();                      // refills the stage consumed one task ago
            if (!bar_wait_bounded(full + stage, parity, failed)) failed = true;
            const unsigned char* st = ring + stage * kStage3;
            // ldmatrix row address: lanes 8i..8i+7 give the rows of matrix i = atom row i of the lane block, for
            // row pairs (lane % 4); thread (g, t) then holds word t of the atom of row pair g % 4
            const uint32_t lm = s32(st) + (lane & 3) * kUnitStride3 + ((lane >> 3) * A + kNB * hq) * 16;
            const unsigned char* sc = st + (g & 3) * kUnitStride3 + A * 64 + hq * (kNB / 2) * 8;
            float r0 = 0.f, r1 = 0.f;
#pragma unroll
            for (int jj = 0; jj < kNB / 4; ++jj) {
                // scale groups 2 jj and 2 jj + 1 side by side: two independent accumulator chains.  Lane blocks
                // past the end of a short last slice multiply stale bytes by zero activations.
                if (4 * jj < nb) {
                    const int ja = 2 * jj, jb = 2 * jj + 1;
                    int ca[4] = {0, negsum[ja], 0, negsum[ja] * 16};
                    int cb[4] = {0, negsum[jb], 0, negsum[jb] * 16};
                    uint32_t wa[4], wb[4], wc[4], wd[4];
                    ldmatrix4(wa, lm + (4 * jj) * 16);
                    ldmatrix4(wb, lm + (4 * jj + 2) * 16);
                    ldmatrix4(wc, lm + (4 * jj + 1) * 16);
                    ldmatrix4(wd, lm + (4 * jj + 3) * 16);
                    mma_u8s8(ca, wa[0] & mask0, wa[0] & mask1, wa[1] & mask0, wa[1] & mask1, b[4 * jj][0], b[4 * jj][1]);
                    mma_u8s8(cb, wb[0] & mask0, wb[0] & mask1, wb[1] & mask0, wb[1] & mask1, b[4 * jj + 2][0], b[4 * jj + 2][1]);
                    mma_u8s8(ca, wa[2] & mask0, wa[2] & mask1, wa[3] & mask0, wa[3] & mask1, b[4 * jj][2], b[4 * jj][3]);
                    mma_u8s8(cb, wb[2] & mask0, wb[2] & mask1, wb[3] & mask0, wb[3] & mask1, b[4 * jj + 2][2], b[4 * jj + 2][3]);
                    mma_u8s8(ca, wc[0] & mask0, wc[0] & mask1, wc[1] & mask0, wc[1] & mask1, b[4 * jj + 1][0], b[4 * jj + 1][1]);
                    mma_u8s8(cb, wd[0] & mask0, wd[0] & mask1, wd[1] & mask0, wd[1] & mask1, b[4 * jj + 3][0], b[4 * jj + 3][1]);
                    mma_u8s8(ca, wc[2] & mask0, wc[2] & mask1, wc[3] & mask0, wc[3] & mask1, b[4 * jj + 1][2], b[4 * jj + 1][3]);
                    mma_u8s8(cb, wd[2] & mask0, wd[2] & mask1, wd[3] & mask0, wd[3] & mask1, b[4 * jj + 3][2], b[4 * jj + 3][3]);
                    {
                        const uint2 q = *reinterpret_cast<const uint2*>(sc + ja * 8);
                        const uint32_t apair = __byte_perm(q.x, q.y, alpha_sel);     // (scale of row g, scale of row g + 8)
                        const float2 af = __half22float2(*reinterpret_cast<const __half2*>(&apair));
                        r0 = fmaf((float)((ca[0] << 8) + ca[1]), af.x * xscale[ja], r0);
                        r1 = fmaf((float)((ca[2] << 8) + ca[3]), af.y * xscale[ja], r1);
                    }
                    if (4 * jj + 2 < nb) {
                        const uint2 q = *reinterpret_cast<const uint2*>(sc + jb * 8);
                        const uint32_t apair = __byte_perm(q.x, q.y, alpha_sel);
                        const float2 af = __half22float2(*reinterpret_cast<const __half2*>(&apair));
                        r0 = fmaf((float)((cb[0] << 8) + cb[1]), af.x * xscale[jb], r0);
                        r1 = fmaf((float)((cb[2] << 8) + cb[3]), af.y * xscale[jb], r1);
                    }
                }
            }
            r1 *= 0.0625f;
            // every warp of the team releases the stage; it is refilled when all four have
            __syncwarp();
            if (lane == 0) bar_arrive(empty + stage);
            // planes: lanes g and g ^ 4 hold plane 1 and plane 2 of the same rows
            r0 += __shfl_xor_sync(0xffffffffu, r0, 16);
            r1 += __shfl_xor_sync(0xffffffffu, r1, 16);
            if (g < 4 && batch_lane) {
                float* pp = partial + ((size_t)t * rows_cap + 8 * cq + 2 * g) * (kTeamWarps * S) + kTeamWarps * cs + hq;
                pp[0] = failed ? __int_as_float(0x7fc00000) : r0;
                pp[kTeamWarps * S] = failed ? __int_as_float(0x7fc00000) : r1;
            }
            if (++stage == depth) { stage = 0; parity ^= 1u; }
            if (++cq == nq) { cq = 0; ++cs; }
        }
        if (!spec) break;
        // Earlier work of the stream is complete after this wait: if x still reads as it did, the pass stands.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
        int stale = 0;
#pragma unroll 4
        for (int c = (int)threadIdx.x; c < nchunks; c += cthreads) {
            const uint4 now = __ldcg(reinterpret_cast<const uint4*>(X) + c);
            const uint4 was = first_read[c];
            stale |= (now.x != was.x) | (now.y != was.y) | (now.z != was.z) | (now.w != was.w);
        }
        if (!__syncthreads_or(stale)) break;
    }
    if (failed && lane == 0) atomicExch(status_word, (int)PTQTP_ERR_CUDA);
    __syncthreads();                                     // all partial sums are in shared memory
    const int rows = 8 * nq;
    for (int idx = threadIdx.x; idx < m * rows; idx += cthreads) {
        const int mi = idx / rows, r = idx - mi * rows;
        const int row = 8 * q0 + r;
        const float* pp = partial + ((size_t)mi * rows_cap + r) * (kTeamWarps * S);
        float acc = 0.f;
        for (int s = 0; s < kTeamWarps * S; ++s) acc += pp[s];
        if (row < L.n) Y[(size_t)mi * L.n + row] = __float2half_rn(acc);
    }
}

}  // namespace

// PTQTP_ERR_SHAPE when the activations of (K, M) leave no room for a two-stage ring in shared memory.
// warps: 4, 8 or 16 (one, two or four teams; 0 = 4, or 8 for three slices and more or when a CTA streams many units):
// small CTAs let the CTAs of consecutive launches share an SM, so that the head of one launch overlaps the
// streaming of another.
// ctas_per_sm: CTAs of this launch per SM, 1 or 2 (0 = 1).
ptqtp_status launch_gemv3(const Layout2& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int warps,
                          int ctas_per_sm, int depth, cudaStream_t st) {
    if (m < 1 || m > kMaxBatch3) return PTQTP_ERR_SHAPE;
    if (ctas_per_sm < 0 || ctas_per_sm > 2 || depth < 0 || depth == 1 || depth > 8) return PTQTP_ERR_CONFIG;
    if (warps != 0 && warps != 4 && warps != 8 && warps != 16) return PTQTP_ERR_CONFIG;
    const int nquads = (L.nrp + 3) / 4;
    const int per_sm = ctas_per_sm == 2 ? 2 : 1;
    const int grid = min(per_sm * sm_count(), nquads);
    const int rows_cap = 8 * ((nquads + grid - 1) / grid);
    if (warps == 0) {
        warps = L.slices >= 3 || (long)((nquads + grid - 1) / grid) * L.slices >= 64 ? 8 : 4;
        if (m >= 2) warps = m == 2 && L.slices <= 2 ? 8 : 16;   // converting M rows of x is shared by the CTA's threads
    }
    if (warps * per_sm > 16) return PTQTP_ERR_CONFIG;
    const int teams = warps / kTeamWarps;
    const size_t budget = (size_t)(228 / per_sm - 1) * 1024;            // 228 KB per SM, 1 KB of it reserved per CTA
    const bool auto_depth = depth == 0;
    // speculative execution keeps a second copy of x in shared memory: it is dropped when M rows of x leave no
    // room for it beside a two-stage ring
    int speculate = speculation_enabled() ? 1 : 0;
    if (speculate && smem_layout3(L.k, m, L.slices, rows_cap, teams, auto_depth ? 2 : depth, 1).total > budget) speculate = 0;
    if (auto_depth) {
        depth = 3;
        while (depth > 2 && smem_layout3(L.k, m, L.slices, rows_cap, teams, depth, speculate).total > budget) --depth;
    }
    const size_t smem = smem_layout3(L.k, m, L.slices, rows_cap, teams, depth, speculate).total;
    if (smem > budget) return !auto_depth && depth > 2 ? PTQTP_ERR_CONFIG : PTQTP_ERR_SHAPE;
    int* status_word = nullptr;                           // shared with the batch-1 CUDA-core kernel (ptqtp_kernel_status)
    if (gemv_status_word(&status_word) != PTQTP_OK) return PTQTP_ERR_CUDA;
    const ptqtp_status cs = configure_once<gemv3_kernel>();
    if (cs != PTQTP_OK) return cs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(teams * kTeamWarps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_enabled() && !consume_pack(st) ? 1 : 0;   // plain right after a pack on this stream
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv3_kernel, L, static_cast<const unsigned char*>(packed),
                                       reinterpret_cast<const __half*>(X), reinterpret_cast<__half*>(Y), m, rows_cap,
                                       nquads / grid, nquads % grid, teams, depth, speculate, status_word);
    if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

}  // namespace ptqtp
