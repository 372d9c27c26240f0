// Dual-trit-plane layer for up to 64 activation rows per launch on packed format 3 (the batch-1 layout), on the
// fifth-generation tensor cores (tcgen05.mma, accumulators in tensor memory):
//     Y[m] = alpha1 (.) (T1 X[m]) + alpha2 (.) (T2 X[m]),   m < M <= 64.
//
// A CTA owns 128 weight rows (8 tiles per superblock, contiguous in the blob); row i is lane i of every MMA.  Ten
// warps: eight decode (two threads per row, half of a group's columns each), one issues the MMAs, one copies the
// code stages.  Per scale group of 128 columns:
//   * the decoders turn their row's 2-bit codes into fp16 trits (-1, 0, +1): a mask per plane, two byte permutes that
//     put two code bytes under the exponent of 1024, one fp16 FMA that maps 1024 + code * 2^s to code - 1; the trits
//     go to tensor memory (tcgen05.st, one lane per row, 64 columns per plane): the A operand never passes through
//     shared memory;
//   * the activations of the group, fp16 as given (no quantisation), are the B operand: M rows padded to a multiple
//     of 16, in shared memory as K-major core matrices (8 rows x 16 bytes), fetched with 16-byte cp.async one group
//     ahead;
//   * an elected lane of the MMA warp issues 16 MMAs of 128 x NPAD x 16 (8 k-steps for each plane, in two halves of
//     four k-steps that are decoded and multiplied alternately) into two fp32 accumulators and commits each half to
//     an mbarrier; the trits are exact in fp16, so each accumulator is the fp32 sum of +-x;
//   * the decoders read their lane of both accumulators (tcgen05.ld, half of the columns each) and add
//     alpha1 * d1 + alpha2 * d2 in fp32 to their running sums.
// The code stages are copied with 16-byte cp.async that regroup the lane entries of the tiles (made for warp-MMA
// fragments) so that a warp of row threads reads 16 consecutive entries: no bank conflicts.
// Two CTAs share an SM (256 of the 512 tensor-memory columns and 78 to 103 KB of shared memory each), so one CTA's
// decode and epilogue run under the other's MMAs.  Matrices with few rows split K over a cluster of up to 8 CTAs;
// the partial sums meet in distributed shared memory and are added in rank order (no atomics, reproducible).
//
// Waits on mbarriers are bounded: a wait that gives up marks the launch failed (status word, NaN rows), the CTA
// still takes part in the cluster barriers and frees its tensor memory.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kRows6 = 128;                            // weight rows (= MMA rows) per CTA
constexpr int kDecoders6 = 2 * kRows6;                 // decoding threads: one per row and plane
constexpr int kThreads6 = kDecoders6 + 64;             // + the warp that issues the MMAs + the warp that copies the codes
constexpr int kBlockTiles6 = 8;                        // tiles per CTA and superblock: 128 weight rows
constexpr int kStage6 = kBlockTiles6 * kTile3;         // 34816 bytes
constexpr int kStages6 = 2;
// A stage in shared memory: the 16-byte lane entries of the block's eight tiles regrouped as [chunk][t][tile][row pair]
// (a warp of row threads then reads 16 consecutive entries: no bank conflicts), then the tiles' scale quads.
constexpr int kLaneT6 = 64 * 16;                       // bytes between the entries t and t + 1 of a row pair
constexpr int kChunk6 = 4 * kLaneT6;                   // bytes between chunks
constexpr int kStageScales6 = 8 * kChunk6;             // 32768: offset of the scale quads (256 bytes per tile)
constexpr int kTmemCols6 = 256;                        // D: columns 0 .. 2 NPAD - 1; A: columns 128 .. 255
constexpr int kACol6 = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
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
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ uint32_t prmt2(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One arrival for the whole (converged) warp: arrivals on one mbarrier are serialised, 256 of them cost more than
// the work they separate.  The warp barrier orders every lane's earlier operations before lane 0's release.
__device__ __forceinline__ void warp_arrive(uint32_t bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]));
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr));
}
// One lane of a converged warp.
__device__ __forceinline__ uint32_t elect_one() {
    uint32_t leader;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(leader));
    return leader;
}
// The loads above complete here; the registers pass through so that no use of them can be scheduled earlier.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&a)[8], uint32_t (&b)[8]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                   "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7])
                 :: "memory");
}

// Shared-memory matrix descriptor, K-major, no swizzle: core matrices of 8 rows x 16 bytes (128 contiguous bytes);
// lbo = bytes between the two core matrices of a k-step, sbo = bytes between 8-row groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3fffu) | (uint64_t)((lbo >> 4) & 0x3fffu) << 16 |
           (uint64_t)((sbo >> 4) & 0x3fffu) << 32 | (uint64_t)1 << 46;
}

__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// Shared memory (all dynamic): the ring of code stages (the first doubles as the partial-sum exchange of a cluster),
// two activation buffers of one scale group each (16 chunks of 8 columns x NPAD rows x 16 bytes), the mbarriers.
template <int NPAD>
struct Smem6 {
    static constexpr int x_buf = 16 * NPAD * 16;
    static constexpr int x_off = kStages6 * kStage6;
    static constexpr int bar_off = x_off + 2 * x_buf;          // six mbarriers, the word that receives the tensor-
    static constexpr int total = bar_off + 128;                // memory address, the give-up flag
};

// The copies of one activation group (128 columns of every row of X) into an activation buffer: chunk kc (8 columns)
// of row n goes to kc * NPAD * 16 + n * 16.  A decoder owns NPAD / 16 chunks, the same ones for every group (adjacent
// threads take the two halves of a 32-byte sector); XChunks holds their offsets.
template <int NPAD>
struct XChunks {
    uint32_t src[NPAD / 16];     // offset in X, in halves, without the group's 128 gg; 0xffffffff: a row past m
    uint32_t dst[NPAD / 16];     // byte offset in the buffer
    __device__ __forceinline__ void init(int k, int m) {
#pragma unroll
        for (int i = 0; i < NPAD / 16; ++i) {
            const int q = i * kDecoders6 + (int)threadIdx.x;
            const int n = (q >> 1) % NPAD, kc = 2 * ((q >> 1) / NPAD) + (q & 1);
            src[i] = n < m ? (uint32_t)(n * k + 8 * kc) : 0xffffffffu;
            dst[i] = (uint32_t)(kc * (NPAD * 16) + n * 16);
        }
    }
    __device__ __forceinline__ void fetch(const __half* __restrict__ X, int gg, uint32_t buf) const {
#pragma unroll
        for (int i = 0; i < NPAD / 16; ++i)
            if (src[i] != 0xffffffffu) cp_async16(buf + dst[i], X + src[i] + 128 * gg);
    }
};

// Wait for a phase of an mbarrier (the suspending form: a waiting thread takes no issue slots; polling without
// suspension was measured 30 % slower).  Gives up after `limit` polls or when another thread of the CTA has given up.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool wait_phase(uint32_t bar, uint32_t parity, int limit, volatile int* failed) {
    if (mbar_test_wait(bar, parity)) return true;        // the usual case: the phase is long complete
    for (int i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 31) == 31 && *failed) return false;
    }
    *failed = 1;
    return false;
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    // volatile: stays ahead of the tensor-memory stores that follow in program order, so the loads of a step are
    // all in flight before the arithmetic on the first of them
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// A quarter of the 128 columns of one scale group of this thread's row, both planes: the two 16-column chunks
// c = c_first and c_first + 2, as fp16 trits into tensor memory (8 columns per chunk and plane).  The row's code sits
// at the same two bits of every byte (mask0 for plane 0, two bits higher for plane 1); the byte permute puts two code
// bytes under the exponent of 1024 (0x64 high bytes), so a half holds 1024 + code * 2^s exactly, and one fp16 FMA
// maps it to code - 1.  The masks and permutes run on the integer pipe, the FMAs on the fp16 pipe.  H: which half of
// a lane entry holds the group (groups 0, 1 of a superblock: words 0 and 2; groups 2, 3: words 1 and 3).
template <int H>
__device__ __forceinline__ void decode_two_chunks(uint32_t lane_entry, int c_first, uint32_t mask0, __half2 scale0,
                                                  __half2 bias0, __half2 scale1, __half2 bias1, uint32_t a_cols) {
    const uint32_t mask1 = mask0 << 2;
    uint4 v[2][2];
#pragma unroll
    for (int cq = 0; cq < 2; ++cq)
#pragma unroll
        for (int tt = 0; tt < 2; ++tt) v[cq][tt] = lds128(lane_entry + (c_first + 2 * cq) * kChunk6 + tt * kLaneT6);
#pragma unroll
    for (int cq = 0; cq < 2; ++cq) {
        const int c = c_first + 2 * cq;
        uint32_t r0[8], r1[8];
#pragma unroll
        for (int tt = 0; tt < 2; ++tt) {
            const uint32_t w[2] = {H ? v[cq][tt].y : v[cq][tt].x, H ? v[cq][tt].w : v[cq][tt].z};
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                const int col = 4 * s + 2 * tt;                 // columns 8 s + 4 tt .. + 3 of the chunk: two 32-bit columns
                const uint32_t c0 = w[s] & mask0, c1 = w[s] & mask1;
                const uint32_t lo0 = prmt2(c0, 0x64646464u, 0x4140u), hi0 = prmt2(c0, 0x64646464u, 0x4342u);
                const uint32_t lo1 = prmt2(c1, 0x64646464u, 0x4140u), hi1 = prmt2(c1, 0x64646464u, 0x4342u);
                const __half2 a0 = __hfma2(*reinterpret_cast<const __half2*>(&lo0), scale0, bias0);
                const __half2 b0 = __hfma2(*reinterpret_cast<const __half2*>(&hi0), scale0, bias0);
                const __half2 a1 = __hfma2(*reinterpret_cast<const __half2*>(&lo1), scale1, bias1);
                const __half2 b1 = __hfma2(*reinterpret_cast<const __half2*>(&hi1), scale1, bias1);
                r0[col] = *reinterpret_cast<const uint32_t*>(&a0);
                r0[col + 1] = *reinterpret_cast<const uint32_t*>(&b0);
                r1[col] = *reinterpret_cast<const uint32_t*>(&a1);
                r1[col + 1] = *reinterpret_cast<const uint32_t*>(&b1);
            }
        }
        tmem_st8(a_cols + 8 * c, r0);
        tmem_st8(a_cols + 64 + 8 * c, r1);
    }
}

// Warps 0-7: two threads per weight row; each decodes half of a group's columns (both planes), reads half of the
// accumulator columns in the scale epilogue and fetches its share of the activations.  Warp 8 issues the MMAs (the
// whole warp runs the loop so that the operands stay in uniform registers; one elected lane issues).  Warp 9 keeps
// the ring of code stages full.  They meet on mbarriers only (h = 0: k-steps 0-3 of a group, h = 1: k-steps 4-7):
//   code_full[s]  (32 arrivals)  stage s holds the block's tiles of a superblock (one arrival per copying lane)
//   code_free[s]  (8 arrivals: one per decoding warp) every decoder is done with stage s
//   a_full[h]     (8 arrivals)   half h of the group's trits is in tensor memory; for h = 0 also: the group's
//                                activations are in shared memory and the accumulators of the group before are read
//   a_free[h]     (MMA commit)   the 8 MMAs of half h are done; for h = 1: the group's accumulators are complete
// The first half of group g + 1 is decoded under the MMAs of the second half of group g, the second half under the
// MMAs of the first; the two CTAs of an SM fill each other's remaining gaps.
template <int NPAD>
__global__ void __launch_bounds__(kThreads6, 2)
gemm6_kernel(Layout3 L, const unsigned char* __restrict__ packed, const __half* __restrict__ X, __half* __restrict__ Y,
             int m, int csize, int spin_limit, int inject, int* status_word) {
    extern __shared__ __align__(128) unsigned char smem[];
    using SM = Smem6<NPAD>;
    constexpr int HALF = NPAD / 2;                       // accumulator columns per decoder of a row
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::bar_off);
    const uint32_t code_full = smem_u32(bars), code_free = smem_u32(bars + 2), a_full = smem_u32(bars + 4),
                   a_free = smem_u32(bars + 6);
    uint32_t& tmem_slot = *reinterpret_cast<uint32_t*>(bars + 8);
    volatile int* failed = reinterpret_cast<volatile int*>(bars + 9);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int crank = (int)blockIdx.x % csize, blk = (int)blockIdx.x / csize;
    const int rb0 = blk * kBlockTiles6;
    const int tiles = min(kBlockTiles6, L.nrb - rb0);
    const int groups = L.k / 128;
    // this CTA's superblocks: a balanced split of the superblocks over the cluster
    const int sb_base = L.sbs / csize, sb_rem = L.sbs % csize;
    const int sb_lo = crank * sb_base + min(crank, sb_rem);
    const int sb_hi = sb_lo + sb_base + (crank < sb_rem ? 1 : 0);
    const int gg_lo = 4 * sb_lo, gg_end = min(4 * sb_hi, groups);
    const unsigned char* codes = packed + L.codes_off;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(kTmemCols6) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(bars + s, 32);
            mbar_init(bars + 2 + s, kDecoders6 / 32);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(bars + 4 + h, kDecoders6 / 32);
            mbar_init(bars + 6 + h, 1);
        }
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // rows m .. NPAD - 1 of the activation buffers stay zero
    for (int i = tid; i < 2 * SM::x_buf / 16; i += kThreads6)
        reinterpret_cast<uint4*>(smem + SM::x_off)[i] = make_uint4(0u, 0u, 0u, 0u);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot;
    const uint32_t xbuf0 = smem_u32(smem + SM::x_off);

    float y[HALF];
#pragma unroll
    for (int i = 0; i < HALF; ++i) y[i] = 0.f;
    const int hc = (warp >> 2) & 1, row_in = 32 * (warp & 3) + lane;        // decoders only

    if (warp == 9) {
        // ---- the ring of code stages: 16-byte asynchronous copies that regroup the lane entries ----
        bool ok = true;
        for (int sb = sb_lo; sb < sb_hi && ok; ++sb) {
            const int sl = sb - sb_lo, stage = sl & 1;
            if (sl >= kStages6) ok = wait_phase(code_free + 8 * stage, (uint32_t)((sl >> 1) - 1) & 1u, spin_limit, failed);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const unsigned char* src = codes + tile_offset3(L, rb0, sb);
            const uint32_t dst = smem_u32(smem + stage * kStage6);
            for (int tile = 0; tile < tiles; ++tile) {
                const unsigned char* ts = src + (size_t)tile * kTile3;
                const uint32_t td = dst + (uint32_t)(((lane & 3) * 64 + tile * 8 + (lane >> 2)) * 16);
#pragma unroll
                for (int c = 0; c < 8; ++c) cp_async16(td + c * kChunk6, ts + c * 512 + lane * 16);     // lane entry (c, lane)
                if (lane < 16) cp_async16(dst + kStageScales6 + tile * 256 + lane * 16, ts + kTileCodes3 + lane * 16);
            }
            // the stage's mbarrier counts one arrival per lane, made when the lane's copies have landed
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(code_full + 8 * stage) : "memory");
        }
        cp_async_wait_all();
    } else if (warp == 8) {
        // ---- the MMAs ----
        const uint32_t idesc = (1u << 4) | ((uint32_t)(NPAD >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t leader = elect_one();
        bool ok = true;
        for (int gg = gg_lo, pass = 0; gg < gg_end && ok; ++gg, ++pass) {
            const uint64_t bdesc = smem_desc(xbuf0 + (pass & 1) * SM::x_buf, NPAD * 16, 128);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                ok = wait_phase(a_full + 8 * h, (uint32_t)pass & 1u, spin_limit, failed);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                if (leader) {
#pragma unroll
                    for (int p = 0; p < 2; ++p)
#pragma unroll
                        for (int j = 4 * h; j < 4 * h + 4; ++j)     // a k-step further on: two chunks of NPAD * 16 bytes
                            mma_f16_ts(tbase + p * NPAD, tbase + kACol6 + 64 * p + 8 * j, bdesc + (uint64_t)(2 * j * NPAD),
                                       idesc, j > 0 ? 1u : 0u);
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 ::"r"(a_free + 8 * h) : "memory");
                }
                __syncwarp();
            }
        }
    } else {
        // ---- two threads per weight row ----
        const uint32_t tlane = tbase + ((uint32_t)((warp & 3) * 32) << 16);      // this warp's 32 lanes
        // thread -> (tile of the block, row pair g of the tile, member of the pair)
        const int tl = row_in >> 4, g = (lane >> 1) & 7, mem = lane & 1;
        // the row's codes: plane 0 at bits 4 mem .. 4 mem + 1 of every byte, plane 1 two bits higher
        const uint32_t mask0 = 0x03030303u << (4 * mem);
        const __half2 scale0 = __float2half2_rn(mem ? 0.0625f : 1.f), bias0 = __float2half2_rn(mem ? -65.f : -1025.f);
        const __half2 scale1 = __float2half2_rn(mem ? 0.015625f : 0.25f), bias1 = __float2half2_rn(mem ? -17.f : -257.f);
        bool ok = true;
        __half2 alpha_prev = __float2half2_rn(0.f);

        XChunks<NPAD> xc;
        xc.init(L.k, m);
        if (gg_lo < gg_end) xc.fetch(X, gg_lo, xbuf0);
        cp_async_commit();
        const uint32_t a_cols = tlane + kACol6;
        __half2 alpha = alpha_prev;
        int pass = 0;
        for (int gg = gg_lo; gg <= gg_end && gg_lo < gg_end; ++gg, ++pass) {
            const bool live = gg < gg_end;                  // the last round only reads the last group's accumulators
            const int sb = gg >> 2, G = gg & 3, sl = sb - sb_lo, stage = sl & 1;
            const unsigned char* stage_base = smem + stage * kStage6;
            const uint32_t lane_entry = smem_u32(stage_base) + 2 * (G & 1) * kLaneT6 + (tl * 8 + g) * 16;
            if (live) {
                // first half of the group's k-steps: under the MMAs of the second half of the group before
                if (G == 0) ok = ok && !(inject && pass == 0) && wait_phase(code_full + 8 * stage, (uint32_t)(sl >> 1) & 1u, spin_limit, failed);
                if (pass > 0) ok = ok && wait_phase(a_free, (uint32_t)(pass - 1) & 1u, spin_limit, failed);
                if (!__all_sync(0xffffffffu, ok)) { *failed = 1; break; }
                tc_fence_after();
                alpha = *reinterpret_cast<const __half2*>(stage_base + kStageScales6 + tl * 256 + 8 * (4 * g + G) + 4 * mem);
                if (G >> 1) decode_two_chunks<1>(lane_entry, hc, mask0, scale0, bias0, scale1, bias1, a_cols);
                else decode_two_chunks<0>(lane_entry, hc, mask0, scale0, bias0, scale1, bias1, a_cols);
            }
            if (pass > 0) {
                // accumulators of the previous group: y += alpha1 d1 + alpha2 d2 on this thread's half of the columns
                ok = ok && wait_phase(a_free + 8, (uint32_t)(pass - 1) & 1u, spin_limit, failed);
                if (!__all_sync(0xffffffffu, ok)) { *failed = 1; break; }
                tc_fence_after();
                const float a1 = __low2float(alpha_prev), a2 = __high2float(alpha_prev);
#pragma unroll
                for (int c0 = 0; c0 < HALF; c0 += 8) {
                    uint32_t d1[8], d2[8];
                    tmem_ld8(tlane + hc * HALF + c0, d1);
                    tmem_ld8(tlane + NPAD + hc * HALF + c0, d2);
                    tmem_ld_wait(d1, d2);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        y[c0 + i] = fmaf(a1, __uint_as_float(d1[i]), fmaf(a2, __uint_as_float(d2[i]), y[c0 + i]));
                }
            }
            if (!live) break;
            alpha_prev = alpha;
            cp_async_wait_all();                            // this group's activations (queued one round ago)
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            warp_arrive(a_full);
            // the next group's activations, after the fence (it would wait for copies queued before it): their
            // buffer was last read by the MMAs of the previous group, which are done
            if (gg + 1 < gg_end) xc.fetch(X, gg + 1, xbuf0 + ((pass + 1) & 1) * SM::x_buf);
            cp_async_commit();
            // second half: under the MMAs of the first
            if (G >> 1) decode_two_chunks<1>(lane_entry, 4 + hc, mask0, scale0, bias0, scale1, bias1, a_cols);
            else decode_two_chunks<0>(lane_entry, 4 + hc, mask0, scale0, bias0, scale1, bias1, a_cols);
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            warp_arrive(a_full + 8);
            if (G == 3 || gg + 1 == gg_end) warp_arrive(code_free + 8 * stage);
        }
        cp_async_wait_all();
    }
    __syncthreads();
    const bool bad = *failed != 0;
    if (bad) {
        if (tid == 0) atomicExch(status_word, (int)PTQTP_ERR_CUDA);
        // copies and MMAs whose waits gave up may still be in flight: give them time before the memory is reused
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
#pragma unroll
        for (int i = 0; i < HALF; ++i) y[i] = __int_as_float(0x7fc00000);
    }
    const int row = 16 * rb0 + row_in;
    if (csize == 1) {
        if (tid < kDecoders6 && row < L.n) {
#pragma unroll
            for (int i = 0; i < HALF; ++i)
                if (hc * HALF + i < m) Y[(size_t)(hc * HALF + i) * L.n + row] = __float2half_rn(y[i]);
        }
    } else {
        // partial sums of the cluster meet in shared memory; rank r adds its share of the columns in rank order
        float* P = reinterpret_cast<float*>(smem);
        if (tid < kDecoders6) {
#pragma unroll
            for (int i = 0; i < HALF; ++i) P[(hc * HALF + i) * kRows6 + row_in] = y[i];
        }
        cluster_sync_all();
        if (tid < kDecoders6) {
            const int per = NPAD / csize;
            for (int i = crank * per + hc; i < (crank + 1) * per && i < m; i += 2) {
                float s = 0.f;
                for (int r = 0; r < csize; ++r) s += ld_cluster_f32(smem_u32(P + i * kRows6 + row_in), (uint32_t)r);
                if (row < L.n) Y[(size_t)i * L.n + row] = __float2half_rn(s);
            }
        }
        cluster_sync_all();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(kTmemCols6) : "memory");
}

template <int NPAD>
ptqtp_status launch_n6(const Layout3& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int csize,
                       cudaStream_t st) {
    ptqtp_status s = configure_once<gemm6_kernel<NPAD>>();
    if (s != PTQTP_OK) return s;
    int* status_word = nullptr;                           // shared with the GEMV kernels (ptqtp_kernel_status)
    if (gemv_status_word(&status_word) != PTQTP_OK) return PTQTP_ERR_CUDA;
    const int blocks = (L.nrb + kBlockTiles6 - 1) / kBlockTiles6;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks * csize);
    cfg.blockDim = dim3(kThreads6);
    cfg.dynamicSmemBytes = Smem6<NPAD>::total;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm6_kernel<NPAD>, L, static_cast<const unsigned char*>(packed),
                                       reinterpret_cast<const __half*>(X), reinterpret_cast<__half*>(Y), m, csize,
                                       wait_poll_limit(), take_injected_wait_failure() ? 1 : 0, status_word);
    if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

}  // namespace

// 1 <= m <= 64 rows of X (16-byte aligned) on format 3.  ksplit: CTAs of a cluster that share the columns of a row
// block (1, 2, 4 or 8; 0 = library choice: enough CTAs to occupy the device, no more than there are superblocks).
ptqtp_status launch_gemm6(const Layout3& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int ksplit,
                          cudaStream_t st) {
    if (m < 1 || m > 64) return PTQTP_ERR_SHAPE;
    if (ksplit != 0 && ksplit != 1 && ksplit != 2 && ksplit != 4 && ksplit != 8) return PTQTP_ERR_CONFIG;
    if (ksplit == 0) {
        const int blocks = (L.nrb + kBlockTiles6 - 1) / kBlockTiles6;
        ksplit = 1;
        while (ksplit < 8 && blocks * ksplit < sm_count() && 2 * ksplit <= L.sbs) ksplit *= 2;
    }
    const int npad = (m + 15) / 16 * 16;
    switch (npad) {
        case 16: return launch_n6<16>(L, packed, m, X, Y, ksplit, st);
        case 32: return launch_n6<32>(L, packed, m, X, Y, ksplit, st);
        case 48: return launch_n6<48>(L, packed, m, X, Y, ksplit, st);
        default: return launch_n6<64>(L, packed, m, X, Y, ksplit, st);
    }
}

}  // namespace ptqtp
