// Dual-trit-plane layer for up to 64 activation rows per launch on packed format 3 (the batch-1 layout), on the
// fifth-generation tensor cores (tcgen05.mma, accumulators in tensor memory):
//     Y[m] = alpha1 (.) (T1 X[m]) + alpha2 (.) (T2 X[m]),   m < M <= 64.
//
// A CTA of 128 threads owns 128 weight rows (8 tiles per superblock, contiguous in the blob); thread i is row i of
// every MMA.  Per scale group of 128 columns:
//   * each thread turns its row's 2-bit codes into fp16 trits (-1, 0, +1) with a byte-permute lookup -- the code in
//     the high nibble of a selector byte picks the high byte of the fp16 value, the low nibble picks a zero byte --
//     and writes them to tensor memory (tcgen05.st, one lane per row, 64 columns per plane): the A operand never
//     passes through shared memory;
//   * the activations of the group, fp16 as given (no quantisation), are the B operand: M rows padded to a multiple
//     of 16, in shared memory as K-major core matrices (8 rows x 16 bytes), fetched with 16-byte cp.async one group
//     ahead;
//   * one thread issues 16 MMAs of 128 x NPAD x 16 (8 k-steps for each plane) into two fp32 accumulators and commits
//     them to an mbarrier; the trits are exact in fp16, so each accumulator is the fp32 sum of +-x;
//   * every thread reads its lane of both accumulators (tcgen05.ld) and adds alpha1 * d1 + alpha2 * d2 in fp32 to its
//     NPAD running sums.
// Two CTAs share an SM (256 of the 512 tensor-memory columns and about 100 KB of shared memory each), so one CTA's
// decode and epilogue run under the other's MMAs.  Matrices with few rows split K over a cluster of up to 8 CTAs;
// the partial sums meet in distributed shared memory and are added in rank order (no atomics, reproducible).
//
// Waits on mbarriers are bounded: a wait that gives up marks the launch failed (status word, NaN rows), the CTA
// still takes part in the cluster barriers and frees its tensor memory.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kThreads6 = 128;
constexpr int kBlockTiles6 = 8;                        // tiles per CTA and superblock: 128 weight rows
constexpr int kStage6 = kBlockTiles6 * kTile3;         // 34816 bytes
constexpr int kStages6 = 2;
constexpr int kTmemCols6 = 256;                        // D: columns 0 .. 2 NPAD - 1; A: columns 128 .. 255
constexpr int kACol6 = 128;
constexpr uint32_t kTritLut6 = 0x003C00BCu;            // byte q of the table = high byte of fp16(q - 1); byte 3 = 0

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
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Bulk copy global -> this CTA's shared memory, completion counted in bytes on an mbarrier (no multicast).
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, 0, %2;" : "=r"(d) : "r"(a), "r"(sel));
    return d;
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
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
    static constexpr int bar_off = x_off + 2 * x_buf;          // mbarriers: one per stage, one for the MMAs; then the
    static constexpr int total = bar_off + 64;                 // word that receives the tensor-memory address
};

// Queue the copies of activation group gg (columns 128 gg ..) into an activation buffer: chunk kc (8 columns) of
// row n goes to kc * NPAD * 16 + n * 16.  Adjacent threads take the two halves of a 32-byte sector.
template <int NPAD>
__device__ __forceinline__ void fetch_x(const __half* __restrict__ X, int k, int m, int gg, uint32_t buf) {
#pragma unroll
    for (int q0 = 0; q0 < 16 * NPAD; q0 += kThreads6) {
        const int q = q0 + (int)threadIdx.x;
        const int n = (q >> 1) % NPAD, kc = 2 * ((q >> 1) / NPAD) + (q & 1);
        if (n < m) cp_async16(buf + kc * (NPAD * 16) + n * 16, X + (size_t)n * k + 128 * gg + 8 * kc);
    }
}

template <int NPAD>
__global__ void __launch_bounds__(kThreads6, 2)
gemm6_kernel(Layout3 L, const unsigned char* __restrict__ packed, const __half* __restrict__ X, __half* __restrict__ Y,
             int m, int csize, int spin_limit, int inject, int* status_word) {
    extern __shared__ __align__(128) unsigned char smem[];
    using SM = Smem6<NPAD>;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + SM::bar_off);
    uint64_t& mma_bar = full_bar[kStages6];
    uint32_t& tmem_slot = *reinterpret_cast<uint32_t*>(full_bar + kStages6 + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int crank = (int)blockIdx.x % csize, blk = (int)blockIdx.x / csize;
    const int rb0 = blk * kBlockTiles6;
    const int tiles = min(kBlockTiles6, L.nrb - rb0);
    const uint32_t stage_bytes = (uint32_t)tiles * kTile3;
    const int groups = L.k / 128;
    // this CTA's superblocks: a balanced split of the superblocks over the cluster
    const int sb_base = L.sbs / csize, sb_rem = L.sbs % csize;
    const int sb_lo = crank * sb_base + min(crank, sb_rem);
    const int sb_hi = sb_lo + sb_base + (crank < sb_rem ? 1 : 0);
    const unsigned char* codes = packed + L.codes_off;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(kTmemCols6) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < kStages6; ++s) mbar_init(&full_bar[s], 1);
        mbar_init(&mma_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // rows m .. NPAD - 1 of the activation buffers stay zero
    for (int i = tid; i < 2 * SM::x_buf / 16; i += kThreads6)
        reinterpret_cast<uint4*>(smem + SM::x_off)[i] = make_uint4(0u, 0u, 0u, 0u);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot;
    const uint32_t tlane = tbase + ((uint32_t)(warp * 32) << 16);       // this warp's 32 lanes
    const uint32_t xbuf0 = smem_u32(smem + SM::x_off);

    if (tid == 0) {
        for (int s = 0; s < kStages6 && sb_lo + s < sb_hi; ++s) {
            mbar_expect_tx(smem_u32(&full_bar[s]), stage_bytes);
            bulk_copy_g2s(smem_u32(smem + s * kStage6), codes + tile_offset3(L, rb0, sb_lo + s), stage_bytes,
                          smem_u32(&full_bar[s]));
        }
    }
    int gg = 4 * sb_lo;                                  // global group index of the pass at hand
    const int gg_end = min(4 * sb_hi, groups);
    if (gg < gg_end) fetch_x<NPAD>(X, L.k, m, gg, xbuf0);
    cp_async_commit();

    // thread -> (tile of the block, row pair g of the tile, member of the pair)
    const int tl = 2 * warp + (lane >> 4), g = (lane >> 1) & 7, mem = lane & 1;
    const uint32_t sh = 4u - 4u * (uint32_t)mem;         // brings the row's plane-1 code to bits 4-5 of each byte
    const uint32_t idesc = (1u << 4) | ((uint32_t)(NPAD >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    float y[NPAD];
#pragma unroll
    for (int i = 0; i < NPAD; ++i) y[i] = 0.f;
    bool failed = false;
    int pass = 0;

    for (; gg < gg_end; ++gg, ++pass) {
        const int sb = gg >> 2, G = gg & 3, sl = sb - sb_lo, stage = sl % kStages6;
        const unsigned char* tile = smem + stage * kStage6 + tl * kTile3;
        if (G == 0) {
            const bool ok = !(inject && pass == 0) &&
                            mbar_wait_bounded(smem_u32(&full_bar[stage]), (uint32_t)(sl / kStages6) & 1u, spin_limit);
            if (!__syncthreads_and(ok)) { failed = true; break; }
        }
        // (1) the next group's activations into the other buffer (its last reader, the MMAs two passes back, is done)
        if (gg + 1 < gg_end) fetch_x<NPAD>(X, L.k, m, gg + 1, xbuf0 + ((pass + 1) & 1) * SM::x_buf);
        cp_async_commit();

        // (2) decode this row's 128 columns of both planes into tensor memory
        const int u = G & 1, h = G >> 1;
        const __half2 alpha = *reinterpret_cast<const __half2*>(tile + kTileCodes3 + 8 * (4 * g + G) + 4 * mem);
        // (tiles past the matrix hold whatever the stage held: the lookup yields finite values for any bits, such a
        // row only feeds its own accumulator lane and is never stored; the stores are warp-wide instructions)
        {
#pragma unroll
            for (int o = 0; o < 4; ++o) {
                uint32_t r1[16], r2[16];
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
#pragma unroll
                    for (int tt = 0; tt < 2; ++tt) {
                        const uint4 v = *reinterpret_cast<const uint4*>(tile + (2 * o + cc) * 512 + (4 * g + 2 * u + tt) * 16);
                        const uint32_t w[2] = {h ? v.y : v.x, h ? v.w : v.z};
#pragma unroll
                        for (int s = 0; s < 2; ++s) {
                            const uint32_t c = w[s] << sh;
                            const uint32_t s1 = (c & 0x30303030u) | 0x03030303u;
                            const uint32_t s2 = ((c >> 2) & 0x30303030u) | 0x03030303u;
                            const int wq = 4 * cc + 2 * s + tt;             // word of the octet: columns 4 wq .. 4 wq + 3
                            r1[2 * wq] = prmt(kTritLut6, s1);
                            r1[2 * wq + 1] = prmt(kTritLut6, s1 >> 16);
                            r2[2 * wq] = prmt(kTritLut6, s2);
                            r2[2 * wq + 1] = prmt(kTritLut6, s2 >> 16);
                        }
                    }
                }
                tmem_st16(tlane + kACol6 + 16 * o, r1);
                tmem_st16(tlane + kACol6 + 64 + 16 * o, r2);
            }
        }
        // (3) activations of this group landed; operands visible to the tensor core
        cp_async_wait_all_but_one();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc_fence_before();
        __syncthreads();
        // (4) one thread issues the MMAs; the stage is free once the last group of its superblock is decoded
        if (tid == 0) {
            tc_fence_after();
            const uint32_t xb = xbuf0 + (pass & 1) * SM::x_buf;
#pragma unroll
            for (int p = 0; p < 2; ++p)
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    mma_f16_ts(tbase + p * NPAD, tbase + kACol6 + 64 * p + 8 * j,
                               smem_desc(xb + 2 * j * (NPAD * 16), NPAD * 16, 128), idesc, j > 0 ? 1u : 0u);
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                         ::"r"(smem_u32(&mma_bar)) : "memory");
            if ((G == 3 || gg + 1 == gg_end) && sb + kStages6 < sb_hi) {
                mbar_expect_tx(smem_u32(&full_bar[stage]), stage_bytes);
                bulk_copy_g2s(smem_u32(smem + stage * kStage6), codes + tile_offset3(L, rb0, sb + kStages6), stage_bytes,
                              smem_u32(&full_bar[stage]));
            }
        }
        // (5) wait for the MMAs, (6) scale epilogue
        {
            const bool ok = mbar_wait_bounded(smem_u32(&mma_bar), (uint32_t)pass & 1u, spin_limit);
            if (!__syncthreads_and(ok)) { failed = true; break; }
        }
        tc_fence_after();
        const float a1 = __low2float(alpha), a2 = __high2float(alpha);
#pragma unroll
        for (int c0 = 0; c0 < NPAD; c0 += 16) {
            uint32_t d1[16], d2[16];
            tmem_ld16(tlane + c0, d1);
            tmem_ld16(tlane + NPAD + c0, d2);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int i = 0; i < 16; ++i)
                y[c0 + i] = fmaf(a1, __uint_as_float(d1[i]), fmaf(a2, __uint_as_float(d2[i]), y[c0 + i]));
        }
        tc_fence_before();
    }
    cp_async_wait_all();

    if (failed) {
        if (tid == 0) atomicExch(status_word, (int)PTQTP_ERR_CUDA);
        // a copy whose wait gave up may still be in flight: give it time to land before the memory is reused
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
#pragma unroll
        for (int i = 0; i < NPAD; ++i) y[i] = __int_as_float(0x7fc00000);
    }
    const int row = 16 * rb0 + tid;
    if (csize == 1) {
        if (row < L.n) {
#pragma unroll
            for (int i = 0; i < NPAD; ++i)
                if (i < m) Y[(size_t)i * L.n + row] = __float2half_rn(y[i]);
        }
    } else {
        // partial sums of the cluster meet in shared memory; rank r adds its share of the columns in rank order
        __syncthreads();
        float* P = reinterpret_cast<float*>(smem);
#pragma unroll
        for (int i = 0; i < NPAD; ++i) P[i * kThreads6 + tid] = y[i];
        cluster_sync_all();
        const int per = NPAD / csize;
        for (int i = crank * per; i < (crank + 1) * per && i < m; ++i) {
            float s = 0.f;
            for (int r = 0; r < csize; ++r) s += ld_cluster_f32(smem_u32(P + i * kThreads6 + tid), (uint32_t)r);
            if (row < L.n) Y[(size_t)i * L.n + row] = __float2half_rn(s);
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
