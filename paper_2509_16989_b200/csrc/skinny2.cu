// Small-batch dual-trit-plane GEMM for sm_100a on packed format 2:  Y[m,:] = layer(X[m,:]), 1 <= M <= 64.
//
// The planes are decoded once and reused for several batch rows, which the integer-dot-product decode of the
// batch-1 kernel cannot afford (its dp4a pipe is already the bound at M = 1).  Here the contraction runs on the
// tensor cores with int8 warp MMAs (mma.sync m16n8k32, u8 codes x s8 activations, s32 accumulators, measured
// 8 cycles per MMA per scheduler on sm_100):
//
//   * MMA rows.  A warp step covers four consecutive row pairs ("quad") of one 1024-column half slice.  MMA row
//     r = 4 * field + (row pair in quad): a lane (g = lane / 4, t = lane % 4) reads the code word of row pair
//     g % 4 and masks out field g / 4 (rows 0-7) and field 2 + g / 4 (rows 8-15); the byte-sized codes q * 4^f
//     are the u8 A operand as they stand.
//   * MMA k.  The k index is a summation index, so its 32 slots are assigned to columns freely: lane t owns the
//     16-column atom t of a 64-column lane block; one 128-bit shared-memory load of codes and one of activations
//     feed two MMAs.  Four MMAs (two lane blocks) complete one 128-column scale group.
//   * MMA n.  Column 2j is the high byte and column 2j + 1 the low byte of batch row j's block-fixed-point
//     activations (15-bit: X = 256 hi + lo with both bytes signed), so one MMA serves four batch rows; unused
//     columns read a row of zeros.
//   * After each scale group the s32 sums become fp32, are multiplied by the group's scales, the block scale of
//     x and 4^-f, and added to per-lane row sums; the two planes of a row sit in lanes 16 apart and meet in one
//     shuffle per slice.  Slices are summed through shared memory in fixed order (deterministic).
//   * The CTA / warp / slice decomposition, the cp.async ring and the programmatic dependent launch are those of
//     the batch-1 kernel, with half slices (1024 columns) in place of slices so that 16 warps fit; a ring slot
//     holds the four half units of a quad in a bank-conflict-free arrangement.
//   * At most 8 batch rows per pass (shared memory holds their activations for all K); larger M runs several
//     passes, re-reading the planes (from L2 when the matrix fits).
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kHalf = 1024;                  // columns per half slice
constexpr int kSI = 18;                      // 16-byte chunks between the atom rows i of a half unit in a ring slot
constexpr int kSU = 81;                      // chunks per half unit in a ring slot: 4 * 18 code chunks, 4 scale chunks, pad
constexpr int kScaleChunk = 72;              // first scale chunk of a half unit
constexpr int kQuadSlot = 4 * kSU * 16;      // bytes per ring slot (four half units)
constexpr int kSkinnyMaxWarps = 16;

__device__ __forceinline__ void cp16(void* dst_smem, const void* src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp8(void* dst_smem, const void* src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// c += A (16x32 u8, row) * B (32x8 s8, col)
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct SkinnySmem {
    size_t row_stride;       // bytes between activation rows: K + 64 (rows 16 apart in bank space)
    size_t meta_off, partial_off, ring_off, total;
};
__host__ __device__ inline SkinnySmem skinny_smem(int k, int slices, int mt, int mt_pad, int rows_cap, int warps, int depth) {
    SkinnySmem s;
    s.row_stride = (size_t)k + 64;
    s.meta_off = (size_t)(2 * mt + 1) * s.row_stride;                        // 2 byte planes per batch row + a zero row
    s.partial_off = s.meta_off + (size_t)mt_pad * (k / kGroup) * 8;
    s.ring_off = (s.partial_off + (size_t)rows_cap * mt * slices * 4 + 15) / 16 * 16;
    s.total = s.ring_off + (size_t)warps * depth * kQuadSlot;
    return s;
}

// Convert 8 activations of one batch row to 15-bit block fixed point (blocks of 128 columns, 16 threads each).
//   hi, lo : byte planes of this batch row;  meta : (2^-s as float bits, sum_j X_j) per block
__device__ __forceinline__ void convert_row8(uint4 raw, int col, bool valid, unsigned char* hi, unsigned char* lo,
                                             int2* meta) {
    const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
    const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t mxb = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const uint32_t a = rw[e] & 0x7fff7fffu;
        mxb = max(mxb, max(a & 0xffffu, a >> 16));
    }
#pragma unroll
    for (int o = 1; o < 16; o <<= 1) mxb = max(mxb, __shfl_xor_sync(0xffffffffu, mxb, o));
    int s = 0;
    if (mxb != 0u) {
        const int ef = (int)(mxb >> 10);
        const int ex = ef ? ef - 15 : (31 - __clz((int)mxb)) - 24;
        s = 13 - ex;                                   // block maximum in [2^13, 2^14): hi stays within [-64, 64]
    }
    const float scale = __uint_as_float((uint32_t)(127 + s) << 23);
    int H[8], Lo[8];
    int sum = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 v = __half22float2(h2[e]);
        const int X0 = __float_as_int(fmaf(v.x, scale, 12582912.f)) - 0x4B400000;
        const int X1 = __float_as_int(fmaf(v.y, scale, 12582912.f)) - 0x4B400000;
        sum += X0 + X1;
        Lo[2 * e] = (int)(signed char)(X0 & 0xff);
        Lo[2 * e + 1] = (int)(signed char)(X1 & 0xff);
        H[2 * e] = (X0 - Lo[2 * e]) >> 8;
        H[2 * e + 1] = (X1 - Lo[2 * e + 1]) >> 8;
    }
#pragma unroll
    for (int o = 1; o < 16; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    uint32_t hw[2], lw[2];
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        lw[w] = __byte_perm(__byte_perm(Lo[4 * w], Lo[4 * w + 1], 0x0040), __byte_perm(Lo[4 * w + 2], Lo[4 * w + 3], 0x0040), 0x5410);
        hw[w] = __byte_perm(__byte_perm(H[4 * w], H[4 * w + 1], 0x0040), __byte_perm(H[4 * w + 2], H[4 * w + 3], 0x0040), 0x5410);
    }
    if (valid) {
        *reinterpret_cast<uint2*>(hi + col) = make_uint2(hw[0], hw[1]);
        *reinterpret_cast<uint2*>(lo + col) = make_uint2(lw[0], lw[1]);
        if (((col >> 3) & 15) == 0) meta[col >> 7] = make_int2((int)((uint32_t)(127 - s) << 23), sum);
    }
}

// NT = MMA n-tiles per pass (4 batch rows each); mt = batch rows of this pass (<= 4 NT).
template <int NT>
__global__ void __launch_bounds__(kSkinnyMaxWarps * 32, 1)
skinny2_kernel(Layout2 L, const unsigned char* __restrict__ packed, const __half* __restrict__ X, __half* __restrict__ Y,
               int mt, int rows_cap) {
    extern __shared__ __align__(16) unsigned char smem[];
    asm volatile("griddepcontrol.launch_dependents;");

    const int warps = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tig = lane & 3, u = g & 3, plane = g >> 2;
    const int S = (L.k + kHalf - 1) / kHalf;                       // half slices
    const int ngroups = L.k / kGroup;
    const SkinnySmem sm = skinny_smem(L.k, S, mt, 4 * NT, rows_cap, warps, 2);
    unsigned char* xq = smem;                                           // rows 2j (hi), 2j+1 (lo), then a zero row
    int2* meta = reinterpret_cast<int2*>(smem + sm.meta_off);           // [4 NT][K/128]
    float* partial = reinterpret_cast<float*>(smem + sm.partial_off);   // [rows_cap][mt][S]
    unsigned char* ring = smem + sm.ring_off + (size_t)warp * 2 * kQuadSlot;

    // this CTA's quads of row pairs, and this warp's share of their half slices
    const int nq = (L.nrp + 3) / 4;
    const int q0 = (int)((long long)blockIdx.x * nq / gridDim.x);
    const int q1 = (int)((long long)(blockIdx.x + 1) * nq / gridDim.x);
    const int Wc = min(S, warps), mw = warps / Wc;
    const int sl_lane = warp % Wc, wi = warp / Wc;
    const bool idle = wi >= mw;
    const int n_sl = idle ? 0 : (S - sl_lane + Wc - 1) / Wc;
    const int n_q = idle ? 0 : max(0, (q1 - q0 - wi + mw - 1) / mw);
    const unsigned char* codes = packed + L.codes_off;

    // producer: all lanes copy the four half units of a quad into a ring slot.  Lane -> (atom rows ip and
    // ip + 2, lane block ll) of each half unit.
    const int ip = lane >> 4, ll = lane & 15;
    int pt = n_q > 0 ? 0 : n_sl, pj = 0, pslot = 0;
    auto issue = [&]() {
        if (pt < n_sl) {
            const int hs = sl_lane + pt * Wc;                                  // half slice
            const int sl = hs >> 1, l0 = (hs & 1) * 16;
            const int A = sl == L.slices - 1 ? L.last_active : 32;             // lane blocks of the slice
            const int Ah = min(16, A - l0);                                    // ... of this half
            const int q = q0 + wi + pj * mw;
            unsigned char* dst = ring + pslot * kQuadSlot;
#pragma unroll
            for (int uu = 0; uu < 4; ++uu) {
                const int rp = min(4 * q + uu, L.nrp - 1);                     // row pairs past the end re-read the last one
                const unsigned char* src = codes + unit_offset(L, rp, sl);
                unsigned char* d = dst + uu * (kSU * 16);
                if (ll < Ah) {
                    cp16(d + (ip * kSI + ll) * 16, src + (ip * A + l0 + ll) * 16);
                    cp16(d + ((ip + 2) * kSI + ll) * 16, src + ((ip + 2) * A + l0 + ll) * 16);
                }
                if (lane < Ah / 2) cp8(d + kScaleChunk * 16 + lane * 8, src + A * 64 + (l0 / 2 + lane) * 8);
            }
            if (++pj == n_q) { pj = 0; ++pt; }
        }
        cp_commit();
        pslot ^= 1;
    };
    // The packed planes do not depend on earlier work of the stream: fill the ring, then wait for that work.
    issue();
    issue();
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // activations of this pass: block fixed point, two byte planes per batch row; unused rows/records are zero
    {
        const int tasks_per_row = L.k / 8;
        for (int base = (threadIdx.x & ~31); base < mt * tasks_per_row; base += blockDim.x) {      // warp-uniform
            // K/8 is a multiple of 16: a block's 16 threads always lie in one half warp and one batch row
            const int task = base + lane;
            const bool valid = task < mt * tasks_per_row;
            const int mi = valid ? task / tasks_per_row : 0, col = valid ? (task % tasks_per_row) * 8 : 0;
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (valid) raw = __ldg(reinterpret_cast<const uint4*>(X + (size_t)mi * L.k + col));
            convert_row8(raw, col, valid, xq + (size_t)(2 * mi) * sm.row_stride,
                         xq + (size_t)(2 * mi + 1) * sm.row_stride, meta + (size_t)mi * ngroups);
        }
        unsigned char* zrow = xq + (size_t)(2 * mt) * sm.row_stride;
        for (int i = threadIdx.x * 16; i < (int)sm.row_stride; i += blockDim.x * 16)
            *reinterpret_cast<uint4*>(zrow + i) = make_uint4(0u, 0u, 0u, 0u);
        for (int i = mt * ngroups + threadIdx.x; i < 4 * NT * ngroups; i += blockDim.x) meta[i] = make_int2(0, 0);
    }
    __syncthreads();

    // per-lane constants: masks of the two fields this lane extracts, their 4^-f, the B rows it reads
    const uint32_t maskA = 0x03030303u << (2 * plane), maskB = maskA << 4;       // fields plane and 2 + plane
    const float kA = plane ? 0.25f : 1.0f, kB = kA * 0.0625f;
    const int shA = 2 * plane, shB = shA + 4;
    const uint32_t alpha_sel = plane ? 0x7632u : 0x5410u;                        // (alpha_plane[row 0], alpha_plane[row 1])
    uint32_t brow[NT], mrow[NT];                                                 // shared-memory byte offsets
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int n = 8 * nt + g;
        brow[nt] = (uint32_t)((size_t)(n < 2 * mt ? n : 2 * mt) * sm.row_stride) + 16 * tig;
        mrow[nt] = (uint32_t)sm.meta_off + (uint32_t)(4 * nt + tig) * ngroups * 8;
    }
    const uint32_t unit_off = (uint32_t)(ring - smem) + u * (kSU * 16);

    int cslot = 0;
    for (int t = 0; t < n_sl; ++t) {
        const int hs = sl_lane + t * Wc;
        const int sl = hs >> 1, l0 = (hs & 1) * 16;
        const int A = sl == L.slices - 1 ? L.last_active : 32;
        const int groups_here = min(16, A - l0) / 2;
        for (int j = 0; j < n_q; ++j) {
            cp_wait<1>();
            __syncwarp();
            const unsigned char* unit = smem + unit_off + cslot * kQuadSlot;
            const unsigned char* cptr = unit + (tig * kSI) * 16;
            const unsigned char* sptr = unit + kScaleChunk * 16;
            const unsigned char* xptr[NT];
            const unsigned char* mptr[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                xptr[nt] = smem + brow[nt] + hs * kHalf;
                mptr[nt] = smem + mrow[nt] + hs * 64;                  // 8 groups of 8 bytes per half slice
            }
            float yA[NT], yB[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) { yA[nt] = 0.f; yB[nt] = 0.f; }
            for (int gl = 0; gl < groups_here; ++gl) {                 // one 128-column scale group per iteration
                int c[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) { c[nt][0] = 0; c[nt][1] = 0; c[nt][2] = 0; c[nt][3] = 0; }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint4 cw = *reinterpret_cast<const uint4*>(cptr + h * 16);
                    uint4 xb[NT];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) xb[nt] = *reinterpret_cast<const uint4*>(xptr[nt] + h * 64);
                    const uint32_t a0 = cw.x & maskA, a1 = cw.x & maskB, a2 = cw.y & maskA, a3 = cw.y & maskB;
                    const uint32_t e0 = cw.z & maskA, e1 = cw.z & maskB, e2 = cw.w & maskA, e3 = cw.w & maskB;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        mma_u8s8(c[nt], a0, a1, a2, a3, xb[nt].x, xb[nt].y);
                        mma_u8s8(c[nt], e0, e1, e2, e3, xb[nt].z, xb[nt].w);
                    }
                }
                // scale epilogue of the group: (alpha of this lane's plane for row 0, row 1) of row pair u
                const uint2 sc = *reinterpret_cast<const uint2*>(sptr);
                const uint32_t apair = __byte_perm(sc.x, sc.y, alpha_sel);
                const float2 al = __half22float2(*reinterpret_cast<const __half2*>(&apair));
                const float wA = al.x * kA, wB = al.y * kB;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int2 rec = *reinterpret_cast<const int2*>(mptr[nt]);       // (2^-s, sum X) of batch row 4 nt + tig
                    const float cm = __int_as_float(rec.x);
                    const int QA = (c[nt][0] << 8) + c[nt][1] - (rec.y << shA);
                    const int QB = (c[nt][2] << 8) + c[nt][3] - (rec.y << shB);
                    yA[nt] = fmaf(cm * wA, (float)QA, yA[nt]);
                    yB[nt] = fmaf(cm * wB, (float)QB, yB[nt]);
                    xptr[nt] += 128;
                    mptr[nt] += 8;
                }
                cptr += 32;
                sptr += 8;
            }
            // every lane has consumed the slot: refill it
            __syncwarp();
            issue();
            cslot ^= 1;
            // the two planes of a row are 16 lanes apart
            const int ql = wi + j * mw;                          // quad index within the CTA
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const float rA = yA[nt] + __shfl_xor_sync(0xffffffffu, yA[nt], 16);
                const float rB = yB[nt] + __shfl_xor_sync(0xffffffffu, yB[nt], 16);
                const int mi = 4 * nt + tig;
                if (lane < 16 && mi < mt) {
                    float* p = partial + ((size_t)((ql * 4 + u) * 2) * mt + mi) * S + hs;
                    p[0] = rA;
                    p[(size_t)mt * S] = rB;
                }
            }
        }
    }
    cp_wait<0>();
    __syncthreads();
    const int rows = 8 * (q1 - q0);
    for (int idx = threadIdx.x; idx < rows * mt; idx += blockDim.x) {
        const int mi = idx / rows, r = idx % rows;
        const int row = 8 * q0 + r;
        float tsum = 0.f;
        for (int s = 0; s < S; ++s) tsum += partial[((size_t)r * mt + mi) * S + s];
        if (row < L.n) Y[(size_t)mi * L.n + row] = __float2half_rn(tsum);
    }
}

template <int NT>
ptqtp_status launch_nt(const Layout2& L, const void* packed, const uint16_t* X, uint16_t* Y, int mt, int grid, int warps,
                       int rows_cap, size_t smem, cudaStream_t st) {
    auto kern = skinny2_kernel<NT>;
    static thread_local size_t configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    if (smem > 48 * 1024 && smem > configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
        configured[dev] = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_enabled() ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, L, static_cast<const unsigned char*>(packed),
                                       reinterpret_cast<const __half*>(X), reinterpret_cast<__half*>(Y), mt, rows_cap);
    if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

}  // namespace

ptqtp_status launch_skinny2(const Layout2& L, const void* packed, int m, const uint16_t* X, uint16_t* Y,
                            cudaStream_t st) {
    const int S = (L.k + kHalf - 1) / kHalf;                       // half slices
    const int nq = (L.nrp + 3) / 4;
    const int grid = min(sm_count(), nq);
    const int rows_cap = 8 * ((nq + grid - 1) / grid);
    const size_t budget = 227 * 1024;
    // warps: a multiple of the slice count, at most 8; batch rows per pass: the most that fit, at most 8
    int warps = S <= kSkinnyMaxWarps ? S * (kSkinnyMaxWarps / S) : kSkinnyMaxWarps;
    int mt = min(m, 8);
    for (;;) {
        const int nt = mt > 4 ? 2 : 1;
        if (skinny_smem(L.k, S, mt, 4 * nt, rows_cap, warps, 2).total <= budget) break;
        if (mt > 1) { mt = mt > 4 ? 4 : mt / 2; continue; }
        if (warps > 1 && warps > S) { warps -= S <= kSkinnyMaxWarps ? S : 1; continue; }
        if (warps > 1) { --warps; continue; }
        return PTQTP_ERR_SHAPE;
    }
    for (int m0 = 0; m0 < m; m0 += mt) {
        const int cur = min(mt, m - m0);
        const int nt = cur > 4 ? 2 : 1;
        const size_t smem = skinny_smem(L.k, S, cur, 4 * nt, rows_cap, warps, 2).total;
        const uint16_t* Xp = X + (size_t)m0 * L.k;
        uint16_t* Yp = Y + (size_t)m0 * L.n;
        ptqtp_status s = nt == 1 ? launch_nt<1>(L, packed, Xp, Yp, cur, grid, warps, rows_cap, smem, st)
                                 : launch_nt<2>(L, packed, Xp, Yp, cur, grid, warps, rows_cap, smem, st);
        if (s != PTQTP_OK) return s;
    }
    return PTQTP_OK;
}

}  // namespace ptqtp
