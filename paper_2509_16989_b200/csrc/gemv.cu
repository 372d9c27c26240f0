// Batch-1 dual-trit-plane GEMV for sm_100a:  y = alpha1 (.) (T1 x) + alpha2 (.) (T2 x).
//
// The work is organised around the byte stream of the packed planes:
//   * a warp owns R output rows and walks K in 1024-column slices; per slice and row it issues ONE
//     128-bit load per lane (512 contiguous bytes per warp: both planes of 1024 columns of that row)
//     and keeps a ring of D such steps in flight, across tile boundaries, so HBM latency is covered
//     by the warp's own loads; the first loads are issued before x is staged;
//   * x is staged once per CTA into shared memory, already arranged in the (pair, bit-position)
//     order the decode consumes, so the inner loop reads it with conflict-free 128-bit LDS and
//     reuses it for both planes and all R rows;
//   * decode is one LOP3 per two trits: a code q = trit + 1 in {0,1,2} sitting in the fp16 mantissa
//     field IS the fp16 subnormal q * 2^(p-24) (p = its bit position), for both halves of the word
//     at once.  The activation paired with bit position p is pre-multiplied by 2^(s-p), so the
//     product code * x' equals q * x * 2^(s-24) exactly, whatever the position;
//   * accumulation (template ARITH): 0 = every product is added into an fp32 accumulator by a
//     mixed-precision FMA (fp16 operands, fp32 accumulate): additions only carry fp32 rounding;
//     1 = HFMA2 chains of 4 (8 columns) flushed into fp32 by mixed-precision adds; 2 = chains of 8;
//   * sum_j t_j x_j = sum_j q_j x_j - sum_j x_j: every accumulator starts at minus the lane block's
//     sum of x (staged with x), so the +1 offset of the codes costs no instruction;
//   * the group scales (the only multiplies of the method) are applied in fp32 per lane, whose 32
//     columns lie inside one 128-column group; rows are reduced across lanes by warp shuffles and,
//     when K is split across the warps of a CTA, through shared memory.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;

__device__ __forceinline__ __half2 as_h2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }
__device__ __forceinline__ uint32_t as_u32(__half2 v) { return *reinterpret_cast<uint32_t*>(&v); }

// acc32 += lo(h) + hi(h): two mixed-precision adds (fp16 operand, fp32 accumulate).
__device__ __forceinline__ float flush(float acc, __half2 h) {
    const uint32_t u = as_u32(h);
    const unsigned short lo = (unsigned short)(u & 0xffffu), hi = (unsigned short)(u >> 16);
    asm("add.f32.f16 %0, %1, %0;" : "+f"(acc) : "h"(lo));
    asm("add.f32.f16 %0, %1, %0;" : "+f"(acc) : "h"(hi));
    return acc;
}

// acc32 += lo(m)*lo(x) + hi(m)*hi(x): two mixed-precision FMAs (fp16 operands, fp32 accumulate).
__device__ __forceinline__ float mixed_fma2(float acc, uint32_t m, uint32_t x) {
    unsigned short ml, mh, xl, xh;
    asm("mov.b32 {%0,%1}, %2;" : "=h"(ml), "=h"(mh) : "r"(m));
    asm("mov.b32 {%0,%1}, %2;" : "=h"(xl), "=h"(xh) : "r"(x));
    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc) : "h"(ml), "h"(xl));
    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc) : "h"(mh), "h"(xh));
    return acc;
}

// acc32 += sum over the 16 columns of one code word of q * x' (x' pre-scaled per bit position).
template <int ARITH>
__device__ __forceinline__ float word_dot(uint32_t w, const uint32_t* X, float acc32) {
    const uint32_t u = w >> 10;
    const uint32_t m[8] = {w & 0x00030003u, w & 0x000C000Cu, w & 0x00300030u, w & 0x00C000C0u,
                           w & 0x03000300u, u & 0x00030003u, u & 0x000C000Cu, u & 0x00300030u};
    if (ARITH == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) acc32 = mixed_fma2(acc32, m[i], X[i]);
        return acc32;
    } else if (ARITH == 1) {
        __half2 a = __hmul2(as_h2(m[0]), as_h2(X[0]));
        __half2 b = __hmul2(as_h2(m[4]), as_h2(X[4]));
#pragma unroll
        for (int i = 1; i < 4; ++i) {
            a = __hfma2(as_h2(m[i]), as_h2(X[i]), a);
            b = __hfma2(as_h2(m[4 + i]), as_h2(X[4 + i]), b);
        }
        return flush(flush(acc32, a), b);
    } else {
        __half2 a = __hmul2(as_h2(m[0]), as_h2(X[0]));
#pragma unroll
        for (int i = 1; i < 8; ++i) a = __hfma2(as_h2(m[i]), as_h2(X[i]), a);
        return flush(acc32, a);
    }
}

// Stage x for the whole K into shared memory in decode order.
//   xs   : [slice][4][32 lanes] uint4  -- 16 half2 per lane block: word w (0,1), bit position i (0..7):
//          (x[16w+i], x[16w+8+i]) * 2^(s - pos(i)),  pos(i) = 2i for i <= 4, 2i-10 for i >= 5
//   meta : [slice][32 lanes] float2    -- (2^(24-s), -2^(s-24) * sum of the lane block's 32 activations)
// s is chosen per lane block so that max|x| * 2^s lies in [2^14, 2^15): no overflow, full precision.
// Two adjacent threads share a lane block (16 columns each).
__device__ __forceinline__ void stage_x(const Layout& L, const __half* __restrict__ x, uint4* xs, float2* meta) {
    const int half_blocks = L.slices * 64;
    for (int hb = threadIdx.x; hb < half_blocks; hb += kThreads) {
        const int c = hb >> 1, w = hb & 1;
        const int k0 = c * kLaneK + 16 * w;
        alignas(16) __half xv[16];
        if (k0 < L.k) {
            const uint4* p = reinterpret_cast<const uint4*>(x + k0);
            reinterpret_cast<uint4*>(xv)[0] = __ldg(p);
            reinterpret_cast<uint4*>(xv)[1] = __ldg(p + 1);
        } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) xv[e] = __ushort_as_half(0);
        }
        float xf[16];
        float mx = 0.f, sum = 0.f;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            xf[e] = __half2float(xv[e]);
            mx = fmaxf(mx, fabsf(xf[e]));
            sum += xf[e];
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        // exponent of the block maximum; fp16 inputs keep it within [-24, 15] (14 if the block is all zero)
        const int ex = mx > 0.f ? (int)((__float_as_uint(mx) >> 23) & 0xffu) - 127 : 14;
        const int s = 14 - min(max(ex, -24), 15);
        alignas(16) __half2 out[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int pos = i <= 4 ? 2 * i : 2 * i - 10;
            const float sc = __uint_as_float((uint32_t)(127 + s - pos) << 23);
            out[i] = __floats2half2_rn(xf[i] * sc, xf[8 + i] * sc);
        }
        const int slice = c >> 5, lane = c & 31;
        xs[(slice * 4 + 2 * w) * 32 + lane] = reinterpret_cast<uint4*>(out)[0];
        xs[(slice * 4 + 2 * w + 1) * 32 + lane] = reinterpret_cast<uint4*>(out)[1];
        if (w == 0)
            meta[c] = make_float2(__uint_as_float((uint32_t)(127 + 24 - s) << 23),
                                  -sum * __uint_as_float((uint32_t)(127 + s - 24) << 23));
    }
}

template <int R>
struct Step {
    uint4 w[R];
    uint32_t a[R];
};

template <int R, int WS, int D, int ARITH>
__global__ void __launch_bounds__(kThreads)
gemv_kernel(Layout L, const unsigned char* __restrict__ packed, const __half* __restrict__ x,
            __half* __restrict__ y, int tiles) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint4* xs = reinterpret_cast<uint4*>(smem);
    float2* meta = reinterpret_cast<float2*>(smem + (size_t)L.slices * 2048);
    float* red = reinterpret_cast<float*>(smem + (size_t)L.slices * (2048 + 256));   // [kWarps][R]

    constexpr int kRowsPerCta = R * (kWarps / WS);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ks = warp % WS, rsub = warp / WS;
    const int nsl = L.slices / WS;                      // launcher guarantees slices % WS == 0
    const int s_begin = ks * nsl, s_end = s_begin + nsl;
    const uint4* codes = reinterpret_cast<const uint4*>(packed + L.codes_off) + lane;
    const uint32_t* scales = reinterpret_cast<const uint32_t*>(packed + L.scales_off) + (lane >> 2);

    // load cursor (runs D steps ahead of the compute cursor)
    int ltile = blockIdx.x, ls = s_begin;
    Step<R> ring[D];
    auto issue = [&](Step<R>& st) {
        if (ltile < tiles) {
            const int row0 = ltile * kRowsPerCta + rsub * R;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int row = min(row0 + r, L.n - 1);        // rows past N re-read the last row; never stored
                st.w[r] = __ldcs(codes + ((size_t)row * L.slices + ls) * 32);
                st.a[r] = __ldcs(scales + (size_t)row * L.groups_pad + ls * kGroupsPerSlice);
            }
            if (++ls == s_end) { ls = s_begin; ltile += gridDim.x; }
        }
    };
#pragma unroll
    for (int d = 0; d < D; ++d) issue(ring[d]);

    stage_x(L, x, xs, meta);
    __syncthreads();

    int ctile = blockIdx.x, cs = s_begin;
    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.f;

    while (ctile < tiles) {
#pragma unroll
        for (int d = 0; d < D; ++d) {
            if (ctile >= tiles) break;
            const Step<R> cur = ring[d];
            issue(ring[d]);
            uint32_t X[16];
#pragma unroll
            for (int v = 0; v < 4; ++v)
                *reinterpret_cast<uint4*>(&X[4 * v]) = xs[(cs * 4 + v) * 32 + lane];
            const float2 m = meta[cs * 32 + lane];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                // accumulators start at -sum(x): sum_j q_j x_j - sum_j x_j = sum_j t_j x_j (2^(s-24) units)
                float s1 = word_dot<ARITH>(cur.w[r].x, X, m.y);
                s1 = word_dot<ARITH>(cur.w[r].y, X + 8, s1);
                float s2 = word_dot<ARITH>(cur.w[r].z, X, m.y);
                s2 = word_dot<ARITH>(cur.w[r].w, X + 8, s2);
                const float2 a = __half22float2(as_h2(cur.a[r]));
                acc[r] = fmaf(m.x, fmaf(a.y, s2, a.x * s1), acc[r]);   // + 2^(24-s) (alpha1 S1 + alpha2 S2)
            }
            if (++cs == s_end) {
                // tile finished: reduce each row over the lanes (and over the K-splitting warps)
                const int row0 = ctile * kRowsPerCta + rsub * R;
#pragma unroll
                for (int r = 0; r < R; ++r) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
                }
                if (WS == 1) {
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < R; ++r)
                            if (row0 + r < L.n) y[row0 + r] = __float2half_rn(acc[r]);
                    }
                } else {
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < R; ++r) red[warp * R + r] = acc[r];
                    }
                    __syncthreads();
                    if (ks == 0 && lane < R) {
                        float t = 0.f;
#pragma unroll
                        for (int q = 0; q < WS; ++q) t += red[(rsub * WS + q) * R + lane];
                        if (row0 + lane < L.n) y[row0 + lane] = __float2half_rn(t);
                    }
                    __syncthreads();
                }
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] = 0.f;
                cs = s_begin;
                ctile += gridDim.x;
            }
        }
    }
}

template <int R, int WS, int D, int ARITH>
ptqtp_status launch_one(const Layout& L, const void* packed, const uint16_t* x, uint16_t* y, int ctas_per_sm,
                        cudaStream_t st) {
    constexpr int kRowsPerCta = R * (kWarps / WS);
    if (L.slices % WS != 0) return PTQTP_ERR_CONFIG;
    const int tiles = (L.n + kRowsPerCta - 1) / kRowsPerCta;
    const size_t smem = (size_t)L.slices * (2048 + 256) + kWarps * R * sizeof(float);
    if (smem > 227 * 1024) return PTQTP_ERR_SHAPE;
    auto kern = gemv_kernel<R, WS, D, ARITH>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    }
    int grid = ctas_per_sm * sm_count();
    if (grid > tiles) grid = tiles;
    kern<<<grid, kThreads, smem, st>>>(L, static_cast<const unsigned char*>(packed),
                                       reinterpret_cast<const __half*>(x), reinterpret_cast<__half*>(y), tiles);
    return check_launch();
}

}  // namespace

ptqtp_status launch_gemv(const Layout& L, const void* packed, const uint16_t* x, uint16_t* y, int rows_per_warp,
                         int k_split, int ctas_per_sm, int depth, int arith, cudaStream_t st) {
    // Library defaults: enough warps to fill the machine first, then more rows per warp.
    if (k_split == 0) {
        const long want = (long)sm_count() * 16;
        k_split = 1;
        while (k_split < 8 && (long)L.n * k_split < want && L.slices % (2 * k_split) == 0) k_split *= 2;
    }
    if (rows_per_warp == 0) {
        const long want = (long)sm_count() * 24;
        rows_per_warp = (long)L.n * k_split >= 2 * want ? 2 : 1;
    }
    if (ctas_per_sm == 0) ctas_per_sm = 4;
    if (depth == 0) depth = rows_per_warp == 1 ? 4 : 2;
    if (arith < 0) arith = 0;
    if (ctas_per_sm < 1 || ctas_per_sm > 32) return PTQTP_ERR_CONFIG;
#define PTQTP_CASE(RR, WW, DD, AA) \
    if (rows_per_warp == RR && k_split == WW && depth == DD && arith == AA) \
        return launch_one<RR, WW, DD, AA>(L, packed, x, y, ctas_per_sm, st);
#define PTQTP_CASES_A(RR, WW, DD) PTQTP_CASE(RR, WW, DD, 0) PTQTP_CASE(RR, WW, DD, 1) PTQTP_CASE(RR, WW, DD, 2)
#define PTQTP_CASES_W(RR, DD) \
    PTQTP_CASES_A(RR, 1, DD) PTQTP_CASES_A(RR, 2, DD) PTQTP_CASES_A(RR, 4, DD) PTQTP_CASES_A(RR, 8, DD)
    PTQTP_CASES_W(1, 2) PTQTP_CASES_W(1, 4) PTQTP_CASES_W(1, 8)
    PTQTP_CASES_W(2, 1) PTQTP_CASES_W(2, 2) PTQTP_CASES_W(2, 4)
    PTQTP_CASES_W(4, 1) PTQTP_CASES_W(4, 2)
#undef PTQTP_CASES_W
#undef PTQTP_CASES_A
#undef PTQTP_CASE
    return PTQTP_ERR_CONFIG;
}

}  // namespace ptqtp
