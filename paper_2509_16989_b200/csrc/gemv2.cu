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
//   * A CTA owns a contiguous range of row pairs.  Warp w is bound to the 2048-column slice (w mod S) and keeps
//     that slice's X (32 registers per lane) for its whole life; lanes own 64 consecutive columns, so a lane's
//     four accumulator pairs (2 rows x 2 planes) see one scale group half and get the group's scales
//     (the method's only multiplies) in an fp32 epilogue.
//   * Each warp streams its slice units (2048 code bytes + 128 scale bytes, contiguous in HBM) through a
//     private shared-memory ring with cp.async, several units in flight, issued before x is staged.  A lane
//     reads back only bytes it copied itself, so no barrier is needed inside the stream.
//   * Rows are reduced over the lanes by shuffles, over the slices through shared memory in a fixed order
//     (deterministic), rounded once to fp16.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kSlot = 2048 + 256;          // ring slot: 128 atoms of 16 B + one 8-byte scale quad per lane

__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(void* dst_smem, const void* src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

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

// Convert x to block fixed point in shared memory.
//   xhi, xlo : [K/64 blocks][16 words]  bytes of hi_j / lo_j in column order
//   meta     : [K/64 blocks] (2^-s as float, sum_j X_j as int)
// Eight adjacent threads share a 64-column block (8 columns each).
__device__ __forceinline__ void stage_x(int K, const __half* __restrict__ x, uint32_t* xhi, uint32_t* xlo,
                                        int2* meta) {
    const int threads = blockDim.x;
    for (int wbase = (threadIdx.x & ~31) * 8; wbase < K; wbase += threads * 8) {     // warp-uniform loop
        const int base = wbase + (threadIdx.x & 31) * 8;
        uint4 raw = make_uint4(0u, 0u, 0u, 0u);
        if (base < K) raw = __ldg(reinterpret_cast<const uint4*>(x + base));
        const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
        float f[8];
        float mx = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 v = __half22float2(h2[e]);
            f[2 * e] = v.x;
            f[2 * e + 1] = v.y;
            mx = fmaxf(mx, fmaxf(fabsf(v.x), fabsf(v.y)));
        }
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        // exponent of the block maximum: fp16 inputs keep it within [-24, 15]
        int s = 0;
        if (mx > 0.f) {
            int ex = (int)((__float_as_uint(mx) >> 23) & 0xffu) - 127;
            ex = min(max(ex, -24), 15);
            s = 14 - ex;
        }
        const float scale = __uint_as_float((uint32_t)(127 + s) << 23);
        int X[8];
        int sum = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            X[e] = __float2int_rn(f[e] * scale);
            X[e] = min(max(X[e], -32767), 32767);
            sum += X[e];
        }
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        uint32_t hw[2], lw[2];
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            hw[w] = 0u;
            lw[w] = 0u;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int v = X[4 * w + b];
                hw[w] |= (uint32_t)((v >> 8) & 0xff) << (8 * b);
                lw[w] |= (uint32_t)(v & 0xff) << (8 * b);
            }
        }
        if (base < K) {
            const int blk = base >> 6, tt = (base >> 3) & 7;
            *reinterpret_cast<uint2*>(xhi + blk * 16 + 2 * tt) = make_uint2(hw[0], hw[1]);
            *reinterpret_cast<uint2*>(xlo + blk * 16 + 2 * tt) = make_uint2(lw[0], lw[1]);
            if (tt == 0) meta[blk] = make_int2((int)((uint32_t)(127 - s) << 23), sum);
        }
    }
}

template <int D>
__global__ void __launch_bounds__(512, 1)
gemv2_kernel(Layout2 L, const unsigned char* __restrict__ packed, const __half* __restrict__ x,
             __half* __restrict__ y, int rows_cap) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int nblk = L.k / kLane2;
    uint32_t* xhi = reinterpret_cast<uint32_t*>(smem);
    uint32_t* xlo = xhi + nblk * 16;
    int2* meta = reinterpret_cast<int2*>(xlo + nblk * 16);
    float* partial = reinterpret_cast<float*>(meta + nblk);                 // [rows_cap][slices]
    const int warps = blockDim.x >> 5;
    const size_t ring_off = ((size_t)nblk * 136 + (size_t)rows_cap * L.slices * 4 + 15) / 16 * 16;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* ring = smem + ring_off + (size_t)warp * D * kSlot;

    // this CTA's row pairs, and this warp's share of their slice units
    const int rp0 = (int)((long long)blockIdx.x * L.nrp / gridDim.x);
    const int rp1 = (int)((long long)(blockIdx.x + 1) * L.nrp / gridDim.x);
    const int S = L.slices;
    const int Wc = min(S, warps);                       // slice lanes among the warps
    const int m = warps / Wc;                           // warps sharing a slice lane
    const int sl_lane = warp % Wc, wi = warp / Wc;
    const bool idle = wi >= m;
    const int n_sl = idle ? 0 : (S - sl_lane + Wc - 1) / Wc;
    const int n_rp = idle ? 0 : max(0, (rp1 - rp0 - wi + m - 1) / m);
    const int total = n_sl * n_rp;
    const unsigned char* codes = packed + L.codes_off;

    // prefetch cursor
    int pt = 0, pj = 0, pq = 0;
    auto issue = [&](int slot) {
        if (pq < total) {
            const int sl = sl_lane + pt * Wc, rp = rp0 + wi + pj * m;
            const int active = sl == S - 1 ? L.last_active : 32;
            const unsigned char* src = codes + (size_t)rp * L.strip + (size_t)sl * kUnit2;
            unsigned char* dst = ring + slot * kSlot;
            if (lane < active) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    cp_async16(dst + (i * 32 + lane) * 16, src + ((size_t)i * active + lane) * 16);
                cp_async8(dst + 2048 + lane * 8, src + (size_t)active * 64 + (lane >> 1) * 8);
            }
            ++pq;
            if (++pj == n_rp) { pj = 0; ++pt; }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int d = 0; d < D; ++d) issue(d);

    stage_x(L.k, x, xhi, xlo, meta);
    __syncthreads();

    uint32_t xh[16], xl[16];
    float c = 0.f;
    int neg[4] = {0, 0, 0, 0};
    int ct = 0, cj = 0;
    bool live = false;
    for (int q = 0; q < total; ++q) {
        const int slot = q % D;
        const int sl = sl_lane + ct * Wc, rp = rp0 + wi + cj * m;
        if (cj == 0) {                                  // new slice: load this lane's X block
            const int active = sl == S - 1 ? L.last_active : 32;
            live = lane < active;
            const int blk = sl * 32 + (live ? lane : 0);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const uint4 a = *reinterpret_cast<const uint4*>(xhi + blk * 16 + 4 * v);
                const uint4 b = *reinterpret_cast<const uint4*>(xlo + blk * 16 + 4 * v);
                xh[4 * v] = a.x; xh[4 * v + 1] = a.y; xh[4 * v + 2] = a.z; xh[4 * v + 3] = a.w;
                xl[4 * v] = b.x; xl[4 * v + 1] = b.y; xl[4 * v + 2] = b.z; xl[4 * v + 3] = b.w;
            }
            const int2 mt = meta[blk];
            c = __int_as_float(mt.x);
#pragma unroll
            for (int f = 0; f < 4; ++f) neg[f] = -(mt.y << (2 * f));
        }
        cp_async_wait<D - 1>();
        const unsigned char* buf = ring + slot * kSlot;
        float y0 = 0.f, y1 = 0.f;
        if (live) {
            int ah[4] = {0, 0, 0, 0};
            int al[4] = {neg[0], neg[1], neg[2], neg[3]};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 cw = *reinterpret_cast<const uint4*>(buf + (i * 32 + lane) * 16);
                const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
                for (int ww = 0; ww < 4; ++ww) {
#pragma unroll
                    for (int f = 0; f < 4; ++f) {
                        const uint32_t mk = w[ww] & (0x03030303u << (2 * f));
                        ah[f] = dot_us(mk, xh[4 * i + ww], ah[f]);
                        al[f] = dot_uu(mk, xl[4 * i + ww], al[f]);
                    }
                }
            }
            const uint2 sc = *reinterpret_cast<const uint2*>(buf + 2048 + lane * 8);
            const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&sc.x));   // alpha1, alpha2 of row 0
            const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&sc.y));   // ... of row 1
            float F[4];
#pragma unroll
            for (int f = 0; f < 4; ++f) F[f] = (float)((ah[f] << 8) + al[f]);              // 4^f * sum_j t_j X_j
            y0 = c * fmaf(s0.x, F[0], 0.25f * (s0.y * F[1]));
            y1 = (0.0625f * c) * fmaf(s1.x, F[2], 0.25f * (s1.y * F[3]));
        }
        issue(slot);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            y0 += __shfl_xor_sync(0xffffffffu, y0, o);
            y1 += __shfl_xor_sync(0xffffffffu, y1, o);
        }
        if (lane == 0) {
            float* p = partial + (size_t)(rp - rp0) * 2 * S + sl;
            p[0] = y0;
            p[S] = y1;
        }
        if (++cj == n_rp) { cj = 0; ++ct; }
    }
    cp_async_wait<0>();
    __syncthreads();
    const int rows = 2 * (rp1 - rp0);
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        const int row = 2 * rp0 + r;
        float t = 0.f;
        for (int s = 0; s < S; ++s) t += partial[(size_t)r * S + s];
        if (row < L.n) y[row] = __float2half_rn(t);
    }
}

size_t smem_bytes(const Layout2& L, int rows_cap, int warps, int depth) {
    const size_t nblk = (size_t)L.k / kLane2;
    const size_t ring_off = (nblk * 136 + (size_t)rows_cap * L.slices * 4 + 15) / 16 * 16;
    return ring_off + (size_t)warps * depth * kSlot;
}

template <int D>
ptqtp_status launch_d(const Layout2& L, const void* packed, const uint16_t* x, uint16_t* y, int grid, int warps,
                      int rows_cap, size_t smem, cudaStream_t st) {
    auto kern = gemv2_kernel<D>;
    static thread_local size_t configured[64] = {};       // per device: largest dynamic smem already allowed
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    if (smem > 48 * 1024 && smem > configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
        configured[dev] = smem;
    }
    kern<<<grid, warps * 32, smem, st>>>(L, static_cast<const unsigned char*>(packed),
                                         reinterpret_cast<const __half*>(x), reinterpret_cast<__half*>(y), rows_cap);
    return check_launch();
}

}  // namespace

ptqtp_status launch_gemv2(const Layout2& L, const void* packed, const uint16_t* x, uint16_t* y, int warps, int depth,
                          cudaStream_t st) {
    const int S = L.slices;
    if (warps == 0) {
        // the multiple of the slice count closest below 16 warps, so every slice lane has as many warps
        warps = S <= 16 ? S * (16 / S) : 16;
    }
    if (warps < 1 || warps > 16) return PTQTP_ERR_CONFIG;
    const int grid = min(sm_count(), L.nrp);
    const int rows_cap = 2 * ((L.nrp + grid - 1) / grid);
    const size_t budget = 227 * 1024;
    if (depth == 0) {
        depth = 4;
        while (depth > 2 && smem_bytes(L, rows_cap, warps, depth) > budget) --depth;
    }
    const size_t smem = smem_bytes(L, rows_cap, warps, depth);
    if (smem > budget) return depth > 2 || warps > 1 ? PTQTP_ERR_CONFIG : PTQTP_ERR_SHAPE;
    switch (depth) {
        case 2: return launch_d<2>(L, packed, x, y, grid, warps, rows_cap, smem, st);
        case 3: return launch_d<3>(L, packed, x, y, grid, warps, rows_cap, smem, st);
        case 4: return launch_d<4>(L, packed, x, y, grid, warps, rows_cap, smem, st);
        case 6: return launch_d<6>(L, packed, x, y, grid, warps, rows_cap, smem, st);
        case 8: return launch_d<8>(L, packed, x, y, grid, warps, rows_cap, smem, st);
    }
    return PTQTP_ERR_CONFIG;
}

}  // namespace ptqtp
