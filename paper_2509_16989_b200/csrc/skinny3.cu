// Small-batch dual-trit-plane GEMM with a caller-provided workspace (format 2):  Y[m,:] = layer(X[m,:]), M <= 64.
//
// Same contraction as gemv3.cu (int8 warp MMAs on masked codes x block-fixed-point activations), organised so
// that the packed planes are read from HBM exactly once for any M and any K:
//
//   * A first kernel converts X once into the workspace: for every 1024-column half slice the rows
//     (2j = high byte, 2j + 1 = low byte of batch row j) as 1024 contiguous bytes each, and one record
//     (2^-s, sum of the block's integers) per batch row and 128-column block.  (In gemv3.cu every CTA repeats
//     this conversion for its one to four rows.)
//   * The main kernel gives each warp one quad of four row pairs per round and walks the half slices in order,
//     the whole CTA in step: the activation tile of a step (one half slice, up to 16 batch rows) is copied from
//     the workspace (L2-resident) into shared memory by all threads, double buffered, while the warps' code
//     units stream through per-warp ring slots.  A warp keeps the row sums of its quad for all
//     batch rows in registers across the half slices, so no partial sums go through shared memory and the
//     result is written once at the end of the round.
//   * The main kernel issues its first code copies before griddepcontrol.wait, i.e. while the conversion kernel
//     (or whatever precedes it on the stream) is still running.
#include <cuda_fp16.h>
#include <mutex>
#include "ptqtp_internal.h"

// Workspace of ptqtp_gemm_skinny_static: a fixed array in device memory, owned by the library, present on every
// GPU that loads it until the process exits.  In host code this name is only a handle for the runtime (its
// device address comes from cudaGetSymbolAddress); device code may name it directly.
static __device__ __align__(256) unsigned char g_static_workspace[PTQTP_STATIC_WORKSPACE_BYTES];

namespace ptqtp {

namespace {

constexpr int kHalf = 1024;                  // columns per half slice
constexpr int kSI = 18;                      // 16-byte chunks between the atom rows i of a half unit in a ring slot
constexpr int kSU = 81;                      // chunks per half unit in a ring slot
constexpr int kScaleChunk = 72;              // first scale chunk of a half unit
constexpr int kQuadSlot = 4 * kSU * 16;      // bytes per ring slot (four half units)
constexpr int kTileRow = kHalf + 64;         // bytes between activation rows of a tile (rows 16 apart in bank space)
constexpr int kMaxWarps3 = 16;

__device__ __forceinline__ void cp16(void* dst_smem, const void* src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp8(void* dst_smem, const void* src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Workspace layout for (K, M): activation rows, then records.
struct Ws3 {
    int halves;              // ceil(K / 1024)
    int m_pad;               // M rounded up to 4, 8, 16, 32 or 64 (whole MMA n-tile groups)
    size_t meta_off, total;
};
__host__ __device__ inline Ws3 ws3_layout(int k, int m) {
    Ws3 w;
    w.halves = (k + kHalf - 1) / kHalf;
    w.m_pad = m <= 4 ? 4 : m <= 8 ? 8 : m <= 16 ? 16 : m <= 32 ? 32 : 64;
    w.meta_off = (size_t)w.halves * 2 * w.m_pad * kHalf;
    w.total = w.meta_off + (size_t)w.m_pad * (k / kGroup) * 8;
    return w;
}

// ---- kernel 1: X (fp16 [M, K]) -> workspace.  One thread per 8 columns of one (padded) batch row; the 16
// threads of a 128-column block agree on the block scale by shuffles.  Padding rows and columns are written as
// zeros on every call (the workspace keeps whatever the previous call left).
__global__ void __launch_bounds__(256)
convert3_kernel(const __half* __restrict__ X, unsigned char* __restrict__ ws, int k, int m) {
    const Ws3 w = ws3_layout(k, m);
    const int tasks_per_row = w.halves * (kHalf / 8);
    const long long task = (long long)blockIdx.x * blockDim.x + threadIdx.x;        // grid covers m_pad * tasks_per_row exactly
    const int mi = (int)(task / tasks_per_row), col = (int)(task % tasks_per_row) * 8;
    const bool valid = mi < m && col < k;
    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
    if (valid) raw = __ldg(reinterpret_cast<const uint4*>(X + (size_t)mi * k + col));
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
        s = 13 - ex;                                   // block maximum in [2^13, 2^14): high byte within [-64, 64]
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
    for (int q = 0; q < 2; ++q) {
        lw[q] = __byte_perm(__byte_perm(Lo[4 * q], Lo[4 * q + 1], 0x0040), __byte_perm(Lo[4 * q + 2], Lo[4 * q + 3], 0x0040), 0x5410);
        hw[q] = __byte_perm(__byte_perm(H[4 * q], H[4 * q + 1], 0x0040), __byte_perm(H[4 * q + 2], H[4 * q + 3], 0x0040), 0x5410);
    }
    if (!valid) { hw[0] = hw[1] = lw[0] = lw[1] = 0u; }
    const int hs = col / kHalf, ch = col % kHalf;
    unsigned char* row_hi = ws + ((size_t)hs * 2 * w.m_pad + 2 * mi) * kHalf;
    *reinterpret_cast<uint2*>(row_hi + ch) = make_uint2(hw[0], hw[1]);
    *reinterpret_cast<uint2*>(row_hi + kHalf + ch) = make_uint2(lw[0], lw[1]);
    if (col < k && ((col >> 3) & 15) == 0) {
        int2* meta = reinterpret_cast<int2*>(ws + w.meta_off);
        meta[(size_t)mi * (k / kGroup) + (col >> 7)] = valid ? make_int2((int)((uint32_t)(127 - s) << 23), sum) : make_int2(0, 0);
    }
}

// ---- kernel 2.  NTT = MMA n-tiles in total (M padded to 4 NTT batch rows); a step handles NTG = min(NTT, 4).
template <int NTT>
__global__ void __launch_bounds__(kMaxWarps3 * 32, 1)
skinny3_kernel(Layout2 L, const unsigned char* __restrict__ packed, const unsigned char* __restrict__ ws,
               __half* __restrict__ Y, int m, int q_base, int q_rem, int depth) {
    constexpr int NTG = NTT < 4 ? NTT : 4;
    constexpr int NG = NTT / NTG;
    constexpr int kTileRows = 8 * NTG * kTileRow;                       // activation rows of a tile
    constexpr int kTileBytes = kTileRows + 4 * NTG * 64;                // + (2^-s, sum X) of 4 NTG batch rows x 8 groups
    extern __shared__ __align__(16) unsigned char smem[];
    asm volatile("griddepcontrol.launch_dependents;");

    // the last warp only copies activation tiles; the others ("compute warps") stream and contract codes
    const int warps = (blockDim.x >> 5) - 1, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool loader = warp == warps;
    const int g = lane >> 2, tig = lane & 3, u = g & 3, plane = g >> 2;
    const Ws3 w = ws3_layout(L.k, m);
    const int halves = w.halves, ngroups = L.k / kGroup;
    unsigned char* tile = smem;                                          // [2][8 NTG rows][kTileRow]
    unsigned char* ring = smem + 2 * kTileBytes + (size_t)(loader ? 0 : warp) * depth * kQuadSlot;
    const int2* meta = reinterpret_cast<const int2*>(ws + w.meta_off);

    // this CTA's quads (balanced partition from the host) and the rounds needed to give every quad a warp
    const int q0 = (int)blockIdx.x * q_base + min((int)blockIdx.x, q_rem);
    const int nq_cta = q_base + ((int)blockIdx.x < q_rem ? 1 : 0);
    const int rounds = (nq_cta + warps - 1) / warps;
    const unsigned char* codes = packed + L.codes_off;

    // codes of (quad, half slice) -> ring slot; lane -> (atom rows ip and ip + 2, lane block ll) of each half unit
    const int ip = lane >> 4, ll = lane & 15;
    auto issue_codes = [&](int q, int hs, int slot) {
        const int sl = hs >> 1, l0 = (hs & 1) * 16;
        const int A = sl == L.slices - 1 ? L.last_active : 32;
        const int Ah = min(16, A - l0);
        unsigned char* dst = ring + slot * kQuadSlot;
#pragma unroll
        for (int uu = 0; uu < 4; ++uu) {
            const int rp = min(4 * q + uu, L.nrp - 1);                   // row pairs past the end re-read the last one
            const unsigned char* src = codes + unit_offset(L, rp, sl);
            unsigned char* d = dst + uu * (kSU * 16);
            if (ll < Ah) {
                cp16(d + (ip * kSI + ll) * 16, src + (ip * A + l0 + ll) * 16);
                cp16(d + ((ip + 2) * kSI + ll) * 16, src + ((ip + 2) * A + l0 + ll) * 16);
            }
            if (lane < Ah / 2) cp8(d + kScaleChunk * 16 + lane * 8, src + A * 64 + (l0 / 2 + lane) * 8);
        }
    };
    // activation tile of (half slice, n-tile group) -> tile buffer, copied by the loader warp
    auto issue_tile = [&](int hs, int ng, int buf) {
        const unsigned char* src = ws + ((size_t)hs * 2 * w.m_pad + 8 * NTG * ng) * kHalf;
        unsigned char* dst = tile + buf * kTileBytes;
        for (int c = lane; c < 8 * NTG * (kHalf / 16); c += 32)
            cp16(dst + (c >> 6) * kTileRow + (c & 63) * 16, src + (size_t)c * 16);
        // the records of the tile's batch rows for the (up to) 8 groups of the half slice
        for (int c = lane; c < 4 * NTG * 8; c += 32) {
            const int row = c >> 3, gi = hs * 8 + (c & 7);
            if (gi < ngroups) cp8(dst + kTileRows + c * 8, meta + (size_t)(4 * NTG * ng + row) * ngroups + gi);
        }
    };

    const int steps = rounds * halves * NG;              // activation-tile steps
    const int code_steps = rounds * halves;              // (round, half slice) pairs: one ring slot each
    // codes of code step cs for this warp (if it has a quad in that round) -> ring slot cs % depth
    auto issue_code_step = [&](int cs) {
        if (!loader && cs < code_steps) {
            const int r = cs / halves, hs = cs - r * halves;
            const int ql = r * warps + warp;
            if (ql < nq_cta) issue_codes(q0 + ql, hs, cs % depth);
        }
        cp_commit();
    };
    // wait until at most depth - 2 of this thread's copy groups are pending: the codes of the next code step have
    // landed, younger ones may still be in flight
    auto wait_codes = [&]() {
        if (depth >= 3) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else cp_wait_all();
    };
    for (int d = 0; d < depth - 1; ++d) issue_code_step(d);
    // everything above reads only the packed planes; the workspace and Y belong to the stream order
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (loader) {
        if (steps > 0) issue_tile(0, 0, 0);
        cp_commit();
        cp_wait_all();
    } else {
        wait_codes();
    }
    __syncthreads();

    const uint32_t maskA = 0x03030303u << (2 * plane), maskB = maskA << 4;       // fields plane and 2 + plane
    const float kA = plane ? 0.25f : 1.0f, kB = kA * 0.0625f;
    const int shA = 2 * plane, shB = shA + 4;
    const uint32_t alpha_sel = plane ? 0x7632u : 0x5410u;

    int t = 0, cs = 0, slot = 0;
    for (int r = 0; r < rounds; ++r) {
        const int ql = r * warps + warp;                 // this warp's quad of the round, if any
        const bool has = !loader && ql < nq_cta;
        const int q = q0 + ql;
        float yA[NTT], yB[NTT];
#pragma unroll
        for (int nt = 0; nt < NTT; ++nt) { yA[nt] = 0.f; yB[nt] = 0.f; }
        for (int hs = 0; hs < halves; ++hs) {
            const int sl = hs >> 1, l0 = (hs & 1) * 16;
            const int A = sl == L.slices - 1 ? L.last_active : 32;
            const int groups_here = min(16, A - l0) / 2;
            // keep depth - 1 code steps in flight
            if (!loader) issue_code_step(cs + depth - 1);
#pragma unroll
            for (int ng = 0; ng < NG; ++ng) {
                if (loader) {                            // the next step's activation tile into the other buffer
                    int nng = ng + 1, nhs = hs;
                    if (nng == NG) { nng = 0; if (++nhs == halves) nhs = 0; }
                    if (t + 1 < steps) issue_tile(nhs, nng, (t + 1) & 1);
                    cp_commit();
                }
                if (has) {
                    const unsigned char* unit = ring + slot * kQuadSlot + u * (kSU * 16);
                    const unsigned char* cptr = unit + (tig * kSI) * 16;
                    const unsigned char* sptr = unit + kScaleChunk * 16;
                    const unsigned char* xptr = tile + (t & 1) * kTileBytes + g * kTileRow + 16 * tig;
                    const unsigned char* mptr = tile + (t & 1) * kTileBytes + kTileRows + tig * 64;
#pragma unroll 2
                    for (int gl = 0; gl < groups_here; ++gl) {       // one 128-column scale group per iteration
                        int c[NTG][4];
#pragma unroll
                        for (int nt = 0; nt < NTG; ++nt) { c[nt][0] = 0; c[nt][1] = 0; c[nt][2] = 0; c[nt][3] = 0; }
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint4 cw = *reinterpret_cast<const uint4*>(cptr + h * 16);
                            const uint32_t a0 = cw.x & maskA, a1 = cw.x & maskB, a2 = cw.y & maskA, a3 = cw.y & maskB;
                            const uint32_t e0 = cw.z & maskA, e1 = cw.z & maskB, e2 = cw.w & maskA, e3 = cw.w & maskB;
#pragma unroll
                            for (int nt = 0; nt < NTG; ++nt) {
                                const uint4 xb = *reinterpret_cast<const uint4*>(xptr + nt * 8 * kTileRow + h * 64);
                                mma_u8s8(c[nt], a0, a1, a2, a3, xb.x, xb.y);
                                mma_u8s8(c[nt], e0, e1, e2, e3, xb.z, xb.w);
                            }
                        }
                        const uint2 sc = *reinterpret_cast<const uint2*>(sptr);
                        const uint32_t apair = __byte_perm(sc.x, sc.y, alpha_sel);
                        const float2 al = __half22float2(*reinterpret_cast<const __half2*>(&apair));
                        const float wA = al.x * kA, wB = al.y * kB;
#pragma unroll
                        for (int nt = 0; nt < NTG; ++nt) {
                            const int2 rec = *reinterpret_cast<const int2*>(mptr + nt * 256);   // batch row 4 (NTG ng + nt) + tig
                            const float cm = __int_as_float(rec.x);
                            const int QA = (c[nt][0] << 8) + c[nt][1] - (rec.y << shA);
                            const int QB = (c[nt][2] << 8) + c[nt][3] - (rec.y << shB);
                            yA[NTG * ng + nt] = fmaf(cm * wA, (float)QA, yA[NTG * ng + nt]);
                            yB[NTG * ng + nt] = fmaf(cm * wB, (float)QB, yB[NTG * ng + nt]);
                        }
                        cptr += 32;
                        sptr += 8;
                        xptr += 128;
                        mptr += 8;
                    }
                }
                // the next tile and the next codes have landed and everybody is done with this step's tile
                if (loader) cp_wait_all(); else wait_codes();
                __syncthreads();
                ++t;
            }
            ++cs;
            slot = slot + 1 == depth ? 0 : slot + 1;
        }
        // the two planes of a row are 16 lanes apart; lanes 0-15 write the quad's rows for batch rows 4 nt + tig
#pragma unroll
        for (int nt = 0; nt < NTT; ++nt) {
            const float rA = yA[nt] + __shfl_xor_sync(0xffffffffu, yA[nt], 16);
            const float rB = yB[nt] + __shfl_xor_sync(0xffffffffu, yB[nt], 16);
            const int mi = 4 * nt + tig, row = 8 * q + 2 * u;
            if (has && lane < 16 && mi < m) {
                if (row < L.n) Y[(size_t)mi * L.n + row] = __float2half_rn(rA);
                if (row + 1 < L.n) Y[(size_t)mi * L.n + row + 1] = __float2half_rn(rB);
            }
        }
    }
}

size_t smem3(int ntt, int compute_warps, int depth) {
    const int ntg = ntt < 4 ? ntt : 4;
    return (size_t)2 * (8 * ntg * kTileRow + 4 * ntg * 64) + (size_t)compute_warps * depth * kQuadSlot;
}

template <int NTT>
ptqtp_status launch3(const Layout2& L, const void* packed, const unsigned char* ws, uint16_t* Y, int m, int grid,
                     int warps, int nq, cudaStream_t st) {
    auto kern = skinny3_kernel<NTT>;
    const int depth = smem3(NTT, warps, 3) <= 227 * 1024 ? 3 : 2;         // ring slots per compute warp
    const size_t smem = smem3(NTT, warps, depth);
    const ptqtp_status cs = configure_once<skinny3_kernel<NTT>>(false);
    if (cs != PTQTP_OK) return cs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3((warps + 1) * 32);                               // + the tile loader warp
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_enabled() ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, L, static_cast<const unsigned char*>(packed), ws,
                                       reinterpret_cast<__half*>(Y), m, nq / grid, nq % grid, depth);
    if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

}  // namespace

size_t skinny3_workspace_bytes(int k, int m) { return ws3_layout(k, m).total; }

// Device address of the library-owned workspace on the current device.  Looked up once per device, with that
// device current, and cached; nothing is allocated.
ptqtp_status static_workspace_address(void** out) {
    static std::mutex lock;
    static void* cached[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return PTQTP_ERR_CONFIG;
    std::lock_guard<std::mutex> guard(lock);
    if (!cached[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (e != cudaSuccess || !p) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
        cached[dev] = p;
    }
    *out = cached[dev];
    return PTQTP_OK;
}

ptqtp_status launch_skinny3(const Layout2& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, void* workspace,
                            cudaStream_t st) {
    const Ws3 w = ws3_layout(L.k, m);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    // kernel 1: one thread per 8 columns of every padded batch row (a multiple of 128 threads in total)
    const long long tasks = (long long)w.m_pad * w.halves * (kHalf / 8);
    convert3_kernel<<<(unsigned)(tasks / 256), 256, 0, st>>>(reinterpret_cast<const __half*>(X), ws, L.k, m);
    ptqtp_status s = check_launch();
    if (s != PTQTP_OK) return s;
    // kernel 2: one CTA per SM, one quad per compute warp and round; as many as the CTA with most quads needs
    const int nq = (L.nrp + 3) / 4;
    const int grid = min(sm_count(), nq);
    const int per_cta = (nq + grid - 1) / grid;
    const int rounds = (per_cta + kMaxWarps3 - 2) / (kMaxWarps3 - 1);     // one of the 16 warps only loads tiles
    const int warps = (per_cta + rounds - 1) / rounds;                    // compute warps
    switch (w.m_pad / 4) {
        case 1: return launch3<1>(L, packed, ws, Y, m, grid, warps, nq, st);
        case 2: return launch3<2>(L, packed, ws, Y, m, grid, warps, nq, st);
        case 4: return launch3<4>(L, packed, ws, Y, m, grid, warps, nq, st);
        case 8: return launch3<8>(L, packed, ws, Y, m, grid, warps, nq, st);
        default: return launch3<16>(L, packed, ws, Y, m, grid, warps, nq, st);
    }
}

}  // namespace ptqtp
