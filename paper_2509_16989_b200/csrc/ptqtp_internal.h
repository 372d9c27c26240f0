// Internal declarations shared by the translation units of libptqtp (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <mutex>
#include <stdint.h>
#include <stddef.h>
#include "ptqtp.h"

namespace ptqtp {

constexpr int kGroup = 128;          // input columns per scale pair (Sec. 2.3, G = 128)
constexpr int kSliceK = 1024;        // input columns covered by one 512-byte chunk
constexpr int kChunkBytes = 512;     // one warp-wide 128-bit load
constexpr int kLaneK = 32;           // input columns per 16-byte lane block
constexpr int kGroupsPerSlice = kSliceK / kGroup;   // 8
constexpr uint32_t kVersion = 1;

// Byte layout of a packed blob; see the format description in ptqtp.h.
struct Layout {
    int n, k, k_pad, slices, groups_pad;
    size_t codes_off, scales_off, total;
};

struct Header {                       // first bytes of the 256-byte header
    char magic[8];
    uint32_t version, format;
    int32_t n, k, group, k_pad;
    uint64_t codes_off, scales_off, total;
};
static_assert(sizeof(Header) <= PTQTP_HEADER_BYTES, "header must fit its slot");

inline bool shape_ok(const ptqtp_shape* s) {
    return s && s->n_out > 0 && s->k_in > 0 && s->group == kGroup && s->k_in % kGroup == 0 &&
           (s->format == PTQTP_FORMAT_V1 || s->format == PTQTP_FORMAT_V2 || s->format == PTQTP_FORMAT_V3);
}

inline Layout make_layout(const ptqtp_shape* s) {
    Layout L;
    L.n = s->n_out;
    L.k = s->k_in;
    L.k_pad = (s->k_in + kSliceK - 1) / kSliceK * kSliceK;
    L.slices = L.k_pad / kSliceK;
    L.groups_pad = L.k_pad / kGroup;
    L.codes_off = PTQTP_HEADER_BYTES;
    L.scales_off = L.codes_off + (size_t)L.n * L.slices * kChunkBytes;
    L.total = L.scales_off + (size_t)L.n * L.groups_pad * 4;
    return L;
}

// ---- format 2: row-pair interleaved, 2048-column slices (see ptqtp.h) ----
constexpr int kSlice2 = 2048;        // input columns per slice of format 2
constexpr int kLane2 = 64;           // input columns per lane block of format 2
constexpr int kUnit2 = 2176;         // bytes of a full slice unit: 2048 code bytes + 128 scale bytes

struct Layout2 {
    int n, k, nrp;                   // rows, columns, row pairs = ceil(n / 2)
    int slices;                      // ceil(k / 2048)
    int last_active;                 // 64-column lane blocks in the last slice (1..32)
    int last_unit;                   // bytes of the last slice's unit (multiple of 16)
    size_t strip;                    // bytes of one row pair over all slices: (slices - 1) * 2176 + last_unit
    size_t codes_off, total;
};

inline Layout2 make_layout2(const ptqtp_shape* s) {
    Layout2 L;
    L.n = s->n_out;
    L.k = s->k_in;
    L.nrp = (s->n_out + 1) / 2;
    L.slices = (s->k_in + kSlice2 - 1) / kSlice2;
    const int last_cols = s->k_in - (L.slices - 1) * kSlice2;
    L.last_active = last_cols / kLane2;
    L.last_unit = (last_cols + last_cols / 16 + 15) / 16 * 16;
    L.strip = (size_t)(L.slices - 1) * kUnit2 + L.last_unit;
    L.codes_off = PTQTP_HEADER_BYTES;
    L.total = L.codes_off + (size_t)L.nrp * L.strip;
    return L;
}

// Byte offset (from codes_off) of the slice unit of row pair rp and slice s.  Slice-major: all units of slice 0,
// then all units of slice 1, ...; the units of one slice for consecutive row pairs are contiguous.
__host__ __device__ inline size_t unit_offset(const Layout2& L, int rp, int s) {
    return (size_t)s * L.nrp * kUnit2 + (size_t)rp * (s == L.slices - 1 ? L.last_unit : kUnit2);
}

// ---- format 3: tiles of 8 row pairs x 512 columns in tensor-core fragment order (see ptqtp.h) ----
constexpr int kSuper3 = 512;         // input columns per tile (four scale groups)
constexpr int kTileRp3 = 8;          // row pairs per tile
constexpr int kTileCodes3 = 4096;    // code bytes of a tile
constexpr int kTile3 = 4352;         // bytes of a tile: 4096 code bytes + 32 scale quads of 8 bytes

struct Layout3 {
    int n, k, nrp;                   // rows, columns, row pairs = ceil(n / 2)
    int nrb;                         // row blocks = ceil(nrp / 8)
    int sbs;                         // superblocks = ceil(k / 512)
    size_t codes_off, total;
};

inline Layout3 make_layout3(const ptqtp_shape* s) {
    Layout3 L;
    L.n = s->n_out;
    L.k = s->k_in;
    L.nrp = (s->n_out + 1) / 2;
    L.nrb = (L.nrp + kTileRp3 - 1) / kTileRp3;
    L.sbs = (s->k_in + kSuper3 - 1) / kSuper3;
    L.codes_off = PTQTP_HEADER_BYTES;
    L.total = L.codes_off + (size_t)L.nrb * L.sbs * kTile3;
    return L;
}

// Byte offset (from codes_off) of tile (superblock sb, row block rb): superblock-major, so the tiles of one
// superblock for consecutive row blocks are contiguous.
__host__ __device__ inline size_t tile_offset3(const Layout3& L, int rb, int sb) {
    return ((size_t)sb * L.nrb + rb) * kTile3;
}

inline size_t packed_total(const ptqtp_shape* s) {
    return s->format == PTQTP_FORMAT_V3 ? make_layout3(s).total
         : s->format == PTQTP_FORMAT_V2 ? make_layout2(s).total : make_layout(s).total;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void set_last_cuda_error(cudaError_t e);
ptqtp_status check_launch();          // cudaGetLastError -> status

// Launchers (each validates nothing: api.cu has done it).
ptqtp_status launch_pack(const Layout& L, const int8_t* T1, const int8_t* T2, const uint16_t* a1,
                         const uint16_t* a2, void* packed, int32_t* dev_status, cudaStream_t st);
ptqtp_status launch_unpack(const Layout& L, const void* packed, int8_t* T1, int8_t* T2, uint16_t* a1,
                           uint16_t* a2, int32_t* dev_status, cudaStream_t st);
ptqtp_status launch_gemv(const Layout& L, const void* packed, const uint16_t* x, uint16_t* y,
                         int rows_per_warp, int k_split, int ctas_per_sm, int depth, int arith, cudaStream_t st);
ptqtp_status launch_pack2(const Layout2& L, const int8_t* T1, const int8_t* T2, const uint16_t* a1,
                          const uint16_t* a2, void* packed, int32_t* dev_status, cudaStream_t st);
ptqtp_status launch_unpack2(const Layout2& L, const void* packed, int8_t* T1, int8_t* T2, uint16_t* a1,
                            uint16_t* a2, int32_t* dev_status, cudaStream_t st);
ptqtp_status launch_gemv2(const Layout2& L, const void* packed, const uint16_t* x, uint16_t* y, int warps,
                          int ctas_per_sm, int depth, int units, cudaStream_t st, bool gated = false);
ptqtp_status launch_pack3(const Layout3& L, const int8_t* T1, const int8_t* T2, const uint16_t* a1,
                          const uint16_t* a2, void* packed, int32_t* dev_status, cudaStream_t st);
ptqtp_status launch_unpack3(const Layout3& L, const void* packed, int8_t* T1, int8_t* T2, uint16_t* a1,
                            uint16_t* a2, int32_t* dev_status, cudaStream_t st);
// The matrices ("jobs") of one launch of the format-3 batch-1 kernel: they share x (and therefore K).
constexpr int kMaxJobs4 = 4;
struct Jobs4 {
    const unsigned char* codes[kMaxJobs4];    // first tile of each packed blob
    ::__half* y[kMaxJobs4];
    int n[kMaxJobs4], nrp[kMaxJobs4], nrb[kMaxJobs4];
    int rb_base[kMaxJobs4], rb_rem[kMaxJobs4], rb_off[kMaxJobs4];   // balanced partition of each job over the grid
    int count, k, sbs;
};
void add_job4(Jobs4& J, const Layout3& L, const void* packed, uint16_t* y);
ptqtp_status launch_gemv4_jobs(Jobs4& J, const uint16_t* x, int warps, int ctas_per_sm, int depth, int units,
                               cudaStream_t st, int gated);
// warps: per CTA (0 = library choice, -1 = as many as fit); depth: tiles in flight per warp (0 = library choice)
ptqtp_status launch_gemv4(const Layout3& L, const void* packed, const uint16_t* x, uint16_t* y, int warps,
                          int ctas_per_sm, int depth, int units, cudaStream_t st, bool gated = false);
// 2 <= m <= 4 rows on format 3; PTQTP_ERR_SHAPE when (K, m) leaves no room in shared memory
ptqtp_status launch_gemv5(const Layout3& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int warps, int depth,
                          cudaStream_t st);
// 1 <= m <= 64 rows on format 3, tcgen05 kernel; ksplit = CTAs per cluster sharing the columns (0 = library choice)
ptqtp_status launch_gemm6(const Layout3& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int ksplit,
                          cudaStream_t st);
size_t decompose_workspace_bytes(long long rows, int t_max);
void decompose_offsets(long long rows, int t_max, size_t* delta_off, size_t* err_off, size_t* a1_off, size_t* a2_off,
                       size_t* lam_off);
ptqtp_status launch_decompose(const float* W, int n, int k, int G, int t_max, double eps, int canonicalize, int8_t* T1,
                              int8_t* T2, uint16_t* alpha1, uint16_t* alpha2, void* workspace, cudaStream_t st);
size_t skinny3_workspace_bytes(int k, int m);
ptqtp_status launch_skinny3(const Layout2& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, void* workspace,
                            cudaStream_t st);
ptqtp_status static_workspace_address(void** out);
ptqtp_status copy_gemv2_status(int32_t* status_host, cudaStream_t st);
ptqtp_status gemv_status_word(int** out);      // device address of the word copy_gemv2_status reads
// 1 <= m <= 4 on the tensor-core path; PTQTP_ERR_SHAPE when (K, m) leaves no room for its ring in shared memory
ptqtp_status launch_gemv3(const Layout2& L, const void* packed, int m, const uint16_t* X, uint16_t* Y, int warps,
                          int ctas_per_sm, int depth, cudaStream_t st);
int sm_count();
bool speculation_enabled();       // speculative read of x before the dependency wait (ptqtp_set_overlap(2))
bool overlap_enabled();           // programmatic dependent launch of the GEMV kernels (ptqtp_set_overlap)
int wait_poll_limit();            // polls of an mbarrier before a bounded wait gives up (ptqtp_set_wait_limit)
bool take_injected_wait_failure();   // test hook: true once per armed failure (ptqtp_test_fail_next_wait)
bool consume_pack(cudaStream_t st);   // true once after ptqtp_pack on this stream: the next GEMV launch is plain

// Once per kernel and device, process-wide: the largest shared-memory carveout (consecutive launches with
// different carveouts cannot share an SM, and these kernels make no use of L1) and the opt-in maximum of
// dynamic shared memory.  Both attributes belong to the process, so they are set under a lock and never lowered.
// with_carveout = false leaves the carveout preference alone (kernels that want L1).
template <auto Kern>
inline ptqtp_status configure_once(bool with_carveout = true) {
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PTQTP_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!done[dev]) {
        cudaError_t e = with_carveout ? cudaFuncSetAttribute(Kern, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared)
                                      : cudaSuccess;
        if (e == cudaSuccess) e = cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) { set_last_cuda_error(e); (void)cudaGetLastError(); return PTQTP_ERR_CUDA; }
        done[dev] = true;
    }
    return PTQTP_OK;
}


}  // namespace ptqtp
