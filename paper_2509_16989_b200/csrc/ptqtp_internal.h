// Internal declarations shared by the translation units of libptqtp (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
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
           s->format == PTQTP_FORMAT_V1;
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
ptqtp_status launch_gemm_skinny(const Layout& L, const void* packed, int m, const uint16_t* X,
                                uint16_t* Y, cudaStream_t st);
int sm_count();

}  // namespace ptqtp
