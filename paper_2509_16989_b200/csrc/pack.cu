// Pack / unpack kernels of the PTQTP-B200 v1 format (layout described in ptqtp.h).
// One thread handles one 16-byte lane block: 32 columns of one row, both planes.
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

__device__ __forceinline__ uint32_t encode16(const int8_t* t, bool* bad) {
    // 16 trits (column offsets e' = 0..15) -> one word; code q = trit + 1 at bits [16*(e'/8) + 2*(e'%8)].
    uint32_t w = 0;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        uint32_t q = (uint32_t)((int)t[e] + 1);
        if (q > 2u) { *bad = true; q = 1u; }
        w |= q << (16 * (e >> 3) + 2 * (e & 7));
    }
    return w;
}

__global__ void pack_kernel(Layout L, const int8_t* __restrict__ T1, const int8_t* __restrict__ T2,
                            const uint16_t* __restrict__ a1, const uint16_t* __restrict__ a2,
                            unsigned char* __restrict__ packed, int32_t* dev_status) {
    const size_t blocks_per_row = (size_t)L.slices * 32;
    const size_t total = (size_t)L.n * blocks_per_row;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (size_t b = (size_t)blockIdx.x * blockDim.x + threadIdx.x; b < total; b += stride) {
        const int row = (int)(b / blocks_per_row);
        const int in_row = (int)(b % blocks_per_row);          // slice*32 + lane
        const int k0 = in_row * kLaneK;
        alignas(16) int8_t t1[32], t2[32];
        if (k0 < L.k) {                                       // K % 128 == 0, so a block is all in or all out
            const int4* p1 = reinterpret_cast<const int4*>(T1 + (size_t)row * L.k + k0);
            const int4* p2 = reinterpret_cast<const int4*>(T2 + (size_t)row * L.k + k0);
            reinterpret_cast<int4*>(t1)[0] = p1[0];
            reinterpret_cast<int4*>(t1)[1] = p1[1];
            reinterpret_cast<int4*>(t2)[0] = p2[0];
            reinterpret_cast<int4*>(t2)[1] = p2[1];
        } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) { t1[e] = 0; t2[e] = 0; }
        }
        uint4 out;
        out.x = encode16(t1, &bad);
        out.y = encode16(t1 + 16, &bad);
        out.z = encode16(t2, &bad);
        out.w = encode16(t2 + 16, &bad);
        *reinterpret_cast<uint4*>(packed + L.codes_off + b * 16) = out;
        if ((in_row & 3) == 0) {                              // first lane block of a 128-column group
            const int g = k0 / kGroup;
            uint32_t pair = 0;
            if (k0 < L.k) {
                const size_t si = (size_t)row * (L.k / kGroup) + g;
                pair = (uint32_t)a1[si] | ((uint32_t)a2[si] << 16);
            }
            *reinterpret_cast<uint32_t*>(packed + L.scales_off + ((size_t)row * L.groups_pad + g) * 4) = pair;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < PTQTP_HEADER_BYTES / 4) {
        Header h;
        const char m[8] = {'P', 'T', 'Q', 'T', 'P', 'B', '2', '\0'};
        for (int i = 0; i < 8; ++i) h.magic[i] = m[i];
        h.version = kVersion; h.format = PTQTP_FORMAT_V1;
        h.n = L.n; h.k = L.k; h.group = kGroup; h.k_pad = L.k_pad;
        h.codes_off = L.codes_off; h.scales_off = L.scales_off; h.total = L.total;
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(&h);
        const int i = threadIdx.x;
        reinterpret_cast<uint32_t*>(packed)[i] = i < (int)(sizeof(Header) / 4) ? hw[i] : 0u;
    }
    if (bad && dev_status) atomicExch(dev_status, (int)PTQTP_ERR_TRIT);
}

__device__ __forceinline__ void decode16(uint32_t w, int8_t* t) {
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const uint32_t q = (w >> (16 * (e >> 3) + 2 * (e & 7))) & 3u;
        t[e] = (int8_t)((int)q - 1);
    }
}

__global__ void unpack_kernel(Layout L, const unsigned char* __restrict__ packed, int8_t* __restrict__ T1,
                              int8_t* __restrict__ T2, uint16_t* __restrict__ a1, uint16_t* __restrict__ a2,
                              int32_t* dev_status) {
    if (blockIdx.x == 0 && threadIdx.x == 0 && dev_status) {
        const Header* h = reinterpret_cast<const Header*>(packed);
        const char m[8] = {'P', 'T', 'Q', 'T', 'P', 'B', '2', '\0'};
        bool ok = h->version == kVersion && h->format == PTQTP_FORMAT_V1 && h->n == L.n && h->k == L.k &&
                  h->group == kGroup && h->k_pad == L.k_pad && h->codes_off == L.codes_off &&
                  h->scales_off == L.scales_off && h->total == L.total;
        for (int i = 0; i < 8; ++i) ok = ok && h->magic[i] == m[i];
        if (!ok) atomicExch(dev_status, (int)PTQTP_ERR_FORMAT);
    }
    const size_t blocks_per_row = (size_t)L.slices * 32;
    const size_t total = (size_t)L.n * blocks_per_row;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t b = (size_t)blockIdx.x * blockDim.x + threadIdx.x; b < total; b += stride) {
        const int row = (int)(b / blocks_per_row);
        const int in_row = (int)(b % blocks_per_row);
        const int k0 = in_row * kLaneK;
        if (k0 >= L.k) continue;
        const uint4 in = *reinterpret_cast<const uint4*>(packed + L.codes_off + b * 16);
        alignas(16) int8_t t1[32], t2[32];
        decode16(in.x, t1);
        decode16(in.y, t1 + 16);
        decode16(in.z, t2);
        decode16(in.w, t2 + 16);
        int4* p1 = reinterpret_cast<int4*>(T1 + (size_t)row * L.k + k0);
        int4* p2 = reinterpret_cast<int4*>(T2 + (size_t)row * L.k + k0);
        p1[0] = reinterpret_cast<int4*>(t1)[0];
        p1[1] = reinterpret_cast<int4*>(t1)[1];
        p2[0] = reinterpret_cast<int4*>(t2)[0];
        p2[1] = reinterpret_cast<int4*>(t2)[1];
        if ((in_row & 3) == 0) {
            const int g = k0 / kGroup;
            const uint32_t pair =
                *reinterpret_cast<const uint32_t*>(packed + L.scales_off + ((size_t)row * L.groups_pad + g) * 4);
            const size_t si = (size_t)row * (L.k / kGroup) + g;
            a1[si] = (uint16_t)(pair & 0xffffu);
            a2[si] = (uint16_t)(pair >> 16);
        }
    }
}

int grid_for(size_t items, int threads) {
    size_t g = (items + threads - 1) / threads;
    const size_t cap = (size_t)sm_count() * 16;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

}  // namespace

ptqtp_status launch_pack(const Layout& L, const int8_t* T1, const int8_t* T2, const uint16_t* a1,
                         const uint16_t* a2, void* packed, int32_t* dev_status, cudaStream_t st) {
    const size_t items = (size_t)L.n * L.slices * 32;
    pack_kernel<<<grid_for(items, 256), 256, 0, st>>>(L, T1, T2, a1, a2, static_cast<unsigned char*>(packed),
                                                     dev_status);
    return check_launch();
}

ptqtp_status launch_unpack(const Layout& L, const void* packed, int8_t* T1, int8_t* T2, uint16_t* a1,
                           uint16_t* a2, int32_t* dev_status, cudaStream_t st) {
    const size_t items = (size_t)L.n * L.slices * 32;
    unpack_kernel<<<grid_for(items, 256), 256, 0, st>>>(L, static_cast<const unsigned char*>(packed), T1, T2,
                                                       a1, a2, dev_status);
    return check_launch();
}

}  // namespace ptqtp
