// Pack / unpack kernels of the PTQTP-B200 format 3 (layout described in ptqtp.h).
// One thread handles one 16-byte lane entry of a tile chunk: four code words = 16 columns of one row pair.
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

// Position of a lane entry: tile (superblock sb, row block rb), chunk c (0..7), row pair g (0..7) and t (0..3).
struct Entry3 {
    int sb, rb, c, g, t;
    size_t off;                       // byte offset of the entry from the start of the codes
};

// Entries are numbered in storage order: tile (superblock-major), chunk, lane.
__device__ __forceinline__ Entry3 entry_of(const Layout3& L, size_t e) {
    Entry3 p;
    const size_t tile = e >> 8;                         // 256 entries per tile
    const int r = (int)(e & 255);
    p.sb = (int)(tile / L.nrb);
    p.rb = (int)(tile % L.nrb);
    p.c = r >> 5;
    p.g = (r >> 2) & 7;
    p.t = r & 3;
    p.off = tile * kTile3 + (size_t)r * 16;
    return p;
}

// First column of word (s, h) of an entry: k-step 2c + s of the superblock, group 2h + t/2, half t%2.
__device__ __forceinline__ int word_col(const Entry3& p, int s, int h) {
    return p.sb * kSuper3 + 128 * (2 * h + (p.t >> 1)) + 8 * (2 * p.c + s) + 4 * (p.t & 1);
}

__device__ __forceinline__ uint32_t code3(int t, bool* bad) {
    uint32_t q = (uint32_t)(t + 1);
    if (q > 2u) { *bad = true; q = 1u; }
    return q;
}

// The four trits (as int8x4) of one plane, one row, columns col .. col + 3; trit 0 outside the matrix.
__device__ __forceinline__ uint32_t load4(const int8_t* T, const Layout3& L, int row, int col) {
    if (row >= L.n || col >= L.k) return 0u;            // K is a multiple of 128: four columns are in or out together
    return *reinterpret_cast<const uint32_t*>(T + (size_t)row * L.k + col);
}

__global__ void pack3_kernel(Layout3 L, const int8_t* __restrict__ T1, const int8_t* __restrict__ T2,
                             const uint16_t* __restrict__ a1, const uint16_t* __restrict__ a2,
                             unsigned char* __restrict__ packed, int32_t* dev_status) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned char* codes = packed + L.codes_off;
    bool bad = false;

    const size_t n_tiles = (size_t)L.nrb * L.sbs;
    for (size_t e = tid; e < n_tiles * 256; e += stride) {
        const Entry3 p = entry_of(L, e);
        const int row = 2 * (p.rb * kTileRp3 + p.g);
        uint32_t w[4];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int col = word_col(p, s, h);
                const uint32_t v[4] = {load4(T1, L, row, col), load4(T2, L, row, col), load4(T1, L, row + 1, col),
                                       load4(T2, L, row + 1, col)};
                uint32_t word = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    uint32_t byte = 0;
#pragma unroll
                    for (int f = 0; f < 4; ++f) byte |= code3((int)(int8_t)(v[f] >> (8 * b)), &bad) << (2 * f);
                    word |= byte << (8 * b);
                }
                w[2 * s + h] = word;
            }
        }
        *reinterpret_cast<uint4*>(codes + p.off) = make_uint4(w[0], w[1], w[2], w[3]);
    }

    // scale quads: 32 per tile, quad 4 g + t = row pair g of the tile, group t of the superblock
    const int groups = L.k / kGroup;
    for (size_t q = tid; q < n_tiles * 32; q += stride) {
        const size_t tile = q >> 5;
        const int l = (int)(q & 31), g = l >> 2, t = l & 3;
        const int sb = (int)(tile / L.nrb), rb = (int)(tile % L.nrb);
        const int grp = 4 * sb + t;
        uint16_t s[4] = {0, 0, 0, 0};
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = 2 * (rb * kTileRp3 + g) + r;
            if (row < L.n && grp < groups) {
                s[2 * r] = a1[(size_t)row * groups + grp];
                s[2 * r + 1] = a2[(size_t)row * groups + grp];
            }
        }
        *reinterpret_cast<uint2*>(codes + tile * kTile3 + kTileCodes3 + l * 8) =
            make_uint2((uint32_t)s[0] | ((uint32_t)s[1] << 16), (uint32_t)s[2] | ((uint32_t)s[3] << 16));
    }

    if (blockIdx.x == 0 && threadIdx.x < PTQTP_HEADER_BYTES / 4) {
        Header h;
        const char m[8] = {'P', 'T', 'Q', 'T', 'P', 'B', '2', '\0'};
        for (int i = 0; i < 8; ++i) h.magic[i] = m[i];
        h.version = kVersion; h.format = PTQTP_FORMAT_V3;
        h.n = L.n; h.k = L.k; h.group = kGroup; h.k_pad = L.sbs * kSuper3;
        h.codes_off = L.codes_off; h.scales_off = kTile3; h.total = L.total;
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(&h);
        const int i = threadIdx.x;
        reinterpret_cast<uint32_t*>(packed)[i] = i < (int)(sizeof(Header) / 4) ? hw[i] : 0u;
    }
    if (bad && dev_status) atomicExch(dev_status, (int)PTQTP_ERR_TRIT);
}

__global__ void unpack3_kernel(Layout3 L, const unsigned char* __restrict__ packed, int8_t* __restrict__ T1,
                               int8_t* __restrict__ T2, uint16_t* __restrict__ a1, uint16_t* __restrict__ a2,
                               int32_t* dev_status) {
    if (blockIdx.x == 0 && threadIdx.x == 0 && dev_status) {
        const Header* h = reinterpret_cast<const Header*>(packed);
        const char m[8] = {'P', 'T', 'Q', 'T', 'P', 'B', '2', '\0'};
        bool ok = h->version == kVersion && h->format == PTQTP_FORMAT_V3 && h->n == L.n && h->k == L.k &&
                  h->group == kGroup && h->k_pad == L.sbs * kSuper3 && h->codes_off == L.codes_off &&
                  h->scales_off == (uint64_t)kTile3 && h->total == L.total;
        for (int i = 0; i < 8; ++i) ok = ok && h->magic[i] == m[i];
        if (!ok) atomicExch(dev_status, (int)PTQTP_ERR_FORMAT);
    }
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned char* codes = packed + L.codes_off;

    const size_t n_tiles = (size_t)L.nrb * L.sbs;
    for (size_t e = tid; e < n_tiles * 256; e += stride) {
        const Entry3 p = entry_of(L, e);
        const int row = 2 * (p.rb * kTileRp3 + p.g);
        const uint4 in = *reinterpret_cast<const uint4*>(codes + p.off);
        const uint32_t w[4] = {in.x, in.y, in.z, in.w};
#pragma unroll
        for (int s = 0; s < 2; ++s) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int col = word_col(p, s, h);
                if (col >= L.k) continue;
                const uint32_t word = w[2 * s + h];
                uint32_t out[4] = {0u, 0u, 0u, 0u};      // int8x4 of (row, plane 1), (row, plane 2), (row+1, ...)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const uint32_t byte = (word >> (8 * b)) & 0xffu;
#pragma unroll
                    for (int f = 0; f < 4; ++f)
                        out[f] |= ((uint32_t)((int)((byte >> (2 * f)) & 3u) - 1) & 0xffu) << (8 * b);
                }
                if (row < L.n) {
                    *reinterpret_cast<uint32_t*>(T1 + (size_t)row * L.k + col) = out[0];
                    *reinterpret_cast<uint32_t*>(T2 + (size_t)row * L.k + col) = out[1];
                }
                if (row + 1 < L.n) {
                    *reinterpret_cast<uint32_t*>(T1 + (size_t)(row + 1) * L.k + col) = out[2];
                    *reinterpret_cast<uint32_t*>(T2 + (size_t)(row + 1) * L.k + col) = out[3];
                }
            }
        }
    }

    const int groups = L.k / kGroup;
    for (size_t q = tid; q < n_tiles * 32; q += stride) {
        const size_t tile = q >> 5;
        const int l = (int)(q & 31), g = l >> 2, t = l & 3;
        const int sb = (int)(tile / L.nrb), rb = (int)(tile % L.nrb);
        const int grp = 4 * sb + t;
        if (grp >= groups) continue;
        const uint2 s = *reinterpret_cast<const uint2*>(codes + tile * kTile3 + kTileCodes3 + l * 8);
        const uint32_t v[2] = {s.x, s.y};
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = 2 * (rb * kTileRp3 + g) + r;
            if (row < L.n) {
                a1[(size_t)row * groups + grp] = (uint16_t)(v[r] & 0xffffu);
                a2[(size_t)row * groups + grp] = (uint16_t)(v[r] >> 16);
            }
        }
    }
}

int grid_for3(size_t items, int threads) {
    size_t g = (items + threads - 1) / threads;
    const size_t cap = (size_t)sm_count() * 16;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

}  // namespace

ptqtp_status launch_pack3(const Layout3& L, const int8_t* T1, const int8_t* T2, const uint16_t* a1,
                          const uint16_t* a2, void* packed, int32_t* dev_status, cudaStream_t st) {
    const size_t items = (size_t)L.nrb * L.sbs * 256;
    pack3_kernel<<<grid_for3(items, 256), 256, 0, st>>>(L, T1, T2, a1, a2, static_cast<unsigned char*>(packed),
                                                        dev_status);
    return check_launch();
}

ptqtp_status launch_unpack3(const Layout3& L, const void* packed, int8_t* T1, int8_t* T2, uint16_t* a1,
                            uint16_t* a2, int32_t* dev_status, cudaStream_t st) {
    const size_t items = (size_t)L.nrb * L.sbs * 256;
    unpack3_kernel<<<grid_for3(items, 256), 256, 0, st>>>(L, static_cast<const unsigned char*>(packed), T1, T2,
                                                          a1, a2, dev_status);
    return check_launch();
}

}  // namespace ptqtp
