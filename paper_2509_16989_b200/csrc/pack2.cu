// Pack / unpack kernels of the PTQTP-B200 format 2 (layout described in ptqtp.h).
// One thread handles one 16-byte atom: 16 columns of one row pair, both planes.
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

// Position of an atom: row pair, slice, sub-block i (0..3) and lane block (0..active-1).
struct Atom {
    int rp, slice, i, lane, active;
    size_t unit_off;                 // byte offset of the slice unit from the start of the codes
};

__device__ __forceinline__ int active_of(const Layout2& L, int slice) {
    return slice == L.slices - 1 ? L.last_active : 32;
}

// Atoms are numbered row pair major, then slice, then (i, lane) in storage order.
__device__ __forceinline__ Atom atom_of(const Layout2& L, size_t a) {
    const size_t atoms_per_rp = (size_t)(L.k / 16);
    Atom t;
    t.rp = (int)(a / atoms_per_rp);
    int r = (int)(a % atoms_per_rp);
    t.slice = r / 128;                                  // a full slice holds 128 atoms
    r -= t.slice * 128;
    t.active = active_of(L, t.slice);
    t.i = r / t.active;
    t.lane = r % t.active;
    t.unit_off = unit_offset(L, t.rp, t.slice);
    return t;
}

__device__ __forceinline__ uint32_t code_of(int8_t t, bool* bad) {
    uint32_t q = (uint32_t)((int)t + 1);
    if (q > 2u) { *bad = true; q = 1u; }
    return q;
}

__global__ void pack2_kernel(Layout2 L, const int8_t* __restrict__ T1, const int8_t* __restrict__ T2,
                             const uint16_t* __restrict__ a1, const uint16_t* __restrict__ a2,
                             unsigned char* __restrict__ packed, int32_t* dev_status) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned char* codes = packed + L.codes_off;
    bool bad = false;

    const size_t n_atoms = (size_t)L.nrp * (L.k / 16);
    for (size_t a = tid; a < n_atoms; a += stride) {
        const Atom t = atom_of(L, a);
        const int c0 = t.slice * kSlice2 + t.lane * kLane2 + t.i * 16;
        alignas(16) int8_t v[4][16];                   // [row 0 plane 1, row 0 plane 2, row 1 plane 1, row 1 plane 2]
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = 2 * t.rp + r;
            if (row < L.n) {
                *reinterpret_cast<int4*>(v[2 * r]) = *reinterpret_cast<const int4*>(T1 + (size_t)row * L.k + c0);
                *reinterpret_cast<int4*>(v[2 * r + 1]) = *reinterpret_cast<const int4*>(T2 + (size_t)row * L.k + c0);
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) { v[2 * r][e] = 0; v[2 * r + 1][e] = 0; }
            }
        }
        uint32_t w[4];
#pragma unroll
        for (int ww = 0; ww < 4; ++ww) {
            uint32_t word = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int e = 4 * ww + b;
                const uint32_t byte = code_of(v[0][e], &bad) | (code_of(v[1][e], &bad) << 2) |
                                      (code_of(v[2][e], &bad) << 4) | (code_of(v[3][e], &bad) << 6);
                word |= byte << (8 * b);
            }
            w[ww] = word;
        }
        *reinterpret_cast<uint4*>(codes + t.unit_off + ((size_t)t.i * t.active + t.lane) * 16) =
            make_uint4(w[0], w[1], w[2], w[3]);
    }

    // scale quads: one per row pair and 128-column group, after the codes of their slice unit
    const int groups = L.k / kGroup;
    const size_t n_quads = (size_t)L.nrp * groups;
    for (size_t q = tid; q < n_quads; q += stride) {
        const int rp = (int)(q / groups), g = (int)(q % groups);
        const int slice = g / 16, gl = g % 16;
        const int active = active_of(L, slice);
        uint16_t s[4] = {0, 0, 0, 0};
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = 2 * rp + r;
            if (row < L.n) {
                s[2 * r] = a1[(size_t)row * groups + g];
                s[2 * r + 1] = a2[(size_t)row * groups + g];
            }
        }
        unsigned char* dst = codes + unit_offset(L, rp, slice) + (size_t)active * 64 + gl * 8;
        *reinterpret_cast<uint2*>(dst) = make_uint2((uint32_t)s[0] | ((uint32_t)s[1] << 16),
                                                    (uint32_t)s[2] | ((uint32_t)s[3] << 16));
    }

    // padding bytes at the end of a last unit whose content is not a multiple of 16 bytes
    const int last_content = L.last_active * 64 + L.last_active * 4;
    if (last_content < L.last_unit) {
        for (size_t rp = tid; rp < (size_t)L.nrp; rp += stride) {
            unsigned char* dst = codes + unit_offset(L, (int)rp, L.slices - 1);
            for (int b = last_content; b < L.last_unit; ++b) dst[b] = 0;
        }
    }

    if (blockIdx.x == 0 && threadIdx.x < PTQTP_HEADER_BYTES / 4) {
        Header h;
        const char m[8] = {'P', 'T', 'Q', 'T', 'P', 'B', '2', '\0'};
        for (int i = 0; i < 8; ++i) h.magic[i] = m[i];
        h.version = kVersion; h.format = PTQTP_FORMAT_V2;
        h.n = L.n; h.k = L.k; h.group = kGroup; h.k_pad = L.slices * kSlice2;
        h.codes_off = L.codes_off; h.scales_off = L.strip; h.total = L.total;
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(&h);
        const int i = threadIdx.x;
        reinterpret_cast<uint32_t*>(packed)[i] = i < (int)(sizeof(Header) / 4) ? hw[i] : 0u;
    }
    if (bad && dev_status) atomicExch(dev_status, (int)PTQTP_ERR_TRIT);
}

__global__ void unpack2_kernel(Layout2 L, const unsigned char* __restrict__ packed, int8_t* __restrict__ T1,
                               int8_t* __restrict__ T2, uint16_t* __restrict__ a1, uint16_t* __restrict__ a2,
                               int32_t* dev_status) {
    if (blockIdx.x == 0 && threadIdx.x == 0 && dev_status) {
        const Header* h = reinterpret_cast<const Header*>(packed);
        const char m[8] = {'P', 'T', 'Q', 'T', 'P', 'B', '2', '\0'};
        bool ok = h->version == kVersion && h->format == PTQTP_FORMAT_V2 && h->n == L.n && h->k == L.k &&
                  h->group == kGroup && h->k_pad == L.slices * kSlice2 && h->codes_off == L.codes_off &&
                  h->scales_off == L.strip && h->total == L.total;
        for (int i = 0; i < 8; ++i) ok = ok && h->magic[i] == m[i];
        if (!ok) atomicExch(dev_status, (int)PTQTP_ERR_FORMAT);
    }
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned char* codes = packed + L.codes_off;

    const size_t n_atoms = (size_t)L.nrp * (L.k / 16);
    for (size_t a = tid; a < n_atoms; a += stride) {
        const Atom t = atom_of(L, a);
        const int c0 = t.slice * kSlice2 + t.lane * kLane2 + t.i * 16;
        const uint4 in = *reinterpret_cast<const uint4*>(codes + t.unit_off + ((size_t)t.i * t.active + t.lane) * 16);
        const uint32_t w[4] = {in.x, in.y, in.z, in.w};
        alignas(16) int8_t v[4][16];
#pragma unroll
        for (int ww = 0; ww < 4; ++ww) {
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const uint32_t byte = (w[ww] >> (8 * b)) & 0xffu;
#pragma unroll
                for (int f = 0; f < 4; ++f) v[f][4 * ww + b] = (int8_t)((int)((byte >> (2 * f)) & 3u) - 1);
            }
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = 2 * t.rp + r;
            if (row < L.n) {
                *reinterpret_cast<int4*>(T1 + (size_t)row * L.k + c0) = *reinterpret_cast<const int4*>(v[2 * r]);
                *reinterpret_cast<int4*>(T2 + (size_t)row * L.k + c0) = *reinterpret_cast<const int4*>(v[2 * r + 1]);
            }
        }
    }

    const int groups = L.k / kGroup;
    const size_t n_quads = (size_t)L.nrp * groups;
    for (size_t q = tid; q < n_quads; q += stride) {
        const int rp = (int)(q / groups), g = (int)(q % groups);
        const int slice = g / 16, gl = g % 16;
        const int active = active_of(L, slice);
        const uint2 s = *reinterpret_cast<const uint2*>(codes + unit_offset(L, rp, slice) +
                                                        (size_t)active * 64 + gl * 8);
        const uint32_t v[2] = {s.x, s.y};
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = 2 * rp + r;
            if (row < L.n) {
                a1[(size_t)row * groups + g] = (uint16_t)(v[r] & 0xffffu);
                a2[(size_t)row * groups + g] = (uint16_t)(v[r] >> 16);
            }
        }
    }
}

int grid_for2(size_t items, int threads) {
    size_t g = (items + threads - 1) / threads;
    const size_t cap = (size_t)sm_count() * 16;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

}  // namespace

ptqtp_status launch_pack2(const Layout2& L, const int8_t* T1, const int8_t* T2, const uint16_t* a1,
                          const uint16_t* a2, void* packed, int32_t* dev_status, cudaStream_t st) {
    const size_t items = (size_t)L.nrp * (L.k / 16);
    pack2_kernel<<<grid_for2(items, 256), 256, 0, st>>>(L, T1, T2, a1, a2, static_cast<unsigned char*>(packed),
                                                        dev_status);
    return check_launch();
}

ptqtp_status launch_unpack2(const Layout2& L, const void* packed, int8_t* T1, int8_t* T2, uint16_t* a1,
                            uint16_t* a2, int32_t* dev_status, cudaStream_t st) {
    const size_t items = (size_t)L.nrp * (L.k / 16);
    unpack2_kernel<<<grid_for2(items, 256), 256, 0, st>>>(L, static_cast<const unsigned char*>(packed), T1, T2,
                                                          a1, a2, dev_status);
    return check_launch();
}

}  // namespace ptqtp
