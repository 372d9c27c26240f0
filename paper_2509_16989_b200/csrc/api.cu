// C ABI of libptqtp: argument validation and dispatch.  Declarations and contracts: include/ptqtp.h.
#include <string.h>
#include "ptqtp_internal.h"

namespace ptqtp {

static thread_local int g_last_cuda_error = 0;

void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

ptqtp_status check_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return PTQTP_ERR_CUDA;
    }
    return PTQTP_OK;
}

int sm_count() {
    // cached per device; a failed query falls back to the B200 count
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached = n;
        cached_dev = dev;
    }
    return cached;
}

static ptqtp_status check_packed(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, Layout* L) {
    if (!shape || !packed) return PTQTP_ERR_NULL;
    if (!shape_ok(shape)) return PTQTP_ERR_SHAPE;
    *L = make_layout(shape);
    if (!aligned16(packed)) return PTQTP_ERR_ALIGN;
    if (packed_bytes < L->total) return PTQTP_ERR_SIZE;
    return PTQTP_OK;
}

}  // namespace ptqtp

using namespace ptqtp;

extern "C" {

size_t ptqtp_packed_size(const ptqtp_shape* shape) {
    if (!shape_ok(shape)) return 0;
    return make_layout(shape).total;
}

ptqtp_status ptqtp_pack(const ptqtp_shape* shape, const int8_t* T1, const int8_t* T2, const uint16_t* alpha1,
                        const uint16_t* alpha2, void* packed, size_t packed_bytes, int32_t* dev_status,
                        void* stream) {
    if (!T1 || !T2 || !alpha1 || !alpha2) return PTQTP_ERR_NULL;
    Layout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(T1) || !aligned16(T2) || !aligned16(alpha1) || !aligned16(alpha2)) return PTQTP_ERR_ALIGN;
    if (dev_status && (reinterpret_cast<uintptr_t>(dev_status) & 3u)) return PTQTP_ERR_ALIGN;
    return launch_pack(L, T1, T2, alpha1, alpha2, packed, dev_status, static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_unpack(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, int8_t* T1,
                          int8_t* T2, uint16_t* alpha1, uint16_t* alpha2, int32_t* dev_status, void* stream) {
    if (!T1 || !T2 || !alpha1 || !alpha2) return PTQTP_ERR_NULL;
    Layout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(T1) || !aligned16(T2) || !aligned16(alpha1) || !aligned16(alpha2)) return PTQTP_ERR_ALIGN;
    if (dev_status && (reinterpret_cast<uintptr_t>(dev_status) & 3u)) return PTQTP_ERR_ALIGN;
    return launch_unpack(L, packed, T1, T2, alpha1, alpha2, dev_status, static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_gemv_cfg(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, const uint16_t* x,
                            uint16_t* y, int32_t rows_per_warp, int32_t k_split, int32_t ctas_per_sm,
                            int32_t depth, int32_t arith, void* stream) {
    if (!x || !y) return PTQTP_ERR_NULL;
    Layout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(x) || !aligned16(y)) return PTQTP_ERR_ALIGN;
    if (rows_per_warp < 0 || k_split < 0 || ctas_per_sm < 0 || depth < 0 || arith < -1) return PTQTP_ERR_CONFIG;
    return launch_gemv(L, packed, x, y, rows_per_warp, k_split, ctas_per_sm, depth, arith,
                       static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_gemv(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, const uint16_t* x,
                        uint16_t* y, void* stream) {
    return ptqtp_gemv_cfg(shape, packed, packed_bytes, x, y, 0, 0, 0, 0, -1, stream);
}

ptqtp_status ptqtp_gemm_skinny(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, int32_t m,
                               const uint16_t* X, uint16_t* Y, void* stream) {
    if (!X || !Y) return PTQTP_ERR_NULL;
    Layout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (m < 1 || m > PTQTP_MAX_BATCH) return PTQTP_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(Y)) return PTQTP_ERR_ALIGN;
    return launch_gemm_skinny(L, packed, m, X, Y, static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_gemv_host(const ptqtp_shape* shape, const void* packed, size_t packed_bytes,
                             const uint16_t* x_host, uint16_t* y_host, uint16_t* x_dev, uint16_t* y_dev,
                             void* stream) {
    if (!x_host || !y_host || !x_dev || !y_dev) return PTQTP_ERR_NULL;
    Layout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(x_dev) || !aligned16(y_dev)) return PTQTP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(x_dev, x_host, (size_t)L.k * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    s = launch_gemv(L, packed, x_dev, y_dev, 0, 0, 0, 0, -1, st);
    if (s != PTQTP_OK) return s;
    e = cudaMemcpyAsync(y_host, y_dev, (size_t)L.n * 2, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

ptqtp_status ptqtp_parse_header(const void* header_host, size_t bytes, ptqtp_shape* shape) {
    if (!header_host || !shape) return PTQTP_ERR_NULL;
    if (bytes < sizeof(Header)) return PTQTP_ERR_SIZE;
    Header h;
    memcpy(&h, header_host, sizeof(Header));
    if (memcmp(h.magic, "PTQTPB2\0", 8) != 0 || h.version != kVersion || h.format != PTQTP_FORMAT_V1)
        return PTQTP_ERR_FORMAT;
    ptqtp_shape s = {h.n, h.k, h.group, (int32_t)h.format};
    if (!shape_ok(&s)) return PTQTP_ERR_FORMAT;
    const Layout L = make_layout(&s);
    if (h.k_pad != L.k_pad || h.codes_off != L.codes_off || h.scales_off != L.scales_off || h.total != L.total)
        return PTQTP_ERR_FORMAT;
    *shape = s;
    return PTQTP_OK;
}

const char* ptqtp_status_string(ptqtp_status status) {
    switch (status) {
        case PTQTP_OK: return "ok";
        case PTQTP_ERR_NULL: return "null pointer";
        case PTQTP_ERR_SHAPE: return "bad shape (N, K > 0, K % 128 == 0, group == 128, 1 <= M <= 64)";
        case PTQTP_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case PTQTP_ERR_SIZE: return "packed buffer too small";
        case PTQTP_ERR_TRIT: return "plane entry outside {-1,0,1}";
        case PTQTP_ERR_FORMAT: return "packed header does not match";
        case PTQTP_ERR_CUDA: return "CUDA runtime error";
        case PTQTP_ERR_CONFIG: return "unsupported launch configuration";
    }
    return "unknown status";
}

int ptqtp_last_cuda_error(void) { return g_last_cuda_error; }

int ptqtp_version(void) { return 100; }

}  // extern "C"
