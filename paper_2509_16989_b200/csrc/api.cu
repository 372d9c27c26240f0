// C ABI of libptqtp: argument validation and dispatch.  Declarations and contracts: include/ptqtp.h.
#include <string.h>
#include <atomic>
#include <mutex>
#include <vector>
#include "ptqtp_internal.h"

namespace ptqtp {

static thread_local int g_last_cuda_error = 0;
// Process-wide settings, read by every launch and written by their setters from any thread.
static std::atomic<int> g_overlap{0};                  // ptqtp_set_overlap: plain launches unless the caller opts in
static std::atomic<int> g_wait_limit{1 << 22};         // ptqtp_set_wait_limit
static std::atomic<int> g_fail_waits{0};               // ptqtp_test_fail_next_wait

bool overlap_enabled() { return g_overlap.load(std::memory_order_relaxed) != 0; }
int wait_poll_limit() { return g_wait_limit.load(std::memory_order_relaxed); }
bool take_injected_wait_failure() {
    int n = g_fail_waits.load(std::memory_order_relaxed);
    while (n > 0)
        if (g_fail_waits.compare_exchange_weak(n, n - 1)) return true;
    return false;
}

// Streams on which ptqtp_pack was the library's last call: the next GEMV launch there is a plain launch, so that
// it reads the packed planes only after the pack kernel has completed (a dependent launch reads them earlier).
static std::mutex g_pack_mutex;
static std::vector<cudaStream_t> g_pack_streams;
static bool g_pack_overflow = false;
void note_pack(cudaStream_t st) {
    std::lock_guard<std::mutex> lock(g_pack_mutex);
    for (cudaStream_t s : g_pack_streams)
        if (s == st) return;
    if (g_pack_streams.size() < 256) g_pack_streams.push_back(st); else g_pack_overflow = true;
}
bool consume_pack(cudaStream_t st) {
    std::lock_guard<std::mutex> lock(g_pack_mutex);
    if (g_pack_overflow) {                              // too many streams to remember: be plain once everywhere
        g_pack_overflow = false;
        g_pack_streams.clear();
        return true;
    }
    for (size_t i = 0; i < g_pack_streams.size(); ++i) {
        if (g_pack_streams[i] == st) {
            g_pack_streams.erase(g_pack_streams.begin() + i);
            return true;
        }
    }
    return false;
}
bool speculation_enabled() { return g_overlap.load(std::memory_order_relaxed) >= 2; }

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

// Layout of either format, as selected by shape->format.
struct AnyLayout {
    bool v2, v3;
    Layout l1;
    Layout2 l2;
    Layout3 l3;
};

static ptqtp_status check_packed(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, AnyLayout* L) {
    if (!shape || !packed) return PTQTP_ERR_NULL;
    if (!shape_ok(shape)) return PTQTP_ERR_SHAPE;
    L->v2 = shape->format == PTQTP_FORMAT_V2;
    L->v3 = shape->format == PTQTP_FORMAT_V3;
    if (L->v3) L->l3 = make_layout3(shape); else if (L->v2) L->l2 = make_layout2(shape); else L->l1 = make_layout(shape);
    if (!aligned16(packed)) return PTQTP_ERR_ALIGN;
    if (packed_bytes < packed_total(shape)) return PTQTP_ERR_SIZE;
    return PTQTP_OK;
}

static int default_gemv_arith() { return 3; }

static ptqtp_status gemv_any(const AnyLayout& L, const void* packed, const uint16_t* x, uint16_t* y, int p0, int p1,
                             int p2, int p3, int p4, cudaStream_t st) {
    if (L.v3) {
        if (p4 != -1 && p4 != 5) return PTQTP_ERR_CONFIG;
        return launch_gemv4(L.l3, packed, x, y, p1, p2, p3, p0, st);
    }
    if (L.v2) {
        if ((p4 != -1 && p4 != 3 && p4 != 4) || (p0 != 0 && p4 == 4)) return PTQTP_ERR_CONFIG;
        if (p4 == 4) {                       // tensor-core kernel
            const ptqtp_status s = launch_gemv3(L.l2, packed, 1, x, y, p1, p2, p3, st);
            return s == PTQTP_ERR_SHAPE ? PTQTP_ERR_CONFIG : s;
        }
        if (p2 > 4) return PTQTP_ERR_CONFIG;
        if (p4 == -1 && p0 == 0 && p1 == 0 && p2 == 0 && p3 == 0 && default_gemv_arith() == 4) {
            const ptqtp_status s = launch_gemv3(L.l2, packed, 1, x, y, 0, 0, 0, st);
            if (s != PTQTP_ERR_SHAPE) return s;          // very long K: the CUDA-core kernel takes it
        }
        return launch_gemv2(L.l2, packed, x, y, p1, p2, p3, p0, st);
    }
    return launch_gemv(L.l1, packed, x, y, p0, p1, p2, p3, p4, st);
}

}  // namespace ptqtp

using namespace ptqtp;

extern "C" {

size_t ptqtp_packed_size(const ptqtp_shape* shape) {
    if (!shape_ok(shape)) return 0;
    return packed_total(shape);
}

ptqtp_status ptqtp_pack(const ptqtp_shape* shape, const int8_t* T1, const int8_t* T2, const uint16_t* alpha1,
                        const uint16_t* alpha2, void* packed, size_t packed_bytes, int32_t* dev_status,
                        void* stream) {
    if (!T1 || !T2 || !alpha1 || !alpha2) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(T1) || !aligned16(T2) || !aligned16(alpha1) || !aligned16(alpha2)) return PTQTP_ERR_ALIGN;
    if (dev_status && (reinterpret_cast<uintptr_t>(dev_status) & 3u)) return PTQTP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    note_pack(st);
    return L.v3 ? launch_pack3(L.l3, T1, T2, alpha1, alpha2, packed, dev_status, st)
         : L.v2 ? launch_pack2(L.l2, T1, T2, alpha1, alpha2, packed, dev_status, st)
                : launch_pack(L.l1, T1, T2, alpha1, alpha2, packed, dev_status, st);
}

ptqtp_status ptqtp_unpack(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, int8_t* T1,
                          int8_t* T2, uint16_t* alpha1, uint16_t* alpha2, int32_t* dev_status, void* stream) {
    if (!T1 || !T2 || !alpha1 || !alpha2) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(T1) || !aligned16(T2) || !aligned16(alpha1) || !aligned16(alpha2)) return PTQTP_ERR_ALIGN;
    if (dev_status && (reinterpret_cast<uintptr_t>(dev_status) & 3u)) return PTQTP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return L.v3 ? launch_unpack3(L.l3, packed, T1, T2, alpha1, alpha2, dev_status, st)
         : L.v2 ? launch_unpack2(L.l2, packed, T1, T2, alpha1, alpha2, dev_status, st)
                : launch_unpack(L.l1, packed, T1, T2, alpha1, alpha2, dev_status, st);
}

ptqtp_status ptqtp_gemv_cfg(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, const uint16_t* x,
                            uint16_t* y, int32_t rows_per_warp, int32_t k_split, int32_t ctas_per_sm,
                            int32_t depth, int32_t arith, void* stream) {
    if (!x || !y) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(x) || !aligned16(y)) return PTQTP_ERR_ALIGN;
    if (rows_per_warp < 0 || k_split < -1 || ctas_per_sm < 0 || depth < 0 || arith < -1) return PTQTP_ERR_CONFIG;
    if (k_split < 0 && !L.v2 && !L.v3) return PTQTP_ERR_CONFIG;
    return gemv_any(L, packed, x, y, rows_per_warp, k_split, ctas_per_sm, depth, arith,
                    static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_gemv(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, const uint16_t* x,
                        uint16_t* y, void* stream) {
    return ptqtp_gemv_cfg(shape, packed, packed_bytes, x, y, 0, 0, 0, 0, -1, stream);
}

ptqtp_status ptqtp_gemv_swiglu(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, const uint16_t* x,
                               uint16_t* y, void* stream) {
    if (!x || !y) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!L.v2 && !L.v3) return PTQTP_ERR_CONFIG;
    if (shape->n_out % 2) return PTQTP_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return PTQTP_ERR_ALIGN;
    if (L.v3) return launch_gemv4(L.l3, packed, x, y, 0, 0, 0, 0, static_cast<cudaStream_t>(stream), true);
    return launch_gemv2(L.l2, packed, x, y, 0, 0, 0, 0, static_cast<cudaStream_t>(stream), true);
}

static bool decompose_args_ok(int32_t n, int32_t k, int32_t group, int32_t t_max) {
    return n > 0 && k > 0 && group >= 1 && group <= PTQTP_DECOMPOSE_MAX_GROUP && k % group == 0 && t_max >= 1 &&
           t_max <= PTQTP_DECOMPOSE_MAX_SWEEPS;
}

size_t ptqtp_decompose_workspace_size(int32_t n, int32_t k, int32_t group, int32_t t_max) {
    if (!decompose_args_ok(n, k, group, t_max)) return 0;
    return decompose_workspace_bytes((long long)n * (k / group), t_max);
}

ptqtp_status ptqtp_decompose_layout(int32_t n, int32_t k, int32_t group, int32_t t_max, ptqtp_decompose_offsets* out) {
    if (!out) return PTQTP_ERR_NULL;
    if (!decompose_args_ok(n, k, group, t_max)) return PTQTP_ERR_SHAPE;
    out->sweeps_offset = 0;
    decompose_offsets((long long)n * (k / group), t_max, &out->delta_offset, &out->error_offset, &out->alpha1_offset,
                      &out->alpha2_offset, &out->lambda_offset);
    out->total_bytes = decompose_workspace_bytes((long long)n * (k / group), t_max);
    return PTQTP_OK;
}

ptqtp_status ptqtp_decompose(const float* W, int32_t n, int32_t k, int32_t group, int32_t t_max, double eps,
                             int32_t canonicalize, int8_t* T1, int8_t* T2, uint16_t* alpha1, uint16_t* alpha2,
                             void* workspace, size_t workspace_bytes, void* stream) {
    if (!W || !T1 || !T2 || !alpha1 || !alpha2 || !workspace) return PTQTP_ERR_NULL;
    if (!decompose_args_ok(n, k, group, t_max) || !(eps >= 0.0)) return PTQTP_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(T1) || !aligned16(T2) || !aligned16(alpha1) || !aligned16(alpha2) || !aligned16(workspace))
        return PTQTP_ERR_ALIGN;
    if (workspace_bytes < decompose_workspace_bytes((long long)n * (k / group), t_max)) return PTQTP_ERR_SIZE;
    return launch_decompose(W, n, k, group, t_max, eps, canonicalize ? 1 : 0, T1, T2, alpha1, alpha2, workspace,
                            static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_gemv_multi(int32_t count, const ptqtp_shape* shapes, const void* const* packed,
                              const size_t* packed_bytes, const uint16_t* x, uint16_t* const* y, int32_t epilogue,
                              void* stream) {
    if (!shapes || !packed || !packed_bytes || !x || !y) return PTQTP_ERR_NULL;
    if (count < 1 || count > kMaxJobs4) return PTQTP_ERR_SHAPE;
    if (epilogue != PTQTP_EPILOGUE_NONE && epilogue != PTQTP_EPILOGUE_GATED_PAIR) return PTQTP_ERR_CONFIG;
    if (!aligned16(x)) return PTQTP_ERR_ALIGN;
    const bool pair = epilogue == PTQTP_EPILOGUE_GATED_PAIR;
    if (pair && (count != 2 || shapes[0].n_out != shapes[1].n_out)) return PTQTP_ERR_SHAPE;
    Jobs4 J = {};
    for (int j = 0; j < count; ++j) {
        AnyLayout L;
        ptqtp_status s = check_packed(&shapes[j], packed[j], packed_bytes[j], &L);
        if (s != PTQTP_OK) return s;
        if (!L.v3) return PTQTP_ERR_CONFIG;
        if (shapes[j].k_in != shapes[0].k_in) return PTQTP_ERR_SHAPE;
        uint16_t* yj = pair && j == 1 ? y[0] : y[j];     // the pair has one output
        if (!yj) return PTQTP_ERR_NULL;
        if (!aligned16(yj)) return PTQTP_ERR_ALIGN;
        add_job4(J, L.l3, packed[j], yj);
    }
    return launch_gemv4_jobs(J, x, 0, 0, 0, 0, static_cast<cudaStream_t>(stream), pair ? 2 : 0);
}

// Small batch on format 3.  path 5: up to four rows per pass over the planes on the warp-MMA kernel whose MMA columns
// are the rows (two rows cost about a batch-1 pass, four about one and a half); when four rows of x leave no room in
// shared memory its passes take two rows, or one on the batch-1 kernel.  path 6: the tcgen05 kernel, all rows in one
// pass.  path 0: whichever the measured costs below make cheaper -- the tcgen05 kernel has a fixed cost of several
// microseconds and a cost per byte that grows slowly with the rows, the passes cost a batch-1 call each.
static bool tcgen05_is_cheaper(const Layout3& L3, int m) {
    if (m < 5) return false;
    const double mb = (double)L3.total / 1e6;
    const int npad = (m + 15) / 16 * 16;
    const double us6 = 7.5 + mb * (0.52 + 0.015 * npad);
    const double rate4 = L3.k > 8192 ? 1.15 : 2.1, rate2 = 2.0 * rate4;           // MB per microsecond of a pass
    const int full = m / 4, rest = m % 4;
    const double us5 = full * (1.2 + mb / rate4) + (rest > 2 ? 1.2 + mb / rate4 : rest > 0 ? 1.2 + mb / rate2 : 0.0);
    return us6 < us5;
}
static ptqtp_status skinny_v3(const Layout3& L3, const ptqtp_shape* shape, const void* packed, int m, const uint16_t* X,
                              uint16_t* Y, int path, int k_split, cudaStream_t st) {
    if (path == 6 || (path == 0 && tcgen05_is_cheaper(L3, m))) return launch_gemm6(L3, packed, m, X, Y, k_split, st);
    int per_pass = m < 4 ? m : 4;
    int done = 0;
    while (done < m) {
        const uint16_t* Xp = X + (size_t)done * shape->k_in;
        uint16_t* Yp = Y + (size_t)done * shape->n_out;
        const int rows = m - done < per_pass ? m - done : per_pass;
        ptqtp_status sp = rows == 1 ? launch_gemv4(L3, packed, Xp, Yp, 0, 0, 0, 0, st)
                                    : launch_gemv5(L3, packed, rows, Xp, Yp, 0, 0, st);
        if (sp == PTQTP_ERR_SHAPE && rows > 1 && done == 0) { per_pass = per_pass > 2 ? 2 : 1; continue; }   // nothing launched yet
        if (sp != PTQTP_OK) return sp;
        done += rows;
    }
    return PTQTP_OK;
}

ptqtp_status ptqtp_gemm_skinny(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, int32_t m,
                               const uint16_t* X, uint16_t* Y, void* stream) {
    if (!X || !Y) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (m < 1 || m > PTQTP_MAX_BATCH) return PTQTP_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(Y)) return PTQTP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (L.v2) {
        // Up to four rows cost about the same as one on the register-stationary tensor-core kernel; more rows take
        // one pass per four (ptqtp_gemm_skinny_ws reads the planes only once).  When four rows of x leave no room in
        // shared memory the passes take three, two or, on the batch-1 kernel, one row.
        if (m >= 2) {
            int per_pass = m < 4 ? m : 4;
            int done = 0;
            while (done < m) {
                const uint16_t* Xp = X + (size_t)done * shape->k_in;
                uint16_t* Yp = Y + (size_t)done * shape->n_out;
                const int rows = m - done < per_pass ? m - done : per_pass;
                ptqtp_status sp = rows == 1 ? launch_gemv2(L.l2, packed, Xp, Yp, 0, 0, 0, 0, st)
                                            : launch_gemv3(L.l2, packed, rows, Xp, Yp, 0, 0, 0, st);
                if (sp == PTQTP_ERR_SHAPE && rows > 1 && done == 0) { --per_pass; continue; }   // nothing launched yet
                if (sp != PTQTP_OK) return sp;
                done += rows;
            }
            return PTQTP_OK;
        }
        return launch_gemv2(L.l2, packed, X, Y, 0, 0, 0, 0, st);
    }
    if (L.v3) return skinny_v3(L.l3, shape, packed, m, X, Y, 0, 0, st);
    // format 1 is a batch-1 layout
    if (m != 1) return PTQTP_ERR_CONFIG;
    return gemv_any(L, packed, X, Y, 0, 0, 0, 0, -1, st);
}

ptqtp_status ptqtp_gemm_skinny_cfg(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, int32_t m,
                                   const uint16_t* X, uint16_t* Y, int32_t path, int32_t k_split, void* stream) {
    if (!X || !Y) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (m < 1 || m > PTQTP_MAX_BATCH) return PTQTP_ERR_SHAPE;
    if (!L.v3 || (path != 0 && path != 5 && path != 6)) return PTQTP_ERR_CONFIG;
    if (!aligned16(X) || !aligned16(Y)) return PTQTP_ERR_ALIGN;
    return skinny_v3(L.l3, shape, packed, m, X, Y, path, k_split, static_cast<cudaStream_t>(stream));
}

size_t ptqtp_gemm_skinny_workspace_size(const ptqtp_shape* shape, int32_t m) {
    if (!shape_ok(shape) || shape->format != PTQTP_FORMAT_V2 || m < 1 || m > PTQTP_MAX_BATCH) return 0;
    return skinny3_workspace_bytes(shape->k_in, m);
}

ptqtp_status ptqtp_gemm_skinny_ws(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, int32_t m,
                                  const uint16_t* X, uint16_t* Y, void* workspace, size_t workspace_bytes,
                                  void* stream) {
    if (!X || !Y || !workspace) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (m < 1 || m > PTQTP_MAX_BATCH) return PTQTP_ERR_SHAPE;
    if (!L.v2) return PTQTP_ERR_CONFIG;
    if (!aligned16(X) || !aligned16(Y) || !aligned16(workspace)) return PTQTP_ERR_ALIGN;
    if (workspace_bytes < skinny3_workspace_bytes(shape->k_in, m)) return PTQTP_ERR_SIZE;
    return launch_skinny3(L.l2, packed, m, X, Y, workspace, static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_gemm_skinny_static(const ptqtp_shape* shape, const void* packed, size_t packed_bytes, int32_t m,
                                      const uint16_t* X, uint16_t* Y, void* stream) {
    if (!X || !Y) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (m < 1 || m > PTQTP_MAX_BATCH) return PTQTP_ERR_SHAPE;
    if (!L.v2) return PTQTP_ERR_CONFIG;
    if (!aligned16(X) || !aligned16(Y)) return PTQTP_ERR_ALIGN;
    if (skinny3_workspace_bytes(shape->k_in, m) > (size_t)PTQTP_STATIC_WORKSPACE_BYTES) return PTQTP_ERR_SIZE;
    void* workspace = nullptr;
    s = static_workspace_address(&workspace);
    if (s != PTQTP_OK) return s;
    return launch_skinny3(L.l2, packed, m, X, Y, workspace, static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_gemv_host(const ptqtp_shape* shape, const void* packed, size_t packed_bytes,
                             const uint16_t* x_host, uint16_t* y_host, uint16_t* x_dev, uint16_t* y_dev,
                             void* stream) {
    if (!x_host || !y_host || !x_dev || !y_dev) return PTQTP_ERR_NULL;
    AnyLayout L;
    ptqtp_status s = check_packed(shape, packed, packed_bytes, &L);
    if (s != PTQTP_OK) return s;
    if (!aligned16(x_dev) || !aligned16(y_dev)) return PTQTP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(x_dev, x_host, (size_t)shape->k_in * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    // When y_host is pinned memory that the device can address (any pinned allocation under unified addressing),
    // the kernel stores y there itself and the copy back is saved; otherwise y goes through y_dev.
    uint16_t* y_target = y_dev;
    bool direct = false;
    if ((L.v2 || L.v3) && aligned16(y_host)) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, y_host) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
            attr.devicePointer != nullptr) {
            y_target = static_cast<uint16_t*>(attr.devicePointer);
            direct = true;
        } else {
            (void)cudaGetLastError();                    // pageable memory: not an error for this call
        }
    }
    // between its two copies the kernel never overlaps another GEMV: it gets whole SMs
    s = L.v3 ? launch_gemv4(L.l3, packed, x_dev, y_target, -1, 0, 0, 0, st)
      : L.v2 ? launch_gemv2(L.l2, packed, x_dev, y_target, -1, 0, 0, 0, st)
             : gemv_any(L, packed, x_dev, y_dev, 0, 0, 0, 0, -1, st);
    if (s != PTQTP_OK) return s;
    if (!direct) {
        e = cudaMemcpyAsync(y_host, y_dev, (size_t)shape->n_out * 2, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    }
    return PTQTP_OK;
}

ptqtp_status ptqtp_parse_header(const void* header_host, size_t bytes, ptqtp_shape* shape) {
    if (!header_host || !shape) return PTQTP_ERR_NULL;
    if (bytes < sizeof(Header)) return PTQTP_ERR_SIZE;
    Header h;
    memcpy(&h, header_host, sizeof(Header));
    if (memcmp(h.magic, "PTQTPB2\0", 8) != 0 || h.version != kVersion ||
        (h.format != PTQTP_FORMAT_V1 && h.format != PTQTP_FORMAT_V2 && h.format != PTQTP_FORMAT_V3))
        return PTQTP_ERR_FORMAT;
    ptqtp_shape s = {h.n, h.k, h.group, (int32_t)h.format};
    if (!shape_ok(&s)) return PTQTP_ERR_FORMAT;
    if (h.format == PTQTP_FORMAT_V1) {
        const Layout L = make_layout(&s);
        if (h.k_pad != L.k_pad || h.codes_off != L.codes_off || h.scales_off != L.scales_off || h.total != L.total)
            return PTQTP_ERR_FORMAT;
    } else if (h.format == PTQTP_FORMAT_V3) {
        const Layout3 L = make_layout3(&s);
        if (h.k_pad != L.sbs * kSuper3 || h.codes_off != L.codes_off || h.scales_off != (uint64_t)kTile3 ||
            h.total != L.total)
            return PTQTP_ERR_FORMAT;
    } else {
        const Layout2 L = make_layout2(&s);
        if (h.k_pad != L.slices * kSlice2 || h.codes_off != L.codes_off || h.scales_off != L.strip ||
            h.total != L.total)
            return PTQTP_ERR_FORMAT;
    }
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

ptqtp_status ptqtp_kernel_status(int32_t* status_host, void* stream) {
    if (!status_host) return PTQTP_ERR_NULL;
    return copy_gemv2_status(status_host, static_cast<cudaStream_t>(stream));
}

ptqtp_status ptqtp_kernel_status_clear(void* stream) {
    int* word = nullptr;
    ptqtp_status s = gemv_status_word(&word);
    if (s != PTQTP_OK) return s;
    cudaError_t e = cudaMemsetAsync(word, 0, sizeof(int), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { set_last_cuda_error(e); return PTQTP_ERR_CUDA; }
    return PTQTP_OK;
}

int ptqtp_set_overlap(int level) {
    return g_overlap.exchange(level <= 0 ? 0 : level >= 2 ? 2 : 1);
}

int ptqtp_set_wait_limit(int polls) {
    return g_wait_limit.exchange(polls < 1 ? 1 : polls);
}

void ptqtp_test_fail_next_wait(int launches) {
    g_fail_waits.store(launches < 0 ? 0 : launches);
}

int ptqtp_version(void) { return 100; }

}  // extern "C"
