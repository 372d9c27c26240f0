// Small-batch variant Y[m,:] = layer(X[m,:]), 1 <= M <= 64.
// Provisional: one batch-1 pass per row of X (the planes are re-read from L2/HBM M times).
#include "ptqtp_internal.h"

namespace ptqtp {

ptqtp_status launch_gemm_skinny(const Layout& L, const void* packed, int m, const uint16_t* X, uint16_t* Y,
                                cudaStream_t st) {
    for (int i = 0; i < m; ++i) {
        ptqtp_status s = launch_gemv(L, packed, X + (size_t)i * L.k, Y + (size_t)i * L.n, 0, 0, 0, 0, -1, st);
        if (s != PTQTP_OK) return s;
    }
    return PTQTP_OK;
}

}  // namespace ptqtp
