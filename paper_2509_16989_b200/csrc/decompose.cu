// Progressive trit-plane decomposition W ~ alpha1 (.) T1 + alpha2 (.) T2 on the GPU (Algorithm 1 with the inner
// formulas of Algorithm 2 and Appendix C).  The step before the hot path: it produces what ptqtp_pack packs.
//
// Every group-row (G contiguous input columns of one output row, Sec. 2.3 "Batch Processing") is independent
// (Sec. 2.2: "for each i independently"), so one thread owns one group-row and the sweeps of Algorithm 1 are one
// kernel launch each:
//
//   init     t1 = t2 = sign(w) with 0 -> +1, alpha = (1, 1), lambda = 1e-8                     (Alg. 2 init)
//   alpha    S = [t1 t2], A = S^T S + lambda I, b = S^T w                                      (Eq. 3-5)
//            kappa = ||A||_F ||A^-1||_F = ||A||_F^2 / |det A| for the 2 x 2 system             (Eq. 6)
//            kappa >= 1e6: lambda <- min(lambda sqrt(kappa / 1e6), 1), used by this sweep's solve   (Alg. 2, App. C)
//            alpha = A^-1 b by the explicit 2 x 2 inverse                                      (App. B)
//   T        per element the pair (c1, c2) in {-1,0,1}^2 of smallest (w - (alpha1 c1 + alpha2 c2))^2, equal
//            errors resolved towards fewer non-zeros, then towards plane 1                     (Alg. 2 T-step)
//   stop     after the sweep in which the largest ||alpha_t - alpha_{t-1}||_2 over all group-rows falls below eps,
//            or after t_max sweeps                                                             (Alg. 1 last line)
//
// All arithmetic is IEEE double precision with every product and sum rounded on its own (no contraction into
// fused multiply-adds) and the sums over a group-row taken in column order, so a run is reproducible bit for bit
// and independent of the launch shape.  The stopping rule needs the maximum over the whole matrix: each sweep
// leaves it in the workspace (atomic maximum on the bit patterns of non-negative doubles, which order like the
// values), a one-thread kernel between two sweeps turns it into a "done" flag, and the sweeps after that return
// at once -- the call stays asynchronous, with 2 t_max + 1 small launches.
#include <cuda_fp16.h>
#include "ptqtp_internal.h"

namespace ptqtp {

namespace {

constexpr int kDecThreads = 128;

// Workspace: [0] int32 sweeps run, [1] int32 done; from byte 64: (t_max + 1) x u64 largest change of a scale pair per
// sweep (entry t for sweep t, 1-based), t_max x f64 total squared error after each sweep, then per group-row the
// scales alpha1, alpha2 and lambda (f64 each, R entries each).
struct DecLayout {
    size_t delta_off, err_off, a1_off, a2_off, lam_off, total;
};
__host__ __device__ inline DecLayout dec_layout(long long rows, int t_max) {
    DecLayout d;
    d.delta_off = 64;
    d.err_off = d.delta_off + (size_t)(t_max + 1) * 8;
    d.a1_off = (d.err_off + (size_t)t_max * 8 + 63) / 64 * 64;
    d.a2_off = d.a1_off + (size_t)rows * 8;
    d.lam_off = d.a2_off + (size_t)rows * 8;
    d.total = d.lam_off + (size_t)rows * 8;
    return d;
}

__global__ void dec_init_kernel(unsigned char* ws, int t_max) {
    const DecLayout d = dec_layout(0, t_max);
    int* ctl = reinterpret_cast<int*>(ws);
    for (int i = threadIdx.x; i < 16; i += blockDim.x) ctl[i] = 0;
    unsigned long long* delta = reinterpret_cast<unsigned long long*>(ws + d.delta_off);
    double* err = reinterpret_cast<double*>(ws + d.err_off);
    for (int i = threadIdx.x; i <= t_max; i += blockDim.x) delta[i] = 0ull;
    for (int i = threadIdx.x; i < t_max; i += blockDim.x) err[i] = 0.0;
}

// After sweep `sweep`: record it as run and raise the flag when the largest change fell below eps.
__global__ void dec_check_kernel(unsigned char* ws, int t_max, int sweep, double eps) {
    int* ctl = reinterpret_cast<int*>(ws);
    if (ctl[1]) return;
    const unsigned long long* delta = reinterpret_cast<const unsigned long long*>(ws + dec_layout(0, t_max).delta_off);
    ctl[0] = sweep;
    if (__longlong_as_double((long long)delta[sweep]) < eps) ctl[1] = 1;
}

// The nine candidate pairs in tie-break order: fewest non-zeros first, then a non-zero in plane 1.
__constant__ signed char kCand1[9] = {0, 1, -1, 0, 0, 1, -1, 1, -1};
__constant__ signed char kCand2[9] = {0, 0, 0, 1, -1, 1, -1, -1, 1};

// One sweep for every group-row.  Shared memory: w of the CTA's group-rows, element-major ([j][thread], so that
// the threads of a warp read consecutive words), and the trit pairs likewise as one byte each.
__global__ void __launch_bounds__(kDecThreads)
dec_sweep_kernel(const float* __restrict__ W, int8_t* __restrict__ T1, int8_t* __restrict__ T2, unsigned char* __restrict__ ws,
                 long long rows, int G, int t_max, int sweep, double lambda0, double lambda_max, double kappa_thr) {
    const int* ctl = reinterpret_cast<const int*>(ws);
    if (ctl[1]) return;                                 // the stopping rule was met by an earlier sweep
    extern __shared__ __align__(16) unsigned char smem[];
    float* sw = reinterpret_cast<float*>(smem);                         // [G][kDecThreads]
    unsigned char* st = smem + (size_t)G * kDecThreads * 4;             // [G][kDecThreads]: (t1 + 1) | (t2 + 1) << 2
    const DecLayout d = dec_layout(rows, t_max);
    double* A1 = reinterpret_cast<double*>(ws + d.a1_off);
    double* A2 = reinterpret_cast<double*>(ws + d.a2_off);
    double* LAM = reinterpret_cast<double*>(ws + d.lam_off);
    const long long r0 = (long long)blockIdx.x * kDecThreads;
    const int nrows = (int)min((long long)kDecThreads, rows - r0);
    const int tid = threadIdx.x;

    // the CTA's group-rows are contiguous in memory: coalesced reads, transposed into shared memory
    const size_t base = (size_t)r0 * G;
    const int total = nrows * G;
    for (int i = tid; i < total; i += kDecThreads) {
        const int r = i / G, j = i - r * G;
        const float w = W[base + i];
        sw[j * kDecThreads + r] = w;
        unsigned char code;
        if (sweep == 1) {
            const unsigned char s = w >= 0.f ? 2 : 0;   // sign(w) with 0 -> +1, both planes
            code = s | (s << 2);
        } else {
            code = (unsigned char)((T1[base + i] + 1) | ((T2[base + i] + 1) << 2));
        }
        st[j * kDecThreads + r] = code;
    }
    __syncthreads();

    if (tid < nrows) {
        const long long r = r0 + tid;
        double a1_old = 1.0, a2_old = 1.0, lam = lambda0;
        if (sweep > 1) { a1_old = A1[r]; a2_old = A2[r]; lam = LAM[r]; }
        // alpha-step: sums in column order (products of a trit with a number are exact)
        double n11 = 0.0, n22 = 0.0, n12 = 0.0, b1 = 0.0, b2 = 0.0;
        for (int j = 0; j < G; ++j) {
            const unsigned char c = st[j * kDecThreads + tid];
            const double f1 = (double)((int)(c & 3) - 1), f2 = (double)((int)(c >> 2) - 1);
            const double w = (double)sw[j * kDecThreads + tid];
            n11 = __dadd_rn(n11, __dmul_rn(f1, f1));
            n22 = __dadd_rn(n22, __dmul_rn(f2, f2));
            n12 = __dadd_rn(n12, __dmul_rn(f1, f2));
            b1 = __dadd_rn(b1, __dmul_rn(f1, w));
            b2 = __dadd_rn(b2, __dmul_rn(f2, w));
        }
        double A11 = __dadd_rn(n11, lam), A22 = __dadd_rn(n22, lam);
        const double n12sq = __dmul_rn(n12, n12);
        double det = __dsub_rn(__dmul_rn(A11, A22), n12sq);
        const double fro = __dadd_rn(__dadd_rn(__dmul_rn(A11, A11), __dmul_rn(A22, A22)), __dmul_rn(__dmul_rn(2.0, n12), n12));
        const double kappa = __ddiv_rn(fro, fabs(det));
        if (kappa >= kappa_thr) lam = fmin(__dmul_rn(lam, __dsqrt_rn(__ddiv_rn(kappa, kappa_thr))), lambda_max);
        lam = fmax(lam, lambda0);
        A11 = __dadd_rn(n11, lam);
        A22 = __dadd_rn(n22, lam);
        det = __dsub_rn(__dmul_rn(A11, A22), n12sq);
        const double a1 = __ddiv_rn(__dsub_rn(__dmul_rn(A22, b1), __dmul_rn(n12, b2)), det);
        const double a2 = __ddiv_rn(__dsub_rn(__dmul_rn(A11, b2), __dmul_rn(n12, b1)), det);
        // T-step: the level of a candidate is formed first and then subtracted, so that structurally equal
        // candidates (alpha1 == alpha2 in the first sweep) have bit-equal errors and the order decides
        double level[9];
#pragma unroll
        for (int m = 0; m < 9; ++m)
            level[m] = __dadd_rn(__dmul_rn(a1, (double)kCand1[m]), __dmul_rn(a2, (double)kCand2[m]));
        double err = 0.0;
        for (int j = 0; j < G; ++j) {
            const double w = (double)sw[j * kDecThreads + tid];
            double dbest = __dsub_rn(w, level[0]);
            double best = __dmul_rn(dbest, dbest);
            int bm = 0;
#pragma unroll
            for (int m = 1; m < 9; ++m) {
                const double dm = __dsub_rn(w, level[m]);
                const double e = __dmul_rn(dm, dm);
                if (e < best) { best = e; bm = m; }     // strict: an equal error keeps the earlier candidate
            }
            const int c1 = kCand1[bm], c2 = kCand2[bm];
            st[j * kDecThreads + tid] = (unsigned char)((c1 + 1) | ((c2 + 1) << 2));
            // E = sum_j (w_j - (alpha1 t1_j + alpha2 t2_j))^2 with the chosen pair
            const double res = __dsub_rn(w, __dadd_rn(__dmul_rn(a1, (double)c1), __dmul_rn(a2, (double)c2)));
            err = __dadd_rn(err, __dmul_rn(res, res));
        }
        const double d1 = __dsub_rn(a1, a1_old), d2 = __dsub_rn(a2, a2_old);
        const double delta = __dsqrt_rn(__dadd_rn(__dmul_rn(d1, d1), __dmul_rn(d2, d2)));
        A1[r] = a1;
        A2[r] = a2;
        LAM[r] = lam;
        // NaN cannot arise (lambda >= 1e-8 keeps det away from 0); a non-negative double orders like its bit pattern
        atomicMax(reinterpret_cast<unsigned long long*>(ws + d.delta_off) + sweep, (unsigned long long)__double_as_longlong(delta));
        atomicAdd(reinterpret_cast<double*>(ws + d.err_off) + (sweep - 1), err);
    }
    __syncthreads();
    for (int i = tid; i < total; i += kDecThreads) {
        const int r = i / G, j = i - r * G;
        const unsigned char c = st[j * kDecThreads + r];
        T1[base + i] = (int8_t)((int)(c & 3) - 1);
        T2[base + i] = (int8_t)((int)(c >> 2) - 1);
    }
}

// Final pass: optional normal form that leaves W_hat unchanged (both scales non-negative by flipping (alpha_k, t_k),
// then alpha1 >= alpha2 by exchanging the planes of the group-row), and the scales rounded once to fp16.
__global__ void __launch_bounds__(kDecThreads)
dec_finish_kernel(int8_t* __restrict__ T1, int8_t* __restrict__ T2, unsigned char* __restrict__ ws, uint16_t* __restrict__ alpha1,
                  uint16_t* __restrict__ alpha2, long long rows, int G, int t_max, int canonicalize) {
    const DecLayout d = dec_layout(rows, t_max);
    double* A1 = reinterpret_cast<double*>(ws + d.a1_off);
    double* A2 = reinterpret_cast<double*>(ws + d.a2_off);
    // a warp per group-row: the lanes walk its elements
    const long long r = ((long long)blockIdx.x * kDecThreads + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    double a1 = A1[r], a2 = A2[r];
    const bool neg1 = canonicalize && a1 < 0.0, neg2 = canonicalize && a2 < 0.0;
    if (neg1) a1 = -a1;
    if (neg2) a2 = -a2;
    const bool swap = canonicalize && a1 < a2;
    if (canonicalize && (neg1 || neg2 || swap)) {
        const size_t base = (size_t)r * G;
        for (int j = lane; j < G; j += 32) {
            int8_t u = T1[base + j], v = T2[base + j];
            if (neg1) u = (int8_t)-u;
            if (neg2) v = (int8_t)-v;
            T1[base + j] = swap ? v : u;
            T2[base + j] = swap ? u : v;
        }
    }
    if (swap) { const double s = a1; a1 = a2; a2 = s; }
    if (lane == 0) {
        A1[r] = a1;
        A2[r] = a2;
        alpha1[r] = __half_as_ushort(__double2half(a1));
        alpha2[r] = __half_as_ushort(__double2half(a2));
    }
}

}  // namespace

size_t decompose_workspace_bytes(long long rows, int t_max) { return dec_layout(rows, t_max).total; }

void decompose_offsets(long long rows, int t_max, size_t* delta_off, size_t* err_off, size_t* a1_off, size_t* a2_off,
                       size_t* lam_off) {
    const DecLayout d = dec_layout(rows, t_max);
    *delta_off = d.delta_off; *err_off = d.err_off; *a1_off = d.a1_off; *a2_off = d.a2_off; *lam_off = d.lam_off;
}

ptqtp_status launch_decompose(const float* W, int n, int k, int G, int t_max, double eps, int canonicalize, int8_t* T1,
                              int8_t* T2, uint16_t* alpha1, uint16_t* alpha2, void* workspace, cudaStream_t st) {
    const long long rows = (long long)n * (k / G);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    const size_t smem = (size_t)G * kDecThreads * 5;
    ptqtp_status s = configure_once<dec_sweep_kernel>(false);
    if (s != PTQTP_OK) return s;
    const unsigned grid = (unsigned)((rows + kDecThreads - 1) / kDecThreads);
    dec_init_kernel<<<1, 64, 0, st>>>(ws, t_max);
    for (int sweep = 1; sweep <= t_max; ++sweep) {
        dec_sweep_kernel<<<grid, kDecThreads, smem, st>>>(W, T1, T2, ws, rows, G, t_max, sweep, 1e-8, 1.0, 1e6);
        dec_check_kernel<<<1, 1, 0, st>>>(ws, t_max, sweep, eps);
    }
    const unsigned fgrid = (unsigned)((rows * 32 + kDecThreads - 1) / kDecThreads);
    dec_finish_kernel<<<fgrid, kDecThreads, 0, st>>>(T1, T2, ws, alpha1, alpha2, rows, G, t_max, canonicalize);
    return check_launch();
}

}  // namespace ptqtp
