/* CPU oracle in plain C: the fp64 layer product and the progressive trit-plane decomposition.
 * TEST INFRASTRUCTURE ONLY -- never linked into or called by the CUDA library.
 *
 * It restates oracle/layer.py and oracle/decompose.py as scalar loops so that (a) the layer
 * product can be timed on the host cores as the reported CPU baseline and (b) whole
 * LLaMA-shaped matrices can be decomposed in minutes.  Every sum runs sequentially in j and
 * the file is compiled with -ffp-contract=off, so results equal the numpy oracle bit for bit.
 *
 * Layer product: Eq. 1-2 with one scale pair per output row per group of G input columns
 * (Sec. 2.3 "Batch Processing"); a trit contributes +x, -x or nothing (Sec. 4).
 * Decomposition: Algorithm 1 (sweeps over all group-rows, stop when the largest change of a
 * scale pair is below eps), inner formulas of Algorithm 2 / Appendix C, 2x2 inverse of
 * Appendix B ("Computational Complexity").
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* IEEE binary16 bit pattern -> double, exactly. */
static double half_bits_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int frac = h & 0x3ff;
    double v;
    if (expo == 0)
        v = ldexp((double)frac, -24);                 /* zero and subnormals */
    else if (expo == 31)
        v = frac ? NAN : INFINITY;
    else
        v = ldexp((double)(frac + 1024), expo - 25);  /* (1 + frac/1024) * 2^(expo-15) */
    return sign ? -v : v;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* y[m*N + i] = sum_g ( a1[i,g] * sum_{j in g} T1[i,j] x[m,j] + a2[i,g] * sum_{j in g} T2[i,j] x[m,j] )
 * T1,T2: int8 [N*K] row-major; a1,a2: fp16 bits [N*(K/G)]; x: fp16 bits [M*K]; y: double [M*N]. */
void oracle_layer_fp64(const int8_t *T1, const int8_t *T2, const uint16_t *a1, const uint16_t *a2,
                       const uint16_t *x, int N, int K, int G, int M, double *y, int threads)
{
    int ngroups = K / G;
    double *xd = (double *)malloc(sizeof(double) * (size_t)M * K);
    for (size_t q = 0; q < (size_t)M * K; ++q) xd[q] = half_bits_to_double(x[q]);
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int i = 0; i < N; ++i) {
        for (int m = 0; m < M; ++m) {
            const double *xm = xd + (size_t)m * K;
            double acc = 0.0;
            for (int g = 0; g < ngroups; ++g) {
                double s1 = 0.0, s2 = 0.0;
                for (int j = g * G; j < (g + 1) * G; ++j) {
                    int t1 = T1[(size_t)i * K + j];
                    int t2 = T2[(size_t)i * K + j];
                    if (t1 == 1) s1 += xm[j]; else if (t1 == -1) s1 -= xm[j];
                    if (t2 == 1) s2 += xm[j]; else if (t2 == -1) s2 -= xm[j];
                }
                acc += half_bits_to_double(a1[(size_t)i * ngroups + g]) * s1
                     + half_bits_to_double(a2[(size_t)i * ngroups + g]) * s2;
            }
            y[(size_t)m * N + i] = acc;
        }
    }
    free(xd);
}

/* Candidate pairs in tie-break order: 0 = fewest non-zeros first, then plane 1; 1 = meshgrid. */
static const int CAND_SPARSE[9][2] = {{0,0},{1,0},{-1,0},{0,1},{0,-1},{1,1},{-1,-1},{1,-1},{-1,1}};
static const int CAND_MESH[9][2]   = {{-1,-1},{-1,0},{-1,1},{0,-1},{0,0},{0,1},{1,-1},{1,0},{1,1}};

/* One sweep of one group-row: alpha-step then T-step.  Returns the squared error after the T-step. */
static double sweep_group_row(const double *w, int G, int8_t *t1, int8_t *t2, double *pa1, double *pa2,
                              double *plam, double lambda0, double lambda_max, double kappa_thr,
                              const int (*cand)[2], int update_then_solve)
{
    double n11 = 0, n22 = 0, n12 = 0, b1 = 0, b2 = 0;
    for (int j = 0; j < G; ++j) { double f1 = t1[j]; n11 = n11 + f1 * f1; }
    for (int j = 0; j < G; ++j) { double f2 = t2[j]; n22 = n22 + f2 * f2; }
    for (int j = 0; j < G; ++j) { double f1 = t1[j], f2 = t2[j]; n12 = n12 + f1 * f2; }
    for (int j = 0; j < G; ++j) { double f1 = t1[j]; b1 = b1 + f1 * w[j]; }
    for (int j = 0; j < G; ++j) { double f2 = t2[j]; b2 = b2 + f2 * w[j]; }
    double lam = *plam;
    double A11 = n11 + lam, A22 = n22 + lam, A12 = n12;
    double det = A11 * A22 - A12 * A12;
    double kappa = (A11 * A11 + A22 * A22 + 2.0 * A12 * A12) / fabs(det);
    double lam_grown = lam;
    if (kappa >= kappa_thr) {
        lam_grown = lam * sqrt(kappa / kappa_thr);
        if (lam_grown > lambda_max) lam_grown = lambda_max;
    }
    if (lam_grown < lambda0) lam_grown = lambda0;
    if (update_then_solve) {
        lam = lam_grown;
        A11 = n11 + lam;
        A22 = n22 + lam;
    }
    det = A11 * A22 - A12 * A12;
    double a1 = (A22 * b1 - A12 * b2) / det;
    double a2 = (A11 * b2 - A12 * b1) / det;
    *plam = lam_grown;
    *pa1 = a1;
    *pa2 = a2;
    double level[9];
    for (int m = 0; m < 9; ++m) level[m] = a1 * cand[m][0] + a2 * cand[m][1];
    for (int j = 0; j < G; ++j) {
        int best = 0;
        double d0 = w[j] - level[0];
        double best_err = d0 * d0;
        for (int m = 1; m < 9; ++m) {
            double d = w[j] - level[m];
            double e = d * d;
            if (e < best_err) { best_err = e; best = m; }
        }
        t1[j] = (int8_t)cand[best][0];
        t2[j] = (int8_t)cand[best][1];
    }
    double E = 0.0;
    for (int j = 0; j < G; ++j) {
        double r = w[j] - (a1 * (double)t1[j] + a2 * (double)t2[j]);
        E = E + r * r;
    }
    return E;
}

/* Decompose W [N*K] (fp32, row-major).  Outputs: T1,T2 int8 [N*K]; a1,a2 double [N*K/G];
 * err_hist double [T_max] (total squared error after each sweep); delta_hist double [T_max].
 * tie_break: 0 sparse-first, 1 meshgrid.  lambda_order: 0 update-then-solve, 1 solve-then-update.
 * conv_rule: 0 max over group-rows, 1 Frobenius over all, 2 per-group freeze.
 * Returns the number of sweeps run, or -1 on bad arguments. */
int oracle_decompose(const float *W, int N, int K, int G, int T_max, double eps, double lambda0,
                     double lambda_max, double kappa_thr, int tie_break, int lambda_order,
                     int conv_rule, int canonicalize, int8_t *T1, int8_t *T2, double *a1, double *a2,
                     double *err_hist, double *delta_hist, int threads)
{
    if (N <= 0 || K <= 0 || G <= 0 || K % G != 0 || T_max < 1) return -1;
    if (tie_break < 0 || tie_break > 1 || lambda_order < 0 || lambda_order > 1 || conv_rule < 0 || conv_rule > 2)
        return -1;
    const int (*cand)[2] = tie_break == 0 ? CAND_SPARSE : CAND_MESH;
    size_t R = (size_t)N * (K / G);
    double *lam = (double *)malloc(sizeof(double) * R);
    double *err = (double *)malloc(sizeof(double) * R);
    double *delta = (double *)malloc(sizeof(double) * R);
    unsigned char *frozen = (unsigned char *)calloc(R, 1);
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (size_t r = 0; r < R; ++r) {
        for (int j = 0; j < G; ++j) {
            int8_t s = W[r * G + j] >= 0.0f ? 1 : -1;
            T1[r * G + j] = s;
            T2[r * G + j] = s;
        }
        a1[r] = 1.0;
        a2[r] = 1.0;
        lam[r] = lambda0;
        err[r] = 0.0;
    }
    int sweeps = 0;
    for (int t = 1; t <= T_max; ++t) {
        ++sweeps;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 256)
        for (size_t r = 0; r < R; ++r) {
            if (frozen[r]) { delta[r] = 0.0; continue; }
            double wd[1024];
            double *w = G <= 1024 ? wd : (double *)malloc(sizeof(double) * G);
            for (int j = 0; j < G; ++j) w[j] = (double)W[r * G + j];
            double p1, p2;
            err[r] = sweep_group_row(w, G, T1 + r * G, T2 + r * G, &p1, &p2, &lam[r], lambda0, lambda_max,
                                     kappa_thr, cand, lambda_order == 0);
            double d1 = p1 - a1[r], d2 = p2 - a2[r];
            delta[r] = sqrt(d1 * d1 + d2 * d2);
            a1[r] = p1;
            a2[r] = p2;
            if (w != wd) free(w);
        }
        double E = 0.0, dmax = 0.0, dsq = 0.0;
        for (size_t r = 0; r < R; ++r) {
            E = E + err[r];
            if (delta[r] > dmax) dmax = delta[r];
            dsq = dsq + delta[r] * delta[r];
        }
        err_hist[t - 1] = E;
        delta_hist[t - 1] = dmax;
        int stop = 0;
        if (conv_rule == 0) stop = dmax < eps;
        else if (conv_rule == 1) stop = sqrt(dsq) < eps;
        else {
            stop = 1;
            for (size_t r = 0; r < R; ++r) {
                if (delta[r] < eps) frozen[r] = 1;
                if (!frozen[r]) stop = 0;
            }
        }
        if (stop) break;
    }
    if (canonicalize) {
#pragma omp parallel for num_threads(threads) schedule(static)
        for (size_t r = 0; r < R; ++r) {
            if (a1[r] < 0) { a1[r] = -a1[r]; for (int j = 0; j < G; ++j) T1[r * G + j] = (int8_t)-T1[r * G + j]; }
            if (a2[r] < 0) { a2[r] = -a2[r]; for (int j = 0; j < G; ++j) T2[r * G + j] = (int8_t)-T2[r * G + j]; }
            if (a1[r] < a2[r]) {
                double tmp = a1[r]; a1[r] = a2[r]; a2[r] = tmp;
                for (int j = 0; j < G; ++j) { int8_t s = T1[r * G + j]; T1[r * G + j] = T2[r * G + j]; T2[r * G + j] = s; }
            }
        }
    }
    free(lam); free(err); free(delta); free(frozen);
    return sweeps;
}
