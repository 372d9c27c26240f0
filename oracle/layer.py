"""fp64 layer product of the dual-trit-plane linear layer.  Test infrastructure only.

Definition (Eq. 1-2, with one scale pair per output row per group of G input columns as in
the "Batch Processing" paragraph of Sec. 2.3; the forward is described in words in
Sec. 4 "Hardware Efficiency": a trit multiplies by sign flip, identity or zero and the two
planes are superposed):

    y[m, i] = sum_g ( alpha1[i, g] * sum_{j in group g} T1[i, j] * x[m, j]
                    + alpha2[i, g] * sum_{j in group g} T2[i, j] * x[m, j] )

Inputs are widened exactly to fp64 (int8 trits, fp16 scales, fp16 activations); all
arithmetic is fp64.  No blocking, fusion or reordering beyond the formula.
"""
import numpy as np


def _check(T1, T2, alpha1, alpha2, x, G):
    T1 = np.asarray(T1)
    T2 = np.asarray(T2)
    if T1.ndim != 2 or T1.shape != T2.shape:
        raise ValueError("T1 and T2 must be [N, K] and equal in shape")
    N, K = T1.shape
    if K % G != 0:
        raise ValueError("K must be a multiple of the group size")
    a1 = np.asarray(alpha1)
    a2 = np.asarray(alpha2)
    if a1.shape != (N, K // G) or a2.shape != (N, K // G):
        raise ValueError("alpha1, alpha2 must be [N, K/G]")
    x = np.asarray(x)
    if x.shape[-1] != K:
        raise ValueError("x must end in K")
    if np.any((T1 < -1) | (T1 > 1)) or np.any((T2 < -1) | (T2 > 1)):
        raise ValueError("trit-plane entries must lie in {-1, 0, 1}")
    return T1, T2, a1, a2, x, N, K


def layer_fp64(T1, T2, alpha1, alpha2, x, G=128):
    """y = alpha1 (.) (T1 x) + alpha2 (.) (T2 x) in fp64.

    T1, T2: [N, K] integers in {-1,0,1}; alpha1, alpha2: [N, K/G]; x: [K] or [M, K].
    Returns y with shape [N] or [M, N] (fp64).
    """
    T1, T2, a1, a2, x, N, K = _check(T1, T2, alpha1, alpha2, x, G)
    single = x.ndim == 1
    X = np.atleast_2d(x).astype(np.float64)
    a1 = a1.astype(np.float64)
    a2 = a2.astype(np.float64)
    Y = np.zeros((X.shape[0], N), dtype=np.float64)
    for m in range(X.shape[0]):
        for g in range(K // G):
            cols = slice(g * G, (g + 1) * G)
            xg = X[m, cols]
            s1 = (T1[:, cols].astype(np.float64) * xg).sum(axis=1)
            s2 = (T2[:, cols].astype(np.float64) * xg).sum(axis=1)
            Y[m] += a1[:, g] * s1 + a2[:, g] * s2
    return Y[0] if single else Y


def layer_fp64_loops(T1, T2, alpha1, alpha2, x, G=128):
    """The same product as scalar Python loops (tiny cases only; batch 1)."""
    T1, T2, a1, a2, x, N, K = _check(T1, T2, alpha1, alpha2, x, G)
    y = [0.0] * N
    for i in range(N):
        for g in range(K // G):
            s1 = 0.0
            s2 = 0.0
            for j in range(g * G, (g + 1) * G):
                xj = float(x[j])
                t1 = int(T1[i, j])
                t2 = int(T2[i, j])
                if t1 == 1:
                    s1 += xj
                elif t1 == -1:
                    s1 -= xj
                if t2 == 1:
                    s2 += xj
                elif t2 == -1:
                    s2 -= xj
            y[i] += float(a1[i, g]) * s1 + float(a2[i, g]) * s2
    return np.array(y, dtype=np.float64)


def dense_weight(T1, T2, alpha1, alpha2, G=128):
    """W_hat = alpha1 (.) T1 + alpha2 (.) T2 with the scales expanded over their groups."""
    T1 = np.asarray(T1)
    T2 = np.asarray(T2)
    a1 = np.repeat(np.asarray(alpha1).astype(np.float64), G, axis=1)
    a2 = np.repeat(np.asarray(alpha2).astype(np.float64), G, axis=1)
    return a1 * T1.astype(np.float64) + a2 * T2.astype(np.float64)


def parity_metrics(y_test, y_ref, x):
    """The two error measures the GEMV is judged on, per batch row.

    rel_l2  = ||y_test - y_ref||_2 / ||y_ref||_2
    max_abs = max_i |y_test_i - y_ref_i| and its bound 2e-3 * ||x||_inf * sqrt(K)
    """
    yt = np.atleast_2d(np.asarray(y_test, dtype=np.float64))
    yr = np.atleast_2d(np.asarray(y_ref, dtype=np.float64))
    X = np.atleast_2d(np.asarray(x, dtype=np.float64))
    out = []
    for m in range(yr.shape[0]):
        nr = np.linalg.norm(yr[m])
        rel = np.linalg.norm(yt[m] - yr[m]) / nr if nr > 0 else float(np.linalg.norm(yt[m]))
        mab = float(np.max(np.abs(yt[m] - yr[m]))) if yr.shape[1] else 0.0
        bound = 2e-3 * float(np.max(np.abs(X[m]))) * np.sqrt(X.shape[1]) if X.shape[1] else 0.0
        out.append((float(rel), mab, bound))
    return out


def swiglu_fp64(T1, T2, alpha1, alpha2, x, G=128):
    """Gated pair epilogue on top of the layer product, fp64 (batch 1 or [M, K]).

    The matrix holds gate and up projections interleaved by rows: row 2i is gate row i, row 2i+1 is up row i
    (the MLP of the LLaMA / Qwen models the paper quantises computes down(silu(gate(x)) * up(x)); the paper's
    layer, Eq. 1-2, is what produces gate(x) and up(x)).  With t = layer_fp64(...):

        y[i] = silu(t[2i]) * t[2i+1],     silu(g) = g / (1 + exp(-g))

    Returns [N/2] or [M, N/2].
    """
    t = layer_fp64(T1, T2, alpha1, alpha2, x, G)
    if t.shape[-1] % 2:
        raise ValueError("an even number of rows is required (gate and up rows come in pairs)")
    g, u = t[..., 0::2], t[..., 1::2]
    return g / (1.0 + np.exp(-g)) * u
