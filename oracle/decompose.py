"""Progressive trit-plane decomposition W ~ alpha1 (.) T1 + alpha2 (.) T2.  Test infrastructure only.

Follows Algorithm 1 (group structure, sweep order, stopping rule) with the inner formulas of
Algorithm 2 and the prose of Appendix C ("Progressive and Adaptive Regularization"):

  * W [N, K] is cut into group-rows w of G contiguous input columns (Sec. 2.3, "Batch
    Processing": reshape n x d -> (nd/G) x G); every group-row has its own scale pair.
  * init: t1 = t2 = sign(w) with 0 -> +1, alpha = (1, 1), lambda = 1e-8   (Alg. 2 init lines).
  * sweep t = 1..T_max over all group-rows:
      alpha-step  S = [t1 t2], A = S^T S + lambda I_2, b = S^T w               (Eq. 3-5)
                  kappa = ||A||_F ||A^-1||_F                                    (Eq. 6)
                  if kappa >= 1e6: lambda <- min(lambda sqrt(kappa/1e6), 1)     (Alg. 2; App. C)
                  alpha = A^-1 b with the explicit 2x2 inverse                  (App. B, complexity)
      T-step      per element, the pair (c1, c2) in {-1,0,1}^2 that minimises
                  (w_j - (alpha1 c1 + alpha2 c2))^2                             (Alg. 2 T-step)
      stop        when max over group-rows of ||alpha_t - alpha_{t-1}||_2 < eps (Alg. 1 last line)

Readings taken where the text is silent or ambiguous (each is a parameter):

  lambda_order  "update_then_solve" (default): the enlarged lambda is used by the solve of the same
                sweep, once per sweep (App. C prose); "solve_then_update": Alg. 2's line order.
  tie_break     "sparse_first" (default): equal errors are resolved in the order
                (0,0), (+1,0), (-1,0), (0,+1), (0,-1), (+1,+1), (-1,-1), (+1,-1), (-1,+1),
                i.e. fewest non-zeros first, then a non-zero in plane 1;
                "meshgrid": first minimum in the order c1 = -1,0,1 outer, c2 = -1,0,1 inner.
  conv_rule     "max_rows" (default, Alg. 1), "frobenius_all" (Alg. 2: norm over the whole alpha),
                "per_group_freeze" (a group-row stops updating once its own change < eps).
  canonicalize  after convergence, per group-row and without changing W_hat: make both scales
                non-negative by flipping (alpha_k, t_k), then order the pair so alpha1 >= alpha2.

The candidate level alpha1 c1 + alpha2 c2 is formed first and then subtracted from w, as the
T-step formula is written, so that structurally equal candidates (alpha1 == alpha2 at t = 1)
have bit-equal errors and the tie-break, not rounding noise, decides.

All arithmetic is fp64.  Sums over the G elements of a group-row run sequentially in j so that
the C restatement under oracle/c reproduces every bit.  The scales are rounded to fp16 (RNE)
only at the end.
"""
import numpy as np

SPARSE_FIRST = ((0, 0), (1, 0), (-1, 0), (0, 1), (0, -1), (1, 1), (-1, -1), (1, -1), (-1, 1))
MESHGRID = tuple((c1, c2) for c1 in (-1, 0, 1) for c2 in (-1, 0, 1))


def candidate_order(tie_break):
    if tie_break == "sparse_first":
        return SPARSE_FIRST
    if tie_break == "meshgrid":
        return MESHGRID
    raise ValueError("unknown tie_break %r" % (tie_break,))


def _seq_sum(a):
    """Sum over axis 1, sequentially in j (fixed rounding order)."""
    s = np.zeros(a.shape[0], dtype=np.float64)
    for j in range(a.shape[1]):
        s = s + a[:, j]
    return s


def kappa_2x2(A11, A12, A22):
    """kappa = ||A||_F * ||A^-1||_F for symmetric 2x2 A (Eq. 6).

    With A^-1 = adj(A)/det and ||adj(A)||_F = ||A||_F this is ||A||_F^2 / |det A|.
    """
    det = A11 * A22 - A12 * A12
    return (A11 * A11 + A22 * A22 + 2.0 * A12 * A12) / np.abs(det)


def alpha_step(w, t1, t2, lam, kappa_thr=1e6, lambda_max=1.0, lambda_min=1e-8,
               lambda_order="update_then_solve"):
    """Ridge solve of Eq. 3-5 for every group-row; returns (alpha1, alpha2, lambda_next, kappa)."""
    f1 = t1.astype(np.float64)
    f2 = t2.astype(np.float64)
    n11 = _seq_sum(f1 * f1)
    n22 = _seq_sum(f2 * f2)
    n12 = _seq_sum(f1 * f2)
    b1 = _seq_sum(f1 * w)
    b2 = _seq_sum(f2 * w)
    A11 = n11 + lam
    A22 = n22 + lam
    kappa = kappa_2x2(A11, n12, A22)
    grow = kappa >= kappa_thr
    lam_grown = np.where(grow, np.minimum(lam * np.sqrt(kappa / kappa_thr), lambda_max), lam)
    lam_grown = np.maximum(lam_grown, lambda_min)
    if lambda_order == "update_then_solve":
        lam = lam_grown
        A11 = n11 + lam
        A22 = n22 + lam
    elif lambda_order != "solve_then_update":
        raise ValueError("unknown lambda_order %r" % (lambda_order,))
    det = A11 * A22 - n12 * n12
    a1 = (A22 * b1 - n12 * b2) / det
    a2 = (A11 * b2 - n12 * b1) / det
    return a1, a2, lam_grown, kappa


def t_step(w, a1, a2, tie_break="sparse_first"):
    """Per element, the candidate pair of smallest squared error (first in tie-break order)."""
    cands = candidate_order(tie_break)
    best_err = None
    best_m = None
    for m, (c1, c2) in enumerate(cands):
        level = a1 * c1 + a2 * c2
        err = (w - level[:, None]) ** 2
        if best_err is None:
            best_err = err
            best_m = np.zeros(w.shape, dtype=np.int64)
        else:
            better = err < best_err          # strict: an equal error keeps the earlier candidate
            best_err = np.where(better, err, best_err)
            best_m[better] = m
    c1s = np.array([c[0] for c in cands], dtype=np.int8)
    c2s = np.array([c[1] for c in cands], dtype=np.int8)
    return c1s[best_m], c2s[best_m]


def group_error(w, a1, a2, t1, t2):
    """E = sum_j (w_j - alpha1 t1_j - alpha2 t2_j)^2 per group-row."""
    r = w - (a1[:, None] * t1.astype(np.float64) + a2[:, None] * t2.astype(np.float64))
    return _seq_sum(r * r)


def canonicalize_planes(a1, a2, t1, t2):
    """W_hat-preserving normal form: alpha1 >= alpha2 >= 0 per group-row."""
    a1 = a1.copy()
    a2 = a2.copy()
    t1 = t1.copy()
    t2 = t2.copy()
    neg1 = a1 < 0
    a1[neg1] = -a1[neg1]
    t1[neg1] = -t1[neg1]
    neg2 = a2 < 0
    a2[neg2] = -a2[neg2]
    t2[neg2] = -t2[neg2]
    swap = a1 < a2
    a1s = a1[swap].copy()
    a1[swap] = a2[swap]
    a2[swap] = a1s
    t1s = t1[swap].copy()
    t1[swap] = t2[swap]
    t2[swap] = t1s
    return a1, a2, t1, t2


def decompose(W, G=128, T_max=50, eps=1e-4, lambda0=1e-8, lambda_max=1.0, kappa_thr=1e6,
              tie_break="sparse_first", lambda_order="update_then_solve", conv_rule="max_rows",
              canonicalize=True, chunk=8192):
    """Decompose W [N, K] into two trit-planes and group-wise scales.

    Returns a dict:
      T1, T2            int8 [N, K]
      alpha1, alpha2    fp64 [N, K/G] (the iterate alpha_t returned with T_t, no refit)
      alpha1_fp16, alpha2_fp16   the same rounded to fp16
      sweeps            number of sweeps run
      err_history       list over sweeps of the total squared error after the T-step
      err_rows_history  list over sweeps of the per-group-row squared errors
      alpha_history     list over sweeps of (alpha1, alpha2) before canonicalisation
      lambda_history    list over sweeps of the lambda in force after that sweep
      delta_history     list over sweeps of max group-row ||alpha_t - alpha_{t-1}||_2
    """
    W = np.asarray(W)
    if W.ndim != 2:
        raise ValueError("W must be [N, K]")
    N, K = W.shape
    if K % G != 0:
        raise ValueError("K must be a multiple of G")
    w_all = W.astype(np.float64).reshape(N * (K // G), G)
    R = w_all.shape[0]
    t1 = np.where(w_all >= 0, 1, -1).astype(np.int8)
    t2 = t1.copy()
    a1 = np.ones(R, dtype=np.float64)
    a2 = np.ones(R, dtype=np.float64)
    lam = np.full(R, lambda0, dtype=np.float64)
    frozen = np.zeros(R, dtype=bool)
    hist = dict(err_history=[], err_rows_history=[], alpha_history=[], lambda_history=[],
                delta_history=[])
    sweeps = 0
    for _t in range(1, T_max + 1):
        sweeps += 1
        a1_new = a1.copy()
        a2_new = a2.copy()
        err_rows = np.zeros(R, dtype=np.float64)
        for lo in range(0, R, chunk):
            sl = slice(lo, min(lo + chunk, R))
            w = w_all[sl]
            p1, p2, lam_next, _kappa = alpha_step(w, t1[sl], t2[sl], lam[sl], kappa_thr,
                                                  lambda_max, lambda0, lambda_order)
            n1, n2 = t_step(w, p1, p2, tie_break)
            keep = frozen[sl]
            if keep.any():          # only reachable under conv_rule == "per_group_freeze"
                p1 = np.where(keep, a1[sl], p1)
                p2 = np.where(keep, a2[sl], p2)
                n1 = np.where(keep[:, None], t1[sl], n1)
                n2 = np.where(keep[:, None], t2[sl], n2)
                lam_next = np.where(keep, lam[sl], lam_next)
            a1_new[sl] = p1
            a2_new[sl] = p2
            t1[sl] = n1
            t2[sl] = n2
            lam[sl] = lam_next
            err_rows[sl] = group_error(w, p1, p2, n1, n2)
        delta = np.sqrt((a1_new - a1) ** 2 + (a2_new - a2) ** 2)
        a1, a2 = a1_new, a2_new
        hist["err_history"].append(float(_seq_sum(err_rows[None, :])[0]))
        hist["err_rows_history"].append(err_rows)
        hist["alpha_history"].append((a1.copy(), a2.copy()))
        hist["lambda_history"].append(lam.copy())
        hist["delta_history"].append(float(delta.max()) if R else 0.0)
        if conv_rule == "max_rows":
            if R == 0 or delta.max() < eps:
                break
        elif conv_rule == "frobenius_all":
            if np.sqrt(_seq_sum((delta * delta)[None, :])[0]) < eps:
                break
        elif conv_rule == "per_group_freeze":
            frozen |= delta < eps
            if frozen.all():
                break
        else:
            raise ValueError("unknown conv_rule %r" % (conv_rule,))
    if canonicalize:
        a1, a2, t1, t2 = canonicalize_planes(a1, a2, t1, t2)
    out = dict(T1=t1.reshape(N, K), T2=t2.reshape(N, K),
               alpha1=a1.reshape(N, K // G), alpha2=a2.reshape(N, K // G), sweeps=sweeps)
    out["alpha1_fp16"] = out["alpha1"].astype(np.float16)
    out["alpha2_fp16"] = out["alpha2"].astype(np.float16)
    out.update(hist)
    return out


def reconstruction_error(W, T1, T2, alpha1, alpha2, G=128):
    """||W - (alpha1 (.) T1 + alpha2 (.) T2)||_F / ||W||_F in fp64 (scales widened exactly)."""
    W = np.asarray(W, dtype=np.float64)
    a1 = np.repeat(np.asarray(alpha1).astype(np.float64), G, axis=1)
    a2 = np.repeat(np.asarray(alpha2).astype(np.float64), G, axis=1)
    What = a1 * np.asarray(T1, dtype=np.float64) + a2 * np.asarray(T2, dtype=np.float64)
    return float(np.linalg.norm(W - What) / np.linalg.norm(W))
