"""Exhaustive enumerations on tiny rows (K <= 6).  Test infrastructure only.

``tstep_bruteforce``  : Algorithm 1's T-step as it is stated -- the arg-min over WHOLE-ROW plane
                        pairs (all 9^K of them) of ||w - alpha1 c1 - alpha2 c2||^2 for fixed scales.
``global_bruteforce`` : the best error any pair of planes can reach when the scales are refitted by
                        unregularised least squares for that pair (the floor the alternating scheme
                        of Sec. 2.2-2.3 can only approach: it converges to a local minimum).
"""
import itertools
import numpy as np


def tstep_bruteforce(w, a1, a2):
    """Return (min_error, list of all (t1, t2) whole-row pairs attaining it exactly)."""
    w = [float(v) for v in w]
    K = len(w)
    if K > 6:
        raise ValueError("9^K enumeration is for K <= 6")
    trits = (-1, 0, 1)
    best = None
    winners = []
    for t1 in itertools.product(trits, repeat=K):
        for t2 in itertools.product(trits, repeat=K):
            e = 0.0
            for j in range(K):
                level = a1 * t1[j] + a2 * t2[j]
                d = w[j] - level
                e += d * d
            if best is None or e < best:
                best = e
                winners = [(t1, t2)]
            elif e == best:
                winners.append((t1, t2))
    return best, winners


def global_bruteforce(w):
    """min over all 9^K plane pairs of min over (alpha1, alpha2) of ||w - alpha1 t1 - alpha2 t2||^2."""
    w = np.asarray(w, dtype=np.float64)
    K = w.shape[0]
    if K > 6:
        raise ValueError("9^K enumeration is for K <= 6")
    trits = (-1, 0, 1)
    best = float(np.dot(w, w))
    arg = None
    planes = [np.array(t, dtype=np.float64) for t in itertools.product(trits, repeat=K)]
    for t1 in planes:
        for t2 in planes:
            S = np.stack([t1, t2], axis=1)
            theta, _res, _rank, _sv = np.linalg.lstsq(S, w, rcond=None)
            r = w - S @ theta
            e = float(np.dot(r, r))
            if e < best - 1e-15:
                best = e
                arg = (t1.copy(), t2.copy(), theta.copy())
    return best, arg
