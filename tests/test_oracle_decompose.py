"""Pins of the oracle's progressive trit-plane decomposition (CPU only)."""
from fractions import Fraction

import numpy as np
import pytest

from oracle.bruteforce import global_bruteforce, tstep_bruteforce
from oracle.c_oracle import decompose_c
from oracle.decompose import (alpha_step, canonicalize_planes, decompose, group_error, kappa_2x2,
                              reconstruction_error, t_step)
from oracle.layer import dense_weight
from paper_2509_16989_b200.inputs import make_weights
from golden_io import load_worked_2x4


def gaussian(N, K, seed, sigma=0.02):
    return (np.random.default_rng(seed).standard_normal((N, K)) * sigma).astype(np.float32)


# ---------------------------------------------------------------- invariants the paper states

def test_trit_range_and_shapes():
    W = make_weights(16, 512, seed=1)
    r = decompose(W)
    for T in (r["T1"], r["T2"]):
        assert T.dtype == np.int8 and T.shape == W.shape
        assert set(np.unique(T)).issubset({-1, 0, 1})
    assert r["alpha1"].shape == (16, 4) and r["alpha1_fp16"].dtype == np.float16
    assert 1 <= r["sweeps"] <= 50


def test_error_never_increases():
    # Sec. 2.3: no update step increases ||W - W_hat||_F^2.  The T-step is exactly monotone; the
    # ridge alpha-step minimises E + lambda |alpha|^2, so E itself may rise by at most lambda |alpha|^2.
    for seed, W in ((0, gaussian(32, 512, 0)), (1, make_weights(32, 512, seed=1))):
        r = decompose(W, canonicalize=False)
        E = r["err_rows_history"]
        for t in range(1, len(E)):
            a1p, a2p = r["alpha_history"][t - 1]
            lam = r["lambda_history"][t]
            slack = lam * (a1p ** 2 + a2p ** 2)
            assert np.all(E[t] <= E[t - 1] * (1 + 1e-9) + slack)
        tot = r["err_history"]
        assert all(tot[t] <= tot[t - 1] * (1 + 1e-9) for t in range(1, len(tot)))
        assert tot[-1] < 0.05 * float((W.astype(np.float64) ** 2).sum())


def test_tstep_is_monotone_for_fixed_alpha():
    rng = np.random.default_rng(3)
    w = rng.standard_normal((50, 16))
    t1 = rng.integers(-1, 2, (50, 16)).astype(np.int8)
    t2 = rng.integers(-1, 2, (50, 16)).astype(np.int8)
    a1 = rng.standard_normal(50)
    a2 = rng.standard_normal(50)
    n1, n2 = t_step(w, a1, a2)
    assert np.all(group_error(w, a1, a2, n1, n2) <= group_error(w, a1, a2, t1, t2))


# ---------------------------------------------------------------- the alpha-step

def test_alpha_step_equals_library_ridge_solve():
    rng = np.random.default_rng(5)
    R, G = 40, 32
    w = rng.standard_normal((R, G))
    t1 = rng.integers(-1, 2, (R, G)).astype(np.int8)
    t2 = rng.integers(-1, 2, (R, G)).astype(np.int8)
    lam = np.full(R, 1e-3)
    a1, a2, lam_next, kappa = alpha_step(w, t1, t2, lam)
    for r in range(R):
        S = np.stack([t1[r], t2[r]], axis=1).astype(np.float64)
        A = S.T @ S + lam_next[r] * np.eye(2)
        ref = np.linalg.solve(A, S.T @ w[r])
        assert np.allclose([a1[r], a2[r]], ref, rtol=1e-10, atol=1e-12)
        # it is the minimiser of the ridge objective (Eq. 7): perturbing alpha never lowers it
        def obj(th):
            return np.sum((w[r] - S @ th) ** 2) + lam_next[r] * np.sum(th ** 2)
        base = obj(np.array([a1[r], a2[r]]))
        for d in ((1e-3, 0), (-1e-3, 0), (0, 1e-3), (0, -1e-3)):
            assert obj(np.array([a1[r] + d[0], a2[r] + d[1]])) >= base


def test_kappa_closed_form_and_lower_bound():
    rng = np.random.default_rng(6)
    for _ in range(50):
        B = rng.standard_normal((5, 2))
        A = B.T @ B + 0.1 * np.eye(2)
        k = kappa_2x2(A[0, 0], A[0, 1], A[1, 1])
        ref = np.linalg.norm(A, "fro") * np.linalg.norm(np.linalg.inv(A), "fro")
        assert k == pytest.approx(ref, rel=1e-10)
        assert k >= 2 - 1e-12
    assert kappa_2x2(3.0, 0.0, 3.0) == pytest.approx(2.0)


def test_first_sweep_closed_form_and_lambda_growth():
    # Both planes start equal, so S^T S is singular; with lambda > 0 the solve gives
    # alpha1 = alpha2 = sum|w| / (2G + lambda), bit-equal, and kappa >= 1e6 grows lambda once.
    W = gaussian(4, 256, 7)
    r = decompose(W, T_max=1, canonicalize=False)
    a1, a2 = r["alpha_history"][0]
    assert np.array_equal(a1, a2)
    lam = r["lambda_history"][0]
    G = 128
    kappa0 = ((G + 1e-8) ** 2 * 2 + 2 * G * G) / ((G + 1e-8) ** 2 - G * G)
    assert np.allclose(lam, 1e-8 * np.sqrt(kappa0 / 1e6), rtol=1e-6)
    sabs = np.abs(W.astype(np.float64)).reshape(-1, G).sum(axis=1)
    assert np.allclose(a1, sabs / (2 * G + lam), rtol=1e-9)
    assert np.all(lam <= 1.0) and np.all(lam >= 1e-8)


def test_lambda_is_capped():
    W = gaussian(2, 128, 8)
    r = decompose(W, T_max=1, kappa_thr=1e-12, canonicalize=False)   # growth factor ~1e11
    assert np.all(r["lambda_history"][0] == 1.0)
    calm = decompose(W, T_max=1, lambda0=0.5, canonicalize=False)      # kappa ~ 5e2: no growth
    assert np.all(calm["lambda_history"][0] == 0.5)


def test_lambda_order_readings_agree_on_the_planes():
    W = gaussian(16, 256, 9)
    a = decompose(W, lambda_order="update_then_solve")
    b = decompose(W, lambda_order="solve_then_update")
    assert np.array_equal(a["T1"], b["T1"]) and np.array_equal(a["T2"], b["T2"])
    assert np.allclose(a["alpha1"], b["alpha1"], rtol=1e-5)


# ---------------------------------------------------------------- the T-step against 9^K brute force

@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_tstep_matches_whole_row_bruteforce(K):
    # Alg. 1 states the T-step as an arg-min over whole-row plane pairs; the per-element rule of
    # Alg. 2 must reach the same minimum and return one of its minimisers (the tie-break's one).
    rng = np.random.default_rng(100 + K)
    for trial in range(6 if K < 4 else 3):
        w = np.round(rng.standard_normal(K) * 4) / 2 if trial % 2 else rng.standard_normal(K)
        a1, a2 = (1.5, 1.5) if trial == 1 else tuple(rng.standard_normal(2))
        best, winners = tstep_bruteforce(w, a1, a2)
        n1, n2 = t_step(w[None, :], np.array([a1]), np.array([a2]))
        e = float(group_error(w[None, :], np.array([a1]), np.array([a2]), n1, n2)[0])
        assert e == pytest.approx(best, rel=1e-12, abs=1e-300)
        assert (tuple(int(v) for v in n1[0]), tuple(int(v) for v in n2[0])) in winners
        # among all exact minimisers the rule returns the sparsest, then the one with plane 2 emptiest
        key = lambda p: (sum(abs(v) for v in p[0]) + sum(abs(v) for v in p[1]), sum(abs(v) for v in p[1]))
        got = (tuple(int(v) for v in n1[0]), tuple(int(v) for v in n2[0]))
        assert key(got) == min(key(p) for p in winners)


def test_tstep_bruteforce_k6_once():
    w = np.array([0.9, -0.2, 0.05, -1.4, 0.6, 0.31])
    best, winners = tstep_bruteforce(w, 0.7, 0.25)
    n1, n2 = t_step(w[None, :], np.array([0.7]), np.array([0.25]))
    assert float(group_error(w[None, :], np.array([0.7]), np.array([0.25]), n1, n2)[0]) == pytest.approx(best, rel=1e-12)
    assert winners == [(tuple(int(v) for v in n1[0]), tuple(int(v) for v in n2[0]))]


def test_tie_break_orders():
    # alpha1 == alpha2: (1,0) and (0,1) tie, (1,-1) ties with (0,0).
    w = np.array([[1.0, 0.0, 2.0, -1.0]])
    a = np.array([1.0])
    s1, s2 = t_step(w, a, a, "sparse_first")
    assert s1.tolist() == [[1, 0, 1, -1]] and s2.tolist() == [[0, 0, 1, 0]]
    m1, m2 = t_step(w, a, a, "meshgrid")
    assert m1.tolist() == [[0, -1, 1, -1]] and m2.tolist() == [[1, 1, 1, 0]]


# ---------------------------------------------------------------- the whole iteration

def test_worked_example_exact_trits_and_scales():
    g = load_worked_2x4()
    W = np.array([[float(v) for v in row] for row in g["W"]], np.float32)
    r = decompose(W, G=4, canonicalize=False)
    assert r["sweeps"] == g["n_sweeps"]
    T1h, T2h = None, None
    # replay sweep by sweep (the history stores scales and errors; planes are final only)
    for T_max in range(1, g["n_sweeps"] + 1):
        p = decompose(W, G=4, T_max=T_max, canonicalize=False)
        for row in (0, 1):
            ref = g["sweeps"][(T_max, row)]
            assert p["T1"][row].tolist() == ref["T1"], (T_max, row)
            assert p["T2"][row].tolist() == ref["T2"], (T_max, row)
            assert p["alpha1"][row, 0] == pytest.approx(float(ref["alpha"][0]), abs=5e-6)
            assert p["alpha2"][row, 0] == pytest.approx(float(ref["alpha"][1]), abs=5e-6)
            assert p["err_rows_history"][-1][row] == pytest.approx(float(ref["E"]), abs=5e-5)
    assert r["err_history"][-1] == pytest.approx(float(g["Etotal"]), abs=5e-6)
    What = dense_weight(r["T1"], r["T2"], r["alpha1"], r["alpha2"], G=4)
    assert np.allclose(What, [[float(v) for v in row] for row in g["What"]], atol=1e-5)
    assert reconstruction_error(W, r["T1"], r["T2"], r["alpha1"], r["alpha2"], G=4) == pytest.approx(
        float(Fraction(2, 360)) ** 0.5, rel=1e-5)
    c = decompose(W, G=4, canonicalize=True)
    for row in (0, 1):
        assert c["T1"][row].tolist() == g["canon"][row]["T1"]
        assert c["T2"][row].tolist() == g["canon"][row]["T2"]
        assert c["alpha1"][row, 0] == pytest.approx(float(g["canon"][row]["alpha"][0]), abs=5e-6)
        assert c["alpha2"][row, 0] == pytest.approx(float(g["canon"][row]["alpha"][1]), abs=5e-6)
    # C restatement and both lambda-order readings reproduce it too
    cc = decompose_c(W, G=4, canonicalize=False)
    assert np.array_equal(cc["T1"], r["T1"]) and np.array_equal(cc["T2"], r["T2"])
    alt = decompose(W, G=4, canonicalize=False, lambda_order="solve_then_update")
    assert np.array_equal(alt["T1"], r["T1"]) and np.array_equal(alt["T2"], r["T2"])


def test_worked_example_discriminates_tie_break():
    g = load_worked_2x4()
    W = np.array([[float(v) for v in row] for row in g["W"]], np.float32)
    p = decompose(W, G=4, T_max=1, canonicalize=False, tie_break="meshgrid")
    assert p["T1"][0].tolist() != g["sweeps"][(1, 0)]["T1"] or p["T2"][0].tolist() != g["sweeps"][(1, 0)]["T2"]


def test_worked_example_global_optimum_of_row1():
    g = load_worked_2x4()
    w1 = np.array([float(v) for v in g["W"][1]])
    best, _ = global_bruteforce(w1)
    assert best == pytest.approx(float(g["Eglobal_row1"]), rel=1e-9)
    assert float(g["sweeps"][(g["n_sweeps"], 1)]["E"]) > best


def test_fixed_point_is_stable():
    W = gaussian(8, 256, 11)
    r = decompose(W, T_max=200, eps=1e-12, canonicalize=False)
    assert r["sweeps"] < 200
    more = decompose(W, T_max=r["sweeps"] + 3, eps=0.0, canonicalize=False)
    assert np.array_equal(more["T1"], r["T1"]) and np.array_equal(more["T2"], r["T2"])
    assert np.allclose(more["alpha1"], r["alpha1"], rtol=0, atol=1e-12)


def test_never_beats_global_optimum_and_planted_rows():
    rng = np.random.default_rng(12)
    hits = 0
    for trial in range(12):
        K = int(rng.integers(3, 5))
        w = rng.standard_normal(K).astype(np.float32)
        r = decompose(w[None, :], G=K, canonicalize=False)
        best, _ = global_bruteforce(w.astype(np.float64))
        assert r["err_history"][-1] >= best - 1e-7
        hits += r["err_history"][-1] <= best + 1e-7
    assert hits >= 1
    # planted rows w = a1 t1 + a2 t2 are exactly representable: the brute-forcer must find error 0
    t1 = np.array([1, -1, 0, 1], float)
    t2 = np.array([0, 1, -1, 1], float)
    best, _ = global_bruteforce(0.75 * t1 + 0.25 * t2)
    assert best == pytest.approx(0.0, abs=1e-20)


def test_all_zero_group_and_no_nans():
    W = gaussian(4, 256, 13)
    W[1, :128] = 0.0
    W[2, 128:] = 0.0
    r = decompose(W)
    for key in ("alpha1", "alpha2"):
        assert np.all(np.isfinite(r[key]))
    assert np.all(r["T1"][1, :128] == 0) and np.all(r["T2"][1, :128] == 0)
    assert r["alpha1"][1, 0] == 0.0 and r["alpha2"][2, 1] == 0.0
    rc = decompose_c(W)
    assert np.array_equal(rc["T1"], r["T1"]) and np.array_equal(rc["alpha1"], r["alpha1"])


def test_canonicalisation_preserves_what():
    rng = np.random.default_rng(14)
    R, G = 30, 16
    a1 = rng.standard_normal(R)
    a2 = rng.standard_normal(R)
    t1 = rng.integers(-1, 2, (R, G)).astype(np.int8)
    t2 = rng.integers(-1, 2, (R, G)).astype(np.int8)
    b1, b2, u1, u2 = canonicalize_planes(a1, a2, t1, t2)
    assert np.all(b1 >= b2) and np.all(b2 >= 0)
    before = a1[:, None] * t1 + a2[:, None] * t2
    after = b1[:, None] * u1 + b2[:, None] * u2
    assert np.allclose(before, after, rtol=0, atol=1e-15)
    W = gaussian(8, 256, 15)
    raw = decompose(W, canonicalize=False)
    can = decompose(W, canonicalize=True)
    assert np.allclose(dense_weight(raw["T1"], raw["T2"], raw["alpha1"], raw["alpha2"]),
                       dense_weight(can["T1"], can["T2"], can["alpha1"], can["alpha2"]), atol=1e-15)
    assert np.all(can["alpha1"] >= can["alpha2"]) and np.all(can["alpha2"] >= 0)


@pytest.mark.parametrize("conv_rule", ["max_rows", "frobenius_all", "per_group_freeze"])
@pytest.mark.parametrize("tie_break", ["sparse_first", "meshgrid"])
def test_c_restatement_is_bit_identical(conv_rule, tie_break):
    W = make_weights(24, 512, seed=16)
    a = decompose(W, conv_rule=conv_rule, tie_break=tie_break)
    b = decompose_c(W, conv_rule=conv_rule, tie_break=tie_break, threads=3)
    assert a["sweeps"] == b["sweeps"]
    for k in ("T1", "T2", "alpha1", "alpha2"):
        assert np.array_equal(a[k], b[k]), k
    assert a["err_history"] == b["err_history"]


def test_convergence_rules_and_sanity_ranges():
    # Convergence within 50 sweeps (Sec. 2.3) and the error level expected of two trit-planes on
    # Gaussian weights (sanity range only: the paper prints no reconstruction error).
    W = make_weights(64, 1024, seed=17)
    r = decompose_c(W)
    assert r["sweeps"] <= 50 and r["delta_history"][-1] < 1e-4
    err = reconstruction_error(W, r["T1"], r["T2"], r["alpha1_fp16"], r["alpha2_fp16"])
    assert 0.10 < err < 0.25
    frz = decompose_c(W, conv_rule="per_group_freeze")
    assert reconstruction_error(W, frz["T1"], frz["T2"], frz["alpha1_fp16"], frz["alpha2_fp16"]) < 0.25
    one = decompose_c(W, T_max=1)
    assert reconstruction_error(W, one["T1"], one["T2"], one["alpha1_fp16"], one["alpha2_fp16"]) > err
