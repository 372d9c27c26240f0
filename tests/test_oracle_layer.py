"""Pins of the oracle's layer product (CPU only)."""
import numpy as np
import pytest

from oracle.layer import dense_weight, layer_fp64, layer_fp64_loops, parity_metrics
from oracle.c_oracle import layer_fp64_c
from paper_2509_16989_b200.inputs import make_case
from golden_io import load_worked_2x4


def small_case(N=24, K=256, M=1, seed=3):
    return make_case(N, K, seed=seed, M=M)


def test_dense_matmul_crosscheck():
    # Eq. 1-2: the layer is W_hat x with W_hat = alpha1 (.) T1 + alpha2 (.) T2.
    for M in (1, 3):
        c = small_case(M=M, seed=5 + M)
        y = layer_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
        What = dense_weight(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
        ref = np.atleast_2d(c["x"]).astype(np.float64) @ What.T
        ref = ref[0] if M == 1 else ref
        assert np.allclose(y, ref, rtol=1e-12, atol=1e-13)


def test_three_implementations_agree():
    c = small_case(N=7, K=384, seed=11)
    y = layer_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
    yl = layer_fp64_loops(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
    yc = layer_fp64_c(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"], threads=2)
    assert np.allclose(y, yl, rtol=1e-12, atol=1e-14)
    assert np.allclose(y, yc, rtol=1e-12, atol=1e-14)
    cm = small_case(N=5, K=256, M=4, seed=12)
    ym = layer_fp64(cm["T1"], cm["T2"], cm["alpha1"], cm["alpha2"], cm["x"])
    ycm = layer_fp64_c(cm["T1"], cm["T2"], cm["alpha1"], cm["alpha2"], cm["x"], threads=3)
    assert ym.shape == (4, 5) and np.allclose(ym, ycm, rtol=1e-12, atol=1e-14)


def test_gather_special_case():
    # T2 = 0, alpha1 = 1, T1 has one +1 per row -> y is a gather of x.
    N, K = 16, 256
    rng = np.random.default_rng(0)
    x = rng.standard_normal(K).astype(np.float16)
    cols = rng.integers(0, K, N)
    T1 = np.zeros((N, K), np.int8)
    T1[np.arange(N), cols] = 1
    T2 = np.zeros_like(T1)
    ones = np.ones((N, K // 128), np.float16)
    for f in (layer_fp64, layer_fp64_loops, lambda *a: layer_fp64_c(*a, threads=1)):
        y = f(T1, T2, ones, ones, x)
        assert np.array_equal(y, x[cols].astype(np.float64))
    # a single -1 per row in plane 2 with alpha2 = 2 -> y = -2 x[col]
    y = layer_fp64(T2, -T1, ones, 2 * ones, x)
    assert np.array_equal(y, -2.0 * x[cols].astype(np.float64))


def test_all_plus_one_closed_form():
    # T1 = +1 everywhere, T2 = 0: y_i = sum_g alpha1[i,g] * sum_{j in g} x_j.
    c = small_case(N=9, K=512, seed=2)
    T1 = np.ones_like(c["T1"])
    T2 = np.zeros_like(c["T2"])
    gs = c["x"].astype(np.float64).reshape(-1, 128).sum(axis=1)
    ref = c["alpha1"].astype(np.float64) @ gs
    for f in (layer_fp64, lambda *a: layer_fp64_c(*a, threads=2)):
        assert np.allclose(f(T1, T2, c["alpha1"], c["alpha2"], c["x"]), ref, rtol=1e-13, atol=1e-15)


def test_cancellation_and_zero_planes():
    c = small_case(seed=4)
    y = layer_fp64(c["T1"], -c["T1"], c["alpha1"], c["alpha1"], c["x"])
    assert np.array_equal(y, np.zeros(c["N"]))
    z = np.zeros_like(c["T1"])
    assert np.array_equal(layer_fp64(z, z, c["alpha1"], c["alpha2"], c["x"]), np.zeros(c["N"]))
    assert np.array_equal(layer_fp64_c(z, z, c["alpha1"], c["alpha2"], c["x"]), np.zeros(c["N"]))


def test_linearity_in_x_and_scales():
    c = small_case(seed=6)
    d = small_case(seed=7)
    # power-of-two combinations keep fp16 inputs exact
    x2 = (2.0 * c["x"].astype(np.float64) + 0.5 * d["x"].astype(np.float64))
    yc = layer_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
    yd = layer_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], d["x"])
    y2 = layer_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], x2)
    assert np.allclose(y2, 2.0 * yc + 0.5 * yd, rtol=1e-12, atol=1e-14)
    z = np.zeros_like(c["alpha1"])
    y_p1 = layer_fp64(c["T1"], c["T2"], c["alpha1"], z, c["x"])
    y_p2 = layer_fp64(c["T1"], c["T2"], z, c["alpha2"], c["x"])
    assert np.allclose(yc, y_p1 + y_p2, rtol=1e-12, atol=1e-14)
    # swapping the planes together with their scales leaves y unchanged
    ys = layer_fp64(c["T2"], c["T1"], c["alpha2"], c["alpha1"], c["x"])
    assert np.allclose(yc, ys, rtol=1e-12, atol=1e-14)
    # flipping a plane and its scale leaves y unchanged
    yf = layer_fp64(-c["T1"], c["T2"], -c["alpha1"].astype(np.float64), c["alpha2"], c["x"])
    assert np.allclose(yc, yf, rtol=1e-12, atol=1e-14)


def test_group_boundaries_matter():
    # a scale belongs to its own 128 columns: moving a +1 across a group boundary changes alpha.
    N, K = 1, 256
    x = np.zeros(K, np.float16)
    x[127] = 1.0
    x[128] = 1.0
    T1 = np.zeros((N, K), np.int8)
    T2 = np.zeros((N, K), np.int8)
    a1 = np.array([[3.0, 5.0]], np.float16)
    a2 = np.array([[7.0, 11.0]], np.float16)
    T1[0, 127] = 1
    assert layer_fp64(T1, T2, a1, a2, x)[0] == 3.0
    T1[:] = 0
    T1[0, 128] = 1
    assert layer_fp64(T1, T2, a1, a2, x)[0] == 5.0
    T2[0, 127] = -1
    assert layer_fp64(T1, T2, a1, a2, x)[0] == 5.0 - 7.0
    assert layer_fp64_c(T1, T2, a1, a2, x)[0] == 5.0 - 7.0


def test_worked_example_layer_product():
    g = load_worked_2x4()
    final = {r: g["sweeps"][(g["n_sweeps"], r)] for r in (0, 1)}
    T1 = np.array([final[0]["T1"], final[1]["T1"]], np.int8)
    T2 = np.array([final[0]["T2"], final[1]["T2"]], np.int8)
    a1 = np.array([[float(final[0]["alpha"][0])], [float(final[1]["alpha"][0])]])
    a2 = np.array([[float(final[0]["alpha"][1])], [float(final[1]["alpha"][1])]])
    x = np.array([float(v) for v in g["x"]])
    y = layer_fp64(T1, T2, a1, a2, x, G=4)
    assert np.allclose(y, [float(v) for v in g["y"]], rtol=1e-14)
    # the canonicalised planes give the same product
    T1c = np.array([g["canon"][0]["T1"], g["canon"][1]["T1"]], np.int8)
    T2c = np.array([g["canon"][0]["T2"], g["canon"][1]["T2"]], np.int8)
    a1c = np.array([[float(g["canon"][r]["alpha"][0])] for r in (0, 1)])
    a2c = np.array([[float(g["canon"][r]["alpha"][1])] for r in (0, 1)])
    assert np.allclose(layer_fp64(T1c, T2c, a1c, a2c, x, G=4), y, rtol=1e-14)


def test_rejects_bad_inputs():
    c = small_case()
    bad = c["T1"].copy()
    bad[0, 0] = 2
    with pytest.raises(ValueError):
        layer_fp64(bad, c["T2"], c["alpha1"], c["alpha2"], c["x"])
    with pytest.raises(ValueError):
        layer_fp64(c["T1"], c["T2"], c["alpha1"][:, :1], c["alpha2"], c["x"])
    with pytest.raises(ValueError):
        layer_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"][:-1])


def test_parity_metrics_definition():
    y = np.array([3.0, 4.0])
    yt = np.array([3.0, 4.5])
    x = np.array([0.5, -2.0, 1.0, 0.0])
    (rel, mab, bound), = parity_metrics(yt, y, x)
    assert rel == pytest.approx(0.1) and mab == 0.5 and bound == pytest.approx(2e-3 * 2.0 * 2.0)
