"""Pins of the gated pair epilogue of the oracle (CPU only)."""
import numpy as np
import scipy.special

from oracle.layer import layer_fp64, swiglu_fp64
from paper_2509_16989_b200.inputs import make_case


def interleaved_case(n_pairs, K, seed):
    return make_case(2 * n_pairs, K, seed=seed)


def test_equals_the_library_logistic_applied_to_the_layer_rows():
    c = interleaved_case(24, 512, seed=3)
    c["alpha1"] = (c["alpha1"].astype(np.float32) * 40).astype(np.float16)     # gate values of order 1
    t = layer_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
    want = t[0::2] * scipy.special.expit(t[0::2]) * t[1::2]
    got = swiglu_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
    assert got.shape == (24,)
    assert np.allclose(got, want, rtol=1e-13, atol=0)
    assert np.abs(t[0::2]).max() > 0.5                     # the nonlinearity is exercised


def test_closed_forms():
    K = 128
    T1 = np.zeros((4, K), dtype=np.int8)
    T2 = np.zeros((4, K), dtype=np.int8)
    a1 = np.ones((4, 1), dtype=np.float16)
    a2 = np.zeros((4, 1), dtype=np.float16)
    x = np.zeros(K, dtype=np.float16)
    x[0], x[1] = 2.0, 1.0
    # pair 0: gate = +x0 = 2, up = x1 = 1; pair 1: gate = -x0 = -2, up = x1 = 1
    T1[0, 0], T1[1, 1], T1[2, 0], T1[3, 1] = 1, 1, -1, 1
    y = swiglu_fp64(T1, T2, a1, a2, x)
    silu2 = 2.0 / (1.0 + np.exp(-2.0))
    assert np.isclose(y[0], silu2, rtol=1e-15)
    assert np.isclose(y[0] - y[1], 2.0, rtol=1e-15)         # silu(g) - silu(-g) = g
    # a zero gate row gives zero, whatever the up row
    T1[0, 0] = 0
    assert swiglu_fp64(T1, T2, a1, a2, x)[0] == 0.0
    # the up row enters linearly
    T1[0, 0] = 1
    T1[1, 1] = -1
    assert np.isclose(swiglu_fp64(T1, T2, a1, a2, x)[0], -silu2, rtol=1e-15)


def test_batch_rows_are_independent_and_odd_row_counts_are_refused():
    c = make_case(6, 256, seed=5, M=3)
    Y = swiglu_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
    for m in range(3):
        assert np.array_equal(Y[m], swiglu_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"][m]))
    c = make_case(5, 256, seed=5)
    try:
        swiglu_fp64(c["T1"], c["T2"], c["alpha1"], c["alpha2"], c["x"])
        assert False
    except ValueError:
        pass
