"""GPU trit-plane decomposition (ptqtp_decompose) against the CPU oracle: identical planes, scales to 1e-12, the
same number of sweeps and the same error and change histories; the hand-worked 2 x 4 example; degenerate groups."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from golden_io import load_worked_2x4
from oracle.c_oracle import decompose_c
from oracle.decompose import decompose, reconstruction_error
from paper_2509_16989_b200 import binding
from paper_2509_16989_b200.inputs import make_activations, make_weights
from gpu_util import assert_parity, dev, oracle_y

pytestmark = pytest.mark.gpu


def run(W, **kw):
    T1, T2, a1, a2, info = binding.ptqtp_decompose(dev(np.ascontiguousarray(W, dtype=np.float32)), details=True, **kw)
    return dict(T1=T1.cpu().numpy(), T2=T2.cpu().numpy(), alpha1_fp16=a1.cpu().numpy(), alpha2_fp16=a2.cpu().numpy(), **info)


def assert_same(got, ref, what=""):
    assert got["sweeps"] == ref["sweeps"], what
    assert np.array_equal(got["T1"], ref["T1"]) and np.array_equal(got["T2"], ref["T2"]), what
    for k in ("alpha1", "alpha2"):
        assert np.all(np.abs(got[k] - ref[k]) <= 1e-12 * np.maximum(1.0, np.abs(ref[k]))), what
        assert np.array_equal(got[k + "_fp16"].view(np.uint16), ref[k + "_fp16"].view(np.uint16)), what
    assert np.allclose(got["delta_history"], ref["delta_history"], rtol=1e-12, atol=1e-300), what
    assert np.allclose(got["err_history"], ref["err_history"], rtol=1e-10, atol=1e-300), what


def test_worked_2x4_example():
    g = load_worked_2x4()
    W = np.array([[float(v) for v in row] for row in g["W"]], dtype=np.float32)
    out = run(W, group=4)
    assert out["sweeps"] == g["n_sweeps"]
    for row in (0, 1):
        want = g["canon"][row]
        assert list(out["T1"][row]) == want["T1"] and list(out["T2"][row]) == want["T2"]
        assert abs(out["alpha1"][row, 0] - float(want["alpha"][0])) < 5e-6
        assert abs(out["alpha2"][row, 0] - float(want["alpha"][1])) < 5e-6
    # the squared error after every sweep (both rows together), and the final total of 2
    for t in range(1, g["n_sweeps"] + 1):
        want = float(g["sweeps"][(t, 0)]["E"] + g["sweeps"][(t, 1)]["E"])
        assert abs(out["err_history"][t - 1] - want) < 1e-4
    assert abs(out["err_history"][-1] - float(g["Etotal"])) < 1e-5
    # without the normal form the planes of the last sweep come back as they are
    raw = run(W, group=4, canonicalize=False)
    for row in (0, 1):
        last = g["sweeps"][(g["n_sweeps"], row)]
        assert list(raw["T1"][row]) == last["T1"] and list(raw["T2"][row]) == last["T2"]
        assert abs(raw["alpha1"][row, 0] - float(last["alpha"][0])) < 5e-6


@pytest.mark.parametrize("N,K,seed", [(512, 4096, 40), (37, 1152, 41), (1, 128, 42), (130, 256, 43)])
def test_matches_the_cpu_oracle(N, K, seed):
    W = make_weights(N, K, seed=seed)
    assert_same(run(W), decompose_c(W), "N=%d K=%d" % (N, K))
    assert_same(run(W, canonicalize=False), decompose_c(W, canonicalize=False), "raw iterate")


@pytest.mark.parametrize("G", [4, 32, 64, 256])
def test_other_group_sizes_and_sweep_limits(G):
    W = make_weights(48, 1024, seed=50 + G)
    assert_same(run(W, group=G), decompose_c(W, G=G), "G=%d" % G)
    assert_same(run(W, group=G, t_max=3), decompose_c(W, G=G, T_max=3), "three sweeps")
    assert_same(run(W, group=G, eps=1e-2), decompose_c(W, G=G, eps=1e-2), "loose eps")


def test_degenerate_groups():
    rng = np.random.default_rng(7)
    W = (rng.standard_normal((64, 512)) * 0.02).astype(np.float32)
    W[3, 128:256] = 0.0                 # an all-zero group: alpha = 0, planes 0, no NaN
    W[5, :128] = 0.25                   # a constant group
    W[7, 256:384] = np.where(rng.random(128) < 0.5, 0.5, -0.5).astype(np.float32)     # exactly one level
    W[9, :] = 0.0
    W[11, 384:] = np.repeat(np.array([1.0, -2.0, 3.0, 0.0], np.float32), 32)
    W[13, 0] = 1e4                      # a huge outlier
    W[15, :128] = -0.0
    got, ref = run(W), decompose_c(W)
    assert_same(got, ref, "degenerate")
    assert np.all(np.isfinite(got["alpha1"])) and np.all(np.isfinite(got["alpha2"]))
    assert not got["T1"][3, 128:256].any() and not got["T2"][3, 128:256].any()
    assert got["alpha1"][3, 1] == 0.0 and got["alpha2"][3, 1] == 0.0
    # and the numpy oracle agrees on a slice (the C oracle is bit-identical to it)
    sub = decompose(W[:16])
    assert np.array_equal(run(W[:16])["T1"], sub["T1"])


def test_decompose_pack_gemv_pipeline_on_the_gpu():
    # W -> planes on the GPU -> pack -> GEMV, never leaving the device; checked against the oracle's layer product
    # on the same planes and against the dense product at the level of the reconstruction error
    N, K = 1024, 4096
    W = make_weights(N, K, seed=60)
    T1, T2, a1, a2 = binding.ptqtp_decompose(dev(W))
    x = make_activations(K, seed=61)
    for fmt in (binding.FORMAT_V2, binding.FORMAT_V3):
        packed, st = binding.ptqtp_pack(T1, T2, a1, a2, fmt=fmt)
        y = binding.ptqtp_gemv(packed, N, K, dev(x), fmt=fmt)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        c = dict(T1=T1.cpu().numpy(), T2=T2.cpu().numpy(), alpha1=a1.cpu().numpy(), alpha2=a2.cpu().numpy(), x=x)
        assert_parity(y.cpu().numpy(), oracle_y(c), x, "fmt %d" % fmt)
    err = reconstruction_error(W, c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    assert 0.10 < err < 0.25
    dense = W.astype(np.float64) @ x.astype(np.float64)
    assert np.linalg.norm(y.cpu().numpy().astype(np.float64) - dense) / np.linalg.norm(dense) < 2.5 * err


def test_argument_checks():
    L = binding.lib()
    assert L.ptqtp_decompose_workspace_size(8, 256, 128, 50) > 0
    for bad in ((0, 256, 128, 50), (8, 200, 128, 50), (8, 256, 0, 50), (8, 256, 512, 50), (8, 256, 128, 0), (8, 256, 128, 1001)):
        assert L.ptqtp_decompose_workspace_size(*bad) == 0
    W = dev(make_weights(8, 256, seed=1))
    with pytest.raises(binding.PtqtpError) as e:
        binding.ptqtp_decompose(W, group=100)
    assert e.value.status == binding.ERR_SHAPE
