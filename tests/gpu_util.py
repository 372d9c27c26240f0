"""Helpers for the GPU parity tests: tensors on cuda:0 and the parity bar."""
import numpy as np
import torch

from oracle.c_oracle import layer_fp64_c, max_threads
from oracle.layer import parity_metrics
from paper_2509_16989_b200 import binding

REL_L2_TOL = 1e-3          # ||y_gpu - y||_2 / ||y||_2
MAX_ABS_COEF = 2e-3        # max_i |y_gpu_i - y_i| <= 2e-3 * ||x||_inf * sqrt(K)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


FORMATS = (binding.FORMAT_V1, binding.FORMAT_V2, binding.FORMAT_V3)


def pack_case(c, fmt=None):
    packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=fmt)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return packed


def oracle_y(c, rows=None):
    T1, T2, a1, a2 = c["T1"], c["T2"], c["alpha1"], c["alpha2"]
    if rows is not None:
        T1, T2, a1, a2 = T1[rows], T2[rows], a1[rows], a2[rows]
    return layer_fp64_c(T1, T2, a1, a2, c["x"], threads=max_threads())


def assert_parity(y_gpu, y_ref, x, what=""):
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    assert np.all(np.isfinite(y_gpu)), what
    for m, (rel, mab, bound) in enumerate(parity_metrics(y_gpu, y_ref, x)):
        assert rel <= REL_L2_TOL, "%s row %d: rel-L2 %.3e > %.1e" % (what, m, rel, REL_L2_TOL)
        assert mab <= bound, "%s row %d: max-abs %.3e > %.3e" % (what, m, mab, bound)
