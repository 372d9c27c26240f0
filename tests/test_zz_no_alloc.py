"""ptqtp_gemm_skinny_static: the small-batch call for users who cannot allocate device memory at the call site
(plug-ins inside a process whose framework owns the whole GPU memory pool, latency-critical decode loops where
cudaMalloc would stall the device).  Its workspace is a fixed array inside the library.

Checked here through the C ABI: two calls in a row, each against the existing workspace entry point
(ptqtp_gemm_skinny_ws) on the same inputs -- within the parity tolerance of the other GPU tests, and, since both
run the same kernels on the same inputs, bit for bit -- and against the fp64 oracle; sizes beyond the fixed array
are refused.  The file name makes pytest collect it last."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2509_16989_b200 import binding
from paper_2509_16989_b200.inputs import make_case
from gpu_util import REL_L2_TOL, MAX_ABS_COEF, assert_parity, dev, oracle_y

pytestmark = pytest.mark.gpu


def close_to(y_new, y_old, x):
    a = y_new.astype(np.float64)
    b = y_old.astype(np.float64)
    assert np.all(np.isfinite(a))
    for m in range(b.shape[0]):
        rel = np.linalg.norm(a[m] - b[m]) / np.linalg.norm(b[m])
        assert rel <= REL_L2_TOL
        assert np.max(np.abs(a[m] - b[m])) <= MAX_ABS_COEF * np.max(np.abs(x[m].astype(np.float64))) * np.sqrt(x.shape[1])


def test_static_workspace_entry_point_matches_workspace_entry_point_twice():
    L = binding.lib()
    N, K, M = 1000, 4096, 6
    c = make_case(N, K, seed=70, M=M)
    packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]))
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    shape = binding.make_shape(N, K)
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    need = binding.gemm_skinny_workspace_size(N, K, M)
    assert 0 < need <= binding.STATIC_WORKSPACE_BYTES
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    for call, seed in enumerate((71, 72)):                       # two calls in a row, different activations
        x = make_case(N, K, seed=seed, M=M)["x"]
        X = dev(x)
        Y_old = torch.empty((M, N), dtype=torch.float16, device="cuda")
        Y_new = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
        rc = L.ptqtp_gemm_skinny_ws(ctypes.byref(shape), packed.data_ptr(), packed.numel(), M, X.data_ptr(),
                                    Y_old.data_ptr(), ws.data_ptr(), ws.numel(), stream)
        assert rc == binding.OK
        rc = L.ptqtp_gemm_skinny_static(ctypes.byref(shape), packed.data_ptr(), packed.numel(), M, X.data_ptr(),
                                        Y_new.data_ptr(), stream)
        assert rc == binding.OK, binding.status_string(rc)
        torch.cuda.synchronize()
        close_to(Y_new.cpu().numpy(), Y_old.cpu().numpy(), x)
        assert np.array_equal(Y_new.cpu().numpy().view(np.uint16), Y_old.cpu().numpy().view(np.uint16))
        assert_parity(Y_new.cpu().numpy(), oracle_y(dict(c, x=x)), x, "static workspace call %d" % call)


def test_static_workspace_entry_point_refuses_what_does_not_fit():
    L = binding.lib()
    N, K, M = 8, 8192, 64                                         # 2 * 64 * 8192 bytes of activations alone: too large
    assert binding.gemm_skinny_workspace_size(N, K, M) > binding.STATIC_WORKSPACE_BYTES
    c = make_case(N, K, seed=73, M=M)
    packed, _ = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]))
    X = dev(c["x"])
    Y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    shape = binding.make_shape(N, K)
    rc = L.ptqtp_gemm_skinny_static(ctypes.byref(shape), packed.data_ptr(), packed.numel(), M, X.data_ptr(),
                                    Y.data_ptr(), None)
    assert rc == binding.ERR_SIZE
    torch.cuda.synchronize()
    assert not bool(Y.any())                                      # nothing was launched
    with pytest.raises(binding.PtqtpError) as e:
        binding.ptqtp_gemm_skinny_static(packed, N, K, X, Y)
    assert e.value.status == binding.ERR_SIZE
