"""ctypes access to oracle/c/ptqtp_oracle.c (plain C loops).  Test infrastructure only.

``build()`` compiles the C file with gcc into oracle/c/libptqtp_oracle.so (no fast-math, no FMA
contraction, OpenMP over independent rows / group-rows).  The wrappers marshal numpy arrays.
"""
import ctypes
import os
import subprocess

import numpy as np

_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c")
_SRC = os.path.join(_DIR, "ptqtp_oracle.c")
_LIB = os.path.join(_DIR, "libptqtp_oracle.so")
_lib = None

TIE_BREAK = {"sparse_first": 0, "meshgrid": 1}
LAMBDA_ORDER = {"update_then_solve": 0, "solve_then_update": 1}
CONV_RULE = {"max_rows": 0, "frobenius_all": 1, "per_group_freeze": 2}


def build(force=False):
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
           "-fPIC", _SRC, "-o", _LIB, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_max_threads.restype = ctypes.c_int
        lib.oracle_layer_fp64.restype = None
        lib.oracle_layer_fp64.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int] * 4 + [
            ctypes.c_void_p, ctypes.c_int]
        lib.oracle_decompose.restype = ctypes.c_int
        lib.oracle_decompose.argtypes = ([ctypes.c_void_p] + [ctypes.c_int] * 4 + [ctypes.c_double] * 4
                                         + [ctypes.c_int] * 4 + [ctypes.c_void_p] * 6 + [ctypes.c_int])
        _lib = lib
    return _lib


def max_threads():
    return int(_load().oracle_max_threads())


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def layer_fp64_c(T1, T2, alpha1_fp16, alpha2_fp16, x_fp16, G=128, threads=1):
    """fp64 layer product by scalar C loops.  x: [K] or [M, K] fp16; returns [N] or [M, N] fp64."""
    T1 = np.ascontiguousarray(T1, dtype=np.int8)
    T2 = np.ascontiguousarray(T2, dtype=np.int8)
    a1 = np.ascontiguousarray(alpha1_fp16, dtype=np.float16)
    a2 = np.ascontiguousarray(alpha2_fp16, dtype=np.float16)
    x = np.ascontiguousarray(x_fp16, dtype=np.float16)
    N, K = T1.shape
    single = x.ndim == 1
    M = 1 if single else x.shape[0]
    assert T2.shape == (N, K) and a1.shape == (N, K // G) and a2.shape == (N, K // G)
    assert x.shape[-1] == K and K % G == 0
    y = np.empty((M, N), dtype=np.float64)
    _load().oracle_layer_fp64(_ptr(T1), _ptr(T2), _ptr(a1), _ptr(a2), _ptr(x), N, K, G, M, _ptr(y),
                              int(threads))
    return y[0] if single else y


def decompose_c(W, G=128, T_max=50, eps=1e-4, lambda0=1e-8, lambda_max=1.0, kappa_thr=1e6,
                tie_break="sparse_first", lambda_order="update_then_solve", conv_rule="max_rows",
                canonicalize=True, threads=None):
    """The decomposition of oracle.decompose.decompose as C loops (same results, bit for bit)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    T1 = np.empty((N, K), dtype=np.int8)
    T2 = np.empty((N, K), dtype=np.int8)
    a1 = np.empty((N, K // G), dtype=np.float64)
    a2 = np.empty((N, K // G), dtype=np.float64)
    eh = np.zeros(T_max, dtype=np.float64)
    dh = np.zeros(T_max, dtype=np.float64)
    if threads is None:
        threads = max_threads()
    sweeps = _load().oracle_decompose(_ptr(W), N, K, G, T_max, eps, lambda0, lambda_max, kappa_thr,
                                      TIE_BREAK[tie_break], LAMBDA_ORDER[lambda_order],
                                      CONV_RULE[conv_rule], int(bool(canonicalize)), _ptr(T1), _ptr(T2),
                                      _ptr(a1), _ptr(a2), _ptr(eh), _ptr(dh), int(threads))
    if sweeps < 0:
        raise ValueError("oracle_decompose rejected its arguments")
    return dict(T1=T1, T2=T2, alpha1=a1, alpha2=a2, alpha1_fp16=a1.astype(np.float16),
                alpha2_fp16=a2.astype(np.float16), sweeps=sweeps,
                err_history=[float(v) for v in eh[:sweeps]],
                delta_history=[float(v) for v in dh[:sweeps]])
