"""ctypes binding of libptqtp.so: argument marshalling only; every step runs in the CUDA kernels.

torch supplies device memory and streams.  Function names mirror the C ABI (include/ptqtp.h).
There is no CPU path: if the shared library is missing or a call fails, a PtqtpError is raised.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libptqtp.so")

GROUP = 128
FORMAT_V1 = 1
FORMAT_V2 = 2
FORMAT_V3 = 3
DEFAULT_FORMAT = FORMAT_V2
HEADER_BYTES = 256
MAX_BATCH = 64

OK, ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_SIZE, ERR_TRIT, ERR_FORMAT, ERR_CUDA, ERR_CONFIG = (
    0, -1, -2, -3, -4, -5, -6, -7, -8)

EXPORTS = ("ptqtp_packed_size", "ptqtp_pack", "ptqtp_unpack", "ptqtp_gemv", "ptqtp_gemm_skinny", "ptqtp_gemm_skinny_cfg",
           "ptqtp_gemv_host", "ptqtp_gemv_cfg", "ptqtp_parse_header", "ptqtp_status_string",
           "ptqtp_last_cuda_error", "ptqtp_version", "ptqtp_set_overlap", "ptqtp_gemm_skinny_workspace_size", "ptqtp_gemm_skinny_ws",
           "ptqtp_gemm_skinny_static", "ptqtp_kernel_status", "ptqtp_gemv_swiglu", "ptqtp_kernel_status_clear",
           "ptqtp_set_wait_limit", "ptqtp_test_fail_next_wait", "ptqtp_gemv_multi", "ptqtp_decompose",
           "ptqtp_decompose_workspace_size", "ptqtp_decompose_layout")


class PtqtpError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s failed: %s (status %d, cuda error %d)"
                         % (what, status_string(status), status, lib().ptqtp_last_cuda_error()))


class DecomposeOffsets(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in ("sweeps_offset", "delta_offset", "error_offset", "alpha1_offset",
                                               "alpha2_offset", "lambda_offset", "total_bytes")]


class Shape(ctypes.Structure):
    _fields_ = [("n_out", ctypes.c_int32), ("k_in", ctypes.c_int32), ("group", ctypes.c_int32),
                ("format", ctypes.c_int32)]


_lib = None


def lib():
    """Load libptqtp.so (built in-tree by build.py).  Raises if it is absent: no fallback exists."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libptqtp.so not found at %s: run `python -m paper_2509_16989_b200.build`"
                               % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
        sp = ctypes.POINTER(Shape)
        L.ptqtp_packed_size.restype = sz
        L.ptqtp_packed_size.argtypes = [sp]
        L.ptqtp_pack.restype = ctypes.c_int
        L.ptqtp_pack.argtypes = [sp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.ptqtp_unpack.restype = ctypes.c_int
        L.ptqtp_unpack.argtypes = [sp, vp, sz, vp, vp, vp, vp, vp, vp]
        L.ptqtp_gemv.restype = ctypes.c_int
        L.ptqtp_gemv.argtypes = [sp, vp, sz, vp, vp, vp]
        L.ptqtp_gemv_swiglu.restype = ctypes.c_int
        L.ptqtp_gemv_swiglu.argtypes = [sp, vp, sz, vp, vp, vp]
        L.ptqtp_decompose_workspace_size.restype = sz
        L.ptqtp_decompose_workspace_size.argtypes = [i32, i32, i32, i32]
        L.ptqtp_decompose_layout.restype = ctypes.c_int
        L.ptqtp_decompose_layout.argtypes = [i32, i32, i32, i32, ctypes.POINTER(DecomposeOffsets)]
        L.ptqtp_decompose.restype = ctypes.c_int
        L.ptqtp_decompose.argtypes = [vp, i32, i32, i32, i32, ctypes.c_double, i32, vp, vp, vp, vp, vp, sz, vp]
        L.ptqtp_gemv_multi.restype = ctypes.c_int
        L.ptqtp_gemv_multi.argtypes = [i32, sp, ctypes.POINTER(vp), ctypes.POINTER(sz), vp, ctypes.POINTER(vp), i32, vp]
        L.ptqtp_gemm_skinny.restype = ctypes.c_int
        L.ptqtp_gemm_skinny.argtypes = [sp, vp, sz, i32, vp, vp, vp]
        L.ptqtp_gemm_skinny_cfg.restype = ctypes.c_int
        L.ptqtp_gemm_skinny_cfg.argtypes = [sp, vp, sz, i32, vp, vp, i32, i32, vp]
        L.ptqtp_gemm_skinny_workspace_size.restype = sz
        L.ptqtp_gemm_skinny_workspace_size.argtypes = [sp, i32]
        L.ptqtp_gemm_skinny_ws.restype = ctypes.c_int
        L.ptqtp_gemm_skinny_ws.argtypes = [sp, vp, sz, i32, vp, vp, vp, sz, vp]
        L.ptqtp_gemm_skinny_static.restype = ctypes.c_int
        L.ptqtp_gemm_skinny_static.argtypes = [sp, vp, sz, i32, vp, vp, vp]
        L.ptqtp_gemv_host.restype = ctypes.c_int
        L.ptqtp_gemv_host.argtypes = [sp, vp, sz, vp, vp, vp, vp, vp]
        L.ptqtp_gemv_cfg.restype = ctypes.c_int
        L.ptqtp_gemv_cfg.argtypes = [sp, vp, sz, vp, vp, i32, i32, i32, i32, i32, vp]
        L.ptqtp_parse_header.restype = ctypes.c_int
        L.ptqtp_parse_header.argtypes = [vp, sz, sp]
        L.ptqtp_status_string.restype = ctypes.c_char_p
        L.ptqtp_status_string.argtypes = [ctypes.c_int]
        L.ptqtp_last_cuda_error.restype = ctypes.c_int
        L.ptqtp_version.restype = ctypes.c_int
        L.ptqtp_kernel_status.restype = ctypes.c_int
        L.ptqtp_kernel_status.argtypes = [ctypes.POINTER(ctypes.c_int32), vp]
        L.ptqtp_set_overlap.restype = ctypes.c_int
        L.ptqtp_set_overlap.argtypes = [ctypes.c_int]
        L.ptqtp_kernel_status_clear.restype = ctypes.c_int
        L.ptqtp_kernel_status_clear.argtypes = [vp]
        L.ptqtp_set_wait_limit.restype = ctypes.c_int
        L.ptqtp_set_wait_limit.argtypes = [ctypes.c_int]
        L.ptqtp_test_fail_next_wait.restype = None
        L.ptqtp_test_fail_next_wait.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def status_string(status):
    return lib().ptqtp_status_string(int(status)).decode()


def make_shape(N, K, group=GROUP, fmt=None):
    if fmt is None:
        fmt = DEFAULT_FORMAT
    return Shape(int(N), int(K), int(group), int(fmt))


def packed_size(N, K, fmt=None):
    return int(lib().ptqtp_packed_size(ctypes.byref(make_shape(N, K, fmt=fmt))))


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dev(t, dtype, what):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (what, dtype))
    return ctypes.c_void_p(t.data_ptr())


def _check(status, what):
    if status != OK:
        raise PtqtpError(status, what)


def ptqtp_pack(T1, T2, alpha1, alpha2, packed=None, dev_status=None, stream=None, fmt=None):
    """Pack int8 planes [N,K] and fp16 scales [N,K/128] (CUDA tensors).  Returns (packed uint8 tensor, dev_status)."""
    N, K = T1.shape
    shape = make_shape(N, K, fmt=fmt)
    nbytes = packed_size(N, K, fmt=fmt)
    if nbytes == 0:
        raise PtqtpError(ERR_SHAPE, "ptqtp_packed_size")
    if packed is None:
        packed = torch.empty(nbytes, dtype=torch.uint8, device=T1.device)
    if dev_status is None:
        dev_status = torch.zeros(1, dtype=torch.int32, device=T1.device)
    st = lib().ptqtp_pack(ctypes.byref(shape), _dev(T1, torch.int8, "T1"), _dev(T2, torch.int8, "T2"),
                          _dev(alpha1, torch.float16, "alpha1"), _dev(alpha2, torch.float16, "alpha2"),
                          _dev(packed, torch.uint8, "packed"), packed.numel(),
                          _dev(dev_status, torch.int32, "dev_status"), _stream_ptr(stream))
    _check(st, "ptqtp_pack")
    return packed, dev_status


def ptqtp_unpack(packed, N, K, dev_status=None, stream=None, fmt=None):
    """Inverse of ptqtp_pack.  Returns (T1, T2, alpha1, alpha2, dev_status) as CUDA tensors."""
    shape = make_shape(N, K, fmt=fmt)
    dev = packed.device
    T1 = torch.empty((N, K), dtype=torch.int8, device=dev)
    T2 = torch.empty((N, K), dtype=torch.int8, device=dev)
    a1 = torch.empty((N, K // GROUP), dtype=torch.float16, device=dev)
    a2 = torch.empty((N, K // GROUP), dtype=torch.float16, device=dev)
    if dev_status is None:
        dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
    st = lib().ptqtp_unpack(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                            _dev(T1, torch.int8, "T1"), _dev(T2, torch.int8, "T2"),
                            _dev(a1, torch.float16, "alpha1"), _dev(a2, torch.float16, "alpha2"),
                            _dev(dev_status, torch.int32, "dev_status"), _stream_ptr(stream))
    _check(st, "ptqtp_unpack")
    return T1, T2, a1, a2, dev_status


def ptqtp_gemv(packed, N, K, x, y=None, stream=None, fmt=None):
    """y[N] = layer(x[K]) from a packed blob; fp16 CUDA tensors."""
    shape = make_shape(N, K, fmt=fmt)
    if y is None:
        y = torch.empty(N, dtype=torch.float16, device=x.device)
    st = lib().ptqtp_gemv(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                          _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"), _stream_ptr(stream))
    _check(st, "ptqtp_gemv")
    return y


def ptqtp_gemv_cfg(packed, N, K, x, y=None, rows_per_warp=0, k_split=0, ctas_per_sm=0, depth=0, arith=-1,
                   stream=None, fmt=None):
    shape = make_shape(N, K, fmt=fmt)
    if y is None:
        y = torch.empty(N, dtype=torch.float16, device=x.device)
    st = lib().ptqtp_gemv_cfg(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                              _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"),
                              int(rows_per_warp), int(k_split), int(ctas_per_sm), int(depth), int(arith),
                              _stream_ptr(stream))
    _check(st, "ptqtp_gemv_cfg")
    return y


def ptqtp_gemv_swiglu(packed, N, K, x, y=None, stream=None, fmt=FORMAT_V2):
    """y[N/2] = silu(row 2i) * row 2i+1 of the layer applied to x; packed holds gate/up rows interleaved (format 2 or 3)."""
    shape = make_shape(N, K, fmt=fmt)
    if y is None:
        y = torch.empty(N // 2, dtype=torch.float16, device=x.device)
    st = lib().ptqtp_gemv_swiglu(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                                 _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"), _stream_ptr(stream))
    _check(st, "ptqtp_gemv_swiglu")
    return y


def ptqtp_decompose(W, group=GROUP, t_max=50, eps=1e-4, canonicalize=True, stream=None, details=False):
    """Trit-plane decomposition of a CUDA fp32 matrix W [N, K] on the GPU.  Returns (T1, T2, alpha1, alpha2) as CUDA
    tensors (int8 planes, fp16 scales [N, K/group]); with details=True also a dict with the number of sweeps, the
    per-sweep largest scale change and total squared error, and the unrounded fp64 scales (synchronises)."""
    N, K = W.shape
    need = int(lib().ptqtp_decompose_workspace_size(N, K, int(group), int(t_max)))
    if need == 0:
        raise PtqtpError(ERR_SHAPE, "ptqtp_decompose_workspace_size")
    dev = W.device
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    T1 = torch.empty((N, K), dtype=torch.int8, device=dev)
    T2 = torch.empty((N, K), dtype=torch.int8, device=dev)
    a1 = torch.empty((N, K // group), dtype=torch.float16, device=dev)
    a2 = torch.empty((N, K // group), dtype=torch.float16, device=dev)
    st = lib().ptqtp_decompose(_dev(W, torch.float32, "W"), N, K, int(group), int(t_max), float(eps), int(bool(canonicalize)),
                               _dev(T1, torch.int8, "T1"), _dev(T2, torch.int8, "T2"), _dev(a1, torch.float16, "alpha1"),
                               _dev(a2, torch.float16, "alpha2"), _dev(ws, torch.uint8, "workspace"), ws.numel(),
                               _stream_ptr(stream))
    _check(st, "ptqtp_decompose")
    if not details:
        return T1, T2, a1, a2
    off = DecomposeOffsets()
    _check(lib().ptqtp_decompose_layout(N, K, int(group), int(t_max), ctypes.byref(off)), "ptqtp_decompose_layout")
    (stream or torch.cuda.current_stream()).synchronize()
    host = ws.cpu().numpy()
    R = N * (K // group)
    sweeps = int(host[off.sweeps_offset:off.sweeps_offset + 4].view("<i4")[0])
    f64 = lambda o, n: host[o:o + 8 * n].view("<f8").copy()
    info = dict(sweeps=sweeps, delta_history=f64(off.delta_offset + 8, sweeps), err_history=f64(off.error_offset, sweeps),
                alpha1=f64(off.alpha1_offset, R).reshape(N, K // group), alpha2=f64(off.alpha2_offset, R).reshape(N, K // group),
                lam=f64(off.lambda_offset, R).reshape(N, K // group))
    return T1, T2, a1, a2, info


EPILOGUE_NONE, EPILOGUE_GATED_PAIR = 0, 1


def ptqtp_gemv_multi(packed_list, N_list, K, x, ys=None, epilogue=EPILOGUE_NONE, stream=None):
    """One launch for several format-3 matrices that share x: returns the list of outputs (one output for the
    gated pair epilogue: silu(matrix 0) * matrix 1)."""
    count = len(packed_list)
    shapes = (Shape * count)(*[make_shape(N, K, fmt=FORMAT_V3) for N in N_list])
    n_out = 1 if epilogue == EPILOGUE_GATED_PAIR else count
    if ys is None:
        ys = [torch.empty(N_list[j], dtype=torch.float16, device=x.device) for j in range(n_out)]
    ptrs = (ctypes.c_void_p * count)(*[_dev(p, torch.uint8, "packed").value for p in packed_list])
    sizes = (ctypes.c_size_t * count)(*[p.numel() for p in packed_list])
    yp = (ctypes.c_void_p * count)(*([_dev(y, torch.float16, "y").value for y in ys] + [None] * (count - len(ys))))
    st = lib().ptqtp_gemv_multi(count, shapes, ptrs, sizes, _dev(x, torch.float16, "x"), yp, int(epilogue),
                                _stream_ptr(stream))
    _check(st, "ptqtp_gemv_multi")
    return ys


def ptqtp_gemm_skinny(packed, N, K, X, Y=None, stream=None, fmt=None):
    """Y[M,N] = layer applied to each row of X[M,K]; fp16 CUDA tensors, 1 <= M <= 64."""
    shape = make_shape(N, K, fmt=fmt)
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=X.device)
    st = lib().ptqtp_gemm_skinny(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                                 int(M), _dev(X, torch.float16, "X"), _dev(Y, torch.float16, "Y"),
                                 _stream_ptr(stream))
    _check(st, "ptqtp_gemm_skinny")
    return Y


def ptqtp_gemm_skinny_cfg(packed, N, K, X, Y=None, path=0, k_split=0, stream=None):
    """ptqtp_gemm_skinny on format 3 with the kernel chosen by the caller (path 0 / 5 / 6, k_split 0 / 1 / 2 / 4 / 8)."""
    shape = make_shape(N, K, fmt=FORMAT_V3)
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=X.device)
    st = lib().ptqtp_gemm_skinny_cfg(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                                     int(M), _dev(X, torch.float16, "X"), _dev(Y, torch.float16, "Y"), int(path),
                                     int(k_split), _stream_ptr(stream))
    _check(st, "ptqtp_gemm_skinny_cfg")
    return Y


def gemm_skinny_workspace_size(N, K, M, fmt=None):
    return int(lib().ptqtp_gemm_skinny_workspace_size(ctypes.byref(make_shape(N, K, fmt=fmt)), int(M)))


def ptqtp_gemm_skinny_ws(packed, N, K, X, Y=None, workspace=None, stream=None, fmt=None):
    """ptqtp_gemm_skinny with a caller-provided workspace (uint8 CUDA tensor; allocated here if None)."""
    shape = make_shape(N, K, fmt=fmt)
    M = X.shape[0]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=X.device)
    if workspace is None:
        workspace = torch.empty(gemm_skinny_workspace_size(N, K, M, fmt=fmt), dtype=torch.uint8, device=X.device)
    st = lib().ptqtp_gemm_skinny_ws(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(), int(M),
                                    _dev(X, torch.float16, "X"), _dev(Y, torch.float16, "Y"),
                                    _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream))
    _check(st, "ptqtp_gemm_skinny_ws")
    return Y


STATIC_WORKSPACE_BYTES = 512 * 1024


def ptqtp_gemm_skinny_static(packed, N, K, X, Y, stream=None, fmt=None):
    """ptqtp_gemm_skinny_ws on the library's own fixed workspace: for callers that cannot allocate device memory.

    Y must be passed in (this wrapper allocates nothing either).  Raises PtqtpError(ERR_SIZE) when
    gemm_skinny_workspace_size(N, K, M) exceeds STATIC_WORKSPACE_BYTES.  Calls share one array per device:
    do not let two of them overlap on the GPU."""
    shape = make_shape(N, K, fmt=fmt)
    st = lib().ptqtp_gemm_skinny_static(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                                        int(X.shape[0]), _dev(X, torch.float16, "X"), _dev(Y, torch.float16, "Y"),
                                        _stream_ptr(stream))
    _check(st, "ptqtp_gemm_skinny_static")
    return Y


def ptqtp_gemv_host(packed, N, K, x_host, y_host, x_dev, y_dev, stream=None, fmt=None):
    """Host-buffer call: H2D copy of x, GEMV, D2H copy of y, all on `stream` (no sync)."""
    shape = make_shape(N, K, fmt=fmt)
    for t, what in ((x_host, "x_host"), (y_host, "y_host")):
        if t.is_cuda or t.dtype != torch.float16 or not t.is_contiguous():
            raise TypeError("%s must be a contiguous fp16 host tensor" % what)
    st = lib().ptqtp_gemv_host(ctypes.byref(shape), _dev(packed, torch.uint8, "packed"), packed.numel(),
                               ctypes.c_void_p(x_host.data_ptr()), ctypes.c_void_p(y_host.data_ptr()),
                               _dev(x_dev, torch.float16, "x_dev"), _dev(y_dev, torch.float16, "y_dev"),
                               _stream_ptr(stream))
    _check(st, "ptqtp_gemv_host")
    return y_host


def ptqtp_kernel_status(stream=None):
    """Device-side health word of the batch-1 kernel (0 = healthy); synchronises the stream to read it."""
    out = ctypes.c_int32(-1)
    if stream is None:
        stream = torch.cuda.current_stream()
    _check(lib().ptqtp_kernel_status(ctypes.byref(out), ctypes.c_void_p(stream.cuda_stream)), "ptqtp_kernel_status")
    stream.synchronize()
    return int(out.value)


def ptqtp_kernel_status_clear(stream=None):
    """Reset the device-side health word to 0 (enqueued on the stream)."""
    _check(lib().ptqtp_kernel_status_clear(_stream_ptr(stream)), "ptqtp_kernel_status_clear")


def ptqtp_set_wait_limit(polls):
    """Polls after which a bounded wait for a bulk copy gives up; returns the old value."""
    return int(lib().ptqtp_set_wait_limit(int(polls)))


def ptqtp_test_fail_next_wait(launches):
    """Test hook: the next `launches` format-3 batch-1 launches let one bounded wait run out."""
    lib().ptqtp_test_fail_next_wait(int(launches))


def ptqtp_set_overlap(level):
    """Overlap level of consecutive GEMV calls: 0 (default) plain launches, 1 programmatic dependent launch, 2 also
    the speculative read of x.  True/False mean 2/0.  Returns the old level."""
    if level is True:
        level = 2
    return int(lib().ptqtp_set_overlap(int(level)))


def ptqtp_parse_header(header_bytes):
    """Parse a host copy (bytes) of a blob's header; returns (N, K, format)."""
    buf = ctypes.create_string_buffer(bytes(header_bytes), len(header_bytes))
    shape = Shape()
    st = lib().ptqtp_parse_header(ctypes.cast(buf, ctypes.c_void_p), len(header_bytes), ctypes.byref(shape))
    _check(st, "ptqtp_parse_header")
    return shape.n_out, shape.k_in, shape.format
