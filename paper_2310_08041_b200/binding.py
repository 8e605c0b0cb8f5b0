"""ctypes bindings of the C ABI in ``include/qllm.h`` (argument marshalling only).

Device arguments are torch CUDA tensors (torch is used for device memory and
streams, nothing else); host arguments are numpy arrays.  Function names match the
C entry points.  Importing this module loads ``libqllm_b200.so`` and raises if it
is missing: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch  # noqa: F401  (loads the CUDA runtime the library links against)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqllm_b200.so")

QLLM_OK = 0
QLLM_ERR_NULL, QLLM_ERR_SHAPE, QLLM_ERR_BITS, QLLM_ERR_DTYPE = -1, -2, -3, -4
QLLM_ERR_MAP, QLLM_ERR_INFEASIBLE, QLLM_ERR_CUDA, QLLM_ERR_TIMEOUT = -5, -6, -7, -8
QLLM_ERR_ALIGN, QLLM_ERR_UNSUPPORTED, QLLM_ERR_NOMEM = -9, -10, -11
QLLM_F32, QLLM_BF16 = 0, 1

# every symbol include/qllm.h declares
EXPORTS = [
    "qllm_reassemble_quant", "qllm_quantize_rows", "qllm_qgemm", "qllm_qgemm_noalloc", "qllm_qgemm_acc", "qllm_calib_absmax",
    "qllm_build_reassembly", "qllm_build_reassembly_eq5", "qllm_build_reassembly_dist", "qllm_layernorm_rows", "qllm_channel_distance", "qllm_free_reassembly", "qllm_reassembly_map",
    "qllm_reassembly_weights", "qllm_reassembly_stats", "qllm_validate_map", "qllm_fold_previous",
    "qllm_theta_percentile", "qllm_theta_for_extra", "qllm_search_theta",
    "qllm_layer_create", "qllm_layer_destroy", "qllm_layer_forward", "qllm_layer_forward_host",
    "qllm_layer_reassemble_quant", "qllm_layer_qgemm",
    "qllm_layer_workspace", "qllm_layer_keep_byte_weights",
    "qllm_status_string", "qllm_last_cuda_error", "qllm_poll_status", "qllm_launch_count", "qllm_debug_wait_expiry",
]

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2310_08041_b200.build` "
        "(nvcc, sm_100a).  There is no CPU fallback.")
_lib = ctypes.CDLL(LIB_PATH)

_vp, _i, _i64, _f, _d = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_double
_lib.qllm_reassemble_quant.argtypes = [_vp, _i, _i64, _i, _vp, _vp, _f, _vp, _vp, _vp, _i, _vp, _vp, _vp, _vp, _vp]
_lib.qllm_quantize_rows.argtypes = [_vp, _i, _i64, _i, _i, _vp, _vp, _vp, _vp, _vp]
_lib.qllm_qgemm.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i, _i, _i, _i, _i, _vp, _vp]
_lib.qllm_qgemm_noalloc.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i, _i, _i, _i, _i, _vp]
_lib.qllm_qgemm_acc.argtypes = [_vp, _vp, _vp, _i64, _i, _i, _i, _i, _vp]
_lib.qllm_calib_absmax.argtypes = [_vp, _i, _i64, _i, _vp, _vp, _f, _vp, _vp]
_lib.qllm_build_reassembly.argtypes = [_vp, _i, _f, _vp, _i, _vp, _vp, _i, _i, ctypes.POINTER(_vp)]
_lib.qllm_build_reassembly_dist.argtypes = [_vp, _i, _f, _vp, _vp, _i, _vp, _vp, _i, _i, ctypes.POINTER(_vp)]
_lib.qllm_build_reassembly_eq5.argtypes = [_vp, _i, _f, _vp, _i64, _vp, _i, _vp, _vp, _i, _i, _vp, ctypes.POINTER(_vp)]
_lib.qllm_layernorm_rows.argtypes = [_vp, _i, _i64, _i, _vp, _vp, _f, _vp, _vp]
_lib.qllm_channel_distance.argtypes = [_vp, _i64, _vp, _i, _i, _vp, _vp]
_lib.qllm_free_reassembly.argtypes = [_vp]
_lib.qllm_free_reassembly.restype = None
_lib.qllm_reassembly_map.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_i64)]
_lib.qllm_reassembly_weights.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_i64), ctypes.POINTER(_vp),
                                         ctypes.POINTER(_vp), ctypes.POINTER(_vp)]
_lib.qllm_reassembly_stats.argtypes = [_vp, ctypes.POINTER(_i64)]
_lib.qllm_validate_map.argtypes = [_vp, _vp, _i, _i64]
_lib.qllm_theta_percentile.argtypes = [_vp, _i, _d]
_lib.qllm_theta_percentile.restype = _f
_lib.qllm_search_theta.argtypes = [_vp, _i, _i64, _i, _vp, _vp, _f, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp]
_lib.qllm_fold_previous.argtypes = [_vp, _vp, _vp, _i, _vp, _vp, _i, _vp, _vp]
_lib.qllm_theta_for_extra.argtypes = [_vp, _i, _i]
_lib.qllm_theta_for_extra.restype = _f
_lib.qllm_layer_create.argtypes = [_vp, _vp, _vp, _f, _vp, _i, _i, _i, _i64, ctypes.POINTER(_vp)]
_lib.qllm_layer_destroy.argtypes = [_vp]
_lib.qllm_layer_destroy.restype = None
_lib.qllm_layer_forward.argtypes = [_vp, _vp, _i64, _vp, _vp]
_lib.qllm_layer_forward_host.argtypes = [_vp, _vp, _i64, _vp, _vp]
_lib.qllm_layer_reassemble_quant.argtypes = [_vp, _vp, _i64, _vp]
_lib.qllm_layer_qgemm.argtypes = [_vp, _i64, _vp, _vp]
_lib.qllm_layer_workspace.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp),
                                      ctypes.POINTER(ctypes.c_int)]
_lib.qllm_layer_keep_byte_weights.argtypes = [_vp, _i, _vp]
_lib.qllm_status_string.argtypes = [_i]
_lib.qllm_status_string.restype = ctypes.c_char_p
_lib.qllm_launch_count.restype = _i64
_lib.qllm_debug_wait_expiry.argtypes = [_vp, _vp]


class QllmError(RuntimeError):
    def __init__(self, status):
        self.status = status
        msg = _lib.qllm_status_string(status).decode()
        if status == QLLM_ERR_CUDA:
            msg += " [cudaError %d]" % _lib.qllm_last_cuda_error()
        super().__init__("qllm status %d: %s" % (status, msg))


def _check(status):
    if status != QLLM_OK:
        raise QllmError(status)


def _dp(t):
    """Device pointer of a torch tensor (None -> NULL)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device arguments must be contiguous CUDA tensors"
    return t.data_ptr()


def _hp(a):
    return None if a is None else a.ctypes.data_as(_vp)


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _xdtype(t):
    if t.dtype == torch.float32:
        return QLLM_F32
    if t.dtype == torch.bfloat16:
        return QLLM_BF16
    raise QllmError(QLLM_ERR_DTYPE)


# --------------------------------------------------------------------------- device calls
def qllm_reassemble_quant(x, ln_gamma, ln_beta, map_ptr, map_src, map_coef, bits, codes, a_scale, a_zero,
                          a_rowsum=None, ln_eps=1e-5, stream=None):
    M, C = x.shape
    _check(_lib.qllm_reassemble_quant(_dp(x), _xdtype(x), M, C, _dp(ln_gamma), _dp(ln_beta), ln_eps,
                                      _dp(map_ptr), _dp(map_src), _dp(map_coef), bits, _dp(codes),
                                      _dp(a_scale), _dp(a_zero), _dp(a_rowsum), _stream(stream)))


def qllm_quantize_rows(x, bits, codes, a_scale, a_zero, a_rowsum=None, stream=None):
    """Eq. 2 per token row of x [M][C] (no LayerNorm, no map): the run-time stage of a folded layer (Appendix B)."""
    M, C = x.shape
    _check(_lib.qllm_quantize_rows(_dp(x), _xdtype(x), M, C, bits, _dp(codes), _dp(a_scale), _dp(a_zero), _dp(a_rowsum),
                                   _stream(stream)))


def qllm_qgemm(codes, a_scale, a_zero, w_codes, w_scale, w_zero, w_colsum, bias, out, M, N, K, a_bits, w_bits,
               a_rowsum=None, stream=None):
    _check(_lib.qllm_qgemm(_dp(codes), _dp(a_scale), _dp(a_zero), _dp(w_codes), _dp(w_scale), _dp(w_zero),
                           _dp(w_colsum), _dp(bias), _dp(out), M, N, K, a_bits, w_bits, _xdtype(out),
                           _dp(a_rowsum), _stream(stream)))


QLLM_NOALLOC_MAX_M = 65536


def qllm_qgemm_noalloc(codes, a_scale, a_zero, w_codes, w_scale, w_zero, w_colsum, bias, out, M, N, K, a_bits, w_bits,
                       stream=None):
    """qllm_qgemm for callers that must not allocate: the activation row sums are computed into
    a fixed array inside the library (at most QLLM_NOALLOC_MAX_M rows), never into cudaMalloc'd
    scratch.  Calls on one device share that array, so do not overlap them on the GPU."""
    _check(_lib.qllm_qgemm_noalloc(_dp(codes), _dp(a_scale), _dp(a_zero), _dp(w_codes), _dp(w_scale), _dp(w_zero),
                                   _dp(w_colsum), _dp(bias), _dp(out), M, N, K, a_bits, w_bits, _xdtype(out),
                                   _stream(stream)))


def qllm_qgemm_acc(codes, w_codes, acc, M, N, K, a_bits, w_bits, stream=None):
    assert acc.dtype == torch.int32
    _check(_lib.qllm_qgemm_acc(_dp(codes), _dp(w_codes), _dp(acc), M, N, K, a_bits, w_bits, _stream(stream)))


def qllm_calib_absmax(x, ln_gamma, ln_beta, absmax, ln_eps=1e-5, stream=None):
    M, C = x.shape
    _check(_lib.qllm_calib_absmax(_dp(x), _xdtype(x), M, C, _dp(ln_gamma), _dp(ln_beta), ln_eps,
                                  _dp(absmax), _stream(stream)))


def qllm_poll_status():
    return _lib.qllm_poll_status()


def qllm_debug_wait_expiry(gave_up, stream=None):
    """Runs a bounded device-side wait into its (short) limit; gave_up: device int32 tensor, set to 1."""
    _check(_lib.qllm_debug_wait_expiry(_dp(gave_up), _stream(stream)))


def qllm_launch_count():
    return int(_lib.qllm_launch_count())


def qllm_status_string(status):
    return _lib.qllm_status_string(status).decode()


def qllm_last_cuda_error():
    return int(_lib.qllm_last_cuda_error())


# --------------------------------------------------------------------------- host calls
def qllm_theta_percentile(absmax, pct):
    a = np.ascontiguousarray(absmax, np.float32)
    return float(_lib.qllm_theta_percentile(_hp(a), a.shape[0], pct))


def qllm_theta_for_extra(absmax, extra):
    a = np.ascontiguousarray(absmax, np.float32)
    return float(_lib.qllm_theta_for_extra(_hp(a), a.shape[0], extra))


def qllm_search_theta(calib_x, ln_gamma, ln_beta, absmax, W, a_bits, w_bits, P, ln_eps=1e-5, stream=None):
    """calib_x: device tensor [T][C]; ln_gamma, ln_beta (or None), absmax [C], W [N][C]: numpy (host).
    Returns (theta, losses float64[P])."""
    T, C = calib_x.shape
    g = np.ascontiguousarray(ln_gamma, np.float32)
    b = None if ln_beta is None else np.ascontiguousarray(ln_beta, np.float32)
    a = np.ascontiguousarray(absmax, np.float32)
    w = np.ascontiguousarray(W, np.float32)
    assert g.shape == (C,) and a.shape == (C,) and w.shape[1] == C
    theta = ctypes.c_float(0.0)
    losses = np.empty(P, np.float64)
    _check(_lib.qllm_search_theta(_dp(calib_x), _xdtype(calib_x), T, C, _hp(g), None if b is None else _hp(b), ln_eps,
                                  _hp(a), _hp(w), w.shape[0], a_bits, w_bits, P, ctypes.addressof(theta),
                                  _hp(losses), _stream(stream)))
    return float(theta.value), losses


def qllm_fold_previous(map_ptr, map_src, map_coef, W_prev, bias_prev=None):
    """Appendix B: the map applied to the preceding linear layer's output channels (host).  Returns (W_out, bias_out)."""
    p = np.ascontiguousarray(map_ptr, np.int32); s = np.ascontiguousarray(map_src, np.int32)
    c = np.ascontiguousarray(map_coef, np.float32); w = np.ascontiguousarray(W_prev, np.float32)
    C, C_in = p.shape[0] - 1, w.shape[1]
    b = None if bias_prev is None else np.ascontiguousarray(bias_prev, np.float32)
    out = np.empty((C, C_in), np.float32)
    bout = None if b is None else np.empty(C, np.float32)
    _check(_lib.qllm_fold_previous(_hp(p), _hp(s), _hp(c), C, _hp(w), None if b is None else _hp(b), C_in, _hp(out),
                                   None if bout is None else _hp(bout)))
    return out, bout


def qllm_validate_map(map_ptr, map_src, C):
    p = np.ascontiguousarray(map_ptr, np.int32)
    s = np.ascontiguousarray(map_src, np.int32)
    return _lib.qllm_validate_map(_hp(p), _hp(s), C, s.shape[0])


class Reassembly:
    """Owner of a qllm_reassembly_t handle (host data: map + transformed quantized weights)."""

    def __init__(self, handle, C, N):
        self._h = handle
        self.C, self.N = C, N

    def __del__(self):
        self.free()

    def free(self):
        if getattr(self, "_h", None) and _lib is not None:   # at interpreter exit the module may be gone first
            _lib.qllm_free_reassembly(self._h)
            self._h = None

    @property
    def handle(self):
        return self._h

    def stats(self):
        st = (_i64 * 6)()
        _check(_lib.qllm_reassembly_stats(self._h, st))
        return dict(E=st[0], merged_rows=st[1], rounds=st[2], C=st[3], N=st[4], w_bits=st[5])

    def map(self):
        """Copies of (ptr i32[C+1], src i32[nnz], coef f32[nnz])."""
        p, s, c, n = _vp(), _vp(), _vp(), _i64()
        _check(_lib.qllm_reassembly_map(self._h, ctypes.byref(p), ctypes.byref(s), ctypes.byref(c), ctypes.byref(n)))
        nnz = n.value
        ptr = np.ctypeslib.as_array(ctypes.cast(p, ctypes.POINTER(ctypes.c_int32)), (self.C + 1,)).copy()
        src = np.ctypeslib.as_array(ctypes.cast(s, ctypes.POINTER(ctypes.c_int32)), (nnz,)).copy()
        coef = np.ctypeslib.as_array(ctypes.cast(c, ctypes.POINTER(ctypes.c_float)), (nnz,)).copy()
        return ptr, src, coef

    def weights(self):
        """Copies of (w_codes u8[N][row_bytes], w_scale f32[N], w_zero f32[N], w_colsum i32[N])."""
        wc, nb, ws, wz, cs = _vp(), _i64(), _vp(), _vp(), _vp()
        _check(_lib.qllm_reassembly_weights(self._h, ctypes.byref(wc), ctypes.byref(nb), ctypes.byref(ws),
                                            ctypes.byref(wz), ctypes.byref(cs)))
        N = self.N
        codes = np.ctypeslib.as_array(ctypes.cast(wc, ctypes.POINTER(ctypes.c_uint8)), (nb.value,)).copy()
        codes = codes.reshape(N, nb.value // N)
        scale = np.ctypeslib.as_array(ctypes.cast(ws, ctypes.POINTER(ctypes.c_float)), (N,)).copy()
        zero = np.ctypeslib.as_array(ctypes.cast(wz, ctypes.POINTER(ctypes.c_float)), (N,)).copy()
        colsum = np.ctypeslib.as_array(ctypes.cast(cs, ctypes.POINTER(ctypes.c_int32)), (N,)).copy()
        return codes, scale, zero, colsum


def qllm_layernorm_rows(x, ln_gamma, ln_beta, y, ln_eps=1e-5, stream=None):
    """x, ln_gamma, ln_beta (or None), y (float32 [T][C]): device tensors."""
    T, C = x.shape
    _check(_lib.qllm_layernorm_rows(_dp(x), _xdtype(x), T, C, _dp(ln_gamma), _dp(ln_beta), ln_eps, _dp(y), _stream(stream)))


def qllm_channel_distance(y, W, D, stream=None):
    """y float32 [T][C], W float32 [N][C], D float32 [C][C]: device tensors (Eq. 5 table)."""
    T, C = y.shape
    _check(_lib.qllm_channel_distance(_dp(y), T, _dp(W), W.shape[0], C, _dp(D), _stream(stream)))


def qllm_build_reassembly(calib_absmax, theta, W, lr_A=None, lr_B=None, w_bits=4, dist=None, calib_y=None, stream=None):
    """dist: optional host float32 [C][C] distance table (qllm_build_reassembly_dist).  calib_y: optional DEVICE
    float32 tensor [T][C], the layer's input of the calibration tokens: the matching then uses the Eq. 5 distance,
    evaluated on the device (qllm_build_reassembly_eq5)."""
    a = np.ascontiguousarray(calib_absmax, np.float32)
    W = np.ascontiguousarray(W, np.float32)
    N, C = W.shape
    assert a.shape == (C,)
    r = 0
    if lr_A is not None:
        lr_A = np.ascontiguousarray(lr_A, np.float32)
        lr_B = np.ascontiguousarray(lr_B, np.float32)
        r = lr_A.shape[1]
        assert lr_A.shape == (C, r) and lr_B.shape == (r, N)
    h = _vp()
    if calib_y is not None:
        assert dist is None and tuple(calib_y.shape[1:]) == (C,)
        _check(_lib.qllm_build_reassembly_eq5(_hp(a), C, theta, _dp(calib_y), calib_y.shape[0], _hp(W), N, _hp(lr_A),
                                              _hp(lr_B), r, w_bits, _stream(stream), ctypes.byref(h)))
    elif dist is None:
        _check(_lib.qllm_build_reassembly(_hp(a), C, theta, _hp(W), N, _hp(lr_A), _hp(lr_B), r, w_bits, ctypes.byref(h)))
    else:
        d = np.ascontiguousarray(dist, np.float32)
        assert d.shape == (C, C)
        _check(_lib.qllm_build_reassembly_dist(_hp(a), C, theta, _hp(d), _hp(W), N, _hp(lr_A), _hp(lr_B), r, w_bits,
                                               ctypes.byref(h)))
    return Reassembly(h, C, N)


class Layer:
    """Owner of a qllm_layer_t: device-resident map, weights and workspace."""

    def __init__(self, reassembly: Reassembly, ln_gamma, ln_beta, ln_eps, bias, a_bits, x_dtype, out_dtype, max_M):
        g = np.ascontiguousarray(ln_gamma, np.float32)
        b = None if ln_beta is None else np.ascontiguousarray(ln_beta, np.float32)
        bi = None if bias is None else np.ascontiguousarray(bias, np.float32)
        h = _vp()
        _check(_lib.qllm_layer_create(reassembly.handle, _hp(g), _hp(b), ln_eps, _hp(bi), a_bits,
                                      x_dtype, out_dtype, max_M, ctypes.byref(h)))
        self._h = h
        self.C, self.N, self.a_bits, self.max_M = reassembly.C, reassembly.N, a_bits, max_M
        self.x_dtype, self.out_dtype = x_dtype, out_dtype

    def __del__(self):
        self.destroy()

    def destroy(self):
        if getattr(self, "_h", None) and _lib is not None:   # at interpreter exit the module may be gone first
            _lib.qllm_layer_destroy(self._h)
            self._h = None

    def forward(self, x, out, stream=None):
        _check(_lib.qllm_layer_forward(self._h, _dp(x), x.shape[0], _dp(out), _stream(stream)))

    def reassemble_quant(self, x, stream=None):
        _check(_lib.qllm_layer_reassemble_quant(self._h, _dp(x), x.shape[0], _stream(stream)))

    def qgemm(self, M, out, stream=None):
        _check(_lib.qllm_layer_qgemm(self._h, M, _dp(out), _stream(stream)))

    def keep_byte_weights(self, keep=True, stream=None):
        _check(_lib.qllm_layer_keep_byte_weights(self._h, 1 if keep else 0, _stream(stream)))

    def forward_host(self, x_host, out_host, M, stream=None):
        """x_host/out_host: host pointers (ints) or numpy arrays / pinned CPU torch tensors."""
        def hptr(a):
            if isinstance(a, int):
                return a
            if isinstance(a, np.ndarray):
                return a.ctypes.data
            return a.data_ptr()
        _check(_lib.qllm_layer_forward_host(self._h, hptr(x_host), M, hptr(out_host), _stream(stream)))

    def workspace_ptrs(self):
        """(codes, a_scale, a_zero, a_rowsum, lane_bits): device addresses and the code lane width (4 or 8)."""
        c, s, z, r, lanes = _vp(), _vp(), _vp(), _vp(), ctypes.c_int(0)
        _check(_lib.qllm_layer_workspace(self._h, ctypes.byref(c), ctypes.byref(s), ctypes.byref(z), ctypes.byref(r),
                                         ctypes.byref(lanes)))
        return c.value, s.value, z.value, r.value, lanes.value
