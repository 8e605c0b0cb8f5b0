"""CPU oracle of the QLLM quantized linear layer -- TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy wrappers around ``qllm_oracle.cpp`` (plain single-threaded C++,
fp64 internals), which states what the hot path computes from the paper's
definitions: LayerNorm, reassembly-map apply (Eq. 3 / Eq. 4), the Eq. 2 quantizer,
the integer matmul of Eq. 1 on codes, the dequantizing epilogue, and the offline
map builder (Sec. 4.1.1-4.1.2, Appendix A/B).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares nothing with the CUDA library and imports nothing from it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qllm_oracle.cpp")
_LIB = os.path.join(_HERE, "libqllm_oracle.so")
_LIB_OMP = os.path.join(_HERE, "libqllm_oracle_omp.so")
_lib = None
_parallel = False


def build(force: bool = False, parallel: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no fast-math).  The default build is single-threaded: the OpenMP pragmas
    on the loops over token rows are ignored.  parallel=True makes a second library with -fopenmp, in which
    those loops (and nothing else) run on all cores; it exists for the benchmark's all-cores baseline."""
    target = _LIB_OMP if parallel else _LIB
    if force or not os.path.exists(target) or os.path.getmtime(target) < os.path.getmtime(_SRC):
        tmp = target + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC"] + (["-fopenmp"] if parallel else []) +
                              ["-o", tmp, _SRC])
        os.replace(tmp, target)
    return target


def set_parallel(flag: bool) -> None:
    """Switch the wrappers between the single-threaded library (default) and the OpenMP one."""
    global _lib, _parallel
    if flag != _parallel:
        _parallel = flag
        _lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build(parallel=_parallel))
        _lib.orc_theta_percentile.restype = ctypes.c_float
        _lib.orc_theta_for_extra.restype = ctypes.c_float
        _lib.orc_extra_channels.restype = ctypes.c_int64
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def layernorm(x, gamma, beta=None, eps=1e-5):
    """x: float32 [M][C] or uint16 (bfloat16 bit patterns) [M][C] -> float64 [M][C]."""
    x = np.ascontiguousarray(x)
    assert x.dtype in (np.float32, np.uint16)
    M, C = x.shape
    y = np.empty((M, C), np.float64)
    g = _c(gamma, np.float32)
    b = None if beta is None else _c(beta, np.float32)
    lib().orc_layernorm(_p(x), ctypes.c_int(0 if x.dtype == np.float32 else 1), ctypes.c_int64(M),
                        ctypes.c_int(C), _p(g), _p(b), ctypes.c_double(eps), _p(y))
    return y


def channel_absmax(y):
    y = _c(y, np.float64)
    M, C = y.shape
    out = np.empty(C, np.float32)
    lib().orc_channel_absmax(_p(y), ctypes.c_int64(M), ctypes.c_int(C), _p(out))
    return out


def map_apply(y, ptr, src, coef):
    y = _c(y, np.float64)
    M, C_in = y.shape
    ptr = _c(ptr, np.int32); src = _c(src, np.int32); coef = _c(coef, np.float32)
    C_out = ptr.shape[0] - 1
    out = np.empty((M, C_out), np.float64)
    lib().orc_map_apply(_p(y), ctypes.c_int64(M), ctypes.c_int(C_in), ctypes.c_int(C_out),
                        _p(ptr), _p(src), _p(coef), _p(out))
    return out


def quant_rows(v, bits, want_pre=False):
    """Eq. 2 per row.  Returns dict(codes u8 [R][C], scale f32, zero f32, sum i32[, pre, zpre])."""
    v = _c(v, np.float64)
    R, C = v.shape
    codes = np.empty((R, C), np.uint8)
    scale = np.empty(R, np.float32); zero = np.empty(R, np.float32)
    csum = np.empty(R, np.int32)
    pre = np.empty((R, C), np.float64) if want_pre else None
    zpre = np.empty(R, np.float64) if want_pre else None
    lib().orc_quant_rows(_p(v), ctypes.c_int64(R), ctypes.c_int(C), ctypes.c_int(bits), _p(codes),
                         _p(scale), _p(zero), _p(csum), _p(pre), _p(zpre))
    out = dict(codes=codes, scale=scale, zero=zero, sum=csum)
    if want_pre:
        out.update(pre=pre, zpre=zpre)
    return out


def pack4(codes):
    codes = _c(codes, np.uint8)
    R, C = codes.shape
    assert C % 2 == 0
    out = np.empty((R, C // 2), np.uint8)
    lib().orc_pack4(_p(codes), ctypes.c_int64(R), ctypes.c_int(C), _p(out))
    return out


def weight_transform(W, ptr, src, lrA=None, lrB=None):
    """W f32 [N][C_in] -> fp64 [N][C_out] (rows of the map summed; + (A B)^T)."""
    W = _c(W, np.float32)
    N, C_in = W.shape
    ptr = _c(ptr, np.int32); src = _c(src, np.int32)
    C_out = ptr.shape[0] - 1
    r = 0
    if lrA is not None:
        lrA = _c(lrA, np.float32); lrB = _c(lrB, np.float32)
        r = lrA.shape[1]
        assert lrA.shape == (C_out, r) and lrB.shape == (r, N)
    out = np.empty((N, C_out), np.float64)
    lib().orc_weight_transform(_p(W), ctypes.c_int(N), ctypes.c_int(C_in), ctypes.c_int(C_out),
                               _p(ptr), _p(src), _p(lrA), _p(lrB), ctypes.c_int(r), _p(out))
    return out


def int_matmul(qa, qw):
    qa = _c(qa, np.uint8); qw = _c(qw, np.uint8)
    M, K = qa.shape
    N, K2 = qw.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    rc = lib().orc_int_matmul(_p(qa), _p(qw), ctypes.c_int64(M), ctypes.c_int(N), ctypes.c_int(K), _p(acc))
    assert rc == 0, "int32 overflow in the oracle matmul"
    return acc


def int_matmul_at(qa, qw, ms, ns):
    """acc[i] = sum_k qa[ms[i]][k] * qw[ns[i]][k] for a list of (m, n) pairs."""
    qa = _c(qa, np.uint8); qw = _c(qw, np.uint8)
    ms = _c(ms, np.int64); ns = _c(ns, np.int32)
    K = qw.shape[1]
    assert qa.shape[1] == K
    acc = np.empty(ms.shape[0], np.int32)
    rc = lib().orc_int_matmul_at(_p(qa), _p(qw), ctypes.c_int(K), _p(ms), _p(ns),
                                 ctypes.c_int64(ms.shape[0]), _p(acc))
    assert rc == 0
    return acc


def epilogue(acc, K, a_scale, a_zero, a_rowsum, w_scale, w_zero, w_colsum, bias=None):
    acc = _c(acc, np.int32)
    M, N = acc.shape
    out = np.empty((M, N), np.float64)
    b = None if bias is None else _c(bias, np.float32)
    lib().orc_epilogue(_p(acc), ctypes.c_int64(M), ctypes.c_int(N), ctypes.c_int(K),
                       _p(_c(a_scale, np.float32)), _p(_c(a_zero, np.float32)), _p(_c(a_rowsum, np.int32)),
                       _p(_c(w_scale, np.float32)), _p(_c(w_zero, np.float32)), _p(_c(w_colsum, np.int32)),
                       _p(b), _p(out))
    return out


def cast_f32(v):
    v = _c(v, np.float64)
    out = np.empty(v.shape, np.float32)
    lib().orc_cast_f32(_p(v), ctypes.c_int64(v.size), _p(out))
    return out


def cast_bf16(v):
    """fp64 -> bfloat16 bit patterns (uint16), round to nearest even."""
    v = _c(v, np.float64)
    out = np.empty(v.shape, np.uint16)
    lib().orc_cast_bf16(_p(v), ctypes.c_int64(v.size), _p(out))
    return out


def dense_linear(X, W):
    X = _c(X, np.float64); W = _c(W, np.float64)
    M, C = X.shape
    N = W.shape[0]
    out = np.empty((M, N), np.float64)
    lib().orc_dense_linear(_p(X), _p(W), ctypes.c_int64(M), ctypes.c_int(N), ctypes.c_int(C), _p(out))
    return out


def extra_channels(absmax, theta):
    a = _c(absmax, np.float32)
    return int(lib().orc_extra_channels(_p(a), ctypes.c_int(a.shape[0]), ctypes.c_float(theta)))


def theta_percentile(absmax, pct):
    a = _c(absmax, np.float32)
    return float(lib().orc_theta_percentile(_p(a), ctypes.c_int(a.shape[0]), ctypes.c_double(pct)))


def theta_for_extra(absmax, extra):
    a = _c(absmax, np.float32)
    return float(lib().orc_theta_for_extra(_p(a), ctypes.c_int(a.shape[0]), ctypes.c_int(extra)))


class Infeasible(Exception):
    pass


class NeedsMoreRounds(Exception):
    """Eq. 5 distances are defined between undivided channels: one matching round only."""


def channel_distance(y, W):
    """Eq. 5 table D[i][j] = 1/4 ||y_i - y_j||^2 ||W_i - W_j||^2 in fp64.  y [T][C] (fp64), W [N][C] (fp32)."""
    y = _c(y, np.float64); W = _c(W, np.float32)
    T, C = y.shape
    N = W.shape[0]
    assert W.shape[1] == C
    D = np.empty((C, C), np.float64)
    lib().orc_channel_distance(_p(y), ctypes.c_int64(T), _p(W), ctypes.c_int(N), ctypes.c_int(C), _p(D))
    return D


def build_map(absmax, theta, dist=None):
    """Returns (ptr i32[C+1], src i32[nnz], coef f32[nnz], stats dict).  dist: optional Eq. 5 table [C][C]."""
    a = _c(absmax, np.float32)
    C = a.shape[0]
    E = extra_channels(a, theta)
    cap = C + E
    ptr = np.empty(C + 1, np.int32); src = np.empty(cap, np.int32); coef = np.empty(cap, np.float32)
    stats = np.zeros(3, np.int64)
    if dist is None:
        rc = lib().orc_build_map(_p(a), ctypes.c_int(C), ctypes.c_float(theta), _p(ptr), _p(src), _p(coef),
                                 ctypes.c_int64(cap), _p(stats))
    else:
        d = _c(dist, np.float64)
        assert d.shape == (C, C)
        rc = lib().orc_build_map_dist(_p(a), ctypes.c_int(C), ctypes.c_float(theta), _p(d), _p(ptr), _p(src), _p(coef),
                                      ctypes.c_int64(cap), _p(stats))
    if rc == -1:
        raise Infeasible()
    if rc == -4:
        raise NeedsMoreRounds()
    assert rc == 0, rc
    nnz = int(ptr[C])
    return ptr, src[:nnz].copy(), coef[:nnz].copy(), dict(E=int(stats[0]), merged_rows=int(stats[1]),
                                                          rounds=int(stats[2]))


# ---------------------------------------------------------------------------
# Whole-path conveniences (compositions of the steps above, nothing new).
# ---------------------------------------------------------------------------
def prepare_weights(W, ptr, src, w_bits, lrA=None, lrB=None):
    Wr = weight_transform(W, ptr, src, lrA, lrB)
    q = quant_rows(Wr, w_bits)
    return dict(Wr=Wr, codes=q["codes"], scale=q["scale"], zero=q["zero"], colsum=q["sum"])


def reassemble_quant(x, gamma, beta, eps, ptr, src, coef, bits, want_pre=False):
    y = layernorm(x, gamma, beta, eps)
    xr = map_apply(y, ptr, src, coef)
    q = quant_rows(xr, bits, want_pre=want_pre)
    q["xr"] = xr
    return q


# ---------------------------------------------------------------------------
# Adaptive threshold search (Algorithm 1), a composition of the steps above.
# Reading: the reassembly error of Eq. 6 is taken on the layer's own output (the
# calibration tokens through the full-precision layer against the same tokens
# through the reassembled, quantized layer), not on an attention block's output.
# ---------------------------------------------------------------------------
def theta_grid(absmax, P):
    """Algorithm 1: theta_p = min(m) + p / P * (max(m) - min(m)), p = 1..P (float32 values)."""
    m = _c(absmax, np.float32).astype(np.float64)
    lo, hi = float(m.min()), float(m.max())
    return np.array([np.float32(lo + (p / P) * (hi - lo)) for p in range(1, P + 1)], np.float32)


def reassembly_loss(xcal, gamma, beta, eps, W, absmax, theta, a_bits, w_bits):
    """|| Y - Y~ ||_F^2 with Y = LN(x) W^T and Y~ = quant(X^) quant(W^) for the map built at theta
    (Eq. 6 on the layer's output); inf when the channel count cannot be restored."""
    y = layernorm(xcal, gamma, beta, eps)
    Y = dense_linear(y, _c(W, np.float32).astype(np.float64))
    try:
        ptr, src, coef, _ = build_map(absmax, theta)
    except Infeasible:
        return float("inf")
    w = prepare_weights(W, ptr, src, w_bits)
    q = reassemble_quant(xcal, gamma, beta, eps, ptr, src, coef, a_bits)
    acc = int_matmul(q["codes"], w["codes"])
    Yq = epilogue(acc, W.shape[1], q["scale"], q["zero"], q["sum"], w["scale"], w["zero"], w["colsum"])
    return float(((Y - Yq) ** 2).sum())


def search_theta(xcal, gamma, beta, eps, W, absmax, a_bits, w_bits, P):
    """Algorithm 1: returns (theta*, losses[P]); theta* is the first grid point with the smallest loss."""
    grid = theta_grid(absmax, P)
    losses = np.array([reassembly_loss(xcal, gamma, beta, eps, W, absmax, float(t), a_bits, w_bits) for t in grid])
    best = int(np.argmin(losses))          # first occurrence: Algorithm 1 updates only on a strictly smaller loss
    return float(grid[best]), losses


# ---------------------------------------------------------------------------
# Appendix B: the map folded into a preceding linear layer (plain numpy, fp64).
# ---------------------------------------------------------------------------
def fold_previous(W_prev, bias_prev, ptr, src, coef):
    """Row c of the result = sum_j coef_j * row src_j of W_prev [C_src][C_in] (and of its bias): the
    preceding layer's output channels duplicated with 1/T (disassembly) and averaged (assembly).
    Returns (W_out float32 [C][C_in], bias_out float32 [C] or None), sums taken in fp64 in entry order."""
    W = np.asarray(W_prev, np.float32).astype(np.float64)
    b = None if bias_prev is None else np.asarray(bias_prev, np.float32).astype(np.float64)
    C = len(ptr) - 1
    out = np.zeros((C, W.shape[1]), np.float64)
    bout = None if b is None else np.zeros(C, np.float64)
    for c in range(C):
        for j in range(int(ptr[c]), int(ptr[c + 1])):
            cf = float(np.float32(coef[j]))
            out[c] += cf * W[int(src[j])]
            if b is not None:
                bout[c] += cf * b[int(src[j])]
    return out.astype(np.float32), None if bout is None else bout.astype(np.float32)
