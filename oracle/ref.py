"""ctypes loader for libmtmcref, the fp64 CPU oracle (TEST INFRASTRUCTURE ONLY).

Only tests, the smoke check and the benchmark's CPU legs may import this module.
It never imports the CUDA package and shares nothing with it.  Arrays are numpy:
bf16 operands travel as uint16 bit patterns, bias as float32, results as float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mtmc_ref.cpp")
_LIB = os.path.join(_HERE, "libmtmcref.so")

ACT_NONE, ACT_RELU, ACT_GELU_TANH, ACT_SILU = 0, 1, 2, 3

_lib = None


def build(force: bool = False) -> str:
    """Compile oracle/mtmc_ref.cpp -> oracle/libmtmcref.so with g++ (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, vp, dbl, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_double, ctypes.c_int
        L.mtmc_ref_set_threads.argtypes = [ci]
        L.mtmc_ref_get_threads.restype = ci
        L.mtmc_ref_act.argtypes = [ci, dbl]
        L.mtmc_ref_act.restype = dbl
        L.mtmc_ref_fused_linear.argtypes = [vp, vp, vp, i64, i64, i64, ci, vp]
        L.mtmc_ref_fused_linear_residual.argtypes = [vp, vp, vp, vp, ci, i64, i64, i64, ci, vp]
        L.mtmc_ref_e4m3.argtypes = [ctypes.c_uint8]
        L.mtmc_ref_e4m3.restype = dbl
        L.mtmc_ref_fused_linear_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, ci, vp]
        L.mtmc_ref_fused_linear_fp8_points.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, ci, vp, vp, i64, vp]
        L.mtmc_ref_swiglu_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, ctypes.c_float, i64, i64, i64, vp]
        L.mtmc_ref_linear_lse_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, vp, vp]
        L.mtmc_ref_linear_rowmax_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, vp, vp]
        L.mtmc_ref_linear_cross_entropy_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, i64, i64, i64, vp, vp]
        L.mtmc_ref_e8m0.argtypes = [ctypes.c_uint8]
        L.mtmc_ref_e8m0.restype = dbl
        L.mtmc_ref_fused_linear_mxfp8.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, ci, vp]
        L.mtmc_ref_swiglu_mxfp8.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
        L.mtmc_ref_linear_lse_mxfp8.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp]
        L.mtmc_ref_fused_linear_points.argtypes = [vp, vp, vp, i64, i64, i64, ci, vp, vp, i64, vp]
        L.mtmc_ref_swiglu.argtypes = [vp, vp, vp, i64, i64, i64, vp]
        L.mtmc_ref_swiglu_points.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp, i64, vp]
        L.mtmc_ref_linear_lse.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp]
        L.mtmc_ref_linear_lse_rows.argtypes = [vp, vp, vp, i64, i64, i64, vp, i64, vp]
        L.mtmc_ref_linear_rowmax.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp]
        L.mtmc_ref_linear_cross_entropy.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, vp]
        L.mtmc_ref_linear_softmax.argtypes = [vp, vp, vp, i64, i64, i64, vp]
        L.mtmc_ref_linear_softmax_rows.argtypes = [vp, vp, vp, i64, i64, i64, vp, i64, vp]
        L.mtmc_ref_softmax_vector.argtypes = [vp, i64, vp]
        L.mtmc_ref_linear_softmax_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, vp]
        L.mtmc_ref_softmax_vector.restype = None
        L.mtmc_ref_lse_vector.argtypes = [vp, i64]
        L.mtmc_ref_lse_vector.restype = dbl
        L.mtmc_ref_compare.argtypes = [vp, vp, i64, dbl, dbl, vp]
        L.mtmc_ref_compare.restype = i64
        _lib = L
    return _lib


def _bf16(a, shape) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16 or tuple(a.shape) != tuple(shape):
        raise TypeError("bf16 operand must be a uint16 bit-pattern array of shape %r" % (shape,))
    return a


def _bias(b, N):
    if b is None:
        return None, None
    b = np.ascontiguousarray(b)
    if b.dtype != np.float32 or b.shape != (N,):
        raise TypeError("bias must be float32 [N]")
    return b, b.ctypes.data


def _idx(v) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(v, dtype=np.int64))


def _check(rc: int, name: str) -> None:
    if rc != 0:
        raise ValueError("%s rejected its arguments (status %d)" % (name, rc))


def set_threads(n: int) -> None:
    lib().mtmc_ref_set_threads(int(n))


def get_threads() -> int:
    return int(lib().mtmc_ref_get_threads())


def act(kind: int, z: float) -> float:
    return float(lib().mtmc_ref_act(int(kind), float(z)))


def fused_linear(X, W, b, act_kind: int) -> np.ndarray:
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_fused_linear(X.ctypes.data, W.ctypes.data, bp, M, N, K, int(act_kind), out.ctypes.data),
           "mtmc_ref_fused_linear")
    return out


def fused_linear_residual(X, W, b, R, act_kind: int) -> np.ndarray:
    """act(X.W^T + b) + R; R is [M,N] uint16 (bf16 bit patterns) or float32."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    R = np.ascontiguousarray(R)
    if R.shape != (M, N) or R.dtype not in (np.uint16, np.float32):
        raise TypeError("R must be [M,N] uint16 (bf16 bits) or float32")
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_fused_linear_residual(X.ctypes.data, W.ctypes.data, bp, R.ctypes.data, int(R.dtype == np.uint16),
                                                M, N, K, int(act_kind), out.ctypes.data), "mtmc_ref_fused_linear_residual")
    return out


def e4m3(bits: int) -> float:
    return float(lib().mtmc_ref_e4m3(int(bits) & 0xFF))


def _fp8(a, shape) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint8 or tuple(a.shape) != tuple(shape):
        raise TypeError("fp8 operand must be a uint8 bit-pattern array of shape %r" % (shape,))
    return a


def fused_linear_fp8(X, W, b, scale_x: float, scale_w: float, act_kind: int) -> np.ndarray:
    """act(scale_x*scale_w * Xq.Wq^T + b) with E4M3 bit patterns (uint8) for Xq [M,K] and Wq [N,K]."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    bk, bp = _bias(b, N)
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_fused_linear_fp8(X.ctypes.data, W.ctypes.data, bp, float(scale_x), float(scale_w), M, N, K,
                                           int(act_kind), out.ctypes.data), "mtmc_ref_fused_linear_fp8")
    return out


def e8m0(byte: int) -> float:
    """UE8M0 scale byte -> its value, 2^(byte - 127) (255: NaN)."""
    return float(lib().mtmc_ref_e8m0(int(byte) & 0xFF))


def _scales(a, shape) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint8 or tuple(a.shape) != tuple(shape):
        raise TypeError("block scales must be a uint8 array of shape %r" % (shape,))
    return a


def fused_linear_mxfp8(X, SX, W, SW, b, act_kind: int) -> np.ndarray:
    """act(z + b) with block-scaled E4M3 operands: X [M,K], W [N,K] bit patterns, SX [M,K/32], SW [N,K/32] UE8M0 bytes."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    SX, SW = _scales(SX, (M, K // 32)), _scales(SW, (N, K // 32))
    bk, bp = _bias(b, N)
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_fused_linear_mxfp8(X.ctypes.data, SX.ctypes.data, W.ctypes.data, SW.ctypes.data, bp, M, N, K,
                                             int(act_kind), out.ctypes.data), "mtmc_ref_fused_linear_mxfp8")
    return out


def swiglu_mxfp8(X, SX, Wg, SG, Wu, SU) -> np.ndarray:
    M, K = X.shape
    N = Wg.shape[0]
    X, Wg, Wu = _fp8(X, (M, K)), _fp8(Wg, (N, K)), _fp8(Wu, (N, K))
    SX, SG, SU = _scales(SX, (M, K // 32)), _scales(SG, (N, K // 32)), _scales(SU, (N, K // 32))
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_swiglu_mxfp8(X.ctypes.data, SX.ctypes.data, Wg.ctypes.data, SG.ctypes.data, Wu.ctypes.data, SU.ctypes.data,
                                       M, N, K, out.ctypes.data), "mtmc_ref_swiglu_mxfp8")
    return out


def linear_lse_mxfp8(X, SX, W, SW, b) -> np.ndarray:
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    SX, SW = _scales(SX, (M, K // 32)), _scales(SW, (N, K // 32))
    bk, bp = _bias(b, N)
    lse = np.empty(M, dtype=np.float64)
    _check(lib().mtmc_ref_linear_lse_mxfp8(X.ctypes.data, SX.ctypes.data, W.ctypes.data, SW.ctypes.data, bp, M, N, K, lse.ctypes.data),
           "mtmc_ref_linear_lse_mxfp8")
    return lse


def fused_linear_fp8_points(X, W, b, scale_x: float, scale_w: float, act_kind: int, rows, cols) -> np.ndarray:
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    bk, bp = _bias(b, N)
    rows, cols = _idx(rows), _idx(cols)
    out = np.empty(rows.shape[0], dtype=np.float64)
    _check(lib().mtmc_ref_fused_linear_fp8_points(X.ctypes.data, W.ctypes.data, bp, float(scale_x), float(scale_w), M, N, K,
                                                  int(act_kind), rows.ctypes.data, cols.ctypes.data, rows.shape[0],
                                                  out.ctypes.data), "mtmc_ref_fused_linear_fp8_points")
    return out


def swiglu_fp8(X, Wg, Wu, scale_x: float, scale_g: float, scale_u: float) -> np.ndarray:
    """silu(scale_x*scale_g * Xq.Wgq^T) * (scale_x*scale_u * Xq.Wuq^T) with E4M3 bit patterns (uint8)."""
    M, K = X.shape
    N = Wg.shape[0]
    X, Wg, Wu = _fp8(X, (M, K)), _fp8(Wg, (N, K)), _fp8(Wu, (N, K))
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_swiglu_fp8(X.ctypes.data, Wg.ctypes.data, Wu.ctypes.data, float(scale_x), float(scale_g),
                                     float(scale_u), M, N, K, out.ctypes.data), "mtmc_ref_swiglu_fp8")
    return out


def linear_lse_fp8(X, W, b, scale_x: float, scale_w: float, want_logits: bool = False):
    """Row logsumexp of scale_x*scale_w * Xq.Wq^T + b with E4M3 bit patterns (uint8)."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    bk, bp = _bias(b, N)
    lse = np.empty(M, dtype=np.float64)
    logits = np.empty((M, N), dtype=np.float64) if want_logits else None
    _check(lib().mtmc_ref_linear_lse_fp8(X.ctypes.data, W.ctypes.data, bp, float(scale_x), float(scale_w), M, N, K,
                                         lse.ctypes.data, logits.ctypes.data if want_logits else None),
           "mtmc_ref_linear_lse_fp8")
    return (lse, logits) if want_logits else lse


def fused_linear_points(X, W, b, act_kind: int, rows, cols) -> np.ndarray:
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    rows, cols = _idx(rows), _idx(cols)
    out = np.empty(rows.shape[0], dtype=np.float64)
    _check(lib().mtmc_ref_fused_linear_points(X.ctypes.data, W.ctypes.data, bp, M, N, K, int(act_kind),
                                              rows.ctypes.data, cols.ctypes.data, rows.shape[0], out.ctypes.data),
           "mtmc_ref_fused_linear_points")
    return out


def swiglu(X, Wg, Wu) -> np.ndarray:
    M, K = X.shape
    N = Wg.shape[0]
    X, Wg, Wu = _bf16(X, (M, K)), _bf16(Wg, (N, K)), _bf16(Wu, (N, K))
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_swiglu(X.ctypes.data, Wg.ctypes.data, Wu.ctypes.data, M, N, K, out.ctypes.data),
           "mtmc_ref_swiglu")
    return out


def swiglu_points(X, Wg, Wu, rows, cols) -> np.ndarray:
    M, K = X.shape
    N = Wg.shape[0]
    X, Wg, Wu = _bf16(X, (M, K)), _bf16(Wg, (N, K)), _bf16(Wu, (N, K))
    rows, cols = _idx(rows), _idx(cols)
    out = np.empty(rows.shape[0], dtype=np.float64)
    _check(lib().mtmc_ref_swiglu_points(X.ctypes.data, Wg.ctypes.data, Wu.ctypes.data, M, N, K,
                                        rows.ctypes.data, cols.ctypes.data, rows.shape[0], out.ctypes.data),
           "mtmc_ref_swiglu_points")
    return out


def linear_lse(X, W, b, want_logits: bool = False):
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    lse = np.empty(M, dtype=np.float64)
    logits = np.empty((M, N), dtype=np.float64) if want_logits else None
    _check(lib().mtmc_ref_linear_lse(X.ctypes.data, W.ctypes.data, bp, M, N, K, lse.ctypes.data,
                                     logits.ctypes.data if want_logits else None), "mtmc_ref_linear_lse")
    return (lse, logits) if want_logits else lse


def linear_lse_rows(X, W, b, rows) -> np.ndarray:
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    rows = _idx(rows)
    lse = np.empty(rows.shape[0], dtype=np.float64)
    _check(lib().mtmc_ref_linear_lse_rows(X.ctypes.data, W.ctypes.data, bp, M, N, K,
                                          rows.ctypes.data, rows.shape[0], lse.ctypes.data),
           "mtmc_ref_linear_lse_rows")
    return lse


def linear_rowmax(X, W, b):
    """(max over n of X.W^T + b, lowest index attaining it) per row."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    mx = np.empty(M, dtype=np.float64)
    arg = np.empty(M, dtype=np.int64)
    _check(lib().mtmc_ref_linear_rowmax(X.ctypes.data, W.ctypes.data, bp, M, N, K, mx.ctypes.data, arg.ctypes.data),
           "mtmc_ref_linear_rowmax")
    return mx, arg


def linear_cross_entropy(X, W, b, target):
    """(loss, lse) per row: loss = lse - logit[target]."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    target = _idx(target)
    if target.shape != (M,):
        raise TypeError("target must be int64 [M]")
    loss = np.empty(M, dtype=np.float64)
    lse = np.empty(M, dtype=np.float64)
    _check(lib().mtmc_ref_linear_cross_entropy(X.ctypes.data, W.ctypes.data, bp, target.ctypes.data, M, N, K,
                                               loss.ctypes.data, lse.ctypes.data), "mtmc_ref_linear_cross_entropy")
    return loss, lse


def linear_rowmax_fp8(X, W, b, scale_x: float, scale_w: float):
    """(row maximum, lowest column attaining it) of scale_x*scale_w * Xq.Wq^T + b with E4M3 bit patterns (uint8)."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    bk, bp = _bias(b, N)
    mx = np.empty(M, dtype=np.float64)
    arg = np.empty(M, dtype=np.int64)
    _check(lib().mtmc_ref_linear_rowmax_fp8(X.ctypes.data, W.ctypes.data, bp, float(scale_x), float(scale_w), M, N, K,
                                            mx.ctypes.data, arg.ctypes.data), "mtmc_ref_linear_rowmax_fp8")
    return mx, arg


def linear_cross_entropy_fp8(X, W, b, scale_x: float, scale_w: float, target):
    """(loss, lse) per row of the E4M3 layer: loss = lse - logit[target]."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    bk, bp = _bias(b, N)
    target = _idx(target)
    if target.shape != (M,):
        raise TypeError("target must be int64 [M]")
    loss = np.empty(M, dtype=np.float64)
    lse = np.empty(M, dtype=np.float64)
    _check(lib().mtmc_ref_linear_cross_entropy_fp8(X.ctypes.data, W.ctypes.data, bp, float(scale_x), float(scale_w),
                                                   target.ctypes.data, M, N, K, loss.ctypes.data, lse.ctypes.data),
           "mtmc_ref_linear_cross_entropy_fp8")
    return loss, lse


def linear_softmax(X, W, b) -> np.ndarray:
    """softmax over n of X.W^T + b, [M,N] float64."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    P = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_linear_softmax(X.ctypes.data, W.ctypes.data, bp, M, N, K, P.ctypes.data), "mtmc_ref_linear_softmax")
    return P


def linear_softmax_rows(X, W, b, rows) -> np.ndarray:
    """The listed rows of linear_softmax, [len(rows), N] float64."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _bf16(X, (M, K)), _bf16(W, (N, K))
    bk, bp = _bias(b, N)
    rows = _idx(rows)
    P = np.empty((rows.shape[0], N), dtype=np.float64)
    _check(lib().mtmc_ref_linear_softmax_rows(X.ctypes.data, W.ctypes.data, bp, M, N, K,
                                              rows.ctypes.data, rows.shape[0], P.ctypes.data), "mtmc_ref_linear_softmax_rows")
    return P


def linear_softmax_fp8(X, W, b, scale_x: float, scale_w: float) -> np.ndarray:
    """softmax over n of scale_x*scale_w * Xq.Wq^T + b with E4M3 bit patterns (uint8), [M,N] float64."""
    M, K = X.shape
    N = W.shape[0]
    X, W = _fp8(X, (M, K)), _fp8(W, (N, K))
    bk, bp = _bias(b, N)
    P = np.empty((M, N), dtype=np.float64)
    _check(lib().mtmc_ref_linear_softmax_fp8(X.ctypes.data, W.ctypes.data, bp, float(scale_x), float(scale_w), M, N, K,
                                             P.ctypes.data), "mtmc_ref_linear_softmax_fp8")
    return P


def softmax_vector(z) -> np.ndarray:
    z = np.ascontiguousarray(np.asarray(z, dtype=np.float64))
    p = np.empty_like(z)
    lib().mtmc_ref_softmax_vector(z.ctypes.data, z.shape[0], p.ctypes.data)
    return p


def lse_vector(z) -> float:
    z = np.ascontiguousarray(np.asarray(z, dtype=np.float64))
    return float(lib().mtmc_ref_lse_vector(z.ctypes.data, z.shape[0]))


def compare(got, ref, atol: float, rtol: float) -> dict:
    """|got-ref| <= atol + rtol*|ref| element-wise; NaN/Inf on either side fails."""
    got = np.ascontiguousarray(np.asarray(got, dtype=np.float64)).ravel()
    ref = np.ascontiguousarray(np.asarray(ref, dtype=np.float64)).ravel()
    if got.shape != ref.shape:
        raise ValueError("shape mismatch: %r vs %r" % (got.shape, ref.shape))
    stats = np.zeros(4, dtype=np.float64)
    bad = lib().mtmc_ref_compare(got.ctypes.data, ref.ctypes.data, got.shape[0], float(atol), float(rtol),
                                 stats.ctypes.data)
    return {"violations": int(bad), "max_abs_err": float(stats[0]), "max_ratio": float(stats[1]),
            "worst_index": int(stats[2]), "count": int(got.shape[0]), "ok": bad == 0}
