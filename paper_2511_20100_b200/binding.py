"""Thin ctypes binding to libmtmcfused.so: argument marshalling only.

Same names as the C ABI (include/mtmc_fused.h).  torch supplies device memory and
the stream; every step of the computation runs inside the library's kernels.
There is no fallback: a missing library, a missing GPU or a non-Blackwell GPU is
an error.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MTMC_LIB_VARIANT=trace loads the build with device-side trace stamps (libmtmcfused_trace.so, see build.py)
VARIANT = os.environ.get("MTMC_LIB_VARIANT", "")
LIB_PATH = os.path.join(_HERE, "libmtmcfused%s.so" % ("_" + VARIANT if VARIANT else ""))

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_UNSUPPORTED_DEVICE, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_WORKSPACE, ERR_DEVICE_CHECK = 1, 2, 3, 4, 5, 6, 7
ACT = {"none": 0, "relu": 1, "gelu_tanh": 2, "silu": 3}
OUT_DTYPE = {"fp32": 0, "bf16": 1}
OP = {"fused_linear": 0, "swiglu": 1, "linear_lse": 2, "linear_rowmax": 3, "linear_cross_entropy": 4,
      "fused_linear_mxfp8": 5, "swiglu_mxfp8": 6, "linear_lse_mxfp8": 7, "linear_softmax": 8}

EXPORTS = [
    "mtmc_fused_linear", "mtmc_fused_linear_residual", "mtmc_fused_linear_fp8", "mtmc_swiglu", "mtmc_linear_lse",
    "mtmc_linear_lse_noalloc", "mtmc_linear_rowmax", "mtmc_linear_cross_entropy", "mtmc_linear_softmax",
    "mtmc_linear_softmax_strided", "mtmc_linear_softmax_fp8",
    "mtmc_fused_linear_host", "mtmc_swiglu_host", "mtmc_linear_lse_host",
    "mtmc_fused_linear_host_async", "mtmc_swiglu_host_async", "mtmc_linear_lse_host_async", "mtmc_host_sync",
    "mtmc_set_stream", "mtmc_set_workspace", "mtmc_workspace_bytes", "mtmc_check_status",
    "mtmc_last_error", "mtmc_launch_count", "mtmc_device_alloc_count", "mtmc_last_kernel_name", "mtmc_set_timing", "mtmc_last_kernel_ms",
    "mtmc_fused_linear_mxfp8", "mtmc_swiglu_mxfp8", "mtmc_linear_lse_mxfp8",
    "mtmc_fused_linear_strided", "mtmc_swiglu_strided", "mtmc_linear_lse_strided", "mtmc_linear_rowmax_strided",
    "mtmc_linear_cross_entropy_strided", "mtmc_swiglu_fp8", "mtmc_linear_lse_fp8", "mtmc_linear_rowmax_fp8", "mtmc_linear_cross_entropy_fp8", "mtmc_set_tuning", "mtmc_set_schedule", "mtmc_trace_enabled", "mtmc_set_trace", "mtmc_set_static_weights", "mtmc_version", "mtmc_selftest_timeout",
]

_lib = None


class MtmcError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("libmtmcfused status %d: %s" % (status, message))
        self.status = status


def load() -> ctypes.CDLL:
    """Loads the library (built in-tree by paper_2511_20100_b200.build); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    from . import build as _build
    if _build.needs_build(VARIANT):
        # missing or older than its sources: compile it in-tree (nvcc); there is no other code path to fall back on
        try:
            _build.build(variant=VARIANT)
        except Exception as e:
            raise RuntimeError("libmtmcfused.so is missing or stale at %s and could not be built (%s); "
                               "there is no fallback path" % (LIB_PATH, e))
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
    for name in ("mtmc_fused_linear", "mtmc_fused_linear_host", "mtmc_fused_linear_host_async"):
        getattr(L, name).argtypes = [vp, vp, vp, i64, i64, i64, ci, ci, vp]
    L.mtmc_fused_linear_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, ci, ci, vp]
    L.mtmc_fused_linear_residual.argtypes = [vp, vp, vp, vp, i64, i64, i64, ci, ci, vp]
    L.mtmc_fused_linear_strided.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, ci, ci, vp, i64]
    L.mtmc_fused_linear_mxfp8.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, ci, ci, vp]
    L.mtmc_swiglu_mxfp8.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
    L.mtmc_linear_lse_mxfp8.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp]
    L.mtmc_swiglu_strided.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i64, vp, i64]
    L.mtmc_linear_lse_strided.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, vp]
    L.mtmc_linear_rowmax_strided.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, vp, vp]
    L.mtmc_linear_cross_entropy_strided.argtypes = [vp, i64, vp, i64, vp, vp, i64, i64, i64, vp, vp]
    L.mtmc_swiglu_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, ctypes.c_float, i64, i64, i64, vp]
    L.mtmc_linear_lse_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, vp]
    L.mtmc_linear_rowmax_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, vp, vp]
    L.mtmc_linear_cross_entropy_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, i64, i64, i64, vp, vp]
    for name in ("mtmc_swiglu", "mtmc_swiglu_host", "mtmc_swiglu_host_async", "mtmc_linear_lse", "mtmc_linear_lse_host",
                 "mtmc_linear_lse_host_async", "mtmc_linear_lse_noalloc"):
        getattr(L, name).argtypes = [vp, vp, vp, i64, i64, i64, vp]
    L.mtmc_linear_rowmax.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp]
    L.mtmc_linear_cross_entropy.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp, vp]
    L.mtmc_linear_softmax.argtypes = [vp, vp, vp, i64, i64, i64, ci, vp, vp]
    L.mtmc_linear_softmax_strided.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, ci, vp, i64, vp]
    L.mtmc_linear_softmax_fp8.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, i64, i64, i64, ci, vp, vp]
    L.mtmc_set_stream.argtypes = [vp]
    L.mtmc_set_workspace.argtypes = [vp, sz]
    L.mtmc_workspace_bytes.argtypes = [ci, i64, i64, i64]
    L.mtmc_workspace_bytes.restype = sz
    L.mtmc_last_error.restype = ctypes.c_char_p
    L.mtmc_launch_count.restype = i64
    L.mtmc_device_alloc_count.restype = i64
    L.mtmc_last_kernel_name.restype = ctypes.c_char_p
    L.mtmc_set_timing.argtypes = [ci]
    L.mtmc_last_kernel_ms.restype = ctypes.c_float
    L.mtmc_set_tuning.argtypes = [ci, ci, ci]
    L.mtmc_set_static_weights.argtypes = [ci]
    L.mtmc_set_schedule.argtypes = [ci]
    L.mtmc_set_trace.argtypes = [vp, sz]
    _lib = L
    return L


def _check(rc: int) -> None:
    if rc != OK:
        raise MtmcError(rc, load().mtmc_last_error().decode())


def _dev(t: torch.Tensor, dtype, shape, name: str) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor" % name)
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise TypeError("%s must be contiguous %s of shape %r (got %s %r)" % (name, dtype, tuple(shape), t.dtype, tuple(t.shape)))
    return t.data_ptr()


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _use_current_stream(device) -> None:
    """Makes `device` current and hands torch's current stream on it to the library."""
    idx = device.index if device.index is not None else torch.cuda.current_device()
    if torch.cuda.current_device() != idx:
        torch.cuda.set_device(idx)
    handle = _raw_stream(idx) if _raw_stream is not None else torch.cuda.current_stream(idx).cuda_stream
    load().mtmc_set_stream(ctypes.c_void_p(handle))


def mtmc_fused_linear(X, W, b, act="none", out_dtype="bf16", out=None):
    """out = act(X @ W.T + b) on the current CUDA stream; X [M,K], W [N,K] bf16, b [N] fp32 or None."""
    M, K = X.shape
    N = W.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if out is None:
        out = torch.empty((M, N), dtype=odt, device=X.device)
    _use_current_stream(X.device)
    _check(load().mtmc_fused_linear(_dev(X, torch.bfloat16, (M, K), "X"), _dev(W, torch.bfloat16, (N, K), "W"),
                                    None if b is None else _dev(b, torch.float32, (N,), "b"),
                                    M, N, K, ACT[act], OUT_DTYPE[out_dtype], _dev(out, odt, (M, N), "out")))
    return out


def mtmc_fused_linear_residual(X, W, b, R, act="none", out_dtype="bf16", out=None):
    """out = act(X @ W.T + b) + R; R [M,N] in the output dtype; `out` may be R itself (in-place)."""
    M, K = X.shape
    N = W.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if out is None:
        out = torch.empty((M, N), dtype=odt, device=X.device)
    _use_current_stream(X.device)
    _check(load().mtmc_fused_linear_residual(_dev(X, torch.bfloat16, (M, K), "X"), _dev(W, torch.bfloat16, (N, K), "W"),
                                             None if b is None else _dev(b, torch.float32, (N,), "b"),
                                             _dev(R, odt, (M, N), "R"), M, N, K, ACT[act], OUT_DTYPE[out_dtype],
                                             _dev(out, odt, (M, N), "out")))
    return out


def _view2d(t: torch.Tensor, dtype, shape, name: str):
    """Device pointer and row pitch (elements) of a 2-D CUDA tensor whose rows are contiguous."""
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor" % name)
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or t.stride(1) != 1 or t.stride(0) < t.shape[1]:
        raise TypeError("%s must be %s of shape %r with unit column stride (got %s %r, strides %r)" % (
            name, dtype, tuple(shape), t.dtype, tuple(t.shape), tuple(t.stride())))
    return t.data_ptr(), t.stride(0)


def mtmc_fused_linear_strided(X, W, b, act="none", out_dtype="bf16", out=None):
    """mtmc_fused_linear on views: X [M,K], W [N,K] and out [M,N] may be column slices of wider row-major tensors."""
    M, K = X.shape
    N = W.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if out is None:
        out = torch.empty((M, N), dtype=odt, device=X.device)
    _use_current_stream(X.device)
    (xp, ldx), (wp, ldw), (op, ldo) = _view2d(X, torch.bfloat16, (M, K), "X"), _view2d(W, torch.bfloat16, (N, K), "W"), \
        _view2d(out, odt, (M, N), "out")
    _check(load().mtmc_fused_linear_strided(xp, ldx, wp, ldw, None if b is None else _dev(b, torch.float32, (N,), "b"),
                                            M, N, K, ACT[act], OUT_DTYPE[out_dtype], op, ldo))
    return out


def mtmc_fused_linear_mxfp8(X8, SX, W8, SW, b, act="none", out_dtype="bf16", out=None):
    """out = act(z + b) with block-scaled operands: X8 [M,K], W8 [N,K] float8_e4m3fn; SX [M,K/32], SW [N,K/32] uint8 (UE8M0)."""
    M, K = X8.shape
    N = W8.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if out is None:
        out = torch.empty((M, N), dtype=odt, device=X8.device)
    _use_current_stream(X8.device)
    f8 = torch.float8_e4m3fn
    _check(load().mtmc_fused_linear_mxfp8(_dev(X8, f8, (M, K), "X8"), _dev(SX, torch.uint8, (M, K // 32), "SX"),
                                          _dev(W8, f8, (N, K), "W8"), _dev(SW, torch.uint8, (N, K // 32), "SW"),
                                          None if b is None else _dev(b, torch.float32, (N,), "b"),
                                          M, N, K, ACT[act], OUT_DTYPE[out_dtype], _dev(out, odt, (M, N), "out")))
    return out


def mtmc_swiglu_mxfp8(X8, SX, Wg8, SG, Wu8, SU, out=None):
    """out = silu(z_gate) * z_up with block-scaled float8_e4m3fn operands and UE8M0 scales, bf16 [M,N]."""
    M, K = X8.shape
    N = Wg8.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=X8.device)
    _use_current_stream(X8.device)
    f8, u8 = torch.float8_e4m3fn, torch.uint8
    _check(load().mtmc_swiglu_mxfp8(_dev(X8, f8, (M, K), "X8"), _dev(SX, u8, (M, K // 32), "SX"), _dev(Wg8, f8, (N, K), "Wg8"),
                                    _dev(SG, u8, (N, K // 32), "SG"), _dev(Wu8, f8, (N, K), "Wu8"), _dev(SU, u8, (N, K // 32), "SU"),
                                    M, N, K, _dev(out, torch.bfloat16, (M, N), "out")))
    return out


def mtmc_linear_lse_mxfp8(X8, SX, W8, SW, b, lse_out=None):
    """lse_out[m] = logsumexp_n(z[m] + b) with block-scaled float8_e4m3fn operands and UE8M0 scales, fp32 [M]."""
    M, K = X8.shape
    N = W8.shape[0]
    if lse_out is None:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X8.device)
    _use_current_stream(X8.device)
    f8, u8 = torch.float8_e4m3fn, torch.uint8
    _check(load().mtmc_linear_lse_mxfp8(_dev(X8, f8, (M, K), "X8"), _dev(SX, u8, (M, K // 32), "SX"), _dev(W8, f8, (N, K), "W8"),
                                        _dev(SW, u8, (N, K // 32), "SW"), None if b is None else _dev(b, torch.float32, (N,), "b"),
                                        M, N, K, _dev(lse_out, torch.float32, (M,), "lse_out")))
    return lse_out


def mtmc_swiglu_strided(X, Wg, Wu, out=None):
    """mtmc_swiglu on views: X [M,K], Wg / Wu [N,K] and out [M,N] may be column slices of wider row-major tensors."""
    M, K = X.shape
    N = Wg.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    _use_current_stream(X.device)
    (xp, ldx), (gp, ldg), (up, ldu), (op, ldo) = (_view2d(X, torch.bfloat16, (M, K), "X"), _view2d(Wg, torch.bfloat16, (N, K), "Wg"),
                                                  _view2d(Wu, torch.bfloat16, (N, K), "Wu"), _view2d(out, torch.bfloat16, (M, N), "out"))
    _check(load().mtmc_swiglu_strided(xp, ldx, gp, ldg, up, ldu, M, N, K, op, ldo))
    return out


def mtmc_linear_lse_strided(X, W, b, lse_out=None):
    """mtmc_linear_lse with X [M,K] and W [N,K] as views (unit column stride, any row pitch that is a multiple of 8)."""
    M, K = X.shape
    N = W.shape[0]
    if lse_out is None:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X.device)
    _use_current_stream(X.device)
    (xp, ldx), (wp, ldw) = _view2d(X, torch.bfloat16, (M, K), "X"), _view2d(W, torch.bfloat16, (N, K), "W")
    _check(load().mtmc_linear_lse_strided(xp, ldx, wp, ldw, None if b is None else _dev(b, torch.float32, (N,), "b"), M, N, K,
                                          _dev(lse_out, torch.float32, (M,), "lse_out")))
    return lse_out


def mtmc_linear_rowmax_strided(X, W, b):
    """mtmc_linear_rowmax with X and W as views; returns (max fp32 [M], argmax int32 [M])."""
    M, K = X.shape
    N = W.shape[0]
    mx = torch.empty((M,), dtype=torch.float32, device=X.device)
    arg = torch.empty((M,), dtype=torch.int32, device=X.device)
    _use_current_stream(X.device)
    (xp, ldx), (wp, ldw) = _view2d(X, torch.bfloat16, (M, K), "X"), _view2d(W, torch.bfloat16, (N, K), "W")
    _check(load().mtmc_linear_rowmax_strided(xp, ldx, wp, ldw, None if b is None else _dev(b, torch.float32, (N,), "b"), M, N, K,
                                             mx.data_ptr(), arg.data_ptr()))
    return mx, arg


def mtmc_linear_cross_entropy_strided(X, W, b, targets):
    """mtmc_linear_cross_entropy with X and W as views; returns the loss, fp32 [M]."""
    M, K = X.shape
    N = W.shape[0]
    loss = torch.empty((M,), dtype=torch.float32, device=X.device)
    _use_current_stream(X.device)
    (xp, ldx), (wp, ldw) = _view2d(X, torch.bfloat16, (M, K), "X"), _view2d(W, torch.bfloat16, (N, K), "W")
    _check(load().mtmc_linear_cross_entropy_strided(xp, ldx, wp, ldw, None if b is None else _dev(b, torch.float32, (N,), "b"),
                                                    _dev(targets, torch.int64, (M,), "targets"), M, N, K, loss.data_ptr(), None))
    return loss


def mtmc_fused_linear_fp8(X8, W8, b, scale_x, scale_w, act="none", out_dtype="bf16", out=None):
    """out = act(scale_x * scale_w * X8 @ W8.T + b) with float8_e4m3fn operands X8 [M,K], W8 [N,K]."""
    M, K = X8.shape
    N = W8.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if out is None:
        out = torch.empty((M, N), dtype=odt, device=X8.device)
    _use_current_stream(X8.device)
    _check(load().mtmc_fused_linear_fp8(_dev(X8, torch.float8_e4m3fn, (M, K), "X8"), _dev(W8, torch.float8_e4m3fn, (N, K), "W8"),
                                        None if b is None else _dev(b, torch.float32, (N,), "b"),
                                        float(scale_x), float(scale_w), M, N, K, ACT[act], OUT_DTYPE[out_dtype],
                                        _dev(out, odt, (M, N), "out")))
    return out


def mtmc_swiglu_fp8(X8, Wg8, Wu8, scale_x, scale_g, scale_u, out=None):
    """out = silu(scale_x*scale_g * X8 @ Wg8.T) * (scale_x*scale_u * X8 @ Wu8.T), float8_e4m3fn operands, bf16 [M,N]."""
    M, K = X8.shape
    N = Wg8.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=X8.device)
    _use_current_stream(X8.device)
    f8 = torch.float8_e4m3fn
    _check(load().mtmc_swiglu_fp8(_dev(X8, f8, (M, K), "X8"), _dev(Wg8, f8, (N, K), "Wg8"), _dev(Wu8, f8, (N, K), "Wu8"),
                                  float(scale_x), float(scale_g), float(scale_u), M, N, K, _dev(out, torch.bfloat16, (M, N), "out")))
    return out


def mtmc_linear_lse_fp8(X8, W8, b, scale_x, scale_w, lse_out=None):
    """lse_out[m] = logsumexp_n(scale_x*scale_w * X8 @ W8.T + b) with float8_e4m3fn operands, fp32 [M]."""
    M, K = X8.shape
    N = W8.shape[0]
    if lse_out is None:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X8.device)
    _use_current_stream(X8.device)
    f8 = torch.float8_e4m3fn
    _check(load().mtmc_linear_lse_fp8(_dev(X8, f8, (M, K), "X8"), _dev(W8, f8, (N, K), "W8"),
                                      None if b is None else _dev(b, torch.float32, (N,), "b"),
                                      float(scale_x), float(scale_w), M, N, K, _dev(lse_out, torch.float32, (M,), "lse_out")))
    return lse_out


def mtmc_swiglu(X, Wg, Wu, out=None):
    """out = silu(X @ Wg.T) * (X @ Wu.T), bf16 [M,N]."""
    M, K = X.shape
    N = Wg.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    _use_current_stream(X.device)
    _check(load().mtmc_swiglu(_dev(X, torch.bfloat16, (M, K), "X"), _dev(Wg, torch.bfloat16, (N, K), "Wg"),
                              _dev(Wu, torch.bfloat16, (N, K), "Wu"), M, N, K, _dev(out, torch.bfloat16, (M, N), "out")))
    return out


def mtmc_linear_lse(X, W, b, lse_out=None):
    """lse_out[m] = logsumexp_n(X @ W.T + b), fp32 [M]; the logits are never materialised."""
    M, K = X.shape
    N = W.shape[0]
    if lse_out is None:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X.device)
    _use_current_stream(X.device)
    _check(load().mtmc_linear_lse(_dev(X, torch.bfloat16, (M, K), "X"), _dev(W, torch.bfloat16, (N, K), "W"),
                                  None if b is None else _dev(b, torch.float32, (N,), "b"),
                                  M, N, K, _dev(lse_out, torch.float32, (M,), "lse_out")))
    return lse_out


def mtmc_linear_rowmax(X, W, b, max_out=None, argmax_out=None, want_argmax=True):
    """(max_n, argmax_n) of X @ W.T + b per row, fp32 [M] and int32 [M]; the logits are never materialised."""
    M, K = X.shape
    N = W.shape[0]
    if max_out is None:
        max_out = torch.empty((M,), dtype=torch.float32, device=X.device)
    if argmax_out is None and want_argmax:
        argmax_out = torch.empty((M,), dtype=torch.int32, device=X.device)
    _use_current_stream(X.device)
    _check(load().mtmc_linear_rowmax(_dev(X, torch.bfloat16, (M, K), "X"), _dev(W, torch.bfloat16, (N, K), "W"),
                                     None if b is None else _dev(b, torch.float32, (N,), "b"), M, N, K,
                                     _dev(max_out, torch.float32, (M,), "max_out"),
                                     None if argmax_out is None else _dev(argmax_out, torch.int32, (M,), "argmax_out")))
    return max_out, argmax_out


def mtmc_linear_cross_entropy(X, W, b, targets, loss_out=None, lse_out=None, want_lse=False):
    """loss[m] = logsumexp_n(z[m]) - z[m][targets[m]] with z = X @ W.T + b; targets int64 [M] on the device."""
    M, K = X.shape
    N = W.shape[0]
    if loss_out is None:
        loss_out = torch.empty((M,), dtype=torch.float32, device=X.device)
    if lse_out is None and want_lse:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X.device)
    _use_current_stream(X.device)
    _check(load().mtmc_linear_cross_entropy(_dev(X, torch.bfloat16, (M, K), "X"), _dev(W, torch.bfloat16, (N, K), "W"),
                                            None if b is None else _dev(b, torch.float32, (N,), "b"),
                                            _dev(targets, torch.int64, (M,), "targets"), M, N, K,
                                            _dev(loss_out, torch.float32, (M,), "loss_out"),
                                            None if lse_out is None else _dev(lse_out, torch.float32, (M,), "lse_out")))
    return (loss_out, lse_out) if want_lse else loss_out


def mtmc_linear_softmax(X, W, b, out_dtype="fp32", prob_out=None, lse_out=None, want_lse=False):
    """prob[m][n] = softmax over n of z = X @ W.T + b, [M,N] fp32 or bf16; the logits are never written."""
    M, K = X.shape
    N = W.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if prob_out is None:
        prob_out = torch.empty((M, N), dtype=odt, device=X.device)
    if lse_out is None and want_lse:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X.device)
    _use_current_stream(X.device)
    _check(load().mtmc_linear_softmax(_dev(X, torch.bfloat16, (M, K), "X"), _dev(W, torch.bfloat16, (N, K), "W"),
                                      None if b is None else _dev(b, torch.float32, (N,), "b"), M, N, K, OUT_DTYPE[out_dtype],
                                      _dev(prob_out, odt, (M, N), "prob_out"),
                                      None if lse_out is None else _dev(lse_out, torch.float32, (M,), "lse_out")))
    return (prob_out, lse_out) if want_lse else prob_out


def mtmc_linear_softmax_strided(X, W, b, out_dtype="fp32", prob_out=None):
    """mtmc_linear_softmax with X, W and prob_out as row-major views (column slices of wider matrices)."""
    M, K = X.shape
    N = W.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if prob_out is None:
        prob_out = torch.empty((M, N), dtype=odt, device=X.device)
    _use_current_stream(X.device)
    (xp, ldx), (wp, ldw), (op, ldo) = (_view2d(X, torch.bfloat16, (M, K), "X"), _view2d(W, torch.bfloat16, (N, K), "W"),
                                       _view2d(prob_out, odt, (M, N), "prob_out"))
    _check(load().mtmc_linear_softmax_strided(xp, ldx, wp, ldw, None if b is None else _dev(b, torch.float32, (N,), "b"),
                                              M, N, K, OUT_DTYPE[out_dtype], op, ldo, None))
    return prob_out


def mtmc_linear_softmax_fp8(X8, W8, b, scale_x, scale_w, out_dtype="fp32", prob_out=None, lse_out=None, want_lse=False):
    """mtmc_linear_softmax with float8_e4m3fn operands and per-tensor scales."""
    M, K = X8.shape
    N = W8.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if prob_out is None:
        prob_out = torch.empty((M, N), dtype=odt, device=X8.device)
    if lse_out is None and want_lse:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X8.device)
    _use_current_stream(X8.device)
    f8 = torch.float8_e4m3fn
    _check(load().mtmc_linear_softmax_fp8(_dev(X8, f8, (M, K), "X8"), _dev(W8, f8, (N, K), "W8"),
                                          None if b is None else _dev(b, torch.float32, (N,), "b"),
                                          float(scale_x), float(scale_w), M, N, K, OUT_DTYPE[out_dtype],
                                          _dev(prob_out, odt, (M, N), "prob_out"),
                                          None if lse_out is None else _dev(lse_out, torch.float32, (M,), "lse_out")))
    return (prob_out, lse_out) if want_lse else prob_out


def mtmc_linear_rowmax_fp8(X8, W8, b, scale_x, scale_w, max_out=None, argmax_out=None, want_argmax=True):
    """mtmc_linear_rowmax with float8_e4m3fn operands and per-tensor scales."""
    M, K = X8.shape
    N = W8.shape[0]
    if max_out is None:
        max_out = torch.empty((M,), dtype=torch.float32, device=X8.device)
    if argmax_out is None and want_argmax:
        argmax_out = torch.empty((M,), dtype=torch.int32, device=X8.device)
    _use_current_stream(X8.device)
    f8 = torch.float8_e4m3fn
    _check(load().mtmc_linear_rowmax_fp8(_dev(X8, f8, (M, K), "X8"), _dev(W8, f8, (N, K), "W8"),
                                         None if b is None else _dev(b, torch.float32, (N,), "b"),
                                         float(scale_x), float(scale_w), M, N, K, _dev(max_out, torch.float32, (M,), "max_out"),
                                         None if argmax_out is None else _dev(argmax_out, torch.int32, (M,), "argmax_out")))
    return max_out, argmax_out


def mtmc_linear_cross_entropy_fp8(X8, W8, b, scale_x, scale_w, targets, loss_out=None, lse_out=None, want_lse=False):
    """mtmc_linear_cross_entropy with float8_e4m3fn operands and per-tensor scales."""
    M, K = X8.shape
    N = W8.shape[0]
    if loss_out is None:
        loss_out = torch.empty((M,), dtype=torch.float32, device=X8.device)
    if lse_out is None and want_lse:
        lse_out = torch.empty((M,), dtype=torch.float32, device=X8.device)
    _use_current_stream(X8.device)
    f8 = torch.float8_e4m3fn
    _check(load().mtmc_linear_cross_entropy_fp8(_dev(X8, f8, (M, K), "X8"), _dev(W8, f8, (N, K), "W8"),
                                                None if b is None else _dev(b, torch.float32, (N,), "b"),
                                                float(scale_x), float(scale_w), _dev(targets, torch.int64, (M,), "targets"), M, N, K,
                                                _dev(loss_out, torch.float32, (M,), "loss_out"),
                                                None if lse_out is None else _dev(lse_out, torch.float32, (M,), "lse_out")))
    return (loss_out, lse_out) if want_lse else loss_out


def mtmc_linear_lse_noalloc(X, W, b, lse_out):
    """mtmc_linear_lse without any allocation inside the library: the partials go to an
    8 MiB array built into the library image (ceil(N/256) * M <= 1,048,576).  For
    callers that may not allocate device memory -- a request loop that cannot afford
    cudaMalloc's device-wide stall, a plug-in inside a framework that owns the whole
    GPU.  The caller passes every buffer, lse_out included, so this wrapper allocates
    nothing either.  Calls sharing a GPU must not overlap; make the first call on a
    device before any stream capture."""
    M, K = X.shape
    N = W.shape[0]
    _use_current_stream(X.device)
    _check(load().mtmc_linear_lse_noalloc(_dev(X, torch.bfloat16, (M, K), "X"), _dev(W, torch.bfloat16, (N, K), "W"),
                                          None if b is None else _dev(b, torch.float32, (N,), "b"),
                                          M, N, K, _dev(lse_out, torch.float32, (M,), "lse_out")))
    return lse_out


def _host(t: torch.Tensor, dtype, shape, name: str) -> int:
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError("%s must be a CPU tensor" % name)
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise TypeError("%s must be contiguous %s of shape %r" % (name, dtype, tuple(shape)))
    return t.data_ptr()


def mtmc_fused_linear_host(X, W, b, act="none", out_dtype="bf16", out=None, device=0, blocking=True):
    """Host-pointer variant: CPU tensors in, CPU tensor out; copies inside the library.  blocking=False returns at once
    (pinned tensors; the result is valid after mtmc_host_sync())."""
    M, K = X.shape
    N = W.shape[0]
    odt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    if out is None:
        out = torch.empty((M, N), dtype=odt)
    _use_current_stream(torch.device("cuda", device))
    fn = load().mtmc_fused_linear_host if blocking else load().mtmc_fused_linear_host_async
    _check(fn(_host(X, torch.bfloat16, (M, K), "X"), _host(W, torch.bfloat16, (N, K), "W"),
              None if b is None else _host(b, torch.float32, (N,), "b"),
              M, N, K, ACT[act], OUT_DTYPE[out_dtype], _host(out, odt, (M, N), "out")))
    return out


def mtmc_swiglu_host(X, Wg, Wu, out=None, device=0, blocking=True):
    M, K = X.shape
    N = Wg.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16)
    _use_current_stream(torch.device("cuda", device))
    fn = load().mtmc_swiglu_host if blocking else load().mtmc_swiglu_host_async
    _check(fn(_host(X, torch.bfloat16, (M, K), "X"), _host(Wg, torch.bfloat16, (N, K), "Wg"),
              _host(Wu, torch.bfloat16, (N, K), "Wu"), M, N, K, _host(out, torch.bfloat16, (M, N), "out")))
    return out


def mtmc_linear_lse_host(X, W, b, lse_out=None, device=0, blocking=True):
    M, K = X.shape
    N = W.shape[0]
    if lse_out is None:
        lse_out = torch.empty((M,), dtype=torch.float32)
    _use_current_stream(torch.device("cuda", device))
    fn = load().mtmc_linear_lse_host if blocking else load().mtmc_linear_lse_host_async
    _check(fn(_host(X, torch.bfloat16, (M, K), "X"), _host(W, torch.bfloat16, (N, K), "W"),
              None if b is None else _host(b, torch.float32, (N,), "b"),
              M, N, K, _host(lse_out, torch.float32, (M,), "lse_out")))
    return lse_out


def mtmc_fused_linear_host_async(X, W, b, act="none", out_dtype="bf16", out=None, device=0):
    """mtmc_fused_linear_host without waiting for the result (valid after mtmc_host_sync())."""
    return mtmc_fused_linear_host(X, W, b, act, out_dtype, out=out, device=device, blocking=False)


def mtmc_swiglu_host_async(X, Wg, Wu, out=None, device=0):
    return mtmc_swiglu_host(X, Wg, Wu, out=out, device=device, blocking=False)


def mtmc_linear_lse_host_async(X, W, b, lse_out=None, device=0):
    return mtmc_linear_lse_host(X, W, b, lse_out=lse_out, device=device, blocking=False)


def mtmc_host_sync() -> None:
    """Waits for every non-blocking host-pointer call issued so far on the current device."""
    _check(load().mtmc_host_sync())


def mtmc_set_workspace(t: torch.Tensor | None) -> None:
    if t is None:
        _check(load().mtmc_set_workspace(None, 0))
    else:
        _check(load().mtmc_set_workspace(ctypes.c_void_p(t.data_ptr()), t.numel() * t.element_size()))


def mtmc_workspace_bytes(op: str, M: int, N: int, K: int) -> int:
    return int(load().mtmc_workspace_bytes(OP[op], M, N, K))


def mtmc_check_status() -> None:
    _check(load().mtmc_check_status())


def mtmc_selftest_timeout() -> None:
    """Enqueues the bounded-wait self-test kernel; the following mtmc_check_status() raises DEVICE_TIMEOUT."""
    torch.cuda.set_device(torch.cuda.current_device())
    load().mtmc_set_stream(ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    _check(load().mtmc_selftest_timeout())


def mtmc_launch_count() -> int:
    return int(load().mtmc_launch_count())


def mtmc_device_alloc_count() -> int:
    """cudaMalloc calls made by the library in this process so far."""
    return int(load().mtmc_device_alloc_count())


def mtmc_last_kernel_name() -> str:
    """Main kernel launched by this thread's most recent compute call."""
    return load().mtmc_last_kernel_name().decode()


def mtmc_set_timing(enabled: bool) -> None:
    load().mtmc_set_timing(1 if enabled else 0)


def mtmc_last_kernel_ms() -> float:
    return float(load().mtmc_last_kernel_ms())


def mtmc_set_tuning(split_k: int = 0, tile_n: int = 0, cta_pair: int = 0) -> None:
    _check(load().mtmc_set_tuning(int(split_k), int(tile_n), int(cta_pair)))


def mtmc_trace_enabled() -> bool:
    return bool(load().mtmc_trace_enabled())


def mtmc_set_trace(t: torch.Tensor | None) -> None:
    """Hands the trace build a zero-filled int64 CUDA tensor (32 words per CTA), or None to stop tracing."""
    if t is None:
        _check(load().mtmc_set_trace(None, 0))
    else:
        _check(load().mtmc_set_trace(ctypes.c_void_p(t.data_ptr()), t.numel() * t.element_size()))


def mtmc_set_schedule(stream_k: int = 0) -> None:
    """Stream-K schedule of the 256 x 256 pair kernel: 1 wherever legal, -1 never, 0 automatic."""
    _check(load().mtmc_set_schedule(int(stream_k)))


def mtmc_set_static_weights(enabled: bool = True) -> None:
    """Promise that no work in flight writes W: the weight-streaming path may start its W loads early."""
    _check(load().mtmc_set_static_weights(1 if enabled else 0))


def mtmc_version() -> int:
    return int(load().mtmc_version())
