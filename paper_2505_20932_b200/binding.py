"""ctypes binding of ``libqwt2.so``: same names as the C ABI (``include/qwt2.h``), argument
marshalling only.  Tensors are passed as raw device (or host) pointers; PyTorch is used by callers
for memory and streams.  There is no fallback: a missing library raises at import.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqwt2.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2505_20932_b200.build` "
        "(the CUDA library is the product; there is no CPU fallback)")

lib = C.CDLL(LIB_PATH)

# status / enums (mirrors of qwt2.h)
QWT_OK, QWT_ERR_NULL, QWT_ERR_SHAPE, QWT_ERR_ALIGN, QWT_ERR_UNSUPPORTED = 0, 1, 2, 3, 4
QWT_ERR_WORKSPACE, QWT_ERR_CUDA, QWT_ERR_TIMEOUT, QWT_ERR_ARCH, QWT_ERR_TOO_LARGE = 5, 6, 7, 8, 9
QWT_NOALLOC_SCRATCH_BYTES = 6 << 20
QWT_W_INT8, QWT_W_INT4_PACKED = 0, 1
QWT_OUT_INT8_PER_TOKEN, QWT_OUT_BF16, QWT_OUT_FP32, QWT_OUT_INT32_ACC, QWT_OUT_INT8_STATIC = 0, 1, 2, 3, 4

_p, _i32, _i64, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t

# name -> (restype, argtypes); every symbol declared in include/qwt2.h
SIGNATURES = {
    "qwt_version": (C.c_char_p, []),
    "qwt_status_string": (C.c_char_p, [_i32]),
    "qwt_last_cuda_error": (_i32, [C.POINTER(C.c_int)]),
    "qwt_cwac_workspace_bytes": (_sz, [_i64, _i32]),
    "qwt_cwac_calibrate": (_i32, [_p, _p, _i64, _i32, _i64, _p, _p, _p, _p, _sz, _p]),
    "qwt_cwac_stats_accumulate": (_i32, [_p, _p, _i64, _i32, _i64, _p, _p, _sz, _p]),
    "qwt_cwac_solve": (_i32, [_p, _i32, _p, _p, _p, _p]),
    "qwt_cwac_host_staging_bytes": (_sz, [_i64, _i32]),
    "qwt_cwac_calibrate_host": (_i32, [_p, _p, _i64, _i32, _i64, _p, _p, _p, _p, _sz, _p]),
    "qwt_cwac_calibrate_batch_workspace_bytes": (_sz, [_p, _i32]),
    "qwt_cwac_calibrate_batch": (_i32, [_p, _i32, _p, _p, _sz, _p]),
    "qwt_cwac_calibrate_noalloc": (_i32, [_p, _p, _i64, _i32, _i64, _p, _p, _p, _p]),
    "qwt_cwac_fold": (_i32, [_p, _p, _p, _p, _i32, _p, _p, _p]),
    "qwt_cwac_fold_static": (_i32, [_p, _p, _p, _p, _i32, C.c_float, C.c_float, _p, _p, _p]),
    "qwt_qlinear_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32, _i32]),
    "qwt_qlinear_cwac_forward": (_i32, [_p, _p, _p, _i32, _p, _p, _i32, _i32, _i32, _i32, _p, _p, _p, _sz, _p]),
    "qwt_qlinear_cwac_calibrate_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "qwt_qlinear_cwac_calibrate": (_i32, [_p, _p, _p, _i32, _p, _p, _p, _i64, _i32, _i32, _i32, _p, _p, _p, _p, _p,
                                          _sz, _p]),
    "qwt_qlinear_check_status": (_i32, [_p, _p, C.POINTER(_i32)]),
    "qwt_qlinear_host_staging_bytes": (_sz, [_i32, _i32, _i32, _i32, _i32]),
    "qwt_qlinear_cwac_forward_host": (_i32, [_p, _p, _p, _i32, _p, _p, _i32, _i32, _i32, _i32, _p, _p, _p, _sz, _p]),
    "qwt_quantize_rows_u8": (_i32, [_p, _i64, _i32, _i64, _p, _p, _p, _p, _p]),
    "qwt_asym_weight_terms": (_i32, [_p, _p, _i32, _i32, _p, _p]),
    "qwt_qlinear_cwac_forward_asym": (_i32, [_p, _p, _p, _p, _p, _p, _p, _p, _i32, _i32, _i32, _i32, _p, _p, _p, _sz, _p]),
    "qwt_quantize_rows_i8": (_i32, [_p, _i64, _i32, _i64, _i32, _p, _p, _p]),
    "qwt_im2col_i8": (_i32, [_p, _i32, _i32, _i32, _i32, _i32, _i32, _i32, _i32, _p, _p]),
    "qwt_pack_int4": (_i32, [_p, _i64, _i32, _p, _p]),
    "qwt_qconv2d_workspace_bytes": (_sz, [_i32] * 10),
    "qwt_qconv2d_cwac_forward": (_i32, [_p, C.c_float, _p, _p, _p] + [_i32] * 10 + [_p, _p, _p, _sz, _p]),
    "qwt_test_set_wait_limit_ns": (None, [C.c_uint64]),
    "qwt_test_set_phantom_units": (None, [_i32]),
    "qwt_launch_count": (_i64, []),
    "qwt_launch_count_reset": (None, []),
}

for _name, (_res, _args) in SIGNATURES.items():
    _fn = getattr(lib, _name)          # AttributeError here = the library does not export the symbol
    _fn.restype = _res
    _fn.argtypes = _args


class QwtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.qwt_status_string(status).decode()
        if status == QWT_ERR_CUDA:
            e = C.c_int(0)
            lib.qwt_last_cuda_error(C.byref(e))
            msg += f" (cudaError {e.value})"
        super().__init__(f"{where}: {msg} [status {status}]")


def _check(status: int, where: str) -> None:
    if status != QWT_OK:
        raise QwtError(status, where)


def _ptr(t) -> Optional[int]:
    """Raw address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(type(t))


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# --------------------------------------------------------------------------- thin wrappers (same names)

def qwt_version() -> str:
    return lib.qwt_version().decode()


def qwt_status_string(s: int) -> str:
    return lib.qwt_status_string(s).decode()


def qwt_cwac_workspace_bytes(rows: int, channels: int) -> int:
    return lib.qwt_cwac_workspace_bytes(rows, channels)


def qwt_cwac_calibrate(fp_out, q_out, rows, channels, ld, a, b, n_degenerate, workspace, workspace_bytes,
                       stream=None, check=True) -> int:
    s = lib.qwt_cwac_calibrate(_ptr(fp_out), _ptr(q_out), rows, channels, ld, _ptr(a), _ptr(b), _ptr(n_degenerate),
                               _ptr(workspace), workspace_bytes, _stream(stream))
    if check:
        _check(s, "qwt_cwac_calibrate")
    return s


def qwt_cwac_stats_accumulate(fp_out, q_out, rows, channels, ld, stats, workspace, workspace_bytes, stream=None,
                              check=True) -> int:
    s = lib.qwt_cwac_stats_accumulate(_ptr(fp_out), _ptr(q_out), rows, channels, ld, _ptr(stats), _ptr(workspace),
                                      workspace_bytes, _stream(stream))
    if check:
        _check(s, "qwt_cwac_stats_accumulate")
    return s


def qwt_qlinear_cwac_calibrate_workspace_bytes(M, N, K, w_format) -> int:
    return int(lib.qwt_qlinear_cwac_calibrate_workspace_bytes(M, N, K, w_format))


def qwt_qlinear_cwac_calibrate(X, x_scale, W, w_format, w_scale, bias, fp_out, ld, M, N, K, stats, a, b, n_degenerate,
                               workspace, workspace_bytes, stream=None, check=True) -> int:
    s = lib.qwt_qlinear_cwac_calibrate(_ptr(X), _ptr(x_scale), _ptr(W), w_format, _ptr(w_scale), _ptr(bias),
                                       _ptr(fp_out), ld, M, N, K, _ptr(stats), _ptr(a), _ptr(b), _ptr(n_degenerate),
                                       _ptr(workspace), workspace_bytes, _stream(stream))
    if check:
        _check(s, "qwt_qlinear_cwac_calibrate")
    return s


def qwt_cwac_solve(stats, channels, a, b, n_degenerate, stream=None, check=True) -> int:
    s = lib.qwt_cwac_solve(_ptr(stats), channels, _ptr(a), _ptr(b), _ptr(n_degenerate), _stream(stream))
    if check:
        _check(s, "qwt_cwac_solve")
    return s


def qwt_cwac_host_staging_bytes(rows: int, channels: int) -> int:
    return lib.qwt_cwac_host_staging_bytes(rows, channels)


def qwt_cwac_calibrate_host(fp_out, q_out, rows, channels, ld, a, b, n_degenerate, staging, staging_bytes,
                            stream=None, check=True) -> int:
    s = lib.qwt_cwac_calibrate_host(_ptr(fp_out), _ptr(q_out), rows, channels, ld, _ptr(a), _ptr(b),
                                    _ptr(n_degenerate), _ptr(staging), staging_bytes, _stream(stream))
    if check:
        _check(s, "qwt_cwac_calibrate_host")
    return s


class CalibProblem(C.Structure):
    """Mirror of qwt_calib_problem."""
    _fields_ = [("fp_out", _p), ("q_out", _p), ("rows", _i64), ("ld", _i64), ("channels", _i32), ("a", _p), ("b", _p),
                ("w_scale", _p), ("bias", _p), ("fscale", _p), ("fbias", _p)]


def calib_problems(items):
    """items: iterable of (fp_out, q_out, rows, channels, ld, a, b[, w_scale, bias, fscale, fbias]) -> ctypes array."""
    items = list(items)
    arr = (CalibProblem * len(items))()
    for dst, it in zip(arr, items):
        it = tuple(it) + (None,) * (11 - len(it))
        fp, q, rows, ch, ld, a, b, ws, bias, fs, fb = it
        dst.fp_out, dst.q_out, dst.rows, dst.ld, dst.channels = _ptr(fp), _ptr(q), rows, ld, ch
        dst.a, dst.b, dst.w_scale, dst.bias, dst.fscale, dst.fbias = _ptr(a), _ptr(b), _ptr(ws), _ptr(bias), _ptr(fs), _ptr(fb)
    return arr


def qwt_cwac_calibrate_batch_workspace_bytes(problems) -> int:
    return int(lib.qwt_cwac_calibrate_batch_workspace_bytes(C.cast(problems, _p), len(problems)))


def qwt_cwac_calibrate_batch(problems, n_degenerate, workspace, workspace_bytes, stream=None, check=True) -> int:
    s = lib.qwt_cwac_calibrate_batch(C.cast(problems, _p), len(problems), _ptr(n_degenerate), _ptr(workspace),
                                     workspace_bytes, _stream(stream))
    if check:
        _check(s, "qwt_cwac_calibrate_batch")
    return s


def qwt_cwac_calibrate_noalloc(fp_out, q_out, rows, channels, ld, a, b, n_degenerate, stream=None, check=True) -> int:
    """Calibration that takes no workspace: for callers that may not allocate device memory.  The scratch is a
    fixed array inside the library (see include/qwt2.h for its limit and the rule about overlapping calls)."""
    s = lib.qwt_cwac_calibrate_noalloc(_ptr(fp_out), _ptr(q_out), rows, channels, ld, _ptr(a), _ptr(b),
                                       _ptr(n_degenerate), _stream(stream))
    if check:
        _check(s, "qwt_cwac_calibrate_noalloc")
    return s


def qwt_cwac_fold(w_scale, bias, a, b, n, fscale, fbias, stream=None, check=True) -> int:
    s = lib.qwt_cwac_fold(_ptr(w_scale), _ptr(bias), _ptr(a), _ptr(b), n, _ptr(fscale), _ptr(fbias), _stream(stream))
    if check:
        _check(s, "qwt_cwac_fold")
    return s


def qwt_cwac_fold_static(w_scale, bias, a, b, n, S_x, S_r, mult, offset, stream=None, check=True) -> int:
    s = lib.qwt_cwac_fold_static(_ptr(w_scale), _ptr(bias), _ptr(a), _ptr(b), n, S_x, S_r, _ptr(mult), _ptr(offset),
                                 _stream(stream))
    if check:
        _check(s, "qwt_cwac_fold_static")
    return s


def qwt_qlinear_workspace_bytes(M, N, K, wfmt, out_mode) -> int:
    return lib.qwt_qlinear_workspace_bytes(M, N, K, wfmt, out_mode)


def qwt_qlinear_cwac_forward(X, x_scale, W, wfmt, fscale, fbias, M, N, K, out_mode, Y, y_scale, workspace,
                             workspace_bytes, stream=None, check=True) -> int:
    s = lib.qwt_qlinear_cwac_forward(_ptr(X), _ptr(x_scale), _ptr(W), wfmt, _ptr(fscale), _ptr(fbias), M, N, K,
                                     out_mode, _ptr(Y), _ptr(y_scale), _ptr(workspace), workspace_bytes,
                                     _stream(stream))
    if check:
        _check(s, "qwt_qlinear_cwac_forward")
    return s


def qwt_qlinear_check_status(workspace, stream=None, check=True) -> int:
    word = _i32(0)
    s = lib.qwt_qlinear_check_status(_ptr(workspace), _stream(stream), C.byref(word))
    if check:
        _check(s, f"qwt_qlinear_check_status (device word {word.value})")
    return s


def qwt_qlinear_host_staging_bytes(M, N, K, wfmt, out_mode) -> int:
    return lib.qwt_qlinear_host_staging_bytes(M, N, K, wfmt, out_mode)


def qwt_qlinear_cwac_forward_host(X, x_scale, W, wfmt, fscale, fbias, M, N, K, out_mode, Y, y_scale, staging,
                                  staging_bytes, stream=None, check=True) -> int:
    s = lib.qwt_qlinear_cwac_forward_host(_ptr(X), _ptr(x_scale), _ptr(W), wfmt, _ptr(fscale), _ptr(fbias), M, N, K,
                                          out_mode, _ptr(Y), _ptr(y_scale), _ptr(staging), staging_bytes,
                                          _stream(stream))
    if check:
        _check(s, "qwt_qlinear_cwac_forward_host")
    return s


def qwt_quantize_rows_u8(X, rows, cols, ld, Xq, scale, zero, rowsum, stream=None, check=True) -> int:
    s = lib.qwt_quantize_rows_u8(_ptr(X), rows, cols, ld, _ptr(Xq), _ptr(scale), _ptr(zero), _ptr(rowsum), _stream(stream))
    if check:
        _check(s, "qwt_quantize_rows_u8")
    return s


def qwt_asym_weight_terms(W, w_zero, N, K, w_terms, stream=None, check=True) -> int:
    s = lib.qwt_asym_weight_terms(_ptr(W), _ptr(w_zero), N, K, _ptr(w_terms), _stream(stream))
    if check:
        _check(s, "qwt_asym_weight_terms")
    return s


def qwt_qlinear_cwac_forward_asym(X, x_scale, x_zero, x_rowsum, W, w_terms, fscale, fbias, M, N, K, out_mode, Y, y_scale,
                                  workspace, workspace_bytes, stream=None, check=True) -> int:
    s = lib.qwt_qlinear_cwac_forward_asym(_ptr(X), _ptr(x_scale), _ptr(x_zero), _ptr(x_rowsum), _ptr(W), _ptr(w_terms),
                                          _ptr(fscale), _ptr(fbias), M, N, K, out_mode, _ptr(Y), _ptr(y_scale),
                                          _ptr(workspace), workspace_bytes, _stream(stream))
    if check:
        _check(s, "qwt_qlinear_cwac_forward_asym")
    return s


def qwt_quantize_rows_i8(X, rows, cols, ld, qmax, Xq, scale, stream=None, check=True) -> int:
    s = lib.qwt_quantize_rows_i8(_ptr(X), rows, cols, ld, qmax, _ptr(Xq), _ptr(scale), _stream(stream))
    if check:
        _check(s, "qwt_quantize_rows_i8")
    return s


def qwt_im2col_i8(X, batch, H, W, C, kh, kw, stride, pad, patches, stream=None, check=True) -> int:
    s = lib.qwt_im2col_i8(_ptr(X), batch, H, W, C, kh, kw, stride, pad, _ptr(patches), _stream(stream))
    if check:
        _check(s, "qwt_im2col_i8")
    return s


def qwt_pack_int4(codes, rows, cols, packed, stream=None, check=True) -> int:
    s = lib.qwt_pack_int4(_ptr(codes), rows, cols, _ptr(packed), _stream(stream))
    if check:
        _check(s, "qwt_pack_int4")
    return s


def qwt_launch_count() -> int:
    return lib.qwt_launch_count()


def qwt_launch_count_reset() -> None:
    lib.qwt_launch_count_reset()


def qwt_test_set_wait_limit_ns(ns: int) -> None:
    lib.qwt_test_set_wait_limit_ns(int(ns))


def qwt_test_set_phantom_units(n: int) -> None:
    lib.qwt_test_set_phantom_units(int(n))


def qwt_qconv2d_workspace_bytes(batch, H, W, C_, Cout, kh, kw, stride, pad, out_mode) -> int:
    return lib.qwt_qconv2d_workspace_bytes(batch, H, W, C_, Cout, kh, kw, stride, pad, out_mode)


def qwt_qconv2d_cwac_forward(X, x_scale, Wt, fscale, fbias, batch, H, W, C_, Cout, kh, kw, stride, pad, out_mode, Y, y_scale,
                             workspace, workspace_bytes, stream=None, check=True) -> int:
    s = lib.qwt_qconv2d_cwac_forward(_ptr(X), float(x_scale), _ptr(Wt), _ptr(fscale), _ptr(fbias), batch, H, W, C_, Cout,
                                     kh, kw, stride, pad, out_mode, _ptr(Y), _ptr(y_scale), _ptr(workspace),
                                     workspace_bytes, _stream(stream))
    if check:
        _check(s, "qwt_qconv2d_cwac_forward")
    return s
