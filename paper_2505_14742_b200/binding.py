"""Thin ctypes binding of libquaff.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors used as plain device memory (``data_ptr()``); every call is
enqueued on torch's current stream.  bf16 tensors may be ``torch.bfloat16`` or ``torch.uint16`` /
``torch.int16`` bit patterns.  There is no CPU fallback: a missing or unbuilt library raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

QUAFF_OK = 0
QUAFF_ERR_INVALID_ARG = 1
QUAFF_ERR_UNSUPPORTED_SHAPE = 2
QUAFF_ERR_ALIGNMENT = 3
QUAFF_ERR_WORKSPACE_TOO_SMALL = 4
QUAFF_ERR_CUDA = 5
QUAFF_ERR_TIMEOUT = 6
QUAFF_BF16, QUAFF_F32 = 0, 1
QUAFF_WS_PREPARE, QUAFF_WS_MOMENTUM, QUAFF_WS_FWD, QUAFF_WS_BWD, QUAFF_WS_CALIBRATE, QUAFF_WS_HITS, QUAFF_WS_BWD_INT8, QUAFF_WS_BWD_LEAN = 0, 1, 2, 3, 4, 5, 6, 7

EXPORTS = ("quaff_status_string", "quaff_workspace_bytes", "quaff_debug_launch_count", "quaff_debug_force_fwd_tile", "quaff_debug_time_gemm", "quaff_prepare_weight", "quaff_momentum_update", "quaff_lora_down", "quaff_outlier_count", "quaff_select_outliers", "quaff_outlier_hits",
           "quaff_momentum_update_static", "quaff_outlier_colmax", "quaff_momentum_apply", "quaff_quant_act", "quaff_requant_weight_rows", "quaff_qlinear_fwd", "quaff_qlinear_bwd", "quaff_quant_grad", "quaff_qlinear_bwd_int8")

_lib = None
_vp, _i64, _i32, _f32, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_size_t


class QuaffError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


def library_path() -> str:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Load libquaff.so (built in-tree by ``build.build_library``); raises if it is not there."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise FileNotFoundError(f"{path} is missing: run paper_2505_14742_b200.build.build_library() first "
                                    "(there is no fallback path)")
        L = ctypes.CDLL(path)
        L.quaff_status_string.restype = ctypes.c_char_p
        L.quaff_status_string.argtypes = [_i32]
        L.quaff_workspace_bytes.restype = _sz
        L.quaff_workspace_bytes.argtypes = [_i32] * 6
        L.quaff_prepare_weight.restype = _i32
        L.quaff_prepare_weight.argtypes = [_vp, _i64, _i32, _i32, _vp, _i32, _vp, _i64, _vp, _vp, _i64, _vp, _vp]
        L.quaff_momentum_update.restype = _i32
        L.quaff_momentum_update.argtypes = [_vp, _i64, _i32, _i32, _vp, _i32, _vp, _f32, _vp, _vp, _vp, _vp, _sz, _vp]
        L.quaff_momentum_update_static.restype = _i32
        L.quaff_momentum_update_static.argtypes = [_vp, _i64, _i32, _i32, _vp, _i32, _vp, _f32, _vp, _vp, _vp, _vp]
        L.quaff_outlier_colmax.restype = _i32
        L.quaff_outlier_colmax.argtypes = [_vp, _i64, _i32, _i32, _vp, _i32, _vp, _vp, _sz, _vp]
        L.quaff_momentum_apply.restype = _i32
        L.quaff_momentum_apply.argtypes = [_vp, _vp, _i32, _f32, _vp, _vp, _vp]
        L.quaff_quant_act.restype = _i32
        L.quaff_quant_act.argtypes = [_vp, _i64, _i32, _i32, _vp, _i32, _vp, _vp, _i64, _vp, _i64, _i32, _vp, _vp]
        L.quaff_requant_weight_rows.restype = _i32
        L.quaff_requant_weight_rows.argtypes = [_vp, _i64, _i32, _i32, _vp, _vp, _i64, _i32, _vp, _vp]
        L.quaff_outlier_hits.restype = _i32
        L.quaff_outlier_hits.argtypes = [_vp, _i64, _i32, _i32, _i32, _vp, _i32, _vp, _vp, _sz, _vp]
        L.quaff_outlier_count.restype = _i32
        L.quaff_outlier_count.argtypes = [_vp, _i64, _i32, _i32, _i32, _vp, _vp, _sz, _vp]
        L.quaff_select_outliers.restype = _i32
        L.quaff_select_outliers.argtypes = [_vp, _i32, _i32, _vp, _vp, _sz, _vp]
        L.quaff_lora_down.restype = _i32
        L.quaff_lora_down.argtypes = [_vp, _i64, _i32, _i32, _vp, _i32, _vp, _vp, _vp, _sz, _vp]
        L.quaff_qlinear_fwd.restype = _i32
        L.quaff_qlinear_fwd.argtypes = [_i32, _i32, _i32, _vp, _i64, _vp, _i64, _i32, _vp, _vp, _i64, _vp, _vp, _i64, _vp,
                                        _vp, _i64, _vp, _vp, _i32, _f32, _vp, _vp, _i32, _i64, _vp, _vp, _vp, _vp, _sz, _vp]
        L.quaff_qlinear_bwd.restype = _i32
        L.quaff_qlinear_bwd.argtypes = [_i32, _i32, _i32, _vp, _i64, _vp, _i64, _vp, _vp, _i64, _vp, _i32, _vp, _i32, _vp,
                                        _vp, _i64, _vp, _vp, _vp, _i32, _f32, _vp, _i64, _vp, _vp, _i32, _vp, _vp, _vp, _sz, _vp]
        L.quaff_qlinear_bwd_int8.restype = _i32
        L.quaff_qlinear_bwd_int8.argtypes = [_i32, _i32, _i32, _vp, _i64, _vp, _i64, _vp, _vp, _i64, _vp, _i32, _vp, _i32, _vp,
                                             _vp, _i64, _vp, _vp, _vp, _i32, _f32, _vp, _i64, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _sz, _vp]
        L.quaff_quant_grad.restype = _i32
        L.quaff_quant_grad.argtypes = [_vp, _i64, _i32, _i32, _vp, _vp, _i64, _vp, _vp]
        L.quaff_debug_launch_count.restype = ctypes.c_uint64
        L.quaff_debug_launch_count.argtypes = []
        L.quaff_debug_force_fwd_tile.restype = None
        L.quaff_debug_force_fwd_tile.argtypes = [_i32]
        L.quaff_debug_time_gemm.restype = None
        L.quaff_debug_time_gemm.argtypes = [_i32, _vp, _vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().quaff_status_string(int(code)).decode()


def workspace_bytes(which: int, M: int, K: int, N: int, nOp: int, r: int) -> int:
    return int(lib().quaff_workspace_bytes(which, M, K, N, nOp, r))


def quaff_debug_launch_count() -> int:
    return int(lib().quaff_debug_launch_count())


def quaff_debug_force_fwd_tile(tile_n: int) -> None:
    """Force the forward kernel's tile width (128 / 192 / 256); 0 = the library's cost model decides."""
    lib().quaff_debug_force_fwd_tile(int(tile_n))


def quaff_debug_time_gemm(which: int, start: Optional["torch.cuda.Event"], stop: Optional["torch.cuda.Event"]) -> None:
    """Arm (or, with None, disarm) event recording around the next forward (0) / grad-input (1) GEMM launch."""
    lib().quaff_debug_time_gemm(which, start.cuda_event if start is not None else None,
                                stop.cuda_event if stop is not None else None)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensor expected")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(code: int, where: str) -> None:
    if code != QUAFF_OK:
        raise QuaffError(code, where)


def _ld(t: torch.Tensor) -> int:
    return t.stride(0) if t.dim() == 2 else t.numel()


def quaff_outlier_count(X, thr: int, xi, ws) -> None:
    M, K = X.shape
    _check(lib().quaff_outlier_count(_ptr(X), _ld(X), M, K, int(thr), _ptr(xi), _ptr(ws), ws.numel() * ws.element_size(),
                                     _stream()), "quaff_outlier_count")


def quaff_outlier_hits(X, thr: int, O_idx, hits, ws) -> None:
    M, K = X.shape
    nO = 0 if O_idx is None else O_idx.numel()
    _check(lib().quaff_outlier_hits(_ptr(X), _ld(X), M, K, int(thr), _ptr(O_idx), nO, _ptr(hits), _ptr(ws),
                                    ws.numel() * ws.element_size(), _stream()), "quaff_outlier_hits")


def quaff_select_outliers(xi, O_idx, ws) -> None:
    _check(lib().quaff_select_outliers(_ptr(xi), xi.numel(), O_idx.numel(), _ptr(O_idx), _ptr(ws),
                                       ws.numel() * ws.element_size(), _stream()), "quaff_select_outliers")


def quaff_prepare_weight(Wt, O_idx, Wq, dW, W_O, wmax_O) -> None:
    N, K = Wt.shape
    nO = 0 if O_idx is None else O_idx.numel()
    _check(lib().quaff_prepare_weight(_ptr(Wt), _ld(Wt), N, K, _ptr(O_idx), nO, _ptr(Wq), _ld(Wq), _ptr(dW),
                                      _ptr(W_O), _ld(W_O) if W_O is not None else 0, _ptr(wmax_O), _stream()),
           "quaff_prepare_weight")


def quaff_momentum_update(X, O_idx, wmax_O, gamma: float, s_O, ws, colmax_O=None, beta_O=None) -> None:
    M, K = X.shape
    nO = 0 if O_idx is None else O_idx.numel()
    _check(lib().quaff_momentum_update(_ptr(X), _ld(X), M, K, _ptr(O_idx), nO, _ptr(wmax_O), float(gamma), _ptr(s_O),
                                       _ptr(colmax_O), _ptr(beta_O), _ptr(ws), ws.numel() * ws.element_size() if ws is not None else 0,
                                       _stream()), "quaff_momentum_update")


def quaff_momentum_update_static(X, O_idx, wmax_O, gamma: float, s_O, colmax_O=None, beta_O=None) -> None:
    """quaff_momentum_update for callers that cannot allocate a workspace: the scratch is a fixed array
    inside the library (nO <= 4096; calls that overlap on one GPU race on it)."""
    M, K = X.shape
    nO = 0 if O_idx is None else O_idx.numel()
    _check(lib().quaff_momentum_update_static(_ptr(X), _ld(X), M, K, _ptr(O_idx), nO, _ptr(wmax_O), float(gamma),
                                              _ptr(s_O), _ptr(colmax_O), _ptr(beta_O), _stream()),
           "quaff_momentum_update_static")


def quaff_outlier_colmax(X, O_idx, colmax_O, ws) -> None:
    """Column maxima of this GPU's rows over the outlier channels (first half of a token-sharded scale update)."""
    M, K = X.shape
    nO = 0 if O_idx is None else O_idx.numel()
    _check(lib().quaff_outlier_colmax(_ptr(X), _ld(X), M, K, _ptr(O_idx), nO, _ptr(colmax_O), _ptr(ws),
                                      ws.numel() * ws.element_size() if ws is not None else 0, _stream()), "quaff_outlier_colmax")


def quaff_momentum_apply(colmax_O, wmax_O, gamma: float, s_O, beta_O=None) -> None:
    """Eq. 8 and Eq. 7 from given (all-reduced) column maxima."""
    nO = 0 if colmax_O is None else colmax_O.numel()
    _check(lib().quaff_momentum_apply(_ptr(colmax_O), _ptr(wmax_O), nO, float(gamma), _ptr(s_O), _ptr(beta_O), _stream()),
           "quaff_momentum_apply")


def quaff_quant_act(X, O_idx, s_O, Xq, xq_O, dx) -> None:
    M, K = X.shape
    nO = 0 if O_idx is None else O_idx.numel()
    nOp = 0 if xq_O is None else xq_O.shape[1]
    _check(lib().quaff_quant_act(_ptr(X), _ld(X), M, K, _ptr(O_idx), nO, _ptr(s_O), _ptr(Xq), _ld(Xq),
                                 _ptr(xq_O), _ld(xq_O) if xq_O is not None else 0, nOp, _ptr(dx), _stream()),
           "quaff_quant_act")


def quaff_requant_weight_rows(W_O, s_O, wq_O, dw_O) -> None:
    nO = 0 if W_O is None else W_O.shape[0]
    N = dw_O.numel()
    nOp = 0 if wq_O is None else wq_O.shape[1]
    _check(lib().quaff_requant_weight_rows(_ptr(W_O), _ld(W_O) if W_O is not None else 0, nO, N, _ptr(s_O), _ptr(wq_O),
                                           _ld(wq_O) if wq_O is not None else 0, nOp, _ptr(dw_O), _stream()),
           "quaff_requant_weight_rows")


def quaff_lora_down(X, A, T_out, ws, status=None) -> None:
    M, K = X.shape
    _check(lib().quaff_lora_down(_ptr(X), _ld(X), M, K, _ptr(A), A.shape[1], _ptr(T_out), _ptr(status), _ptr(ws),
                                 ws.numel() * ws.element_size(), _stream()), "quaff_lora_down")


def quaff_qlinear_fwd(Xq, xq_O, dx, Wq, dW, wq_O, dw_O, X, A, B, lora_scale: float, T_out, Y, ws,
                      dbg_acc_main=None, dbg_acc_out=None, status=None) -> None:
    M, K = Xq.shape
    N = Wq.shape[0]
    nOp = 0 if xq_O is None else xq_O.shape[1]
    r = 0 if B is None else B.shape[0]
    y_dtype = QUAFF_F32 if Y.dtype == torch.float32 else QUAFF_BF16
    _check(lib().quaff_qlinear_fwd(M, K, N, _ptr(Xq), _ld(Xq), _ptr(xq_O), _ld(xq_O) if xq_O is not None else 0, nOp,
                                   _ptr(dx), _ptr(Wq), _ld(Wq), _ptr(dW), _ptr(wq_O),
                                   _ld(wq_O) if wq_O is not None else 0, _ptr(dw_O),
                                   _ptr(X), _ld(X) if X is not None else 0, _ptr(A), _ptr(B), r, float(lora_scale),
                                   _ptr(T_out), _ptr(Y), y_dtype, _ld(Y), _ptr(dbg_acc_main), _ptr(dbg_acc_out),
                                   _ptr(status), _ptr(ws), ws.numel() * ws.element_size() if ws is not None else 0,
                                   _stream()), "quaff_qlinear_fwd")


def quaff_qlinear_bwd(dY, Wq, dW, wq_O, dw_O, O_idx, s_O, X, T, A, B, lora_scale: float, dX, dA, dB,
                      accumulate: bool, ws, status=None, G_out=None) -> None:
    M, N = dY.shape
    K = Wq.shape[1]
    nOp = 0 if wq_O is None else wq_O.shape[1]
    nO = 0 if O_idx is None else O_idx.numel()
    r = 0 if A is None else A.shape[1]
    _check(lib().quaff_qlinear_bwd(M, K, N, _ptr(dY), _ld(dY), _ptr(Wq), _ld(Wq), _ptr(dW), _ptr(wq_O),
                                   _ld(wq_O) if wq_O is not None else 0, _ptr(dw_O), nOp, _ptr(O_idx), nO, _ptr(s_O),
                                   _ptr(X), _ld(X) if X is not None else 0, _ptr(T), _ptr(A), _ptr(B), r,
                                   float(lora_scale), _ptr(dX), _ld(dX) if dX is not None else 0, _ptr(dA), _ptr(dB),
                                   1 if accumulate else 0, _ptr(G_out), _ptr(status), _ptr(ws),
                                   ws.numel() * ws.element_size() if ws is not None else 0, _stream()),
           "quaff_qlinear_bwd")


def quaff_quant_grad(dY, dW, Zq, dz) -> None:
    """Z = dY * dW[n] quantized per token (the INT8 grad-input variant's first step)."""
    M, N = dY.shape
    _check(lib().quaff_quant_grad(_ptr(dY), _ld(dY), M, N, _ptr(dW), _ptr(Zq), _ld(Zq), _ptr(dz), _stream()), "quaff_quant_grad")


def quaff_qlinear_bwd_int8(dY, Wq, dW, wq_O, dw_O, O_idx, s_O, X, T, A, B, lora_scale: float, dX, dA, dB,
                           accumulate: bool, ws, status=None, G_out=None, dbg_acc=None) -> None:
    """The INT8 grad-input variant of the backward (not the paper's method)."""
    M, N = dY.shape
    K = Wq.shape[1]
    nOp = 0 if wq_O is None else wq_O.shape[1]
    nO = 0 if O_idx is None else O_idx.numel()
    r = 0 if A is None else A.shape[1]
    _check(lib().quaff_qlinear_bwd_int8(M, K, N, _ptr(dY), _ld(dY), _ptr(Wq), _ld(Wq), _ptr(dW), _ptr(wq_O),
                                        _ld(wq_O) if wq_O is not None else 0, _ptr(dw_O), nOp, _ptr(O_idx), nO, _ptr(s_O),
                                        _ptr(X), _ld(X) if X is not None else 0, _ptr(T), _ptr(A), _ptr(B), r,
                                        float(lora_scale), _ptr(dX), _ld(dX), _ptr(dA), _ptr(dB),
                                        1 if accumulate else 0, _ptr(G_out), _ptr(dbg_acc), _ptr(status), _ptr(ws),
                                        ws.numel() * ws.element_size() if ws is not None else 0, _stream()),
           "quaff_qlinear_bwd_int8")
