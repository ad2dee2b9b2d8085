"""numpy front end of the CPU oracle (test infrastructure, not a product path).

Builds ``quaff_oracle.c`` with gcc (no fast-math, no FMA contraction, OpenMP over rows)
and exposes each function on numpy arrays.  bf16 tensors are ``uint16`` bit patterns.
Only tests, the smoke check and the benchmark's CPU legs may import this package; the
CUDA library and its binding never do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "quaff_oracle.c")
_LIB = os.path.join(_HERE, "libquaff_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        # QUAFF_ORACLE_LIB: load this shared object instead (the mutation test points the pins at copies of the
        # oracle with one planted mistake each; nothing else sets it)
        other = os.environ.get("QUAFF_ORACLE_LIB")
        _lib = ctypes.CDLL(other) if other else ctypes.CDLL(build())
        _lib.qo_num_threads.restype = ctypes.c_int
        _lib.qo_int_gemm.restype = ctypes.c_int64
        _lib.qo_qlinear_fwd.restype = ctypes.c_int64
        _lib.qo_qlinear_bwd_int8.restype = ctypes.c_int64
    return _lib


def num_threads() -> int:
    return int(_load().qo_num_threads())


def _p(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"]
    return ctypes.c_void_p(a.ctypes.data)


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


I64 = ctypes.c_int64
I32 = ctypes.c_int
F32 = ctypes.c_float


def prepare_weight(Wt: np.ndarray, O_idx: np.ndarray):
    """Wt[N,K] bf16 bits -> (Wq[N,K] int8, dW[N] f32, W_O[nO,N] bf16 bits, wmax_O[nO] f32)."""
    Wt = _c(Wt, np.uint16)
    O_idx = _c(O_idx, np.int32)
    N, K = Wt.shape
    nO = O_idx.shape[0]
    Wq = np.empty((N, K), np.int8)
    dW = np.empty(N, np.float32)
    W_O = np.empty((nO, N), np.uint16)
    wmax = np.empty(nO, np.float32)
    _load().qo_prepare_weight(_p(Wt), I32(N), I32(K), _p(O_idx), I32(nO), _p(Wq), _p(dW), _p(W_O), _p(wmax))
    return Wq, dW, W_O, wmax


def momentum_update(X: np.ndarray, O_idx: np.ndarray, wmax_O: np.ndarray, gamma: float, s_O: np.ndarray):
    """Returns (s_new, colmax, beta); s_O is not modified."""
    X = _c(X, np.uint16)
    O_idx = _c(O_idx, np.int32)
    wmax_O = _c(wmax_O, np.float32)
    M, K = X.shape
    nO = O_idx.shape[0]
    s = _c(s_O, np.float32).copy()
    cm = np.empty(nO, np.float32)
    be = np.empty(nO, np.float32)
    _load().qo_momentum_update(_p(X), I64(K), I32(M), I32(K), _p(O_idx), I32(nO), _p(wmax_O), F32(gamma),
                               _p(s), _p(cm), _p(be))
    return s, cm, be


def outlier_colmax(X: np.ndarray, O_idx: np.ndarray) -> np.ndarray:
    """Column maxima max_m |X[m, O_i]| of a batch (or of one shard of it), f32 [nO]."""
    X = _c(X, np.uint16)
    O_idx = _c(O_idx, np.int32)
    M, K = X.shape
    cm = np.empty(O_idx.shape[0], np.float32)
    _load().qo_outlier_colmax(_p(X), I64(K), I32(M), _p(O_idx), I32(O_idx.shape[0]), _p(cm))
    return cm


def momentum_apply(colmax_O: np.ndarray, wmax_O: np.ndarray, gamma: float, s_O: np.ndarray):
    """Eq. 8 then Eq. 7 from given column maxima.  Returns (s_new, beta); s_O is not modified."""
    cm = _c(colmax_O, np.float32)
    wmax_O = _c(wmax_O, np.float32)
    s = _c(s_O, np.float32).copy()
    be = np.empty(cm.shape[0], np.float32)
    _load().qo_momentum_apply(_p(cm), _p(wmax_O), I32(cm.shape[0]), F32(gamma), _p(s), _p(be))
    return s, be


def quant_act(X: np.ndarray, O_idx: np.ndarray, s_O: np.ndarray, nOp: int, count_literal: bool = False):
    """Returns (Xq[M,K] int8, xq_O[M,nOp] int8, dx[M] f32[, n_literal_diff])."""
    X = _c(X, np.uint16)
    O_idx = _c(O_idx, np.int32)
    s_O = _c(s_O, np.float32)
    M, K = X.shape
    nO = O_idx.shape[0]
    assert nOp >= nO
    Xq = np.empty((M, K), np.int8)
    xq_O = np.empty((M, max(nOp, 1)), np.int8)
    dx = np.empty(M, np.float32)
    nd = ctypes.c_int64(0)
    _load().qo_quant_act(_p(X), I64(K), I32(M), I32(K), _p(O_idx), I32(nO), _p(s_O), _p(Xq), I64(K),
                         _p(xq_O), I64(max(nOp, 1)), I32(nOp), _p(dx),
                         ctypes.byref(nd) if count_literal else ctypes.c_void_p(0))
    xq_O = xq_O[:, :nOp]
    if count_literal:
        return Xq, xq_O, dx, int(nd.value)
    return Xq, xq_O, dx


def requant_weight_rows(W_O: np.ndarray, s_O: np.ndarray, nOp: int):
    """W_O[nO,N] bf16 bits -> (wq_O[N,nOp] int8, dw_O[N] f32)."""
    W_O = _c(W_O, np.uint16)
    s_O = _c(s_O, np.float32)
    nO, N = W_O.shape
    assert nOp >= nO
    wq = np.empty((N, max(nOp, 1)), np.int8)
    dw = np.empty(N, np.float32)
    _load().qo_requant_weight_rows(_p(W_O), I64(N), I32(nO), I32(N), _p(s_O), _p(wq), I64(max(nOp, 1)), I32(nOp), _p(dw))
    return wq[:, :nOp], dw


def int_gemm(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """C[m,n] = sum_k A[m,k] B[n,k] for int8 A[M,K], B[N,K]; int64 accumulation, int32 result."""
    A = _c(A, np.int8)
    B = _c(B, np.int8)
    M, K = A.shape
    N = B.shape[0]
    C = np.empty((M, N), np.int32)
    ov = _load().qo_int_gemm(_p(A), I64(K), _p(B), I64(K), I32(M), I32(N), I32(K), _p(C), I64(N))
    assert ov == 0, "integer accumulator overflow"
    return C


def qlinear_fwd(Xq, xq_O, dx, Wq, dW, wq_O, dw_O, X, A, B, lora_scale: float, T_in=None):
    """Returns (Y[M,N] f64, T[M,r] bf16 bits, acc1[M,N] i32, acc2[M,N] i32).

    T_in (bf16 bits [M,r]): evaluate the LoRA up-projection on these bits of T instead of rounding X A here."""
    Xq = _c(Xq, np.int8)
    M, K = Xq.shape
    Wq = _c(Wq, np.int8)
    N = Wq.shape[0]
    nOp = xq_O.shape[1]
    xq_O = _c(xq_O if nOp else np.zeros((M, 1), np.int8), np.int8)
    wq_O = _c(wq_O if nOp else np.zeros((N, 1), np.int8), np.int8)
    dx = _c(dx, np.float32)
    dW = _c(dW, np.float32)
    dw_O = _c(dw_O, np.float32)
    r = 0 if A is None else A.shape[1]
    X = _c(X, np.uint16)
    A_ = _c(A, np.uint16) if r else None
    B_ = _c(B, np.uint16) if r else None
    T = np.zeros((M, max(r, 1)), np.uint16)
    if T_in is not None and r:
        T[:, :r] = _c(T_in, np.uint16)
    Y = np.empty((M, N), np.float64)
    a1 = np.empty((M, N), np.int32)
    a2 = np.empty((M, N), np.int32)
    ov = _load().qo_qlinear_fwd(I32(M), I32(K), I32(N), _p(Xq), I64(K), _p(xq_O), I64(xq_O.shape[1]), I32(nOp), _p(dx),
                                _p(Wq), I64(K), _p(dW), _p(wq_O), I64(wq_O.shape[1]), _p(dw_O),
                                _p(X), I64(K), _p(A_), _p(B_), I32(r), F32(lora_scale),
                                _p(T), I32(1 if (T_in is not None and r) else 0), _p(Y), _p(a1), _p(a2))
    assert ov == 0, "integer accumulator overflow"
    return Y, T[:, :r], a1, a2


def lora_down(X, A):
    """T[M,r] = bf16(X A) (bf16 bits) of the whole batch: the forward routine run with no output
    channels, so that only its LoRA down-projection step executes."""
    X = _c(X, np.uint16)
    M, K = X.shape
    r = A.shape[1]
    z8 = np.zeros((1, 1), np.int8)
    zf = np.zeros(1, np.float32)
    T = np.zeros((M, r), np.uint16)
    _load().qo_qlinear_fwd(I32(M), I32(K), I32(0), _p(_c(np.zeros((M, 1), np.int8), np.int8)), I64(1), _p(z8), I64(1), I32(0),
                           _p(_c(np.zeros(M, np.float32), np.float32)), _p(z8), I64(1), _p(zf), _p(z8), I64(1), _p(zf),
                           _p(X), I64(K), _p(_c(A, np.uint16)), _p(np.zeros((r, 1), np.uint16)), I32(r), F32(1.0),
                           _p(T), I32(0), _p(np.zeros(1, np.float64)), _p(None), _p(None))
    return T


def qlinear_bwd(dY, Wq, dW, wq_O, dw_O, O_idx, s_O, X, T, A, B, lora_scale: float,
                want_dX: bool = True, want_dAB: bool = True, G_in=None):
    """Returns (dX[M,K] f64 | None, dA[K,r] f64 | None, dB[r,N] f64 | None, G[M,r] bf16 bits).

    G_in (bf16 bits [M,r]): use these bits of G = bf16(lora_scale dY B^T) instead of rounding the sum here."""
    dY = _c(dY, np.uint16)
    M, N = dY.shape
    Wq = _c(Wq, np.int8)
    K = Wq.shape[1]
    O_idx = _c(O_idx, np.int32)
    nO = O_idx.shape[0]
    nOp = wq_O.shape[1]
    wq_O = _c(wq_O if nOp else np.zeros((N, 1), np.int8), np.int8)
    dW = _c(dW, np.float32)
    dw_O = _c(dw_O, np.float32)
    s_O = _c(s_O, np.float32)
    r = 0 if A is None else A.shape[1]
    X = _c(X, np.uint16)
    T_ = _c(T, np.uint16) if r else None
    A_ = _c(A, np.uint16) if r else None
    B_ = _c(B, np.uint16) if r else None
    dX = np.empty((M, K), np.float64) if want_dX else None
    dA = np.empty((K, r), np.float64) if (want_dAB and r) else None
    dB = np.empty((r, N), np.float64) if (want_dAB and r) else None
    G = np.zeros((M, max(r, 1)), np.uint16)
    G_in_ = _c(G_in, np.uint16) if (G_in is not None and r) else None
    _load().qo_qlinear_bwd(I32(M), I32(K), I32(N), _p(dY), I64(N), _p(Wq), I64(K), _p(dW),
                           _p(wq_O), I64(wq_O.shape[1]), _p(dw_O), I32(nOp), _p(O_idx), I32(nO), _p(s_O),
                           _p(X), I64(K), _p(T_), _p(A_), _p(B_), I32(r), F32(lora_scale),
                           _p(dX), _p(dA), _p(dB), _p(G), _p(G_in_))
    return dX, dA, dB, G[:, :r]


def quant_grad(dY: np.ndarray, dW: np.ndarray):
    """INT8 grad-input variant: Z = dY * dW[n] quantized per token.  Returns (Zq[M,N] int8, dz[M] f32)."""
    dY = _c(dY, np.uint16)
    dW = _c(dW, np.float32)
    M, N = dY.shape
    Zq = np.empty((M, N), np.int8)
    dz = np.empty(M, np.float32)
    _load().qo_quant_grad(_p(dY), I64(N), I32(M), I32(N), _p(dW), _p(Zq), I64(N), _p(dz))
    return Zq, dz


def qlinear_bwd_int8(dY, Wq, dW, wq_O, dw_O, O_idx, s_O, X, T, A, B, lora_scale: float, want_dAB: bool = True, G_in=None):
    """The INT8 grad-input variant (not the paper's method).  Returns (dX[M,K] f64, dA | None, dB | None, G bf16 bits,
    Zq[M,N] int8, dz[M] f32, acc[M,K] int32)."""
    dY = _c(dY, np.uint16)
    M, N = dY.shape
    Wq = _c(Wq, np.int8)
    K = Wq.shape[1]
    O_idx = _c(O_idx, np.int32)
    nO = O_idx.shape[0]
    nOp = wq_O.shape[1]
    wq_O = _c(wq_O if nOp else np.zeros((N, 1), np.int8), np.int8)
    dW = _c(dW, np.float32)
    dw_O = _c(dw_O, np.float32)
    s_O = _c(s_O, np.float32)
    r = 0 if A is None else A.shape[1]
    X = _c(X, np.uint16)
    T_ = _c(T, np.uint16) if r else None
    A_ = _c(A, np.uint16) if r else None
    B_ = _c(B, np.uint16) if r else None
    dX = np.empty((M, K), np.float64)
    dA = np.empty((K, r), np.float64) if (want_dAB and r) else None
    dB = np.empty((r, N), np.float64) if (want_dAB and r) else None
    G = np.zeros((M, max(r, 1)), np.uint16)
    G_in_ = _c(G_in, np.uint16) if (G_in is not None and r) else None
    Zq = np.empty((M, N), np.int8)
    dz = np.empty(M, np.float32)
    acc = np.empty((M, K), np.int32)
    ov = _load().qo_qlinear_bwd_int8(I32(M), I32(K), I32(N), _p(dY), I64(N), _p(Wq), I64(K), _p(dW),
                                     _p(wq_O), I64(wq_O.shape[1]), _p(dw_O), I32(nOp), _p(O_idx), I32(nO), _p(s_O),
                                     _p(X), I64(K), _p(T_), _p(A_), _p(B_), I32(r), F32(lora_scale),
                                     _p(dX), _p(dA), _p(dB), _p(G), _p(G_in_), _p(Zq), _p(dz), _p(acc))
    assert ov == 0, "integer accumulator overflow"
    return dX, dA, dB, G[:, :r], Zq, dz, acc


def outlier_count(X: np.ndarray, thr: int, xi: np.ndarray) -> np.ndarray:
    """Eq. 6 for one calibration sample X[M,K] (bf16 bits): returns xi + indicator (xi is not modified)."""
    X = _c(X, np.uint16)
    M, K = X.shape
    out = _c(xi, np.int32).copy()
    _load().qo_outlier_count(_p(X), I64(K), I32(M), I32(K), I32(int(thr)), _p(out))
    return out


def outlier_hits(X: np.ndarray, thr: int, O_idx: np.ndarray) -> np.ndarray:
    """Hit-rate monitor (Sec. 3.2): [|R and O|, |R|] with R the Eq. 6 outlier channels of this batch X[M,K] (bf16 bits)."""
    X = _c(X, np.uint16)
    M, K = X.shape
    O = _c(O_idx, np.int32)
    hits = np.zeros(2, np.int32)
    _load().qo_outlier_hits(_p(X), I64(K), I32(M), I32(K), I32(int(thr)), _p(O), I32(O.shape[0]), _p(hits))
    return hits


def select_outliers(xi: np.ndarray, nO: int) -> np.ndarray:
    """The nO channels with the largest xi (ties: lower index first), sorted ascending (int32)."""
    xi = _c(xi, np.int32)
    O = np.empty(nO, np.int32)
    _load().qo_select_outliers(_p(xi), I32(xi.shape[0]), I32(nO), _p(O))
    return O

