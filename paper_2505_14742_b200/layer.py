"""One Quaff linear layer on the device: owns the buffers and chains the C-ABI calls of a step.

No arithmetic happens here; every step of the path runs in the library's kernels:
    forward : quaff_momentum_update -> quaff_requant_weight_rows -> quaff_quant_act -> quaff_qlinear_fwd
    backward: quaff_qlinear_bwd
``StepGraph`` records the launches of a whole step (several layers, fixed buffers) into a CUDA graph, so
that a training loop replays ~35 launches per layer with one call instead of enqueueing them one by one.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as Q


def pad32(n: int) -> int:
    return (n + 31) // 32 * 32


class QuaffLinear:
    """Frozen INT8 weight + outlier rows + LoRA adapters + the momentum scale state s_O."""

    def __init__(self, Wt: torch.Tensor, O_idx: Optional[torch.Tensor], A: Optional[torch.Tensor],
                 B: Optional[torch.Tensor], lora_scale: float, gamma: float, max_tokens: int,
                 y_dtype: torch.dtype = torch.bfloat16, debug_acc: bool = False, keep_G: bool = False,
                 int8_grad: bool = False, lean_bwd: bool = False):
        dev = Wt.device
        self.N, self.K = Wt.shape
        self.nO = 0 if O_idx is None else int(O_idx.numel())
        self.nOp = pad32(self.nO)
        self.r = 0 if A is None else int(A.shape[1])
        self.M = max_tokens
        self.gamma = float(gamma)
        self.lora_scale = float(lora_scale)
        self.O_idx = O_idx
        self.A, self.B = A, B
        N, K, M, nO, nOp, r = self.N, self.K, self.M, self.nO, self.nOp, self.r
        i8, f32, bf = torch.int8, torch.float32, torch.bfloat16
        self.Wq = torch.empty((N, K), dtype=i8, device=dev)
        self.dW = torch.empty(N, dtype=f32, device=dev)
        self.W_O = torch.empty((nO, N), dtype=bf, device=dev) if nO else None
        self.wmax_O = torch.empty(nO, dtype=f32, device=dev) if nO else None
        self.s_O = torch.ones(nO, dtype=f32, device=dev) if nO else None
        self.colmax_O = torch.empty(nO, dtype=f32, device=dev) if nO else None
        self.beta_O = torch.empty(nO, dtype=f32, device=dev) if nO else None
        self.wq_O = torch.empty((N, nOp), dtype=i8, device=dev) if nOp else None
        self.dw_O = torch.empty(N, dtype=f32, device=dev)
        self.Xq = torch.empty((M, K), dtype=i8, device=dev)
        self.xq_O = torch.empty((M, nOp), dtype=i8, device=dev) if nOp else None
        self.dx = torch.empty(M, dtype=f32, device=dev)
        self.T = torch.empty((M, r), dtype=bf, device=dev) if r else None
        self.Y = torch.empty((M, N), dtype=y_dtype, device=dev)
        self.dX = torch.empty((M, K), dtype=bf, device=dev)
        self.dA = torch.zeros((K, r), dtype=f32, device=dev) if r else None
        self.dB = torch.zeros((r, N), dtype=f32, device=dev) if r else None
        self.acc_main = torch.empty((M, N), dtype=torch.int32, device=dev) if debug_acc else None
        self.acc_out = torch.empty((M, N), dtype=torch.int32, device=dev) if debug_acc else None
        # G = bf16(lora_scale dY B^T) of the last backward, kept on request (otherwise it lives in the workspace)
        self.G = torch.empty((M, r), dtype=bf, device=dev) if (keep_G and r) else None
        self.status = torch.zeros(4, dtype=torch.int32, device=dev)
        # lean_bwd: a workspace without room for a bf16 copy of the weight: the grad-input GEMM expands the codes in-kernel
        # int8_grad: the backward runs the INT8 grad-input variant (quaff_qlinear_bwd_int8) - not the paper's method
        self.int8_grad = bool(int8_grad)
        ws_bytes = max(Q.workspace_bytes(Q.QUAFF_WS_MOMENTUM, M, K, N, nOp, r),
                       Q.workspace_bytes(Q.QUAFF_WS_FWD, M, K, N, nOp, r),
                       Q.workspace_bytes(Q.QUAFF_WS_BWD_INT8 if int8_grad else (Q.QUAFF_WS_BWD_LEAN if lean_bwd else Q.QUAFF_WS_BWD),
                                         M, K, N, nOp, r), 256)
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        # the LoRA down-projection runs beside the quantization chain, on its own stream and workspace
        self.ws_lora = torch.empty(max(Q.workspace_bytes(Q.QUAFF_WS_FWD, M, K, N, nOp, r), 256), dtype=torch.uint8, device=dev) if r else None
        self.side = torch.cuda.Stream(device=dev) if r else None
        self.side2 = torch.cuda.Stream(device=dev) if nO else None
        Q.quaff_prepare_weight(Wt, O_idx, self.Wq, self.dW, self.W_O, self.wmax_O)

    def forward(self, X: torch.Tensor) -> torch.Tensor:
        M = X.shape[0]
        assert M <= self.M and X.shape[1] == self.K
        Xq, dx, Y = self.Xq[:M], self.dx[:M], self.Y[:M]
        xq_O = self.xq_O[:M] if self.nOp else None
        T = self.T[:M] if self.r else None
        main = torch.cuda.current_stream()
        if self.r:     # T = X A needs only X: fork it off
            self.side.wait_stream(main)
            with torch.cuda.stream(self.side):
                Q.quaff_lora_down(X, self.A, T, self.ws_lora, self.status)
        if self.nO:
            Q.quaff_momentum_update(X, self.O_idx, self.wmax_O, self.gamma, self.s_O, self.ws, self.colmax_O, self.beta_O)
            # the outlier rows of the weight and the activations both need only s_O: side by side
            self.side2.wait_stream(main)
            with torch.cuda.stream(self.side2):
                Q.quaff_requant_weight_rows(self.W_O, self.s_O, self.wq_O, self.dw_O)
        Q.quaff_quant_act(X, self.O_idx, self.s_O, Xq, xq_O, dx)
        if self.nO:
            main.wait_stream(self.side2)
        if self.r:
            main.wait_stream(self.side)
        Q.quaff_qlinear_fwd(Xq, xq_O, dx, self.Wq, self.dW, self.wq_O, self.dw_O, None, None, self.B, self.lora_scale,
                            T, Y, self.ws,
                            self.acc_main[:M] if self.acc_main is not None else None,
                            self.acc_out[:M] if self.acc_out is not None else None, self.status)
        self._X = X
        return Y

    def backward(self, dY: torch.Tensor, accumulate: bool = False, need_dX: bool = True):
        M = dY.shape[0]
        dX = self.dX[:M] if need_dX else None
        T = self.T[:M] if self.r else None
        G = self.G[:M] if self.G is not None else None
        if self.int8_grad:
            Q.quaff_qlinear_bwd_int8(dY, self.Wq, self.dW, self.wq_O, self.dw_O, self.O_idx, self.s_O, self._X, T, self.A, self.B,
                                     self.lora_scale, self.dX[:M], self.dA, self.dB, accumulate, self.ws, self.status, G)
            return self.dX[:M], self.dA, self.dB
        Q.quaff_qlinear_bwd(dY, self.Wq, self.dW, self.wq_O, self.dw_O, self.O_idx, self.s_O, self._X, T, self.A, self.B,
                            self.lora_scale, dX, self.dA, self.dB, accumulate, self.ws, self.status, G)
        return dX, self.dA, self.dB


class StepGraph:
    """CUDA graph of ``body()`` (any sequence of forward / backward calls of QuaffLinear layers, and
    copies, on fixed buffers).  ``body`` must have run at least once before (the first call of an entry
    point sets function attributes and builds nothing a capture may contain), and is captured on a side
    stream; ``replay()`` enqueues the whole recorded step on the current stream."""

    def __init__(self, body):
        self.graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            # thread-local capture mode: CUDA calls of OTHER host threads (a process group's watchdog, a data loader)
            # do not invalidate the capture; what this thread enqueues is checked as strictly as before
            with torch.cuda.graph(self.graph, stream=side, capture_error_mode="thread_local"):
                body()
        torch.cuda.current_stream().wait_stream(side)

    def replay(self) -> None:
        self.graph.replay()
