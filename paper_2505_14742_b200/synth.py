"""Seeded synthetic inputs shaped like the paper's fine-tuning workloads.

This module only *draws numbers*: it holds none of the method's arithmetic (no
scaling factors, no quantization, no GEMM).  It serves both the CUDA path and
the CPU oracle, which otherwise share nothing.  Everything is numpy; bf16
tensors are carried as ``uint16`` bit patterns so that no torch type is needed.

Value structure (paper Sec. 2.2 and Fig. 2): activations are N(0,1) except for
a small, *fixed* set of input channels O whose magnitude is 20-200x larger and
drifts from iteration to iteration; weights are N(0, 0.02); LoRA A is
N(0, 0.02) and LoRA B starts at zero (a non-zero B is available so that the
LoRA branch is exercised).  Real activations of Phi-3 / LLaMA-2 are not
available offline; these tensors stand in for them.

Every tensor is a pure function of (seed, tensor id, layer index, step): the
generator is Philox keyed on those four numbers, so any tensor can be redrawn
independently, in any order, on any machine.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

BASE_SEED = 20250514

# tensor ids (part of the Philox key)
_T_X, _T_W, _T_A, _T_B, _T_DY, _T_OIDX, _T_BASE, _T_DRIFT, _T_S0 = range(1, 10)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, tensor_id: int, layer: int = 0, step: int = 0) -> np.random.Generator:
    key = np.array([np.uint64(seed), np.uint64((tensor_id << 48) | (layer << 32) | step)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def outlier_indices(seed: int, layer: int, K: int, nO: int) -> np.ndarray:
    """The fixed outlier channel set O: nO distinct channels of 0..K-1, sorted (int32)."""
    perm = _rng(seed, _T_OIDX, layer).permutation(K)
    return np.sort(perm[:nO]).astype(np.int32)


def outlier_base(seed: int, layer: int, nO: int, kind: str) -> np.ndarray:
    """Base magnitude of each outlier channel.

    kind: "u30_80", "u20_100" (uniform) or "lognormal200" (exp(ln 40 + 0.8 z), capped at 200).
    """
    g = _rng(seed, _T_BASE, layer)
    if kind == "u30_80":
        return g.uniform(30.0, 80.0, nO)
    if kind == "u20_100":
        return g.uniform(20.0, 100.0, nO)
    if kind == "lognormal200":
        return np.minimum(200.0, np.exp(np.log(40.0) + 0.8 * g.standard_normal(nO)))
    raise ValueError(kind)


def outlier_magnitude(seed: int, layer: int, step: int, base: np.ndarray,
                      late: int = 0, late_step: int = 100) -> np.ndarray:
    """Per-step magnitude: base * (1 + 0.2 u), u ~ U(-1,1) redrawn each step (bounded drift).

    The last ``late`` channels of O stay at magnitude 1 (dormant) before ``late_step``.
    """
    u = _rng(seed, _T_DRIFT, layer, step).uniform(-1.0, 1.0, base.shape[0])
    mag = base * (1.0 + 0.2 * u)
    if late and step < late_step:
        mag[-late:] = 1.0
    return mag


def activations(seed: int, layer: int, step: int, M: int, K: int,
                O_idx: np.ndarray, mag: np.ndarray) -> np.ndarray:
    """X[M,K] as bf16 bits: N(0,1), channels O multiplied by mag."""
    x = _rng(seed, _T_X, layer, step).standard_normal((M, K), dtype=np.float32)
    if len(O_idx):
        x[:, O_idx] *= mag.astype(np.float32)[None, :]
    return f32_to_bf16_bits(x)


def weight(seed: int, layer: int, N: int, K: int, std: float = 0.02) -> np.ndarray:
    """Frozen weight in the nn.Linear layout [N = c_out, K = c_in] as bf16 bits, N(0, std)."""
    w = _rng(seed, _T_W, layer).standard_normal((N, K), dtype=np.float32) * np.float32(std)
    return f32_to_bf16_bits(w)


def lora_A(seed: int, layer: int, K: int, r: int, std: float = 0.02) -> np.ndarray:
    """LoRA down-projection A[K,r] as bf16 bits."""
    a = _rng(seed, _T_A, layer).standard_normal((K, r), dtype=np.float32) * np.float32(std)
    return f32_to_bf16_bits(a)


def lora_B(seed: int, layer: int, r: int, N: int, std: float = 0.0) -> np.ndarray:
    """LoRA up-projection B[r,N] as bf16 bits; std=0 gives the usual zero init."""
    if std == 0.0:
        return np.zeros((r, N), dtype=np.uint16)
    b = _rng(seed, _T_B, layer).standard_normal((r, N), dtype=np.float32) * np.float32(std)
    return f32_to_bf16_bits(b)


def grad_out(seed: int, layer: int, step: int, M: int, N: int, std: float = 1e-2) -> np.ndarray:
    """Upstream gradient dY[M,N] as bf16 bits, N(0, std)."""
    g = _rng(seed, _T_DY, layer, step).standard_normal((M, N), dtype=np.float32) * np.float32(std)
    return f32_to_bf16_bits(g)


def pad_to(n: int, g: int) -> int:
    return ((n + g - 1) // g) * g


@dataclass(frozen=True)
class LayerSpec:
    name: str
    K: int          # c_in
    N: int          # c_out
    nO: int         # |O|
    r: int          # LoRA rank
    late: int = 0   # channels of O that wake up only at step 100


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # index in the list of configurations (also offsets the seed)
    M: int                     # tokens
    layers: Tuple[LayerSpec, ...]
    gamma: float               # momentum of the scale update
    base_kind: str
    steps: int
    lora_alpha: float = 16.0

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index


def _frac(K: int, f: float) -> int:
    return max(1, int(round(f * K)))


WORKLOADS = {
    # tiny single layer: everything is compared, every step
    "tiny": Workload("tiny", 0, 256, (LayerSpec("linear", 512, 512, 8, 8),), 0.9, "u30_80", 10, 8.0),
    # Phi-3-mini attention projections, batch 4 x seq 512
    "phi3_attn": Workload("phi3_attn", 1, 2048,
                          (LayerSpec("qkv_proj", 3072, 9216, 32, 16),
                           LayerSpec("o_proj", 3072, 3072, 32, 16)), 0.2, "u20_100", 50),
    # Phi-3-mini MLP; two members of O are dormant until step 100
    "phi3_mlp": Workload("phi3_mlp", 2, 4096,
                         (LayerSpec("gate_up_proj", 3072, 16384, _frac(3072, 0.01), 16, late=2),
                          LayerSpec("down_proj", 8192, 3072, _frac(8192, 0.01), 16, late=2)),
                         0.2, "u20_100", 200),
    # LLaMA-2-7B decoder block, batch 8 x seq 1024
    "llama7b_block": Workload("llama7b_block", 3, 8192,
                              tuple([LayerSpec(n, 4096, 4096, _frac(4096, 0.005), 64) for n in ("q_proj", "k_proj", "v_proj", "o_proj")]
                                    + [LayerSpec(n, 4096, 11008, _frac(4096, 0.005), 64) for n in ("gate_proj", "up_proj")]
                                    + [LayerSpec("down_proj", 11008, 4096, _frac(11008, 0.005), 64)]),
                              0.2, "lognormal200", 200, 64.0),
}


def sweep_point(M: int, K: int, N: int, r: int, frac: float) -> Workload:
    """One point of the shape sweep (tokens x K x N x rank x outlier fraction)."""
    return Workload(f"sweep_M{M}_K{K}_N{N}_r{r}_f{frac}", 4, M,
                    (LayerSpec("linear", K, N, _frac(K, frac), r),), 0.2, "u20_100", 20, float(r))


@dataclass
class LayerInputs:
    """Frozen, per-layer tensors (bf16 bits unless noted)."""
    spec: LayerSpec
    O_idx: np.ndarray            # int32 [nO]
    base: np.ndarray             # float64 [nO], generator-side only
    W: np.ndarray                # [N,K]
    A: np.ndarray                # [K,r]
    B: np.ndarray                # [r,N]


def layer_inputs(wl: Workload, li: int, b_std: float = 0.0) -> LayerInputs:
    sp = wl.layers[li]
    O_idx = outlier_indices(wl.seed, li, sp.K, sp.nO)
    base = outlier_base(wl.seed, li, sp.nO, wl.base_kind)
    return LayerInputs(sp, O_idx, base,
                       weight(wl.seed, li, sp.N, sp.K),
                       lora_A(wl.seed, li, sp.K, sp.r),
                       lora_B(wl.seed, li, sp.r, sp.N, b_std))


def step_inputs(wl: Workload, li: int, step: int, lin: LayerInputs) -> Tuple[np.ndarray, np.ndarray]:
    """(X[M,K], dY[M,N]) of one step, bf16 bits."""
    sp = lin.spec
    mag = outlier_magnitude(wl.seed, li, step, lin.base, sp.late)
    X = activations(wl.seed, li, step, wl.M, sp.K, lin.O_idx, mag)
    dY = grad_out(wl.seed, li, step, wl.M, sp.N)
    return X, dY
