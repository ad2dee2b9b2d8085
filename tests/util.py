"""Helpers shared by the GPU parity tests: numpy <-> device tensors and the error metrics."""
import numpy as np

from paper_2505_14742_b200 import synth


def f32(bits):
    return synth.bf16_bits_to_f32(bits)


def bf(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def dev_bf16(bits):
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 CUDA tensor with the same bits."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host_bits(t):
    """torch.bfloat16 tensor -> uint16 numpy bit patterns."""
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def host(t):
    import torch
    if t.dtype == torch.bfloat16:
        return f32(host_bits(t)).astype(np.float64)
    return t.detach().cpu().numpy()


def max_rel_err(got, ref):
    """max_ij |got - ref| / max(|ref_ij|, rms(ref) / 64): relative error per element, with a floor
    of 1.6 % of the output's rms so that elements that cancel to ~0 do not divide by nothing."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    floor = max(rms / 64.0, 1e-30)
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), floor))) if ref.size else 0.0


TOL_F32 = 1e-3   # fp32 epilogue, no bf16 rounding anywhere on the path
TOL_BF16 = 2e-2  # bf16 output and / or the bf16 LoRA branch
