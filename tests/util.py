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


def max_rel_err(got, ref, slack=None):
    """max_ij max(|got - ref| - slack_ij, 0) / max(|ref_ij|, rms(ref) / 64): relative error per element,
    with a floor of 1.6 % of the output's rms so that elements that cancel to ~0 do not divide by nothing.

    `slack` (see flip_slack) is the allowance for a bf16 rounding DECISION on an intermediate (T or G)
    that the two sides take from sums of different precision (fp32 tensor-core accumulation against the
    oracle's double): a decision that differs moves that intermediate by one bf16 ulp, and with it one
    term of every output it feeds, however small the (possibly cancelling) sum of all terms is."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if not ref.size:
        return 0.0
    rms = float(np.sqrt(np.mean(ref * ref)))
    floor = max(rms / 64.0, 1e-30)
    err = np.abs(got - ref)
    if slack is not None:
        err = np.maximum(err - slack, 0.0)
    return float(np.max(err / np.maximum(np.abs(ref), floor)))


def flip_slack(inter, other, scale=1.0):
    """Allowance for two one-ulp flips of a bf16 intermediate per output element.

    out[a][b] = scale * sum_m inter[m][a] * other[m][b]  (inter = the bf16-rounded T or G, float array
    [M][r]; other = the matrix it is contracted with, [M][C]); a flipped inter[m][a] changes out[a][b]
    by ulp * |other[m][b]| <= 2^-8 max_m|inter[m][a]| max_m|other[m][b]|.  Returns the [r][C] bound."""
    inter = np.abs(np.asarray(inter, dtype=np.float64))
    other = np.abs(np.asarray(other, dtype=np.float64))
    return 2.0 * abs(scale) * 2.0 ** -8 * np.outer(inter.max(axis=0), other.max(axis=0))


TOL_F32 = 1e-3   # fp32 epilogue, no bf16 rounding anywhere on the path
TOL_BF16 = 2e-2  # bf16 output and / or the bf16 LoRA branch
