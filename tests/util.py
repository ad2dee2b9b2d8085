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


def max_rel_err(got, ref, floor_rel=1e-3):
    """max_ij |got - ref| / max(|ref_ij|, floor_rel * rms(ref)): relative error per element; the floor of a
    thousandth of the output's rms keeps elements that cancel to ~0 from dividing by nothing.  No allowance of any kind."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if not ref.size:
        return 0.0
    rms = float(np.sqrt(np.mean(ref * ref)))
    floor = max(floor_rel * rms, 1e-30)
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), floor)))


def dx_floor(N):
    """Floor (as a fraction of the output's rms) of the metric for dX, a sum of N bf16 products accumulated in fp32 by
    the tensor cores.  Each of the N / 16 accumulation steps of an output element loses up to one unit in the last
    place of the running sum, about N 2^-28 of the output's rms in all whatever the final value is: measured
    2.9e-5 rms on the longest contraction of the workloads (N = 16384), i.e. 2.9e-2 of a 1e-3 rms floor for an
    element that cancels to zero.  Up to N = 2048 the floor is the 1e-3 used everywhere else; beyond, N 2^-21, which
    keeps that accumulation error below a third of the 2e-2 tolerance (N = 16384: 7.8e-3)."""
    return max(1e-3, N * 2.0 ** -21)


def check_bf16_intermediate(got_bits, ref_bits, what):
    """A bf16-rounded intermediate (T = bf16(X A), G = bf16(scale dY B^T)) from the GPU against the oracle's.

    Both round the same exact sum once, the GPU from an fp32 tensor-core accumulation, the oracle from a double
    sum; where the sum lies within the fp32 error of a rounding boundary the two decisions may differ, by ONE unit
    in the last place.  Asserts that no entry is further away than that (one bf16 ulp is at most 2^-7 of the
    value) and that such entries are rare; returns how many entries differ at all."""
    got_bits = np.asarray(got_bits, dtype=np.uint16)
    ref_bits = np.asarray(ref_bits, dtype=np.uint16)
    assert got_bits.shape == ref_bits.shape, what
    err = max_rel_err(f32(got_bits), f32(ref_bits))
    assert err <= 2.0 ** -7, f"{what}: an entry is more than one bf16 ulp from the oracle's ({err:.3e})"
    ndiff = int(np.count_nonzero(got_bits != ref_bits))
    assert ndiff <= max(2, got_bits.size // 100), f"{what}: {ndiff} of {got_bits.size} entries rounded differently"
    return ndiff


TOL_F32 = 1e-3   # fp32 epilogue, no bf16 rounding anywhere on the path
TOL_BF16 = 2e-2  # bf16 output and / or the bf16 LoRA branch
