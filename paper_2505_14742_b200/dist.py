"""Multi-GPU plumbing of the benchmark: one process per GPU, token-sharded replicas.

Per-token quantization makes the rows of a batch independent and the weight is frozen and replicated,
so the path shards over tokens with no collective on the data path: every rank runs the same layers on
its own batch.  What the ranks share is only the clock: a step takes as long as its slowest rank.

A trainer that wants the sharded run to reproduce the single-GPU run over the concatenated batch needs two
tiny reductions per layer and step, both outside the library (which makes no collective call):
``allreduce_colmax_`` between quaff_outlier_colmax and quaff_momentum_apply (then s_O, and with it every
code and accumulator, is bit-identical to the single-GPU run), and ``allreduce_lora_grads_`` after the
backward (the usual data-parallel sum of dA and dB).
"""
from __future__ import annotations

import os


def rank_world():
    """(rank, world size, local rank) from the launcher's environment (torchrun), or a single process."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def batch_index(step: int, rank: int) -> int:
    """Index of the synthetic batch that `rank` processes at `step`: ranks never share a batch."""
    return step + 1000 * rank


def max_over_ranks(value: float, device=None) -> float:
    """The largest `value` over all ranks (the job's time for a step); the value itself in a single process."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world: int, ms_per_step: float) -> float:
    """Units per second of the whole job: all ranks' units over the slowest rank's time."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def allreduce_colmax_(colmax_O):
    """Elementwise MAX over the ranks, in place, of the per-shard column maxima (nO floats): the maximum over all
    tokens is the maximum of the shards' maxima, exactly."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(colmax_O, op=dist.ReduceOp.MAX)
    return colmax_O


def allreduce_lora_grads_(dA, dB):
    """SUM over the ranks, in place, of the LoRA gradients of the shards (r (K + N) floats)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(dA, op=dist.ReduceOp.SUM)
        dist.all_reduce(dB, op=dist.ReduceOp.SUM)
    return dA, dB
