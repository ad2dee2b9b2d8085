"""The benchmark's multi-rank host logic on CPU: two gloo ranks (no GPU needed)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_14742_b200 import dist as qdist, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert qdist.rank_world() == (rank, world, rank)
        # a step takes as long as its slowest rank
        slowest = qdist.max_over_ranks(10.0 + 5.0 * rank)
        # every rank draws its own batch; the same rank and step always draw the same one
        wl = synth.WORKLOADS["tiny"]
        lin = synth.layer_inputs(wl, 0)
        X, _ = synth.step_inputs(wl, 0, qdist.batch_index(3, rank), lin)
        X2, _ = synth.step_inputs(wl, 0, qdist.batch_index(3, rank), lin)
        assert np.array_equal(X, X2)
        digest = torch.tensor([float(X.astype(np.int64).sum())], dtype=torch.float64)
        both = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(both, digest)
        out[rank] = (slowest, [float(b.item()) for b in both])
    finally:
        dist.destroy_process_group()


def test_two_ranks_max_time_and_disjoint_batches():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0
    assert res[0][1] == res[1][1] and res[0][1][0] != res[0][1][1]
    # whole-job rate: both ranks' tokens over the slowest rank's time
    assert qdist.whole_job_rate(256, 2, 15.0) == 2 * 256 / 0.015


def test_single_process_is_identity():
    assert qdist.max_over_ranks(7.5) == 7.5
    assert qdist.batch_index(4, 0) == 4
