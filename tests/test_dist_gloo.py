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


def _shard_worker(rank, world, port, out):
    """Token-sharded step of the oracle on two ranks with the two reductions, against the unsharded oracle."""
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = synth.WORKLOADS["tiny"]
        lin = synth.layer_inputs(wl, 0, b_std=0.02)
        sp = lin.spec
        scale = wl.lora_alpha / sp.r
        X, dY = synth.step_inputs(wl, 0, 0, lin)
        Wq, dW, W_O, wmax = oracle.prepare_weight(lin.W, lin.O_idx)
        s0 = np.full(sp.nO, 1.25, np.float32)
        cut = 100                                                    # uneven shards: rows [0,100) and [100,256)
        rows = slice(0, cut) if rank == 0 else slice(cut, wl.M)
        Xs, dYs = np.ascontiguousarray(X[rows]), np.ascontiguousarray(dY[rows])
        cm = torch.from_numpy(oracle.outlier_colmax(Xs, lin.O_idx))
        qdist.allreduce_colmax_(cm)                                  # MAX over the shards
        s, _ = oracle.momentum_apply(cm.numpy(), wmax, wl.gamma, s0)
        nOp = synth.pad_to(sp.nO, 32)
        Xq, xqo, dx = oracle.quant_act(Xs, lin.O_idx, s, nOp)
        wq, dw = oracle.requant_weight_rows(W_O, s, nOp)
        Y, T, a1, a2 = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, Xs, lin.A, lin.B, scale)
        dX, dA, dB, _ = oracle.qlinear_bwd(dYs, Wq, dW, wq, dw, lin.O_idx, s, Xs, T, lin.A, lin.B, scale)
        tA, tB = torch.from_numpy(dA), torch.from_numpy(dB)
        qdist.allreduce_lora_grads_(tA, tB)                          # SUM over the shards
        out[rank] = (s, Xq, a1, Y, dX, tA.numpy().copy(), tB.numpy().copy())
    finally:
        dist.destroy_process_group()


def test_sharded_step_with_the_two_reductions_reproduces_the_unsharded_step():
    import oracle
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    wl = synth.WORKLOADS["tiny"]
    lin = synth.layer_inputs(wl, 0, b_std=0.02)
    sp = lin.spec
    scale = wl.lora_alpha / sp.r
    X, dY = synth.step_inputs(wl, 0, 0, lin)
    Wq, dW, W_O, wmax = oracle.prepare_weight(lin.W, lin.O_idx)
    s, _, _ = oracle.momentum_update(X, lin.O_idx, wmax, wl.gamma, np.full(sp.nO, 1.25, np.float32))
    nOp = synth.pad_to(sp.nO, 32)
    Xq, xqo, dx = oracle.quant_act(X, lin.O_idx, s, nOp)
    wq, dw = oracle.requant_weight_rows(W_O, s, nOp)
    Y, T, a1, a2 = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, lin.A, lin.B, scale)
    dX, dA, dB, _ = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, lin.O_idx, s, X, T, lin.A, lin.B, scale)
    # the scale state, and with it every code, accumulator and output row, is that of the single-GPU run, bit for bit
    assert np.array_equal(res[0][0], s) and np.array_equal(res[1][0], s)
    assert np.array_equal(np.concatenate([res[0][1], res[1][1]]), Xq)
    assert np.array_equal(np.concatenate([res[0][2], res[1][2]]), a1)
    assert np.array_equal(np.concatenate([res[0][3], res[1][3]]), Y)
    assert np.array_equal(np.concatenate([res[0][4], res[1][4]]), dX)
    # the summed LoRA gradients: the same terms in another order (double sums)
    for rk in (0, 1):
        assert np.allclose(res[rk][5], dA, rtol=1e-12, atol=1e-18) and np.allclose(res[rk][6], dB, rtol=1e-12, atol=1e-18)


def test_single_process_is_identity():
    assert qdist.max_over_ranks(7.5) == 7.5
    assert qdist.batch_index(4, 0) == 4
    t = torch.tensor([1.0, 2.0])
    assert qdist.allreduce_colmax_(t) is t and t.tolist() == [1.0, 2.0]
