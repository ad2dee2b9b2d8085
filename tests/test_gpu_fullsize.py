"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (QuaffLinear layers
replayed through a CUDA graph, no debug dumps on the timed path).

What is cheap for the oracle is compared in full: the scale state s_O, all INT8 activation codes and
step sizes, the re-quantized outlier weight rows, the LoRA gradients.  What costs O(M N K) on the CPU
(INT32 accumulators, Y, dX) is compared on seeded sample rows: per-token quantization makes the rows of
the forward and of the grad-input independent, so the oracle computes exactly those rows.
"""
import numpy as np
import pytest

import oracle
from paper_2505_14742_b200 import synth
from util import TOL_BF16, dev, dev_bf16, f32, flip_slack, host, host_bits, max_rel_err

pytestmark = pytest.mark.gpu


def _run_layer(wl, li, steps, nsample, check_acc, full_grads=True):
    import torch
    from paper_2505_14742_b200 import build
    from paper_2505_14742_b200.layer import QuaffLinear, StepGraph
    build.build_library()
    lin = synth.layer_inputs(wl, li, b_std=0.02)
    sp = lin.spec
    M, K, N, r = wl.M, sp.K, sp.N, sp.r
    scale = wl.lora_alpha / r
    nOp = synth.pad_to(sp.nO, 32)
    layer = QuaffLinear(dev_bf16(lin.W), dev(lin.O_idx), dev_bf16(lin.A), dev_bf16(lin.B), scale, wl.gamma, M)
    Xd = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dYd = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")

    def body():
        layer.forward(Xd)
        layer.backward(dYd)

    Wq, dW, W_O, wmax = oracle.prepare_weight(lin.W, lin.O_idx)
    assert np.array_equal(host(layer.Wq), Wq) and np.array_equal(host(layer.dW), dW)
    s = np.ones(sp.nO, np.float32)
    graph = None
    rng = np.random.default_rng(wl.seed + li)
    for step in range(steps):
        X, dY = synth.step_inputs(wl, li, step, lin)
        Xd.copy_(dev_bf16(X)); dYd.copy_(dev_bf16(dY))
        if graph is None:
            body()                      # first call eagerly (function attributes), then everything through the graph
            torch.cuda.synchronize()
            layer.s_O.fill_(1.0)
            graph = StepGraph(body)
        graph.replay()
        torch.cuda.synchronize()
        assert int(layer.status[0].item()) == 0, "device-side wait timed out"
        s, _, _ = oracle.momentum_update(X, lin.O_idx, wmax, wl.gamma, s)
        assert np.array_equal(host(layer.s_O), s), f"s_O, step {step}"
        Xq, xqo, dx = oracle.quant_act(X, lin.O_idx, s, nOp)
        assert np.array_equal(host(layer.Xq), Xq), f"activation codes, step {step}"
        assert np.array_equal(host(layer.xq_O), xqo) and np.array_equal(host(layer.dx), dx)
        wq, dw = oracle.requant_weight_rows(W_O, s, nOp)
        assert np.array_equal(host(layer.wq_O), wq) and np.array_equal(host(layer.dw_O), dw)
        rows = np.sort(rng.choice(M, nsample, replace=False))
        rows[0], rows[-1] = 0, M - 1                       # first and last row of the first and last tile
        Xs, dYs = np.ascontiguousarray(X[rows]), np.ascontiguousarray(dY[rows])
        oY, oT, o1, o2 = oracle.qlinear_fwd(Xq[rows], xqo[rows], dx[rows], Wq, dW, wq, dw, Xs, lin.A, lin.B, scale)
        Tg = host_bits(layer.T)
        assert max_rel_err(f32(Tg[rows]), f32(oT)) <= TOL_BF16, "T"
        err = max_rel_err(host(layer.Y)[rows], oY, flip_slack(f32(oT).T, f32(lin.B), scale))
        assert err <= TOL_BF16, f"Y rows, step {step}: {err:.3e}"
        odX, _, _, oGs = oracle.qlinear_bwd(dYs, Wq, dW, wq, dw, lin.O_idx, s, Xs, oT, lin.A, lin.B, scale, want_dAB=False)
        err = max_rel_err(host(layer.dX)[rows], odX, flip_slack(f32(oGs).T, f32(lin.A).T))
        assert err <= TOL_BF16, f"dX rows, step {step}: {err:.3e}"
        # LoRA gradients contract over all tokens: T and G of the whole batch from the oracle
        oT_full = oracle.lora_down(X, lin.A)
        if full_grads:
            _, odA, odB, oG_full = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, lin.O_idx, s, X, oT_full, lin.A, lin.B, scale,
                                                      want_dX=False)
            assert max_rel_err(host(layer.dA), odA, flip_slack(f32(oG_full), f32(X)).T) <= TOL_BF16, "dA"
            assert max_rel_err(host(layer.dB), odB, flip_slack(f32(oT_full), f32(dY), scale)) <= TOL_BF16, "dB"
        else:
            # too large for the oracle's loops: dA = X^T G and dB = scale T^T dY on sampled rows / columns, the
            # contraction over all tokens by a float64 matrix product of the oracle's rounded G and T
            Gf = np.empty((M, r), np.float64)
            for m0 in range(0, M, 1024):      # G = bf16(scale dY B^T) from the oracle, a slab of tokens at a time
                sl = slice(m0, min(M, m0 + 1024))
                Gf[sl] = f32(oracle.qlinear_bwd(dY[sl], Wq, dW, wq, dw, lin.O_idx, s, X[sl], oT_full[sl], lin.A, lin.B, scale,
                                                want_dX=False, want_dAB=False)[3])
            ks = np.sort(rng.choice(K, 96, replace=False)); ks[:len(lin.O_idx[:8])] = lin.O_idx[:8]
            ns = np.sort(rng.choice(N, 96, replace=False))
            odA = f32(X[:, ks]).astype(np.float64).T @ Gf
            odB = scale * (f32(oT_full).astype(np.float64).T @ f32(dY[:, ns]).astype(np.float64))
            assert max_rel_err(host(layer.dA)[ks], odA, flip_slack(Gf, f32(X[:, ks])).T) <= TOL_BF16, "dA rows"
            assert max_rel_err(host(layer.dB)[:, ns], odB, flip_slack(f32(oT_full), f32(dY[:, ns]), scale)) <= TOL_BF16, "dB columns"
        if check_acc and step == 0:
            # INT32 accumulators of the same rows through the C ABI's debug dumps (a separate call: the dumps are
            # not on the timed path)
            from paper_2505_14742_b200 import binding as Q
            a1 = torch.empty((nsample, N), dtype=torch.int32, device="cuda")
            a2 = torch.empty((nsample, N), dtype=torch.int32, device="cuda")
            Ys = torch.empty((nsample, N), dtype=torch.bfloat16, device="cuda")
            Ts = torch.empty((nsample, r), dtype=torch.bfloat16, device="cuda")
            Q.quaff_qlinear_fwd(dev(Xq[rows]), dev(xqo[rows]), dev(dx[rows]), layer.Wq, layer.dW, layer.wq_O, layer.dw_O,
                                dev_bf16(Xs), layer.A, layer.B, scale, Ts, Ys, layer.ws, a1, a2, layer.status)
            torch.cuda.synchronize()
            assert np.array_equal(host(a1), o1), "main INT32 accumulator"
            assert np.array_equal(host(a2), o2), "outlier INT32 accumulator"


def test_phi3_attn_qkv_full_size_two_steps():
    _run_layer(synth.WORKLOADS["phi3_attn"], 0, steps=2, nsample=48, check_acc=True)


def test_phi3_attn_o_proj_full_size():
    _run_layer(synth.WORKLOADS["phi3_attn"], 1, steps=1, nsample=48, check_acc=True)


def test_llama7b_down_proj_full_size():
    _run_layer(synth.WORKLOADS["llama7b_block"], 6, steps=1, nsample=24, check_acc=True, full_grads=False)


def test_phi3_mlp_late_outliers_momentum_adaptation():
    """Configuration 'phi3_mlp': two members of O are dormant (magnitude 1) until step 100.  The scale state is
    carried over 112 steps through the momentum / requant / quant_act entry points and compared bit-exactly with
    the oracle at every step (cheap: O(M nO) per step); around the wake-up (steps 99-102, 111) the activation
    codes and the re-quantized rows are compared in full as well, and the late channels' scale must have left 1."""
    import torch
    from paper_2505_14742_b200 import binding as Q, build
    build.build_library()
    wl = synth.WORKLOADS["phi3_mlp"]
    li = 1                                              # down_proj 8192 -> 3072, nO = 82 incl. 2 late
    lin = synth.layer_inputs(wl, li)
    sp = lin.spec
    M, K, N = 512, sp.K, sp.N                           # a 512-token slice of the 4096: the state logic does not depend on M
    nOp = synth.pad_to(sp.nO, 32)
    Wq, dW, W_O, wmax = oracle.prepare_weight(lin.W, lin.O_idx)
    O_d, wmax_d, W_O_d = dev(lin.O_idx), dev(wmax), dev_bf16(W_O)
    s_d = torch.ones(sp.nO, dtype=torch.float32, device="cuda")
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_MOMENTUM, M, K, N, nOp, 0), dtype=torch.uint8, device="cuda")
    Xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
    xqo = torch.empty((M, nOp), dtype=torch.int8, device="cuda")
    dx = torch.empty(M, dtype=torch.float32, device="cuda")
    wq = torch.empty((N, nOp), dtype=torch.int8, device="cuda")
    dw = torch.empty(N, dtype=torch.float32, device="cuda")
    s = np.ones(sp.nO, np.float32)
    for step in range(112):
        mag = synth.outlier_magnitude(wl.seed, li, step, lin.base, sp.late)
        X = synth.activations(wl.seed, li, step, M, K, lin.O_idx, mag)
        Xd = dev_bf16(X)
        Q.quaff_momentum_update(Xd, O_d, wmax_d, wl.gamma, s_d, ws)
        s, _, _ = oracle.momentum_update(X, lin.O_idx, wmax, wl.gamma, s)
        assert np.array_equal(host(s_d), s), f"s_O, step {step}"
        if step in (0, 99, 100, 101, 102, 111):
            Q.quaff_requant_weight_rows(W_O_d, s_d, wq, dw)
            Q.quaff_quant_act(Xd, O_d, s_d, Xq, xqo, dx)
            torch.cuda.synchronize()
            oXq, oxqo, odx = oracle.quant_act(X, lin.O_idx, s, nOp)
            owq, odw = oracle.requant_weight_rows(W_O, s, nOp)
            assert np.array_equal(host(Xq), oXq) and np.array_equal(host(xqo), oxqo) and np.array_equal(host(dx), odx), step
            assert np.array_equal(host(wq), owq) and np.array_equal(host(dw), odw), step
        if step == 99:
            assert np.all(s[-sp.late:] < 12.0), "dormant channels: beta = sqrt(max|x| / max|w|) of an ordinary N(0,1) channel, about 7"
        if step == 111:
            assert np.all(s[-sp.late:] > 25.0), "the late outlier channels (20-100x) have been picked up by the momentum update"


@pytest.mark.parametrize("M,K,N,r,frac", [(512, 2048, 4096, 8, 0.05), (2048, 8192, 2048, 32, 0.01), (32768, 2048, 2048, 64, 0.005)])
def test_shape_sweep_points(M, K, N, r, frac):
    """Points of the shape sweep (tokens x K x N x rank x outlier fraction), one step each; 5 % of 2048 channels is
    nO = 102 (the 128-column forward with nOp = 128)."""
    wl = synth.sweep_point(M, K, N, r, frac)
    _run_layer(wl, 0, steps=1, nsample=16, check_acc=True, full_grads=False)
