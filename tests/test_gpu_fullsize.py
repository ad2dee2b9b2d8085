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
from util import TOL_BF16, check_bf16_intermediate, dev, dev_bf16, dx_floor, host, host_bits, max_rel_err

pytestmark = pytest.mark.gpu


def _run_layer(wl, li, steps, nsample, check_acc, full_grads=True, int8_grad=False, lean_bwd=False, step_inputs=None, extra_rows=()):
    import torch
    from paper_2505_14742_b200 import build
    from paper_2505_14742_b200.layer import QuaffLinear, StepGraph
    build.build_library()
    lin = synth.layer_inputs(wl, li, b_std=0.02)
    sp = lin.spec
    M, K, N, r = wl.M, sp.K, sp.N, sp.r
    scale = wl.lora_alpha / r
    nOp = synth.pad_to(sp.nO, 32)
    # keep_G: the backward writes G into a buffer of the layer instead of its workspace (same kernels, same launches)
    layer = QuaffLinear(dev_bf16(lin.W), dev(lin.O_idx), dev_bf16(lin.A), dev_bf16(lin.B), scale, wl.gamma, M, keep_G=True,
                        int8_grad=int8_grad, lean_bwd=lean_bwd)
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
    none_O, none_s, none_wq = np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros((1, 0), np.int8)
    for step in range(steps):
        X, dY = (step_inputs or synth.step_inputs)(wl, li, step, lin)
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
        rows = np.unique(np.concatenate([rows, np.asarray(extra_rows, dtype=rows.dtype)]))
        Xs, dYs = np.ascontiguousarray(X[rows]), np.ascontiguousarray(dY[rows])
        Tg, Gg = host_bits(layer.T), host_bits(layer.G)
        # the bf16 intermediates of the sampled rows: at most one ulp from the oracle's; everything downstream is
        # compared with the oracle evaluated on the GPU's own T and G bits, with no allowance
        oY, oT, o1, o2 = oracle.qlinear_fwd(Xq[rows], xqo[rows], dx[rows], Wq, dW, wq, dw, Xs, lin.A, lin.B, scale)
        check_bf16_intermediate(Tg[rows], oT, f"T rows, step {step}")
        oY = oracle.qlinear_fwd(Xq[rows], xqo[rows], dx[rows], Wq, dW, wq, dw, Xs, lin.A, lin.B, scale, T_in=Tg[rows])[0]
        err = max_rel_err(host(layer.Y)[rows], oY)
        assert err <= TOL_BF16, f"Y rows, step {step}: {err:.3e}"
        oGs = oracle.qlinear_bwd(dYs, Wq, dW, wq, dw, lin.O_idx, s, Xs, Tg[rows], lin.A, lin.B, scale, want_dX=False, want_dAB=False)[3]
        check_bf16_intermediate(Gg[rows], oGs, f"G rows, step {step}")
        if int8_grad:    # the INT8 grad-input variant against its own oracle function
            odX = oracle.qlinear_bwd_int8(dYs, Wq, dW, wq, dw, lin.O_idx, s, Xs, Tg[rows], lin.A, lin.B, scale, want_dAB=False, G_in=Gg[rows])[0]
        else:
            odX = oracle.qlinear_bwd(dYs, Wq, dW, wq, dw, lin.O_idx, s, Xs, Tg[rows], lin.A, lin.B, scale, want_dAB=False, G_in=Gg[rows])[0]
        err = max_rel_err(host(layer.dX)[rows], odX, dx_floor(N))
        assert err <= TOL_BF16, f"dX rows, step {step}: {err:.3e}"
        # LoRA gradients contract over all tokens
        if full_grads:
            check_bf16_intermediate(Tg, oracle.lora_down(X, lin.A), f"T, step {step}")
            _, odA, odB, _ = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, lin.O_idx, s, X, Tg, lin.A, lin.B, scale, want_dX=False, G_in=Gg)
            ea, eb = max_rel_err(host(layer.dA), odA), max_rel_err(host(layer.dB), odB)
        else:
            # too large for the oracle's loops in full: dA[k][:] depends on column k of X only and dB[:][n] on column n of
            # dY only, so the oracle computes sampled rows of dA and sampled columns of dB over ALL tokens
            ks = np.sort(rng.choice(K, 64, replace=False)); ks[:len(lin.O_idx[:8])] = lin.O_idx[:8]; ks = np.unique(ks)
            ns = np.sort(rng.choice(N, 64, replace=False))
            _, odA, odB, _ = oracle.qlinear_bwd(np.ascontiguousarray(dY[:, ns]), np.zeros((len(ns), len(ks)), np.int8), dW[ns], none_wq,
                                                dw[ns], none_O, none_s, np.ascontiguousarray(X[:, ks]), Tg, np.ascontiguousarray(lin.A[ks]),
                                                np.ascontiguousarray(lin.B[:, ns]), scale, want_dX=False, G_in=Gg)
            ea, eb = max_rel_err(host(layer.dA)[ks], odA), max_rel_err(host(layer.dB)[:, ns], odB)
        assert ea <= TOL_BF16 and eb <= TOL_BF16, f"dA {ea:.3e} dB {eb:.3e}, step {step}"
        if check_acc and step == 0:
            # INT32 accumulators of the same rows through the C ABI's debug dumps (a separate call: the dumps are
            # not on the timed path)
            from paper_2505_14742_b200 import binding as Q
            a1 = torch.empty((len(rows), N), dtype=torch.int32, device="cuda")
            a2 = torch.empty((len(rows), N), dtype=torch.int32, device="cuda")
            Ys = torch.empty((len(rows), N), dtype=torch.bfloat16, device="cuda")
            Ts = torch.empty((len(rows), r), dtype=torch.bfloat16, device="cuda")
            Q.quaff_qlinear_fwd(dev(Xq[rows]), dev(xqo[rows]), dev(dx[rows]), layer.Wq, layer.dW, layer.wq_O, layer.dw_O,
                                dev_bf16(Xs), layer.A, layer.B, scale, Ts, Ys, layer.ws, a1, a2, layer.status)
            torch.cuda.synchronize()
            assert np.array_equal(host(a1), o1), "main INT32 accumulator"
            assert np.array_equal(host(a2), o2), "outlier INT32 accumulator"


def test_phi3_attn_qkv_full_size_two_steps():
    _run_layer(synth.WORKLOADS["phi3_attn"], 0, steps=2, nsample=48, check_acc=True)


def test_phi3_attn_o_proj_full_size():
    _run_layer(synth.WORKLOADS["phi3_attn"], 1, steps=1, nsample=48, check_acc=True)


# LLaMA-2-7B block, 8192 tokens: one layer of each shape (q/k/v/o are 4096 -> 4096, gate/up 4096 -> 11008)
@pytest.mark.parametrize("li", [0, 4, 6], ids=["q_proj", "gate_proj", "down_proj"])
def test_llama7b_block_layers_full_size(li):
    _run_layer(synth.WORKLOADS["llama7b_block"], li, steps=1, nsample=24, check_acc=True, full_grads=False)


# The INT8 grad-input variant (not the paper's method) at full size, against its own oracle function
@pytest.mark.parametrize("wl_name,li", [("llama7b_block", 4), ("phi3_attn", 0)], ids=["llama_gate_proj", "phi3_qkv"])
def test_int8_grad_variant_full_size(wl_name, li):
    _run_layer(synth.WORKLOADS[wl_name], li, steps=1, nsample=24, check_acc=False, full_grads=False, int8_grad=True)


# The backward without a bf16 copy of the weight (codes expanded inside the grad-input GEMM) at full size
@pytest.mark.parametrize("wl_name,li", [("llama7b_block", 6), ("phi3_attn", 0)], ids=["llama_down_proj", "phi3_qkv"])
def test_in_kernel_expansion_full_size(wl_name, li):
    _run_layer(synth.WORKLOADS[wl_name], li, steps=1, nsample=24, check_acc=False, full_grads=False, lean_bwd=True)


# Phi-3 MLP, 4096 tokens: fused gate_up 3072 -> 16384 and down 8192 -> 3072, one forward + backward step each
@pytest.mark.parametrize("li", [0, 1], ids=["gate_up_proj", "down_proj"])
def test_phi3_mlp_layers_full_size(li):
    _run_layer(synth.WORKLOADS["phi3_mlp"], li, steps=1, nsample=24, check_acc=True, full_grads=False)


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


# Sixteen points of the shape sweep (tokens x K x N x rank x outlier fraction): together they take every value of every
# axis, and every pair of values of two axes - M in {512, 2048, 8192, 32768}, K and N in {2048, 4096, 8192}, rank in {8, 32, 64}, 0.5 / 1 / 5 % outlier
# channels.  5 % of 8192 is nO = 410 (nOp = 416 > 128: the forward with all three accumulators resident), 5 % of
# 2048 is nO = 102 (nOp = 128).
SWEEP_POINTS = [(512, 2048, 4096, 8, 0.05), (2048, 8192, 2048, 32, 0.01), (32768, 2048, 2048, 64, 0.005),
                (8192, 8192, 4096, 8, 0.05), (512, 4096, 8192, 64, 0.01), (2048, 4096, 4096, 32, 0.005),
                (8192, 2048, 8192, 32, 0.05), (32768, 4096, 2048, 8, 0.01), (512, 8192, 8192, 32, 0.005),
                (2048, 2048, 2048, 64, 0.05), (8192, 4096, 2048, 64, 0.005), (32768, 8192, 4096, 32, 0.01),
                (2048, 2048, 8192, 8, 0.005), (8192, 2048, 4096, 64, 0.01), (32768, 4096, 8192, 8, 0.05),
                (512, 8192, 2048, 64, 0.005)]


def test_sweep_points_cover_every_axis_value():
    for axis, want in ((0, {512, 2048, 8192, 32768}), (1, {2048, 4096, 8192}), (2, {2048, 4096, 8192}), (3, {8, 32, 64}),
                       (4, {0.005, 0.01, 0.05})):
        assert {p[axis] for p in SWEEP_POINTS} == want
    # ... and every PAIR of values of two different axes occurs together in some point
    import itertools
    axes = ((512, 2048, 8192, 32768), (2048, 4096, 8192), (2048, 4096, 8192), (8, 32, 64), (0.005, 0.01, 0.05))
    for a, b in itertools.combinations(range(5), 2):
        for va in axes[a]:
            for vb in axes[b]:
                assert any(p[a] == va and p[b] == vb for p in SWEEP_POINTS), (a, va, b, vb)


@pytest.mark.parametrize("M,K,N,r,frac", SWEEP_POINTS)
def test_shape_sweep_points(M, K, N, r, frac):
    """One forward + backward step of a sweep point through the graph-replayed layer, against the oracle."""
    wl = synth.sweep_point(M, K, N, r, frac)
    _run_layer(wl, 0, steps=1, nsample=16, check_acc=True, full_grads=False)


def test_tensors_larger_than_two_gib():
    """540672 tokens x 2048 channels: X, Y, dY and dX are 2.2 GB each and the INT8 codes 1.1 GB, so byte offsets of the
    later rows do not fit 32 bits (row 524288 starts at exactly 2^31 bytes).  The batch is a block of 8192 synthetic
    tokens repeated 66 times, each repetition scaled by another power of two (exact in bf16), so that a row fetched from
    or stored to a wrapped address would carry the wrong magnitude.  All codes and step sizes are compared, Y / dX on
    sampled rows on both sides of the 2^31-byte line, dA / dB on sampled columns over all tokens."""
    import dataclasses
    reps, block = 66, 8192
    wl = synth.sweep_point(reps * block, 2048, 2048, 8, 0.005)
    small = dataclasses.replace(wl, M=block)

    def tiled(wl_, li, step, lin):
        Xb, dYb = synth.step_inputs(small, li, step, lin)
        def rep(bits):
            expo = (bits >> 7) & 0xFF
            ok = (expo > 8) & (expo < 240)
            # x 1/4 .. x 4: the exponent field moves, nothing rounds
            scaled = [np.where(ok, (bits.astype(np.int32) + (shift << 7)).astype(np.uint16), bits) for shift in range(-2, 3)]
            out = np.empty((reps, block, bits.shape[1]), np.uint16)
            for t in range(reps):
                out[t] = scaled[t % 5]
            return out.reshape(reps * block, bits.shape[1])
        return rep(Xb), rep(dYb)

    line = (1 << 31) // (2 * 2048)                                   # first row whose byte offset needs 32 bits
    _run_layer(wl, 0, steps=1, nsample=24, check_acc=True, full_grads=False, step_inputs=tiled,
               extra_rows=(line - 1, line, line + 1, 2 * block + 5, reps * block - 2))
