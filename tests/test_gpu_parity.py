"""GPU parity: every C-ABI entry point against the CPU oracle on the same seeded inputs.
INT8 codes, INT32 accumulators, step sizes and scale factors must be bit-exact; dequantized
outputs and gradients within TOL_F32 (fp32 epilogue, no LoRA) or TOL_BF16 (bf16 / LoRA)."""
import numpy as np
import pytest

import oracle
from paper_2505_14742_b200 import synth
from util import TOL_BF16, TOL_F32, bf, check_bf16_intermediate, dev, dev_bf16, dx_floor, f32, host, host_bits, max_rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def Q():
    import torch
    from paper_2505_14742_b200 import binding, build
    build.build_library()
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def _mk_inputs(seed, M, K, N, nO, r, b_std=0.02, zero_rows=()):
    rng = np.random.default_rng(seed)
    O = np.sort(rng.permutation(K)[:nO]).astype(np.int32)
    x = rng.standard_normal((M, K)).astype(np.float32)
    if nO:
        x[:, O] *= rng.uniform(20, 100, nO).astype(np.float32)
    for z in zero_rows:
        x[z] = 0
    X = bf(x)
    Wt = bf(rng.standard_normal((N, K)).astype(np.float32) * 0.02)
    A = bf(rng.standard_normal((K, r)).astype(np.float32) * 0.02) if r else None
    B = bf(rng.standard_normal((r, N)).astype(np.float32) * b_std) if r else None
    dY = bf(rng.standard_normal((M, N)).astype(np.float32) * 1e-2)
    return O, X, Wt, A, B, dY


def _pad32(n):
    return (n + 31) // 32 * 32


# ----------------------------------------------------------------------------- S2 quant_act
@pytest.mark.parametrize("M,K,nO", [(1, 16, 0), (37, 136, 5), (64, 100, 3), (300, 3072, 32), (33, 11008, 55),
                                    (5, 20000, 200), (256, 512, 8)])
def test_quant_act_bit_exact(Q, M, K, nO):
    import torch
    O, X, _, _, _, _ = _mk_inputs(100 + M, M, K, 8, nO, 0, zero_rows=(0,) if M > 3 else ())
    rng = np.random.default_rng(7)
    s = (1.0 + 20.0 * rng.random(nO)).astype(np.float32)
    nOp = _pad32(nO)
    ldx = (K + 7) // 8 * 8 + 8
    ldxq = (K + 15) // 16 * 16 + 16
    Xd = torch.zeros((M, ldx), dtype=torch.bfloat16, device="cuda")
    Xd[:, :K] = dev_bf16(X)
    Xq = torch.full((M, ldxq), -128, dtype=torch.int8, device="cuda")
    xqo = torch.full((M, nOp + 16), -128, dtype=torch.int8, device="cuda") if nOp else None
    dx = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
    Q.quaff_quant_act(Xd[:, :K], dev(O) if nO else None, dev(s) if nO else None, Xq[:, :K],
                      xqo[:, :nOp] if nOp else None, dx)
    torch.cuda.synchronize()
    oXq, oxqo, odx = oracle.quant_act(X, O, s, nOp)
    assert np.array_equal(host(Xq[:, :K]), oXq)
    assert (host(Xq[:, K:]) == -128).all(), "wrote outside the row"
    assert np.array_equal(host(dx), odx)
    if nOp:
        assert np.array_equal(host(xqo[:, :nOp]), oxqo)
        assert (host(xqo[:, nOp:]) == -128).all()


# ----------------------------------------------------------------------------- S1 momentum
@pytest.mark.parametrize("M,K,nO,gamma", [(1, 64, 1, 0.5), (100, 256, 7, 0.9), (2048, 3072, 32, 0.2), (513, 1024, 100, 0.0)])
def test_momentum_update_bit_exact(Q, M, K, nO, gamma):
    import torch
    O, X, Wt, _, _, _ = _mk_inputs(200 + M, M, K, 16, nO, 0)
    _, _, _, wmax = oracle.prepare_weight(Wt, O)
    wmax[0] = 0.0 if nO > 1 else wmax[0]      # a zero weight row must give beta = 1
    s_host = np.ones(nO, np.float32)
    s_dev = dev(s_host.copy())
    cm = torch.empty(nO, dtype=torch.float32, device="cuda")
    be = torch.empty(nO, dtype=torch.float32, device="cuda")
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_MOMENTUM, M, K, 16, _pad32(nO), 0), dtype=torch.uint8, device="cuda")
    Xd = dev_bf16(X)
    for step in range(3):
        Q.quaff_momentum_update(Xd, dev(O), dev(wmax), gamma, s_dev, ws, cm, be)
        torch.cuda.synchronize()
        s_host, ocm, obe = oracle.momentum_update(X, O, wmax, gamma, s_host)
        assert np.array_equal(host(cm), ocm)
        assert np.array_equal(host(be), obe)
        assert np.array_equal(host(s_dev), s_host)


# ----------------------------------------------------------------------------- S3 requant + preprocessing
@pytest.mark.parametrize("nO,N", [(1, 16), (5, 136), (32, 3072), (100, 1000)])
def test_requant_weight_rows_bit_exact(Q, nO, N):
    import torch
    rng = np.random.default_rng(300 + nO)
    W_O = bf(rng.standard_normal((nO, N)).astype(np.float32) * 0.02)
    s = (1.0 + 10.0 * rng.random(nO)).astype(np.float32)
    s[0] = 1.0
    nOp = _pad32(nO)
    wq = torch.full((N, nOp), -128, dtype=torch.int8, device="cuda")
    dw = torch.empty(N, dtype=torch.float32, device="cuda")
    Q.quaff_requant_weight_rows(dev_bf16(W_O), dev(s), wq, dw)
    torch.cuda.synchronize()
    owq, odw = oracle.requant_weight_rows(W_O, s, nOp)
    assert np.array_equal(host(wq), owq)
    assert np.array_equal(host(dw), odw)


@pytest.mark.parametrize("N,K,nO", [(16, 32, 0), (136, 200, 5), (1000, 3072, 32)])
def test_prepare_weight_bit_exact(Q, N, K, nO):
    import torch
    O, _, Wt, _, _, _ = _mk_inputs(400 + N, 1, K, N, nO, 0)
    ldq = (K + 15) // 16 * 16
    Wq = torch.empty((N, ldq), dtype=torch.int8, device="cuda")
    dW = torch.empty(N, dtype=torch.float32, device="cuda")
    W_O = torch.empty((nO, N), dtype=torch.bfloat16, device="cuda") if nO else None
    wmax = torch.empty(nO, dtype=torch.float32, device="cuda") if nO else None
    Q.quaff_prepare_weight(dev_bf16(Wt), dev(O) if nO else None, Wq[:, :K], dW, W_O, wmax)
    torch.cuda.synchronize()
    oWq, odW, oW_O, owmax = oracle.prepare_weight(Wt, O)
    assert np.array_equal(host(Wq[:, :K]), oWq)
    assert np.array_equal(host(dW), odW)
    if nO:
        assert np.array_equal(host_bits(W_O), oW_O)
        assert np.array_equal(host(wmax), owmax)


# ----------------------------------------------------------------------------- S4 + S5 forward
def _oracle_state(O, X, Wt, gamma=0.0):
    Wq, dW, W_O, wmax = oracle.prepare_weight(Wt, O)
    nO = len(O)
    s, _, _ = oracle.momentum_update(X, O, wmax, gamma, np.ones(nO, np.float32))
    nOp = _pad32(nO)
    Xq, xqo, dx = oracle.quant_act(X, O, s, nOp)
    wq, dw = oracle.requant_weight_rows(W_O, s, nOp)
    return Wq, dW, W_O, wmax, s, Xq, xqo, dx, wq, dw


FWD_SHAPES = [(1, 128, 16, 0, 0), (128, 128, 128, 32, 16), (200, 320, 136, 5, 8), (256, 512, 512, 8, 8),
              (384, 1024, 640, 40, 16), (130, 2048, 296, 33, 64), (257, 384, 136, 0, 32), (100, 256, 256, 3, 0),
              (77, 256, 129, 7, 0), (520, 3072, 1032, 32, 16),
              (300, 1024, 392, 150, 16), (513, 640, 520, 128, 8),   # nOp > 128 or K < 4096: 128-column tiles, all accumulators in TMEM
              (130, 4096, 296, 33, 64), (300, 8192, 1032, 100, 16), (1, 4096, 64, 5, 16),
              # 192 to 222 tiles of 256 x 128 are three waves on the 74 CTA pairs, the same area in 256 x 192 tiles two:
              # these take the 192-column forward with the short accumulators in rounds (ragged M and N, LoRA only,
              # outliers only, r = 8, a single main k-block)
              (2048, 256, 3072, 33, 64), (2040, 384, 3016, 0, 32), (2048, 256, 3061, 7, 0), (2048, 128, 3072, 40, 8),
              (200, 11008, 520, 1100, 16)]   # the paper's 10 % budget of down_proj: nO = 1100 outlier channels


@pytest.mark.parametrize("M,K,N,nO,r", FWD_SHAPES)
@pytest.mark.parametrize("y_f32", [True, False])
def test_qlinear_fwd(Q, M, K, N, nO, r, y_f32):
    _check_fwd(Q, M, K, N, nO, r, y_f32)


# Each of the three forward kernels (128-, 192-, 256-column tiles) on the same shapes: several tiles per CTA pair
# (96 to 200 tiles on 74 pairs), ragged M and N, LoRA only, outliers only, a single main k-block, one tiny tile.
FORCED_SHAPES = [(2048, 256, 3072, 33, 64), (2040, 384, 3016, 0, 32), (2048, 256, 3061, 7, 0), (2048, 128, 6400, 40, 8),
                 (300, 1024, 392, 100, 16), (1, 128, 16, 5, 8), (520, 3072, 1032, 32, 16)]


@pytest.mark.parametrize("M,K,N,nO,r", FORCED_SHAPES)
@pytest.mark.parametrize("tile_n", [128, 192, 256])
def test_qlinear_fwd_each_tile_width(Q, M, K, N, nO, r, tile_n):
    Q.quaff_debug_force_fwd_tile(tile_n)
    try:
        _check_fwd(Q, M, K, N, nO, r, (M + tile_n) % 2 == 0)
    finally:
        Q.quaff_debug_force_fwd_tile(0)


def _check_fwd(Q, M, K, N, nO, r, y_f32, y_pad=0):
    import torch
    O, X, Wt, A, B, _ = _mk_inputs(500 + M + N, M, K, N, nO, r)
    Wq, dW, W_O, wmax, s, Xq, xqo, dx, wq, dw = _oracle_state(O, X, Wt)
    nOp = _pad32(nO)
    # Y is a view of a wider buffer with two more rows: whatever lands outside [M][N] shows in the sentinel
    SENT = -777.0
    Ybuf = torch.full((M + 2, N + y_pad), SENT, dtype=torch.float32 if y_f32 else torch.bfloat16, device="cuda")
    Y = Ybuf[:M, :N]
    a1 = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    a2 = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    T = torch.empty((M, r), dtype=torch.bfloat16, device="cuda") if r else None
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(256, Q.workspace_bytes(Q.QUAFF_WS_FWD, M, K, N, nOp, r)), dtype=torch.uint8, device="cuda")
    Q.quaff_qlinear_fwd(dev(Xq), dev(xqo) if nOp else None, dev(dx), dev(Wq), dev(dW), dev(wq) if nOp else None,
                        dev(dw), dev_bf16(X), dev_bf16(A) if r else None, dev_bf16(B) if r else None, 0.5,
                        T, Y, ws, a1, a2, st)
    torch.cuda.synchronize()
    assert host(st)[0] == 0, "device-side wait timed out"
    oY, oT, o1, o2 = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, A, B, 0.5)
    assert np.array_equal(host(a1), o1), "main INT32 accumulator"
    assert np.array_equal(host(a2), o2), "outlier INT32 accumulator"
    if r:
        # T: at most one bf16 ulp from the oracle's, entry by entry; Y is then checked against the oracle's
        # up-projection of the GPU's own T bits, so that no allowance for a differing rounding of T is needed
        Tg = host_bits(T)
        check_bf16_intermediate(Tg, oT, "LoRA down-projection T")
        oY = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, A, B, 0.5, T_in=Tg)[0]
    tol = TOL_F32 if (y_f32 and r == 0) else TOL_BF16
    err = max_rel_err(host(Y), oY)
    assert err <= tol, f"max rel err {err:.3e}"
    assert bool((Ybuf[M:, :] == SENT).all()) and bool((Ybuf[:, N:] == SENT).all()), "write outside Y"


# Row pitches of Y that take the three store paths of the wide forward kernels: 32-byte stores (pitch a multiple of 32
# bytes), 16-byte stores (a multiple of 16 only), element stores (neither); ragged M and N.
@pytest.mark.parametrize("tile_n", [128, 192, 256])
@pytest.mark.parametrize("y_f32,y_pad", [(False, 16), (False, 8), (False, 3), (True, 8), (True, 4), (True, 1)])
def test_qlinear_fwd_padded_output(Q, tile_n, y_f32, y_pad):
    Q.quaff_debug_force_fwd_tile(tile_n)
    try:
        _check_fwd(Q, 300, 512, 1000, 20, 16, y_f32, y_pad)
    finally:
        Q.quaff_debug_force_fwd_tile(0)


# ----------------------------------------------------------------------------- S6-S8 backward
BWD_SHAPES = [(1, 128, 64, 0, 0), (128, 128, 128, 32, 16), (200, 320, 136, 5, 8), (256, 512, 512, 8, 8),
              (384, 640, 1024, 40, 16), (130, 300 // 4 * 4 + 4, 2048, 33, 64), (100, 256, 256, 3, 0),
              (520, 1032, 3072, 32, 16), (300, 2056, 520, 70, 32),
              (200, 11008, 520, 1100, 16)]   # 10 % outlier budget: 2 x 1120 columns of outlier partial products


@pytest.mark.parametrize("M,K,N,nO,r", BWD_SHAPES)
def test_qlinear_bwd(Q, M, K, N, nO, r):
    _check_bwd(Q, M, K, N, nO, r)


# Shapes nobody picked by hand: seeded draws over the supported ranges (ragged everything; K a multiple of 16 and N of 8,
# which the row pitches of the contiguous test buffers need), each through the forward and through both backward paths.
def _random_shape(seed):
    rng = np.random.default_rng(9000 + seed)
    M = int(rng.integers(1, 601))
    K = 16 * int(rng.integers(1, 121))
    N = 8 * int(rng.integers(1, 241))
    nO = int(rng.integers(0, min(K, 140) + 1)) if seed % 4 else 0
    r = 8 * int(rng.integers(0, 9)) if seed % 5 else 0
    return M, K, N, nO, r


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_forward_and_backward(Q, seed):
    M, K, N, nO, r = _random_shape(seed)
    _check_fwd(Q, M, K, N, nO, r, seed % 2 == 0)
    _check_bwd(Q, M, K, N, nO, r)
    if N % 16 == 0:                       # the INT8 grad-input variant takes rows of whole 16-column units
        test_qlinear_bwd_int8(Q, M, K, N, nO, r)


def _check_bwd(Q, M, K, N, nO, r):
    import torch
    K = (K + 7) // 8 * 8
    O, X, Wt, A, B, dY = _mk_inputs(600 + M + N, M, K, N, nO, r)
    Wq, dW, W_O, wmax, s, Xq, xqo, dx, wq, dw = _oracle_state(O, X, Wt)
    nOp = _pad32(nO)
    oY, oT, _, _ = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, A, B, 0.5)
    odX, odA, odB, oG = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, oT, A, B, 0.5)
    dXbuf = torch.full((M + 2, K + 8), -777.0, dtype=torch.bfloat16, device="cuda")     # dX: a view with a sentinel frame
    dX = dXbuf[:M, :K]
    dA = torch.full((K, r), 1.0, dtype=torch.float32, device="cuda") if r else None
    dB = torch.full((r, N), 1.0, dtype=torch.float32, device="cuda") if r else None
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_BWD, M, K, N, nOp, r), dtype=torch.uint8, device="cuda")
    Wq_d = torch.zeros((N, (K + 15) // 16 * 16), dtype=torch.int8, device="cuda")   # row pitch: a multiple of 16
    Wq_d[:, :K] = dev(Wq)
    args = (dev_bf16(dY), Wq_d[:, :K], dev(dW), dev(wq) if nOp else None, dev(dw), dev(O) if nO else None,
            dev(s) if nO else None, dev_bf16(X), dev_bf16(oT) if r else None, dev_bf16(A) if r else None,
            dev_bf16(B) if r else None, 0.5, dX, dA, dB)
    Gd = torch.full((M, r), float("nan"), dtype=torch.bfloat16, device="cuda") if r else None
    Q.quaff_qlinear_bwd(*args, False, ws, st, Gd)
    torch.cuda.synchronize()
    assert host(st)[0] == 0
    if r:
        # G: at most one bf16 ulp from the oracle's, entry by entry; everything downstream of G is then compared with
        # the oracle evaluated on the GPU's own G bits (T is the oracle's on both sides already): no allowance
        Gg = host_bits(Gd)
        check_bf16_intermediate(Gg, oG, "G = bf16(scale dY B^T)")
        odX, odA, odB, _ = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, oT, A, B, 0.5, G_in=Gg)
    err = max_rel_err(host(dX), odX, dx_floor(N))
    assert err <= TOL_BF16, f"dX max rel err {err:.3e}"
    assert bool((dXbuf[M:, :] == -777.0).all()) and bool((dXbuf[:, K:] == -777.0).all()), "write outside dX"
    if nO:
        err_o = max_rel_err(host(dX)[:, O], odX[:, O], dx_floor(N))
        assert err_o <= TOL_BF16, f"dX outlier columns max rel err {err_o:.3e}"
    if r:
        err_a, err_b = max_rel_err(host(dA), odA), max_rel_err(host(dB), odB)
        assert err_a <= TOL_BF16 and err_b <= TOL_BF16, f"dA {err_a:.3e} dB {err_b:.3e}"
    # The same call with a workspace that has no room for a bf16 copy of the weight: the grad-input GEMM then expands the
    # INT8 codes inside the kernel.  Same products in the same order: bit-identical off the outlier columns (those differ
    # in how the two partial products are separated), the same gradients, and within tolerance of the oracle everywhere.
    lean = Q.workspace_bytes(Q.QUAFF_WS_BWD_LEAN, M, K, N, nOp, r)
    assert lean < Q.workspace_bytes(Q.QUAFF_WS_BWD, M, K, N, nOp, r)
    ws_lean = torch.empty(lean, dtype=torch.uint8, device="cuda")
    dXl = torch.full((M + 2, K + 8), -777.0, dtype=torch.bfloat16, device="cuda")
    dAl, dBl = (torch.full_like(dA, 3.0), torch.full_like(dB, 3.0)) if r else (None, None)
    Q.quaff_qlinear_bwd(*args[:12], dXl[:M, :K], dAl, dBl, False, ws_lean, st)
    torch.cuda.synchronize()
    assert host(st)[0] == 0
    assert bool((dXl[M:, :] == -777.0).all()) and bool((dXl[:, K:] == -777.0).all()), "write outside dX (in-kernel expansion)"
    off_O = np.setdiff1d(np.arange(K), O)
    assert np.array_equal(host_bits(dXl[:M, :K].contiguous())[:, off_O], host_bits(dX.contiguous())[:, off_O]), "in-kernel expansion: dX bits"
    err = max_rel_err(host(dXl[:M, :K]), odX, dx_floor(N))
    assert err <= TOL_BF16, f"dX (in-kernel expansion) max rel err {err:.3e}"
    if r:
        assert np.array_equal(host(dAl), host(dA)) and np.array_equal(host(dBl), host(dB))
    # the two halves of the call on their own (other stream layout inside the library): the same kernels, the same bits
    dX2 = torch.full((M, K), float("nan"), dtype=torch.bfloat16, device="cuda")
    Q.quaff_qlinear_bwd(*args[:12], dX2, None, None, False, ws, st)            # dX only
    torch.cuda.synchronize()
    assert host(st)[0] == 0 and np.array_equal(host_bits(dX2), host_bits(dX.contiguous()))
    if r:
        dA2, dB2 = torch.full_like(dA, 2.0), torch.full_like(dB, 2.0)
        Q.quaff_qlinear_bwd(*args[:12], None, dA2, dB2, False, ws, st)         # LoRA gradients only
        torch.cuda.synchronize()
        assert host(st)[0] == 0 and np.array_equal(host(dA2), host(dA)) and np.array_equal(host(dB2), host(dB))
        # gradient accumulation: a second call with accumulate adds the same gradients again
        Q.quaff_qlinear_bwd(*args, True, ws, st)
        torch.cuda.synchronize()
        assert max_rel_err(host(dA), 2 * odA) <= TOL_BF16
        assert max_rel_err(host(dB), 2 * odB) <= TOL_BF16


# ----------------------------------------------------------------------------- whole path, several steps
def test_tiny_workload_all_steps(Q):
    """Configuration 'tiny': 10 iterations of forward + backward with drifting outliers and the
    momentum state carried across steps; everything is compared at every step.  LoRA B is non-zero
    so that the LoRA branch contributes."""
    import torch
    from paper_2505_14742_b200.layer import QuaffLinear
    wl = synth.WORKLOADS["tiny"]
    lin = synth.layer_inputs(wl, 0, b_std=0.02)
    sp = lin.spec
    scale = wl.lora_alpha / sp.r
    layer = QuaffLinear(dev_bf16(lin.W), dev(lin.O_idx), dev_bf16(lin.A), dev_bf16(lin.B), scale, wl.gamma, wl.M,
                        y_dtype=torch.bfloat16, debug_acc=True, keep_G=True)
    Wq, dW, W_O, wmax = oracle.prepare_weight(lin.W, lin.O_idx)
    s = np.ones(sp.nO, np.float32)
    nOp = _pad32(sp.nO)
    for step in range(wl.steps):
        X, dY = synth.step_inputs(wl, 0, step, lin)
        Y = layer.forward(dev_bf16(X))
        dX, dA, dB = layer.backward(dev_bf16(dY))
        torch.cuda.synchronize()
        assert host(layer.status)[0] == 0
        s, _, _ = oracle.momentum_update(X, lin.O_idx, wmax, wl.gamma, s)
        Xq, xqo, dx = oracle.quant_act(X, lin.O_idx, s, nOp)
        wq, dw = oracle.requant_weight_rows(W_O, s, nOp)
        oY, oT, o1, o2 = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, lin.A, lin.B, scale)
        _, _, _, oG = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, lin.O_idx, s, X, oT, lin.A, lin.B, scale, want_dX=False, want_dAB=False)
        Tg, Gg = host_bits(layer.T), host_bits(layer.G)
        check_bf16_intermediate(Tg, oT, f"T at step {step}")
        check_bf16_intermediate(Gg, oG, f"G at step {step}")
        oY = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, lin.A, lin.B, scale, T_in=Tg)[0]
        odX, odA, odB, _ = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, lin.O_idx, s, X, Tg, lin.A, lin.B, scale, G_in=Gg)
        assert np.array_equal(host(layer.s_O), s), f"s_O at step {step}"
        assert np.array_equal(host(layer.Xq), Xq) and np.array_equal(host(layer.xq_O), xqo)
        assert np.array_equal(host(layer.dx), dx)
        assert np.array_equal(host(layer.wq_O), wq) and np.array_equal(host(layer.dw_O), dw)
        assert np.array_equal(host(layer.acc_main), o1) and np.array_equal(host(layer.acc_out), o2)
        assert max_rel_err(host(Y), oY) <= TOL_BF16
        assert max_rel_err(host(dX), odX) <= TOL_BF16
        assert max_rel_err(host(dA), odA) <= TOL_BF16 and max_rel_err(host(dB), odB) <= TOL_BF16


# ----------------------------------------------------------------------------- host-side validation (no launch)
def test_argument_validation(Q):
    import torch
    M, K, N = 32, 64, 48
    X = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    Xq = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    dx = torch.zeros(M, dtype=torch.float32, device="cuda")
    with pytest.raises(Q.QuaffError) as e:
        Q.quaff_quant_act(X[:, 1:], None, None, Xq[:, 1:], None, dx)          # misaligned base
    assert e.value.code == Q.QUAFF_ERR_ALIGNMENT
    O = torch.arange(70, dtype=torch.int32, device="cuda")
    with pytest.raises(Q.QuaffError) as e:
        Q.quaff_quant_act(X, O, dx, Xq, torch.zeros((M, 96), dtype=torch.int8, device="cuda"), dx)   # nO > K
    assert e.value.code == Q.QUAFF_ERR_INVALID_ARG
    with pytest.raises(Q.QuaffError) as e:
        Q.quaff_momentum_update(X, O[:4], dx, 1.5, dx, torch.zeros(256, dtype=torch.uint8, device="cuda"))  # gamma
    assert e.value.code == Q.QUAFF_ERR_INVALID_ARG
    with pytest.raises(Q.QuaffError) as e:
        Q.quaff_momentum_update(X, O[:4], dx, 0.5, dx, torch.zeros(8, dtype=torch.uint8, device="cuda"))
    assert e.value.code == Q.QUAFF_ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()


# ----------------------------------------------------------------------------- split scale update (token shards)
def test_split_momentum_update_matches_the_whole_batch(Q):
    """Column maxima per shard (quaff_outlier_colmax), elementwise maximum (what a MAX all-reduce does), then
    quaff_momentum_apply: the same s_O, bit for bit, as quaff_momentum_update on the whole batch and as the oracle."""
    import torch
    M, K, nO, gamma = 1000, 768, 37, 0.2
    O, X, Wt, _, _, _ = _mk_inputs(901, M, K, 16, nO, 0)
    _, _, _, wmax = oracle.prepare_weight(Wt, O)
    Xd, Od, wd = dev_bf16(X), dev(O), dev(wmax)
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_MOMENTUM, M, K, 16, _pad32(nO), 0), dtype=torch.uint8, device="cuda")
    s_whole, s_split = dev(np.full(nO, 1.5, np.float32)), dev(np.full(nO, 1.5, np.float32))
    cm_whole = torch.empty(nO, dtype=torch.float32, device="cuda")
    Q.quaff_momentum_update(Xd, Od, wd, gamma, s_whole, ws, cm_whole)
    shards = [(0, 300), (300, 301), (301, M)]
    cms = []
    for a, b in shards:
        cm = torch.full((nO,), -1.0, dtype=torch.float32, device="cuda")
        Q.quaff_outlier_colmax(Xd[a:b], Od, cm, ws)
        torch.cuda.synchronize()
        assert np.array_equal(host(cm), oracle.outlier_colmax(X[a:b], O))
        cms.append(cm)
    combined = torch.maximum(torch.maximum(cms[0], cms[1]), cms[2])
    be = torch.empty(nO, dtype=torch.float32, device="cuda")
    Q.quaff_momentum_apply(combined, wd, gamma, s_split, be)
    torch.cuda.synchronize()
    assert np.array_equal(host(combined), host(cm_whole))
    assert np.array_equal(host(s_split), host(s_whole))
    s_or, _, be_or = oracle.momentum_update(X, O, wmax, gamma, np.full(nO, 1.5, np.float32))
    assert np.array_equal(host(s_split), s_or) and np.array_equal(host(be), be_or)


# ----------------------------------------------------------------------------- two host threads, two streams
def test_backward_from_two_host_threads_is_bit_identical_to_serial(Q):
    """Two host threads, each with its own stream, buffers and workspace, call forward + backward at the same time
    (the library's lazily created per-device resources and the side streams of the backward are shared): every
    output equals the serial run's, bit for bit."""
    import threading
    import torch
    M, K, N, nO, r = 640, 1024, 1536, 12, 16
    cases = []
    for seed in (31, 32):
        O, X, Wt, A, B, dY = _mk_inputs(seed, M, K, N, nO, r)
        Wq, dW, W_O, wmax, s, Xq, xqo, dx, wq, dw = _oracle_state(O, X, Wt)
        nOp = _pad32(nO)
        d = dict(Xq=dev(Xq), xqo=dev(xqo), dx=dev(dx), Wq=dev(Wq), dW=dev(dW), wq=dev(wq), dw=dev(dw), X=dev_bf16(X), A=dev_bf16(A),
                 B=dev_bf16(B), dY=dev_bf16(dY), O=dev(O), s=dev(s),
                 ws=torch.empty(max(Q.workspace_bytes(Q.QUAFF_WS_FWD, M, K, N, nOp, r), Q.workspace_bytes(Q.QUAFF_WS_BWD, M, K, N, nOp, r)),
                                dtype=torch.uint8, device="cuda"),
                 st=torch.zeros(4, dtype=torch.int32, device="cuda"))
        cases.append(d)

    def run(d, out):
        T = torch.empty((M, r), dtype=torch.bfloat16, device="cuda")
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dA = torch.empty((K, r), dtype=torch.float32, device="cuda")
        dB = torch.empty((r, N), dtype=torch.float32, device="cuda")
        for _ in range(out["reps"]):
            Q.quaff_qlinear_fwd(d["Xq"], d["xqo"], d["dx"], d["Wq"], d["dW"], d["wq"], d["dw"], d["X"], d["A"], d["B"], 0.5, T, Y, d["ws"],
                                None, None, d["st"])
            Q.quaff_qlinear_bwd(d["dY"], d["Wq"], d["dW"], d["wq"], d["dw"], d["O"], d["s"], d["X"], T, d["A"], d["B"], 0.5, dX, dA, dB,
                                False, d["ws"], d["st"])
        out["res"] = (Y, dX, dA, dB)

    serial = []
    for d in cases:
        o = {"reps": 1}
        run(d, o)
        torch.cuda.synchronize()
        serial.append([host(t) for t in o["res"]])

    outs = [{"reps": 20}, {"reps": 20}]
    errors = []

    def worker(i):
        try:
            with torch.cuda.stream(torch.cuda.Stream()):
                run(cases[i], outs[i])
                torch.cuda.current_stream().synchronize()
        except Exception as e:  # noqa: BLE001
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for i in range(2):
        assert host(cases[i]["st"])[0] == 0
        for got, ref in zip(outs[i]["res"], serial[i]):
            assert np.array_equal(host(got), ref)


# ----------------------------------------------------------------------------- INT8 grad-input variant (not the paper's method)
@pytest.mark.parametrize("M,N", [(1, 16), (37, 144), (300, 3072), (64, 11008), (19, 16384), (5, 9232)])
def test_quant_grad_bit_exact(Q, M, N):
    import torch
    rng = np.random.default_rng(700 + M)
    dY = bf(rng.standard_normal((M, N)).astype(np.float32) * 1e-2)
    if M > 3:
        dY[2] = 0
    dW = (rng.random(N).astype(np.float32) + 0.01) * 1e-3
    ld = N + 16
    Zq = torch.full((M, ld), -128, dtype=torch.int8, device="cuda")
    dz = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
    Q.quaff_quant_grad(dev_bf16(dY), dev(dW), Zq[:, :N], dz)
    torch.cuda.synchronize()
    oZq, odz = oracle.quant_grad(dY, dW)
    assert np.array_equal(host(Zq[:, :N]), oZq)
    assert (host(Zq[:, N:]) == -128).all(), "wrote outside the row"
    assert np.array_equal(host(dz), odz)


@pytest.mark.parametrize("seed", range(16))
def test_random_shapes_of_the_bit_exact_kernels(Q, seed):
    """Seeded draws over the supported sizes for the integer-exact steps: the row width decides how many 16-column units a
    thread holds and whether the ragged-tail variant runs, so widths nobody picked by hand are the point."""
    rng = np.random.default_rng(7000 + seed)
    M = int(rng.integers(1, 301))
    K = int(rng.integers(1, 32769)) if seed % 2 else int(rng.integers(1, 4097))
    nO = int(rng.integers(0, min(K, 300) + 1))
    test_quant_act_bit_exact(Q, M, K, nO)
    test_momentum_update_bit_exact(Q, M, K, max(1, nO), float(rng.integers(0, 11)) / 10.0)
    test_requant_weight_rows_bit_exact(Q, max(1, nO), int(rng.integers(1, 5001)))
    Kw = max(8, min(K, 4096) // 8 * 8)            # the contiguous bf16 weight of that test needs a row pitch of 16 bytes
    test_prepare_weight_bit_exact(Q, int(rng.integers(1, 1201)), Kw, min(nO, Kw))
    test_quant_grad_bit_exact(Q, M, 16 * int(rng.integers(1, 1025)))


def test_quant_grad_rejects_rows_wider_than_it_is_built_for(Q):
    import torch
    dY = torch.zeros((2, 16400), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Q.QuaffError) as e:
        Q.quaff_quant_grad(dY, torch.ones(16400, device="cuda"), torch.empty((2, 16400), dtype=torch.int8, device="cuda"), torch.empty(2, device="cuda"))
    assert e.value.code == Q.QUAFF_ERR_UNSUPPORTED_SHAPE


def test_empty_batch_launches_nothing_and_stores_the_empty_sums(Q):
    """M = 0 is a valid batch: sizes are defined, no output row is touched, and a backward call that does not
    accumulate stores dA = 0 and dB = 0 (sums over no tokens); one that accumulates leaves them alone."""
    import torch
    K, N, nO, nOp, r = 256, 128, 5, 32, 16
    for which in range(8):
        assert 0 <= Q.workspace_bytes(which, 0, K, N, nOp, r) < (1 << 24)
    dev = "cuda"
    u8 = lambda *sh: torch.full(sh, 0x5A, dtype=torch.uint8, device=dev)
    Xq, xqo, Wq, wqo = u8(1, K), u8(1, nOp), u8(N, K), u8(N, nOp)
    dx, dW, dwo, s = (torch.ones(n, device=dev) for n in (1, N, N, nO))
    O = torch.arange(nO, dtype=torch.int32, device=dev)
    bfz = lambda *sh: torch.full(sh, 7.0, dtype=torch.bfloat16, device=dev)
    X, A, B, T, Y, dY, dX = bfz(1, K), bfz(K, r), bfz(r, N), bfz(1, r), bfz(1, N), bfz(1, N), bfz(1, K)
    dA, dB = torch.full((K, r), 3.0, device=dev), torch.full((r, N), 3.0, device=dev)
    ws = torch.empty(max(Q.workspace_bytes(w, 1, K, N, nOp, r) for w in range(8)) + 256, dtype=torch.uint8, device=dev)
    L, p, st = Q.lib(), (lambda t: t.data_ptr()), torch.cuda.current_stream().cuda_stream
    n0 = Q.quaff_debug_launch_count()
    assert L.quaff_quant_act(p(X), K, 0, K, p(O), nO, p(s), p(Xq), K, p(xqo), nOp, nOp, p(dx), st) == 0
    assert L.quaff_lora_down(p(X), K, 0, K, p(A), r, p(T), None, p(ws), ws.numel(), st) == 0
    assert L.quaff_qlinear_fwd(0, K, N, p(Xq), K, p(xqo), nOp, nOp, p(dx), p(Wq), K, p(dW), p(wqo), nOp, p(dwo), p(X), K, p(A), p(B),
                               r, 2.0, p(T), p(Y), Q.QUAFF_BF16, N, None, None, None, p(ws), ws.numel(), st) == 0
    bwd_args = lambda acc: (0, K, N, p(dY), N, p(Wq), K, p(dW), p(wqo), nOp, p(dwo), nOp, p(O), nO, p(s), p(X), K, p(T), p(A), p(B), r,
                            2.0, p(dX), K, p(dA), p(dB), acc, None)
    assert L.quaff_qlinear_bwd(*bwd_args(1), None, p(ws), ws.numel(), st) == 0
    assert L.quaff_qlinear_bwd_int8(*bwd_args(1), None, None, p(ws), ws.numel(), st) == 0
    assert Q.quaff_debug_launch_count() == n0                 # nothing launched so far
    torch.cuda.synchronize()
    assert float(dA.min()) == 3.0 and float(dB.max()) == 3.0  # accumulate: untouched
    for t in (Xq, xqo):
        assert int(t.min()) == 0x5A
    for t in (T, Y, dX):
        assert float(t.float().min()) == 7.0
    assert L.quaff_qlinear_bwd(*bwd_args(0), None, p(ws), ws.numel(), st) == 0
    torch.cuda.synchronize()
    assert float(dA.abs().max()) == 0.0 and float(dB.abs().max()) == 0.0
    dA.fill_(3.0); dB.fill_(3.0)
    assert L.quaff_qlinear_bwd_int8(*bwd_args(0), None, None, p(ws), ws.numel(), st) == 0
    torch.cuda.synchronize()
    assert float(dA.abs().max()) == 0.0 and float(dB.abs().max()) == 0.0
    assert float(dX.float().min()) == 7.0
    # Eq. 8 over no tokens: the column maxima are 0, beta = 1, and Eq. 7 moves s towards 1 (s = 2, gamma = 0.5: 1.5)
    s2, wmax = torch.full((nO,), 2.0, device=dev), torch.ones(nO, device=dev)
    cm, be = torch.full((nO,), -1.0, device=dev), torch.full((nO,), -1.0, device=dev)
    assert L.quaff_momentum_update(p(X), K, 0, K, p(O), nO, p(wmax), 0.5, p(s2), p(cm), p(be), p(ws), ws.numel(), st) == 0
    torch.cuda.synchronize()
    assert s2.tolist() == [1.5] * nO and cm.tolist() == [0.0] * nO and be.tolist() == [1.0] * nO
    os_, ocm, obe = oracle.momentum_update(np.zeros((0, K), np.uint16), np.arange(nO, dtype=np.int32), np.ones(nO, np.float32), 0.5,
                                           np.full(nO, 2.0, np.float32))
    assert os_.tolist() == [1.5] * nO and ocm.tolist() == [0.0] * nO and obe.tolist() == [1.0] * nO


BWD8_SHAPES = [(1, 128, 64, 0, 0), (128, 128, 128, 32, 16), (200, 320, 144, 5, 8), (256, 512, 512, 8, 8),
               (384, 640, 1024, 40, 16), (130, 304, 2048, 33, 64), (100, 256, 256, 3, 0), (520, 1032, 3072, 32, 16),
               (300, 2056, 528, 70, 32), (200, 11008, 528, 1100, 16), (2048, 1000, 1536, 20, 64)]


@pytest.mark.parametrize("M,K,N,nO,r", BWD8_SHAPES)
def test_qlinear_bwd_int8(Q, M, K, N, nO, r):
    """quaff_qlinear_bwd_int8 against its own oracle function: INT32 accumulators bit for bit, G within one ulp, dX, dA,
    dB against the oracle evaluated on the GPU's G bits."""
    import torch
    K = (K + 7) // 8 * 8
    O, X, Wt, A, B, dY = _mk_inputs(800 + M + N, M, K, N, nO, r)
    Wq, dW, W_O, wmax, s, Xq, xqo, dx, wq, dw = _oracle_state(O, X, Wt)
    nOp = _pad32(nO)
    oT = oracle.lora_down(X, A) if r else None
    dXbuf = torch.full((M + 2, K + 8), -777.0, dtype=torch.bfloat16, device="cuda")
    dX = dXbuf[:M, :K]
    dA = torch.full((K, r), 1.0, dtype=torch.float32, device="cuda") if r else None
    dB = torch.full((r, N), 1.0, dtype=torch.float32, device="cuda") if r else None
    Gd = torch.full((M, r), float("nan"), dtype=torch.bfloat16, device="cuda") if r else None
    acc = torch.full((M, K), -7, dtype=torch.int32, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_BWD_INT8, M, K, N, nOp, r), dtype=torch.uint8, device="cuda")
    Wq_d = torch.zeros((N, (K + 15) // 16 * 16), dtype=torch.int8, device="cuda")
    Wq_d[:, :K] = dev(Wq)
    Q.quaff_qlinear_bwd_int8(dev_bf16(dY), Wq_d[:, :K], dev(dW), dev(wq) if nOp else None, dev(dw), dev(O) if nO else None,
                             dev(s) if nO else None, dev_bf16(X), dev_bf16(oT) if r else None, dev_bf16(A) if r else None,
                             dev_bf16(B) if r else None, 0.5, dX, dA, dB, False, ws, st, Gd, acc)
    torch.cuda.synchronize()
    assert host(st)[0] == 0
    Gg = host_bits(Gd) if r else None
    odX, odA, odB, oG, oZq, odz, oacc = oracle.qlinear_bwd_int8(dY, Wq, dW, wq, dw, O, s, X, oT, A, B, 0.5, G_in=Gg)
    assert np.array_equal(host(acc), oacc), "INT32 accumulator of the grad-input"
    if r:
        check_bf16_intermediate(Gg, oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, oT, A, B, 0.5, want_dX=False, want_dAB=False)[3], "G")
    err = max_rel_err(host(dX), odX)
    assert err <= TOL_BF16, f"dX max rel err {err:.3e}"
    assert bool((dXbuf[M:, :] == -777.0).all()) and bool((dXbuf[:, K:] == -777.0).all()), "write outside dX"
    if nO:
        err_o = max_rel_err(host(dX)[:, O], odX[:, O], dx_floor(N))
        assert err_o <= TOL_BF16, f"dX outlier columns max rel err {err_o:.3e}"
    if r:
        err_a, err_b = max_rel_err(host(dA), odA), max_rel_err(host(dB), odB)
        assert err_a <= TOL_BF16 and err_b <= TOL_BF16, f"dA {err_a:.3e} dB {err_b:.3e}"


# ----------------------------------------------------------------------------- state: determinism and checkpoint / resume
def test_checkpoint_resume_and_determinism(Q):
    """The only state a layer carries between steps is s_O (a caller-owned buffer).  Ten steps in one go, and five steps +
    a copy of s_O into a fresh layer + five more steps, end in the same bits everywhere (s_O, codes, Y, dX, dA, dB); so does
    a second run of the ten steps (no floating-point atomics, fixed split-K reduction order)."""
    import torch
    from paper_2505_14742_b200.layer import QuaffLinear
    wl = synth.WORKLOADS["tiny"]
    lin = synth.layer_inputs(wl, 0, b_std=0.02)
    scale = wl.lora_alpha / lin.spec.r

    def make():
        return QuaffLinear(dev_bf16(lin.W), dev(lin.O_idx), dev_bf16(lin.A), dev_bf16(lin.B), scale, wl.gamma, wl.M)

    def run(layer, steps):
        out = None
        for step in steps:
            X, dY = synth.step_inputs(wl, 0, step, lin)
            Y = layer.forward(dev_bf16(X))
            dX, dA, dB = layer.backward(dev_bf16(dY))
            torch.cuda.synchronize()
            out = [host(layer.s_O), host(layer.Xq), host(layer.wq_O), host_bits(Y), host_bits(dX), host(dA), host(dB)]
        return out

    straight = run(make(), range(10))
    again = run(make(), range(10))
    first = make()
    run(first, range(5))
    saved = first.s_O.clone()                     # the checkpoint
    resumed = make()
    resumed.s_O.copy_(saved)
    split = run(resumed, range(5, 10))
    for a, b, c in zip(straight, again, split):
        assert np.array_equal(a, b), "two runs of the same steps differ"
        assert np.array_equal(a, c), "resuming from a saved s_O differs"
