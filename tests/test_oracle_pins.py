"""Pins of the CPU oracle against things other than itself: hand-computed codes (Eq. 1),
closed forms of the momentum update (Eq. 7-8), brute force in Python integers, cases where
the quantized forward (Eq. 9) must equal the exact product, the rounding error bound,
numpy float64 products for the LoRA branch and finite differences for the backward."""
import os

import numpy as np
import pytest

import oracle
from paper_2505_14742_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f32(b):
    return synth.bf16_bits_to_f32(b)


def half_ulp_bf16(t):
    """Half a unit in the last place of bf16 (8 significant bits) at the magnitude of t."""
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(t), 1e-300))) - 8)


def rand_bf(rng, shape, scale=1.0):
    return bf(rng.standard_normal(shape).astype(np.float32) * scale)


# ----------------------------------------------------------------------------- Eq. 1
def _golden_rows():
    rows = []
    for line in open(os.path.join(GOLD, "quant_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        a, b, c = line.split("|")
        rows.append(([float(v) for v in a.split()], [int(v) for v in b.split()], float(c)))
    return rows


@pytest.mark.parametrize("xs,codes,num", _golden_rows())
def test_quant_hand_examples_per_token(xs, codes, num):
    X = bf([xs])
    assert np.array_equal(f32(X)[0], np.float32(xs)), "example must be exact in bf16"
    Xq, xqo, dx = oracle.quant_act(X, np.zeros(0, np.int32), np.zeros(0, np.float32), 0)
    assert Xq[0].tolist() == codes
    assert dx[0] == np.float32(num) / np.float32(127.0)


@pytest.mark.parametrize("xs,codes,num", _golden_rows())
def test_quant_hand_examples_per_output_channel(xs, codes, num):
    # the same rows as a weight: row n of Wt is quantized with its own step size
    Wt = bf([xs, [0.0] * len(xs)])
    Wq, dW, W_O, wmax = oracle.prepare_weight(Wt, np.zeros(0, np.int32))
    assert Wq[0].tolist() == codes and Wq[1].tolist() == [0] * len(xs)
    assert dW[0] == np.float32(num) / np.float32(127.0) and dW[1] == 0.0


def test_quant_outlier_column_is_divided_by_s():
    # x = 100 on the outlier channel, s = 50 -> xhat = 2; the row maximum becomes 4 (channel 0)
    X = bf([[4.0, 100.0, 1.0, -2.0]])
    Xq, xqo, dx = oracle.quant_act(X, np.array([1], np.int32), np.array([50.0], np.float32), 4)
    # r = 127/4 = 31.75: 4 -> 127, 2 -> 63.5 -> 64 (tie to even), 1 -> 31.75 -> 32, -2 -> -63.5 -> -64
    assert Xq[0].tolist() == [127, 64, 32, -64]
    assert xqo[0].tolist() == [64, 0, 0, 0]
    assert dx[0] == np.float32(4.0) / np.float32(127.0)


def test_quant_invariants_random():
    rng = np.random.default_rng(1)
    X = rand_bf(rng, (37, 129))
    X[5] = 0
    O = np.array([3, 77, 128], np.int32)
    s = np.array([1.5, 7.0, 1.0], np.float32)
    Xq, xqo, dx, nd = oracle.quant_act(X, O, s, 8, count_literal=True)
    assert Xq.min() >= -127 and Xq.max() <= 127
    amax = np.abs(Xq.astype(np.int32)).max(axis=1)
    assert (amax[np.arange(37) != 5] == 127).all() and amax[5] == 0 and dx[5] == 0
    assert np.array_equal(xqo[:, :3], Xq[:, O]) and (xqo[:, 3:] == 0).all()
    # Eq. 1 literally divides by Delta; multiplying by 127/amax may flip a rare tie only
    assert nd <= 2
    # step size: the largest |xhat| of the row over 127
    xh = f32(X).astype(np.float64)
    xh[:, O] = (f32(X)[:, O] / s[None, :]).astype(np.float64)
    assert np.allclose(dx, np.abs(xh).max(axis=1) / 127.0, rtol=1e-6)
    # codes are the nearest integers of xhat / Delta
    nz = dx > 0
    assert np.abs(Xq[nz] - xh[nz] / dx[nz, None].astype(np.float64)).max() <= 0.5 + 1e-4


def test_requant_rows_hand_example():
    # W_O (2 outlier rows, 3 output channels), s = (3, 1.5): what = (2*W_O[0], 0.5*W_O[1])
    W_O = bf([[1.0, -0.5, 0.0], [2.0, 4.0, 0.0]])
    s = np.array([3.0, 1.5], np.float32)
    wq, dw = oracle.requant_weight_rows(W_O, s, 4)
    # column 0: what = (2, 1) -> amax 2 -> codes (127, 63.5 -> 64); column 1: (-1, 2) -> (-63.5 -> -64, 127); column 2: zeros
    assert wq.tolist() == [[127, 64, 0, 0], [-64, 127, 0, 0], [0, 0, 0, 0]]
    assert dw.tolist() == [np.float32(2.0) / np.float32(127.0), np.float32(2.0) / np.float32(127.0), 0.0]


def test_requant_s_equal_one_gives_zero():
    rng = np.random.default_rng(2)
    W_O = rand_bf(rng, (5, 33), 0.02)
    wq, dw = oracle.requant_weight_rows(W_O, np.ones(5, np.float32), 8)
    assert not wq.any() and not dw.any()


# ----------------------------------------------------------------------------- Eq. 7-8
def test_beta_exact_values_and_clamp():
    # colmax = 4 * wmax -> beta = 2 exactly; colmax < wmax -> beta = 1; zero weight row -> beta = 1
    X = bf([[8.0, 0.25, 3.0], [-2.0, 0.125, 1.0]])
    O = np.array([0, 1, 2], np.int32)
    wmax = np.array([2.0, 0.5, 0.0], np.float32)
    s, cm, be = oracle.momentum_update(X, O, wmax, 0.0, np.ones(3, np.float32))
    assert cm.tolist() == [8.0, 0.25, 3.0]
    assert be.tolist() == [2.0, 1.0, 1.0]
    assert s.tolist() == [2.0, 1.0, 1.0]          # gamma = 0: s_t = beta ("without momentum")


def test_momentum_gamma_one_is_static():
    rng = np.random.default_rng(3)
    X = rand_bf(rng, (16, 8), 50.0)
    s0 = np.array([1.0, 3.5, 17.25], np.float32)
    s, _, _ = oracle.momentum_update(X, np.array([1, 4, 6], np.int32), np.full(3, 0.05, np.float32), 1.0, s0)
    assert np.array_equal(s, s0)


@pytest.mark.parametrize("gamma", [0.2, 0.9])
def test_momentum_closed_form_constant_input(gamma):
    # constant X -> constant beta -> s_t = beta + gamma^t (s_0 - beta)
    X = bf([[9.0, 1.0], [-36.0, 2.0]])
    O = np.array([0], np.int32)
    wmax = np.array([0.25], np.float32)           # beta = sqrt(36 / 0.25) = 12
    s = np.array([1.0], np.float32)
    for t in range(1, 30):
        s, _, be = oracle.momentum_update(X, O, wmax, gamma, s)
        assert be[0] == 12.0
        expect = 12.0 + (gamma ** t) * (1.0 - 12.0)
        assert abs(float(s[0]) - expect) <= 2e-6 * expect
        assert 1.0 <= s[0] <= 12.0


def test_momentum_touches_only_outlier_columns():
    rng = np.random.default_rng(4)
    X = rand_bf(rng, (20, 10))
    O = np.array([2, 7], np.int32)
    wmax = np.array([0.01, 0.02], np.float32)
    _, cm, _ = oracle.momentum_update(X, O, wmax, 0.5, np.ones(2, np.float32))
    assert np.array_equal(cm, np.abs(f32(X))[:, O].max(axis=0))
    X2 = X.copy()
    X2[:, [0, 1, 3, 4, 5, 6, 8, 9]] = bf(np.float32(1e4))
    _, cm2, _ = oracle.momentum_update(X2, O, wmax, 0.5, np.ones(2, np.float32))
    assert np.array_equal(cm, cm2)


def test_split_momentum_update_equals_the_whole_batch_update():
    """Tokens spread over shards: per-shard column maxima, elementwise maximum, then Eq. 8 / Eq. 7 - the same
    s, bit for bit, as the update on the whole batch (a maximum does not depend on how the rows are grouped)."""
    rng = np.random.default_rng(41)
    X = rand_bf(rng, (37, 24), 30.0)
    O = np.array([0, 5, 11, 23], np.int32)
    wmax = np.array([0.04, 0.0, 0.07, 0.5], np.float32)
    s0 = np.array([1.0, 2.5, 9.0, 1.25], np.float32)
    s_ref, cm_ref, be_ref = oracle.momentum_update(X, O, wmax, 0.2, s0)
    parts = [oracle.outlier_colmax(X[a:b], O) for a, b in ((0, 10), (10, 11), (11, 37))]
    assert np.array_equal(parts[1], np.abs(f32(X[10]))[O])            # a one-row shard: the row itself
    cm = np.maximum(np.maximum(parts[0], parts[1]), parts[2])
    assert np.array_equal(cm, np.abs(f32(X))[:, O].max(axis=0)) and np.array_equal(cm, cm_ref)
    s, be = oracle.momentum_apply(cm, wmax, 0.2, s0)
    assert np.array_equal(s, s_ref) and np.array_equal(be, be_ref)
    # Eq. 8 / Eq. 7 from given maxima: colmax = 9 wmax -> beta = 3; s = 0.5 * 5 + 0.5 * 3 = 4; zero weight row -> beta = 1
    s, be = oracle.momentum_apply(np.array([2.25, 7.0], np.float32), np.array([0.25, 0.0], np.float32), 0.5,
                                  np.array([5.0, 3.0], np.float32))
    assert be.tolist() == [3.0, 1.0] and s.tolist() == [4.0, 2.0]


# ----------------------------------------------------------------------------- weight preprocessing: W_O and max|W_i|
def test_prepare_weight_outlier_rows_and_row_maxima_on_a_non_square_weight():
    """Eq. 8's max|W_i| is taken over row i of W in R^{c_in x c_out}: over ALL outputs of input channel i, i.e. down
    column O_i of the stored [N][K] layout.  A maximum over the wrong axis, or over the codes, fails here."""
    rng = np.random.default_rng(42)
    N, K = 7, 19                                   # non-square, so the two axes cannot be confused
    Wt = rand_bf(rng, (N, K), 0.02)
    Wt[3, 4] = 0x3F40                                # 0.75: the largest entry of input channel 4 sits in output channel 3
    Wt[6, 17] = 0xBF00                              # -0.5: the maximum is over magnitudes
    O = np.array([2, 4, 17], np.int32)
    Wq, dW, W_O, wmax = oracle.prepare_weight(Wt, O)
    assert W_O.shape == (3, N) and wmax.shape == (3,)
    assert np.array_equal(W_O, Wt[:, O].T)                                         # W_O[i][n] = W[O_i][n] = Wt[n][O_i], bit for bit
    assert np.array_equal(wmax, np.abs(f32(Wt))[:, O].max(axis=0))                 # over n, per input channel
    assert wmax[1] == np.float32(0.75) and wmax[2] == np.float32(0.5)
    # and the step sizes are per OUTPUT channel: over k, per row of the stored layout
    assert np.array_equal(dW, np.abs(f32(Wt)).max(axis=1) / np.float32(127.0))


# ----------------------------------------------------------------------------- integer GEMM
def test_int_gemm_brute_force_python_ints():
    rng = np.random.default_rng(5)
    for (M, N, K) in [(1, 1, 1), (3, 5, 7), (8, 8, 8), (2, 9, 33)]:
        A = rng.integers(-127, 128, (M, K)).astype(np.int8)
        B = rng.integers(-127, 128, (N, K)).astype(np.int8)
        C = oracle.int_gemm(A, B)
        for m in range(M):
            for n in range(N):
                assert int(C[m, n]) == sum(int(A[m, k]) * int(B[n, k]) for k in range(K))


def test_int_gemm_extremes():
    K = 16384
    A = np.full((2, K), 127, np.int8)
    B = np.stack([np.full(K, 127, np.int8), np.full(K, -127, np.int8), np.ones(K, np.int8)])
    C = oracle.int_gemm(A, B)
    assert C.tolist() == [[16129 * K, -16129 * K, 127 * K]] * 2


# ----------------------------------------------------------------------------- Eq. 9 as a whole
def _setup(rng, M, K, N, nO, r, s_val=None, b_std=0.02, x_scale=1.0):
    O = np.sort(rng.permutation(K)[:nO]).astype(np.int32)
    x = rng.standard_normal((M, K)).astype(np.float32) * x_scale
    x[:, O] *= rng.uniform(20, 100, nO).astype(np.float32)
    X = bf(x)
    Wt = rand_bf(rng, (N, K), 0.02)
    A = rand_bf(rng, (K, r), 0.02) if r else None
    B = rand_bf(rng, (r, N), b_std) if r else None
    Wq, dW, W_O, wmax = oracle.prepare_weight(Wt, O)
    if s_val is None:
        s, _, _ = oracle.momentum_update(X, O, wmax, 0.0, np.ones(nO, np.float32))
    else:
        s = np.full(nO, s_val, np.float32)
    return O, X, Wt, A, B, Wq, dW, W_O, wmax, s


def _forward(O, X, Wq, dW, W_O, s, A, B, lora_scale, nOp):
    Xq, xqo, dx = oracle.quant_act(X, O, s, nOp)
    wq, dw = oracle.requant_weight_rows(W_O, s, nOp)
    Y, T, a1, a2 = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, A, B, lora_scale)
    return Y, T, a1, a2, (Xq, xqo, dx, wq, dw)


def test_forward_exact_when_quantization_is_lossless():
    """Integer-valued X and W with every row/column maximum equal to 127 (254 on the outlier
    channels, s = 2) quantize without error, so Eq. 9 must return X W exactly (Eq. 3-5)."""
    rng = np.random.default_rng(6)
    M, K, N = 9, 24, 7
    O = np.array([2, 11, 23], np.int32)
    x = rng.integers(-127, 128, (M, K)).astype(np.float32)
    x[:, 0] = 127                                   # every token row reaches 127 off the outliers
    x[:, O] = 2 * rng.integers(-127, 128, (M, 3))   # even, up to 254 -> /2 is an integer <= 127
    w = rng.integers(-127, 128, (N, K)).astype(np.float32)
    w[:, 1] = 127                                   # every output channel reaches 127
    w[:, O] = rng.choice([-127.0, 0.0, 127.0], (N, 3))
    w[:, O[0]] = 127                                # every column of what reaches 127
    X, Wt = bf(x), bf(w)
    assert np.array_equal(f32(X), x) and np.array_equal(f32(Wt), w)
    Wq, dW, W_O, wmax = oracle.prepare_weight(Wt, O)
    s = np.full(3, 2.0, np.float32)
    Y, T, a1, a2, _ = _forward(O, X, Wq, dW, W_O, s, None, None, 0.0, 4)
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.array_equal(Y, exact)
    # brute force of both integer accumulators in Python integers
    xi = x.astype(np.int64)
    xi[:, O] //= 2
    for m in range(M):
        for n in range(N):
            assert int(a1[m, n]) == sum(int(xi[m, k]) * int(w[n, k]) for k in range(K))
            assert int(a2[m, n]) == sum(int(xi[m, O[i]]) * int(w[n, O[i]]) for i in range(3))


def test_forward_s_one_equals_naive_waq():
    """s = 1 makes what = 0, so Eq. 9 must be bit-identical to Eq. 2 (no outlier set at all)."""
    rng = np.random.default_rng(7)
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, 12, 64, 20, 4, 0, s_val=1.0)
    Y, _, a1, a2, _ = _forward(O, X, Wq, dW, W_O, s, None, None, 0.0, 8)
    none = np.zeros(0, np.int32)
    Wq0, dW0, W_O0, _ = oracle.prepare_weight(Wt, none)
    Y0, _, b1, b2, _ = _forward(none, X, Wq0, dW0, W_O0, np.zeros(0, np.float32), None, None, 0.0, 0)
    assert np.array_equal(Y, Y0) and np.array_equal(a1, b1) and not a2.any()
    # and Eq. 2 written out with numpy on the oracle's codes
    Xq, _, dx = oracle.quant_act(X, none, np.zeros(0, np.float32), 0)
    ref = dx.astype(np.float64)[:, None] * (Xq.astype(np.int64) @ Wq0.astype(np.int64).T) * dW0.astype(np.float64)[None, :]
    assert np.allclose(Y0, ref, rtol=1e-14, atol=0)


def test_forward_error_bound_and_outlier_suppression():
    rng = np.random.default_rng(8)
    M, K, N, nO = 32, 256, 48, 6
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, 0)
    assert (s > 1).all()
    Y, _, _, _, (Xq, xqo, dx, wq, dw) = _forward(O, X, Wq, dW, W_O, s, None, None, 0.0, 8)
    x = f32(X).astype(np.float64)
    w = f32(Wt).astype(np.float64)                  # [N,K]
    exact = x @ w.T
    # rounding bound of Eq. 1 applied to both GEMMs of Eq. 9: |x - D q| <= D/2 for each factor
    xh = x.copy()
    xh[:, O] /= s.astype(np.float64)[None, :]
    Dx = dx.astype(np.float64)[:, None]
    DW = dW.astype(np.float64)[None, :]
    Dw = dw.astype(np.float64)[None, :]
    what = (s.astype(np.float64) - 1.0)[None, :] * w[:, O]          # [N,nO]
    slack = 1.0 + 1e-5                                              # fp32 evaluation of the step sizes
    bound = (np.abs(xh) @ np.ones((K, 1))) * (DW / 2) + (Dx / 2) * (np.ones((M, 1)) @ np.abs(w).sum(axis=1)[None, :]) + K * Dx * DW / 4
    bound += (np.abs(xh[:, O]).sum(axis=1)[:, None]) * (Dw / 2) + (Dx / 2) * np.abs(what).sum(axis=1)[None, :] + nO * Dx * Dw / 4
    assert (np.abs(Y - exact) <= bound * slack + 1e-12).all()
    # outlier suppression must reduce the error of naive W8A8 on outlier-bearing data
    none = np.zeros(0, np.int32)
    Wq0, dW0, W_O0, _ = oracle.prepare_weight(Wt, none)
    Y0 = _forward(none, X, Wq0, dW0, W_O0, np.zeros(0, np.float32), None, None, 0.0, 0)[0]
    e_quaff = np.linalg.norm(Y - exact)
    e_naive = np.linalg.norm(Y0 - exact)
    assert e_quaff < 0.5 * e_naive


def test_scaling_identity_on_dequantized_operands():
    """Eq. 4-5: Xhat W + Xhat_O (s_O - 1) W_O = X W; checked through the oracle's codes: the
    dequantized operands must reproduce X W within the rounding bound, and the two terms must
    carry the right channels (a wrong index or a dropped term breaks the agreement)."""
    rng = np.random.default_rng(9)
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, 16, 128, 24, 5, 0)
    Y = _forward(O, X, Wq, dW, W_O, s, None, None, 0.0, 8)[0]
    exact = f32(X).astype(np.float64) @ f32(Wt).astype(np.float64).T
    rel = np.linalg.norm(Y - exact) / np.linalg.norm(exact)
    assert rel < 2e-2
    # dropping the outlier term must be far worse
    s1 = np.ones_like(s)
    wq0, dw0 = oracle.requant_weight_rows(W_O, s1, 8)
    Xq, xqo, dx = oracle.quant_act(X, O, s, 8)
    Ybad = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq0, dw0, X, None, None, 0.0)[0]
    assert np.linalg.norm(Ybad - exact) / np.linalg.norm(exact) > 10 * rel


# ----------------------------------------------------------------------------- LoRA
def test_lora_branch_against_numpy_float64():
    rng = np.random.default_rng(10)
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, 10, 96, 18, 3, 8)
    Y1, T, _, _, _ = _forward(O, X, Wq, dW, W_O, s, A, B, 2.0, 4)
    Y0 = _forward(O, X, Wq, dW, W_O, s, None, None, 0.0, 4)[0]
    t = f32(X).astype(np.float64) @ f32(A).astype(np.float64)
    # T is X A rounded once to bf16: within half a bf16 ulp
    assert (np.abs(f32(T) - t) <= half_ulp_bf16(t)).all()
    lora = 2.0 * (f32(T).astype(np.float64) @ f32(B).astype(np.float64))
    assert np.allclose(Y1 - Y0, lora, rtol=1e-9, atol=1e-12)
    # B = 0 (the usual initialisation): the branch vanishes
    Yz = _forward(O, X, Wq, dW, W_O, s, A, np.zeros_like(B), 2.0, 4)[0]
    assert np.array_equal(Yz, Y0)


def test_supplied_intermediates_T_and_G_are_used_as_given():
    """qlinear_fwd(T_in=...) and qlinear_bwd(G_in=...) evaluate everything downstream of the bf16 intermediate on the
    given bits: with the oracle's own bits nothing changes; with one entry moved by one bf16 ulp the outputs move by
    exactly that entry's term (numpy float64)."""
    rng = np.random.default_rng(43)
    M, K, N, nO, r = 9, 64, 20, 2, 8
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, r)
    nOp = 4
    Xq, xqo, dx = oracle.quant_act(X, O, s, nOp)
    wq, dw = oracle.requant_weight_rows(W_O, s, nOp)
    Y, T, a1, a2 = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, A, B, 0.5)
    Y2, T2, b1, b2 = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, A, B, 0.5, T_in=T)
    assert np.array_equal(Y, Y2) and np.array_equal(T, T2) and np.array_equal(a1, b1) and np.array_equal(a2, b2)
    Tm = T.copy()
    Tm[4, 3] += 1                                              # next bf16 value away from zero
    Y3, T3, _, _ = oracle.qlinear_fwd(Xq, xqo, dx, Wq, dW, wq, dw, X, A, B, 0.5, T_in=Tm)
    assert np.array_equal(T3, Tm)
    d = (f32(Tm).astype(np.float64) - f32(T).astype(np.float64))[4, 3]
    expect = np.zeros_like(Y)
    expect[4] = 0.5 * d * f32(B).astype(np.float64)[3]
    assert d != 0 and np.allclose(Y3 - Y, expect, rtol=1e-9, atol=1e-15)

    dY = rand_bf(rng, (M, N), 1e-2)
    dX, dA, dB, G = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 0.5)
    dX2, dA2, dB2, G2 = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 0.5, G_in=G)
    assert np.array_equal(dX, dX2) and np.array_equal(dA, dA2) and np.array_equal(dB, dB2) and np.array_equal(G, G2)
    Gm = G.copy()
    Gm[2, 5] += 1
    dX3, dA3, dB3, G3 = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 0.5, G_in=Gm)
    assert np.array_equal(G3, Gm) and np.array_equal(dB3, dB)                  # dB does not depend on G
    dg = (f32(Gm).astype(np.float64) - f32(G).astype(np.float64))[2, 5]
    ex = np.zeros_like(dX)
    ex[2] = dg * f32(A).astype(np.float64)[:, 5]                               # dX += G A^T
    assert dg != 0 and np.allclose(dX3 - dX, ex, rtol=1e-9, atol=1e-15)
    ea = np.zeros_like(dA)
    ea[:, 5] = f32(X).astype(np.float64)[2] * dg                               # dA = X^T G
    assert np.allclose(dA3 - dA, ea, rtol=1e-9, atol=1e-15)


# ----------------------------------------------------------------------------- backward
def test_bf16_roundings_are_to_nearest_even_and_single():
    """The three places where the oracle rounds to bf16, on values whose correct rounding is known by hand
    (bf16 keeps 8 significant bits; 1 + 2^-8 lies exactly half way between 1 and 1 + 2^-7):
    T = bf16(X A) and G = bf16(scale dY B^T) round the exact sum ONCE (1 + 2^-8 + 2^-30 is above the half-way point and
    goes up, although it would first collapse onto the tie in fp32 and then go down), ties go to the even neighbour,
    and Wd = bf16(code * Delta_W) rounds the fp32 product the same way."""
    one, up = 0x3F80, 0x3F81                                  # 1.0 and 1 + 2^-7
    ones = bf(np.ones((1, 3), np.float32))
    col = bf(np.array([[1.0], [2.0 ** -8], [2.0 ** -30]], np.float32))
    tie = bf(np.array([[1.0], [2.0 ** -8], [0.0]], np.float32))
    odd = bf(np.array([[1.0 + 2.0 ** -7], [2.0 ** -8], [0.0]], np.float32))   # tie above an odd pattern: up to 1 + 2^-6
    for a_col, want in ((col, up), (tie, one), (odd, 0x3F82)):
        T = oracle.lora_down(ones, a_col)
        assert T.shape == (1, 1) and int(T[0, 0]) == want
        # G = bf16(1 * dY B^T) with dY = ones [1][3], B [1][3] = the same column as a row
        z8 = np.zeros((3, 1), np.int8)
        _, _, _, G = oracle.qlinear_bwd(ones, z8, np.zeros(3, np.float32), np.zeros((3, 0), np.int8), np.zeros(3, np.float32),
                                        np.zeros(0, np.int32), np.zeros(0, np.float32), bf(np.zeros((1, 1), np.float32)),
                                        bf(np.zeros((1, 1), np.float32)), bf(np.zeros((1, 1), np.float32)),
                                        np.ascontiguousarray(a_col.reshape(1, 3)), 1.0, want_dX=False, want_dAB=False)
        assert int(G[0, 0]) == want
    # Wd: code 1 x step 1 + 2^-8 is the tie (down to 1); code 3 x the same step is 3 + 3 * 2^-8 = 1.1000000|11b x 2, above
    # half way (up to 3 + 2^-6 = 3.015625); code -1 mirrors code 1.  dY = identity, so dX is Wd itself.
    Wq = np.array([[1], [3], [-1]], np.int8)
    dW = np.full(3, 1.0 + 2.0 ** -8, np.float32)
    dX, _, _, _ = oracle.qlinear_bwd(bf(np.eye(3, dtype=np.float32)), Wq, dW, np.zeros((3, 0), np.int8), np.zeros(3, np.float32),
                                     np.zeros(0, np.int32), np.zeros(0, np.float32), bf(np.zeros((3, 1), np.float32)),
                                     None, None, None, 1.0, want_dAB=False)
    assert dX[:, 0].tolist() == [1.0, 3.015625, -1.0]


def _dequantized_map(O, Wq, dW, wq, dw, s, K):
    """The linear map of Eq. 9 with the codes held fixed: Y = X @ Weff, Weff[k,n]."""
    Wd = f32(bf(Wq.astype(np.float32) * dW[:, None])).astype(np.float64)          # [N,K]
    wd = f32(bf(wq.astype(np.float32) * dw[:, None])).astype(np.float64)          # [N,nOp]
    Weff = Wd.T.copy()                                                            # [K,N]
    for i, k in enumerate(O):
        Weff[k] = (Weff[k] + wd[:, i]) / float(s[i])
    return Weff


def test_backward_dx_by_finite_differences():
    rng = np.random.default_rng(11)
    M, K, N, nO, r = 6, 40, 14, 3, 4
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, r, b_std=0.0)   # B = 0: G = 0, map is linear
    wq, dw = oracle.requant_weight_rows(W_O, s, 8)
    dY = rand_bf(rng, (M, N), 1e-2)
    T = bf(np.zeros((M, r), np.float32))
    dX, dA, dB, G = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 1.0)
    assert not G.any()
    Weff = _dequantized_map(O, Wq, dW, wq, dw, s, K)
    g = f32(dY).astype(np.float64)

    def loss(x):
        return float(np.sum(g * (x @ Weff)))

    x0 = f32(X).astype(np.float64)
    h = 1.0
    for (m, k) in [(0, 0), (1, int(O[0])), (2, int(O[2])), (5, 39), (3, 17)]:
        e = np.zeros_like(x0)
        e[m, k] = h
        fd = (loss(x0 + e) - loss(x0 - e)) / (2 * h)
        assert abs(fd - dX[m, k]) <= 1e-9 * max(1.0, abs(fd))


def test_backward_matches_full_precision_gradient_statistically():
    rng = np.random.default_rng(12)
    M, K, N, nO = 24, 192, 40, 4
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, 0)
    wq, dw = oracle.requant_weight_rows(W_O, s, 8)
    dY = rand_bf(rng, (M, N), 1e-2)
    dX = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, None, None, None, 0.0)[0]
    full = f32(dY).astype(np.float64) @ f32(Wt).astype(np.float64)
    assert np.linalg.norm(dX - full) / np.linalg.norm(full) < 3e-2
    # per-channel: the outlier columns must carry s_i W_i / s_i = W_i as well
    colerr = np.linalg.norm((dX - full)[:, O], axis=0) / np.linalg.norm(full[:, O], axis=0)
    assert (colerr < 5e-2).all()


def test_backward_lora_grads_against_numpy_float64():
    rng = np.random.default_rng(13)
    M, K, N, nO, r = 12, 48, 20, 2, 4
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, r)
    wq, dw = oracle.requant_weight_rows(W_O, s, 4)
    Y, T, _, _, _ = _forward(O, X, Wq, dW, W_O, s, A, B, 0.5, 4)
    dY = rand_bf(rng, (M, N), 1e-2)
    dX, dA, dB, G = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 0.5)
    g = f32(dY).astype(np.float64)
    gexact = 0.5 * (g @ f32(B).astype(np.float64).T)
    assert (np.abs(f32(G) - gexact) <= half_ulp_bf16(gexact)).all()
    Gd = f32(G).astype(np.float64)
    assert np.allclose(dA, f32(X).astype(np.float64).T @ Gd, rtol=1e-12, atol=1e-15)
    assert np.allclose(dB, 0.5 * (f32(T).astype(np.float64).T @ g), rtol=1e-12, atol=1e-15)
    # dX = (codes-fixed linear map)^T dY + G A^T
    Weff = _dequantized_map(O, Wq, dW, wq, dw, s, K)
    assert np.allclose(dX, g @ Weff.T + Gd @ f32(A).astype(np.float64).T, rtol=1e-10, atol=1e-14)


def test_lora_gradients_by_finite_differences_of_the_forward():
    """dA and dB are the derivatives of sum(dY * Y) w.r.t. A and B of the oracle's own forward,
    up to the bf16 roundings of T and G (2^-9 each)."""
    rng = np.random.default_rng(14)
    M, K, N, nO, r = 8, 32, 12, 2, 4
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, r, b_std=0.05)
    wq, dw = oracle.requant_weight_rows(W_O, s, 4)
    Y, T, _, _, _ = _forward(O, X, Wq, dW, W_O, s, A, B, 1.0, 4)
    dY = rand_bf(rng, (M, N), 1.0)
    _, dA, dB, _ = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 1.0)
    x = f32(X).astype(np.float64)
    a = f32(A).astype(np.float64)
    b = f32(B).astype(np.float64)
    g = f32(dY).astype(np.float64)
    dA_true = x.T @ (g @ b.T)
    dB_true = (x @ a).T @ g
    assert np.linalg.norm(dA - dA_true) / np.linalg.norm(dA_true) < 4e-3
    assert np.linalg.norm(dB - dB_true) / np.linalg.norm(dB_true) < 4e-3


# ----------------------------------------------------------------------------- INT8 grad-input variant (not the paper's method)
def test_quant_grad_hand_examples():
    # Z = dY * Delta_W[n], then Eq. 1 per token.  Row 0: Z = (2.5, 3.5, -0.5, 127) -> amax 127, codes (2, 4, 0, 127): three ties.
    # Row 1: the column scales change which entry is the row maximum: dY = (1, -2, 0.5, 4), Delta_W = (0.5, 0.5, 0.5, 0.5)
    # -> Z = (0.5, -1, 0.25, 2) -> r = 63.5 -> (31.75 -> 32, -63.5 -> -64, 15.875 -> 16, 127).
    dY = bf([[5.0, 7.0, -1.0, 254.0], [1.0, -2.0, 0.5, 4.0], [0.0, 0.0, 0.0, 0.0]])
    dW = np.full(4, 0.5, np.float32)
    Zq, dz = oracle.quant_grad(dY, dW)
    assert Zq.tolist() == [[2, 4, 0, 127], [32, -64, 16, 127], [0, 0, 0, 0]]
    assert dz.tolist() == [1.0, np.float32(2.0) / np.float32(127.0), 0.0]
    # unequal column scales: dY = (8, 1), Delta_W = (0.125, 4) -> Z = (1, 4): the SECOND entry carries the maximum
    Zq, dz = oracle.quant_grad(bf([[8.0, 1.0]]), np.array([0.125, 4.0], np.float32))
    assert Zq.tolist() == [[32, 127]] and dz[0] == np.float32(4.0) / np.float32(127.0)


def test_int8_backward_accumulators_brute_force_and_shared_parts():
    rng = np.random.default_rng(51)
    M, K, N, nO, r = 5, 24, 12, 2, 4
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, r)
    wq, dw = oracle.requant_weight_rows(W_O, s, 4)
    T = oracle.lora_down(X, A)
    dY = rand_bf(rng, (M, N), 1e-2)
    dX8, dA8, dB8, G8, Zq, dz, acc = oracle.qlinear_bwd_int8(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 0.5)
    Zq2, dz2 = oracle.quant_grad(dY, dW)
    assert np.array_equal(Zq, Zq2) and np.array_equal(dz, dz2)
    for m in range(M):
        for k in range(K):
            assert int(acc[m, k]) == sum(int(Zq[m, n]) * int(Wq[n, k]) for n in range(N))
    dX, dA, dB, G = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, T, A, B, 0.5)
    # G, dA, dB and the outlier columns are those of the floating-point backward
    assert np.array_equal(G8, G) and np.array_equal(dA8, dA) and np.array_equal(dB8, dB)
    assert np.allclose(dX8[:, O], dX[:, O], rtol=1e-12, atol=1e-18)
    # the other columns: Dz[m] * acc + G A^T
    rest = np.setdiff1d(np.arange(K), O)
    lora = f32(G).astype(np.float64) @ f32(A).astype(np.float64).T
    assert np.allclose(dX8[:, rest], (dz[:, None].astype(np.float64) * acc.astype(np.float64) + lora)[:, rest], rtol=1e-12, atol=1e-18)


def test_int8_backward_is_exact_when_the_gradient_quantization_is_lossless():
    """Integer-valued weight with column maxima 127 (codes = values, Delta_W = 1) and integer-valued dY with row maxima
    127 (Zq = dY, Dz = 1): the INT8 variant then computes dY W^T exactly, and so does the floating-point backward."""
    rng = np.random.default_rng(52)
    M, K, N = 6, 20, 16
    W = rng.integers(-127, 128, (N, K)).astype(np.float32)
    W[:, 0] = 127.0                                                    # every output channel (row of Wt) has maximum 127
    g = rng.integers(-127, 128, (M, N)).astype(np.float32)
    g[:, 3] = -127.0
    Wt, dY = bf(W), bf(g)
    assert np.array_equal(f32(Wt), W) and np.array_equal(f32(dY), g)
    O = np.zeros(0, np.int32)
    Wq, dW, W_O, wmax = oracle.prepare_weight(Wt, O)
    assert np.array_equal(Wq, W.astype(np.int8)) and (dW == 1.0).all()
    none = np.zeros((N, 0), np.int8)
    X = bf(np.zeros((M, K), np.float32))
    dX8, _, _, _, Zq, dz, acc = oracle.qlinear_bwd_int8(dY, Wq, dW, none, np.zeros(N, np.float32), O, np.zeros(0, np.float32), X, None, None, None, 0.0)
    assert np.array_equal(Zq, g.astype(np.int8)) and (dz == 1.0).all()
    exact = g.astype(np.float64) @ W.astype(np.float64)
    assert np.array_equal(dX8, exact)
    dX = oracle.qlinear_bwd(dY, Wq, dW, none, np.zeros(N, np.float32), O, np.zeros(0, np.float32), X, None, None, None, 0.0)[0]
    assert np.array_equal(dX, exact)


def test_int8_backward_error_bound_against_the_floating_point_backward():
    """Element by element: |dX_int8 - dX_fp| <= (Dz[m] / 2) sum_n |Wq[n][k]|  (rounding of Zq, Eq. 1)
    + 2^-8 sum_n |Z[m][n] Wq[n][k]|  (the bf16 rounding of the dequantized weight on the other side, and of Z in fp32)."""
    rng = np.random.default_rng(53)
    M, K, N, nO = 16, 96, 64, 3
    O, X, Wt, A, B, Wq, dW, W_O, wmax, s = _setup(rng, M, K, N, nO, 0)
    wq, dw = oracle.requant_weight_rows(W_O, s, 4)
    dY = rand_bf(rng, (M, N), 1e-2)
    dX8, _, _, _, Zq, dz, acc = oracle.qlinear_bwd_int8(dY, Wq, dW, wq, dw, O, s, X, None, None, None, 0.0)
    dX = oracle.qlinear_bwd(dY, Wq, dW, wq, dw, O, s, X, None, None, None, 0.0)[0]
    Z = np.abs(f32(dY).astype(np.float64) * dW[None, :].astype(np.float64))
    aW = np.abs(Wq.astype(np.float64))
    bound = 0.5 * dz[:, None].astype(np.float64) * aW.sum(axis=0)[None, :] * (1 + 1e-6) + 2.0 ** -8 * (Z @ aW)
    assert (np.abs(dX8 - dX) <= bound).all()
    # and it is an approximation of the same thing: a few per cent of the gradient's norm
    rest = np.setdiff1d(np.arange(K), O)
    assert np.linalg.norm((dX8 - dX)[:, rest]) / np.linalg.norm(dX[:, rest]) < 3e-2


# ----------------------------------------------------------------------------- generator sanity
def test_synthetic_workload_shapes_and_outliers():
    wl = synth.WORKLOADS["tiny"]
    lin = synth.layer_inputs(wl, 0)
    X, dY = synth.step_inputs(wl, 0, 0, lin)
    assert X.shape == (256, 512) and dY.shape == (256, 512) and lin.W.shape == (512, 512)
    assert len(np.unique(lin.O_idx)) == 8 and (np.diff(lin.O_idx) > 0).all()
    colmax = np.abs(f32(X)).max(axis=0)
    rest = np.delete(colmax, lin.O_idx)
    assert colmax[lin.O_idx].min() > 5 * rest.max()
    X2, _ = synth.step_inputs(wl, 0, 0, lin)
    assert np.array_equal(X, X2)
    X3, _ = synth.step_inputs(wl, 0, 1, lin)
    assert not np.array_equal(X, X3)


# ----------------------------------------------------------------------------- calibration, Eq. 6
def _xi_brute(x_f32, thr):
    """Eq. 6 from its definition in Python integers / Fractions (independent of the C code): |x| in units of 2^-16."""
    from fractions import Fraction
    M, K = x_f32.shape
    a = [[min(int(Fraction(abs(float(v))) * 65536), 2 ** 32 - 1) for v in row] for row in x_f32]
    total = sum(sum(r) for r in a)
    return np.array([1 if max(a[m][k] for m in range(M)) * M * K > thr * total else 0 for k in range(K)], np.int32)


def test_outlier_count_boundary_is_strict():
    # one token, channels [1, 1, 1, x], thr = 2: channel 3 counts iff x > 2 (3 + x) / 4  <=>  x > 3
    for x, hit in ((3.0, 0), (3.015625, 1), (2.984375, 0)):
        X = synth.f32_to_bf16_bits(np.array([[1.0, 1.0, 1.0, x]], np.float32))
        xi = oracle.outlier_count(X, 2, np.zeros(4, np.int32))
        assert xi.tolist() == [0, 0, 0, hit], (x, xi)


def test_outlier_count_fixed_point_truncation_and_accumulation():
    # 2^-17 is below the 2^-16 unit and counts as 0; 2^-10 is 64 units
    X = synth.f32_to_bf16_bits(np.array([[2.0 ** -17, 2.0 ** -10]], np.float32))
    xi = oracle.outlier_count(X, 1, np.array([5, 7], np.int32))       # 64 * 2 > 1 * 64 ; 0 * 2 > 64 is false
    assert xi.tolist() == [5, 8]
    xi = oracle.outlier_count(X, 2, xi)                                 # 64 * 2 > 2 * 64 is false (strict)
    assert xi.tolist() == [5, 8]


def test_outlier_count_saturates_magnitudes_at_two_to_the_32():
    # |x| in units of 2^-16 saturates at 2^32 - 1: 2^20 and 2^16 both count as 2^32 - 1 = S.
    X = synth.f32_to_bf16_bits(np.array([[2.0 ** 20, 2.0 ** 16, 0.0, 0.0]], np.float32))
    xi = oracle.outlier_count(X, 1, np.zeros(4, np.int32))              # S * 4 > 1 * 2S for both; 0 * 4 > 2S is false
    assert xi.tolist() == [1, 1, 0, 0]
    xi = oracle.outlier_count(X, 2, np.zeros(4, np.int32))              # S * 4 > 2 * 2S is false (unsaturated, 2^20 would count)
    assert xi.tolist() == [0, 0, 0, 0]


def test_outlier_count_matches_brute_force_and_finds_planted_channels():
    rng = np.random.default_rng(11)
    for M, K in ((3, 5), (7, 16), (16, 33)):
        x = rng.standard_normal((M, K)).astype(np.float32)
        x[:, rng.integers(K)] *= 300.0
        xb = synth.f32_to_bf16_bits(x)
        xf = synth.bf16_bits_to_f32(xb)
        for thr in (1, 3, 100):
            assert np.array_equal(oracle.outlier_count(xb, thr, np.zeros(K, np.int32)), _xi_brute(xf, thr))
    # the paper's threshold (100 x mean|X|) on the synthetic activations: the planted outlier set is what comes out
    wl = synth.WORKLOADS["tiny"]
    lin = synth.layer_inputs(wl, 0)
    xi = np.zeros(lin.spec.K, np.int32)
    for step in range(8):
        X, _ = synth.step_inputs(wl, 0, step, lin)
        xi = oracle.outlier_count(X, 100, xi)
    # (the threshold is 100 x the mean over ALL channels, outliers included: here about 150, so only the stronger
    # half of the planted channels - magnitude 30..80 times a 3-sigma peak - can cross it)
    assert xi[np.setdiff1d(np.arange(lin.spec.K), lin.O_idx)].max() == 0     # an N(0,1) channel never reaches 100 x mean
    strong = lin.O_idx[lin.base >= 65.0]
    assert len(strong) > 0 and np.all(xi[strong] >= 6), (lin.base, xi[lin.O_idx])
    n_found = int((xi > 0).sum())
    assert set(oracle.select_outliers(xi, n_found).tolist()) <= set(lin.O_idx.tolist())


def test_select_outliers_ties_and_order():
    xi = np.array([2, 5, 5, 0, 5, 1], np.int32)
    assert oracle.select_outliers(xi, 2).tolist() == [1, 2]        # three channels tie at 5: the lower indices win
    assert oracle.select_outliers(xi, 4).tolist() == [0, 1, 2, 4]   # sorted ascending
    assert oracle.select_outliers(xi, 0).tolist() == []
    assert oracle.select_outliers(xi, 6).tolist() == [0, 1, 2, 3, 4, 5]


# ----------------------------------------------------------------------------- hit-rate monitor (Sec. 3.2)
def test_outlier_hits_hand_case():
    # one token; channels 1 and 4 are far above thr x mean: R = {1, 4}.  mean|X| = (4 + 2 * 640) / 6 = 214; thr = 2 -> 428
    X = synth.f32_to_bf16_bits(np.array([[1.0, 640.0, 1.0, 1.0, 640.0, 1.0]], np.float32))
    assert oracle.outlier_hits(X, 2, np.array([1, 4], np.int32)).tolist() == [2, 2]      # every real-time outlier predicted
    assert oracle.outlier_hits(X, 2, np.array([0, 1], np.int32)).tolist() == [1, 2]      # one of two
    assert oracle.outlier_hits(X, 2, np.array([0, 2, 3, 5], np.int32)).tolist() == [0, 2]
    assert oracle.outlier_hits(X, 2, np.zeros(0, np.int32)).tolist() == [0, 2]           # empty O
    assert oracle.outlier_hits(X, 1000, np.array([1, 4], np.int32)).tolist() == [0, 0]   # no channel crosses: rate undefined


def test_outlier_hits_matches_brute_force_sets():
    rng = np.random.default_rng(23)
    for M, K, nO in ((3, 9, 2), (8, 40, 5), (16, 33, 33)):
        x = rng.standard_normal((M, K)).astype(np.float32)
        x[:, rng.choice(K, 3, replace=False)] *= 200.0
        xb = synth.f32_to_bf16_bits(x)
        O = np.sort(rng.choice(K, nO, replace=False)).astype(np.int32)
        for thr in (1, 4, 30):
            R = set(np.flatnonzero(_xi_brute(synth.bf16_bits_to_f32(xb), thr)).tolist())
            got = oracle.outlier_hits(xb, thr, O).tolist()
            assert got == [len(R & set(O.tolist())), len(R)], (M, K, thr, got)
            # the full channel set predicts everything; the complement of O the rest
            assert oracle.outlier_hits(xb, thr, np.arange(K, dtype=np.int32)).tolist() == [len(R), len(R)]
            comp = np.setdiff1d(np.arange(K), O).astype(np.int32)
            assert oracle.outlier_hits(xb, thr, comp)[0] == len(R) - got[0]
