"""GPU parity of the calibration entry points (Eq. 6 counts and the selection of O): integer results, bit-exact."""
import numpy as np
import pytest

import oracle
from paper_2505_14742_b200 import synth
from util import bf, dev, dev_bf16, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def Q():
    from paper_2505_14742_b200 import binding, build
    build.build_library()
    binding.lib()
    return binding


@pytest.mark.parametrize("M,K,thr", [(1, 8, 2), (37, 100, 3), (300, 3072, 100), (257, 11008, 100), (64, 20000, 20)])
def test_outlier_count_bit_exact_over_samples(Q, M, K, thr):
    import torch
    rng = np.random.default_rng(900 + K)
    ldx = (K + 7) // 8 * 8 + 8
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_CALIBRATE, M, K, 0, 0, 0), dtype=torch.uint8, device="cuda")
    xi_d = torch.zeros(K, dtype=torch.int32, device="cuda")
    xi = np.zeros(K, np.int32)
    planted = rng.permutation(K)[: max(1, K // 100)]
    for sample in range(3):
        x = rng.standard_normal((M, K)).astype(np.float32)
        x[:, planted] *= rng.uniform(20, 400, planted.size).astype(np.float32)
        if sample == 1:
            x[0, :4] = [0.0, 1e-7, 70000.0, -2.0 ** -16]         # zero, below the unit, saturating, exactly one unit
        X = bf(x)
        Xd = torch.zeros((M, ldx), dtype=torch.bfloat16, device="cuda")
        Xd[:, :K] = dev_bf16(X)
        Q.quaff_outlier_count(Xd[:, :K], thr, xi_d, ws)
        xi = oracle.outlier_count(X, thr, xi)
        torch.cuda.synchronize()
        assert np.array_equal(host(xi_d), xi), f"sample {sample}"
    assert xi.max() > 0


@pytest.mark.parametrize("K,nO", [(8, 3), (1000, 10), (3072, 32), (11008, 1100), (4096, 4096)])
def test_select_outliers_bit_exact(Q, K, nO):
    import torch
    rng = np.random.default_rng(950 + K)
    xi = rng.integers(0, 6, K).astype(np.int32)          # many ties
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_CALIBRATE, 1, K, 0, 0, 0), dtype=torch.uint8, device="cuda")
    O = torch.full((nO,), -1, dtype=torch.int32, device="cuda")
    Q.quaff_select_outliers(dev(xi), O, ws)
    torch.cuda.synchronize()
    assert np.array_equal(host(O), oracle.select_outliers(xi, nO))


def test_calibration_recovers_the_planted_outlier_set(Q):
    """Calibrate on synthetic samples of the LLaMA-shaped workload (outliers up to 200x, log-normal) with the
    paper's threshold, select O with the layer's budget, and feed it to the weight preprocessing."""
    import torch
    wl = synth.WORKLOADS["llama7b_block"]
    lin = synth.layer_inputs(wl, 0)
    sp = lin.spec
    M = 512
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_CALIBRATE, M, sp.K, 0, 0, 0), dtype=torch.uint8, device="cuda")
    xi_d = torch.zeros(sp.K, dtype=torch.int32, device="cuda")
    xi = np.zeros(sp.K, np.int32)
    for step in range(6):
        mag = synth.outlier_magnitude(wl.seed, 0, step, lin.base)
        X = synth.activations(wl.seed, 0, step, M, sp.K, lin.O_idx, mag)
        Q.quaff_outlier_count(dev_bf16(X), 100, xi_d, ws)
        xi = oracle.outlier_count(X, 100, xi)
    O_d = torch.empty(sp.nO, dtype=torch.int32, device="cuda")
    Q.quaff_select_outliers(xi_d, O_d, ws)
    torch.cuda.synchronize()
    assert np.array_equal(host(xi_d), xi)
    O = host(O_d)
    assert np.array_equal(O, oracle.select_outliers(xi, sp.nO))
    found = set(O[xi[O] > 0].tolist())
    assert found <= set(lin.O_idx.tolist())                   # never a false positive
    assert len(found) >= 0.5 * sp.nO                          # the stronger half of the planted channels crosses 100 x mean


@pytest.mark.parametrize("M,K,nO,thr", [(1, 8, 0, 2), (37, 100, 7, 3), (300, 3072, 32, 20), (257, 11008, 1100, 30), (64, 20000, 20000, 20)])
def test_outlier_hits_bit_exact(Q, M, K, nO, thr):
    """Hit-rate monitor (Sec. 3.2): both integer counts equal the oracle's, on two batches in a row with the same workspace."""
    import torch
    rng = np.random.default_rng(970 + K)
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_HITS, M, K, 0, 0, 0), dtype=torch.uint8, device="cuda")
    planted = rng.permutation(K)[: max(2, K // 100)]
    # O: half of the planted channels plus random others
    O = np.unique(np.concatenate([planted[: planted.size // 2], rng.permutation(K)[:nO]]))[:nO].astype(np.int32) if nO else np.zeros(0, np.int32)
    if nO == K:
        O = np.arange(K, dtype=np.int32)
    hits_d = torch.full((2,), -7, dtype=torch.int32, device="cuda")
    seen = 0
    for batch in range(2):
        x = rng.standard_normal((M, K)).astype(np.float32)
        x[:, planted] *= rng.uniform(50, 400, planted.size).astype(np.float32)
        X = bf(x)
        ldx = (K + 7) // 8 * 8 + 8
        Xd = torch.zeros((M, ldx), dtype=torch.bfloat16, device="cuda")
        Xd[:, :K] = dev_bf16(X)
        Q.quaff_outlier_hits(Xd[:, :K], thr, dev(O) if nO else None, hits_d, ws)
        torch.cuda.synchronize()
        ref = oracle.outlier_hits(X, thr, O)
        assert host(hits_d).tolist() == ref.tolist(), (batch, ref)
        seen += int(ref[1])
    assert seen > 0


def test_hit_rate_of_calibrated_set_on_a_synthetic_stream(Q):
    """Calibrate O on a few samples, then monitor the hit rate over later steps of the same synthetic stream
    (stable outlier channels, drifting magnitudes): the predefined set catches the real-time outliers."""
    import torch
    wl = synth.WORKLOADS["phi3_attn"]
    lin = synth.layer_inputs(wl, 0)
    sp = lin.spec
    M = 256
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_HITS, M, sp.K, 0, 0, 0), dtype=torch.uint8, device="cuda")
    xi_d = torch.zeros(sp.K, dtype=torch.int32, device="cuda")
    for step in range(4):
        mag = synth.outlier_magnitude(wl.seed, 0, step, lin.base)
        Q.quaff_outlier_count(dev_bf16(synth.activations(wl.seed, 0, step, M, sp.K, lin.O_idx, mag)), 100, xi_d, ws)
    O_d = torch.empty(sp.nO, dtype=torch.int32, device="cuda")
    Q.quaff_select_outliers(xi_d, O_d, ws)
    hits_d = torch.zeros(2, dtype=torch.int32, device="cuda")
    tot = np.zeros(2, np.int64)
    for step in range(4, 10):
        mag = synth.outlier_magnitude(wl.seed, 0, step, lin.base)
        X = synth.activations(wl.seed, 0, step, M, sp.K, lin.O_idx, mag)
        Q.quaff_outlier_hits(dev_bf16(X), 100, O_d, hits_d, ws)
        torch.cuda.synchronize()
        h = host(hits_d)
        assert h.tolist() == oracle.outlier_hits(X, 100, host(O_d)).tolist()
        tot += h
    assert tot[1] > 0 and tot[0] >= 0.9 * tot[1]          # the paper reports > 90 % for a calibrated set
