"""quaff_momentum_update_static - the entry point for callers that cannot allocate device scratch
(a plug-in in a framework that owns the memory budget, a step that must not hit cudaMalloc's
device-wide synchronisation) - must give exactly what quaff_momentum_update gives with a
caller-supplied workspace.  Checked on two calls in a row, because the built-in scratch array keeps
the previous call's contents and the entry point has to clear it itself; both are also compared with the
CPU oracle's update.  Collected last on purpose."""
import numpy as np
import pytest

import oracle
from util import bf, dev, dev_bf16, host

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row():
    import torch
    from paper_2505_14742_b200 import binding as Q, build
    build.build_library()
    rng = np.random.default_rng(77)
    M, K, nO, gamma = 700, 1024, 45, 0.2
    O = np.sort(rng.permutation(K)[:nO]).astype(np.int32)
    wmax = (0.05 + 0.05 * rng.random(nO)).astype(np.float32)
    s_ws = dev(np.ones(nO, np.float32))
    s_st = dev(np.ones(nO, np.float32))
    out = {k: torch.empty(nO, dtype=torch.float32, device="cuda") for k in ("cm_ws", "be_ws", "cm_st", "be_st")}
    ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_MOMENTUM, M, K, 16, 64, 0), dtype=torch.uint8, device="cuda")
    s_or = np.ones(nO, np.float32)
    for call in range(2):
        x = rng.standard_normal((M, K)).astype(np.float32)
        x[:, O] *= rng.uniform(20, 100, nO).astype(np.float32) / (1 + 3 * call)   # second call: smaller maxima
        X = dev_bf16(bf(x))
        Q.quaff_momentum_update(X, dev(O), dev(wmax), gamma, s_ws, ws, out["cm_ws"], out["be_ws"])
        Q.quaff_momentum_update_static(X, dev(O), dev(wmax), gamma, s_st, out["cm_st"], out["be_st"])
        torch.cuda.synchronize()
        # bit-exact, like every other check of the scale update
        assert np.array_equal(host(out["cm_st"]), host(out["cm_ws"])), f"column maxima, call {call}"
        assert np.array_equal(host(out["be_st"]), host(out["be_ws"])), f"beta, call {call}"
        assert np.array_equal(host(s_st), host(s_ws)), f"s_O, call {call}"
        # and both against the oracle (Eq. 8, Eq. 7), state carried over the two calls
        s_or, cm_or, be_or = oracle.momentum_update(bf(x), O, wmax, gamma, s_or)
        assert np.array_equal(host(out["cm_st"]), cm_or) and np.array_equal(host(out["be_st"]), be_or), f"oracle, call {call}"
        assert np.array_equal(host(s_st), s_or), f"s_O against the oracle, call {call}"
    assert (host(s_st) > 1.0).all()


def test_static_scratch_variant_rejects_too_many_outlier_channels():
    import torch
    from paper_2505_14742_b200 import binding as Q
    K = 8192
    X = torch.zeros((8, K), dtype=torch.bfloat16, device="cuda")
    O = torch.arange(4097, dtype=torch.int32, device="cuda")
    f = torch.ones(4097, dtype=torch.float32, device="cuda")
    with pytest.raises(Q.QuaffError) as e:
        Q.quaff_momentum_update_static(X, O, f, 0.5, f.clone())
    assert e.value.code == Q.QUAFF_ERR_UNSUPPORTED_SHAPE
    torch.cuda.synchronize()
