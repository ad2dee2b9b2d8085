"""Error behaviour of every C-ABI entry point, as include/quaff.h states it: arguments are checked on the host before
anything is enqueued, and each kind of mistake has its own status code.

The checks run in a child process that sees NO CUDA device (CUDA_VISIBLE_DEVICES is empty), with made-up addresses that
are never dereferenced on the host: a call that is rejected returns its code without touching CUDA, and a call whose
arguments are all valid gets as far as the first CUDA call and reports QUAFF_ERR_CUDA - the library has no CPU path to
fall back to."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import json, sys
from paper_2505_14742_b200 import binding as Q
L = Q.lib()
OK, INV, SHAPE, ALIGN, WS, CUDA = 0, 1, 2, 3, 4, 5
BIG = 1 << 40                                   # "enough workspace"


def P(i):                                       # distinct made-up device addresses, 4096-byte aligned
    return 0x7F0000000000 + i * 0x100000


bad = []


def run(fn, base, cases):
    """base: dict of named arguments in call order, all valid; cases: (changes, expected status)."""
    f = getattr(L, fn)
    names = list(base)
    got = f(*[base[n] for n in names])
    if got != CUDA:
        bad.append((fn, "valid arguments, no device", got, CUDA))
    before = L.quaff_debug_launch_count()
    for changes, want in cases:
        a = dict(base)
        a.update(changes)
        got = f(*[a[n] for n in names])
        if got != want:
            bad.append((fn, {k: (v if not isinstance(v, int) or v < 1 << 32 else hex(v)) for k, v in changes.items()}, got, want))
    if L.quaff_debug_launch_count() != before:
        bad.append((fn, "a rejected call launched something", 0, 0))


M, K, N, nO, nOp, r = 64, 256, 128, 5, 32, 16

run("quaff_prepare_weight",
    dict(Wt=P(1), ldw=K, N=N, K=K, O=P(2), nO=nO, Wq=P(3), ldwq=K, dW=P(4), W_O=P(5), ldwo=N, wmax=P(6), st=None),
    [({"Wt": None}, INV), ({"Wq": None}, INV), ({"dW": None}, INV), ({"N": 0}, INV), ({"K": -1}, INV), ({"ldw": K - 8}, INV),
     ({"ldwq": K - 16}, INV), ({"nO": -1}, INV), ({"nO": K + 1}, INV), ({"O": None}, INV), ({"W_O": None}, INV),
     ({"wmax": None}, INV), ({"ldwo": N - 1}, INV), ({"nO": 4097, "K": 8192, "ldw": 8192, "ldwq": 8192}, SHAPE),
     ({"Wt": P(1) + 2}, ALIGN), ({"Wq": P(3) + 8}, ALIGN), ({"ldw": K + 4}, ALIGN), ({"ldwq": K + 8}, ALIGN)])

mom = dict(X=P(1), ldx=K, M=M, K=K, O=P(2), nO=nO, wmax=P(3), gamma=0.5, s=P(4), colmax=None, beta=None, ws=P(5), wsb=BIG, st=None)
mom_cases = [({"X": None}, INV), ({"M": -1}, INV), ({"K": 0}, INV), ({"ldx": K - 1}, INV), ({"nO": -1}, INV), ({"nO": K + 1}, INV),
             ({"O": None}, INV), ({"gamma": -0.01}, INV), ({"gamma": 1.5}, INV), ({"gamma": float("nan")}, INV),
             ({"wmax": None}, INV), ({"s": None}, INV), ({"nO": 4097, "K": 8192, "ldx": 8192}, SHAPE)]
run("quaff_momentum_update", mom, mom_cases + [({"ws": None}, WS), ({"wsb": 8}, WS)])
mom_static = {k: v for k, v in mom.items() if k not in ("ws", "wsb")}
run("quaff_momentum_update_static", mom_static, mom_cases)

run("quaff_outlier_colmax",
    dict(X=P(1), ldx=K, M=M, K=K, O=P(2), nO=nO, colmax=P(3), ws=P(4), wsb=BIG, st=None),
    [({"X": None}, INV), ({"M": -1}, INV), ({"K": 0}, INV), ({"ldx": K - 1}, INV), ({"nO": K + 1}, INV), ({"O": None}, INV),
     ({"colmax": None}, INV), ({"nO": 4097, "K": 8192, "ldx": 8192}, SHAPE), ({"ws": None}, WS), ({"wsb": 8}, WS)])

run("quaff_momentum_apply",
    dict(colmax=P(1), wmax=P(2), nO=nO, gamma=0.9, s=P(3), beta=None, st=None),
    [({"nO": -1}, INV), ({"gamma": 2.0}, INV), ({"gamma": float("nan")}, INV), ({"colmax": None}, INV), ({"wmax": None}, INV),
     ({"s": None}, INV), ({"nO": 4097}, SHAPE)])

run("quaff_quant_act",
    dict(X=P(1), ldx=K, M=M, K=K, O=P(2), nO=nO, s=P(3), Xq=P(4), ldxq=K, xqo=P(5), ldxo=nOp, nOp=nOp, dx=P(6), st=None),
    [({"X": None}, INV), ({"Xq": None}, INV), ({"dx": None}, INV), ({"M": -1}, INV), ({"K": 0}, INV), ({"nO": K + 1}, INV),
     ({"O": None}, INV), ({"s": None}, INV), ({"nOp": nO - 1}, INV), ({"xqo": None}, INV), ({"ldx": K - 8}, INV),
     ({"ldxq": K - 16}, INV), ({"ldxo": nOp - 16}, INV), ({"X": P(1) + 2}, ALIGN), ({"Xq": P(4) + 4}, ALIGN),
     ({"ldx": K + 4}, ALIGN), ({"ldxq": K + 8}, ALIGN)])

run("quaff_requant_weight_rows",
    dict(W_O=P(1), ldwo=N, nO=nO, N=N, s=P(2), wq=P(3), ldwq=nOp, nOp=nOp, dw=P(4), st=None),
    [({"nO": -1}, INV), ({"N": 0}, INV), ({"nOp": 0}, INV), ({"dw": None}, INV), ({"W_O": None}, INV), ({"s": None}, INV),
     ({"ldwo": N - 1}, INV), ({"wq": None}, INV), ({"ldwq": nOp - 16}, INV), ({"nOp": 40, "ldwq": 48}, SHAPE),
     ({"wq": P(3) + 8}, ALIGN), ({"ldwq": nOp + 8}, ALIGN)])

run("quaff_outlier_count",
    dict(X=P(1), ldx=K, M=M, K=K, thr=100, xi=P(2), ws=P(3), wsb=BIG, st=None),
    [({"X": None}, INV), ({"xi": None}, INV), ({"M": 0}, INV), ({"K": 0}, INV), ({"ldx": K - 8}, INV), ({"thr": -1}, INV),
     ({"X": P(1) + 2}, ALIGN), ({"ldx": K + 4}, ALIGN), ({"ws": None}, WS), ({"ws": P(3) + 4}, WS), ({"wsb": 16}, WS)])

run("quaff_outlier_hits",
    dict(X=P(1), ldx=K, M=M, K=K, thr=100, O=P(2), nO=nO, hits=P(3), ws=P(4), wsb=BIG, st=None),
    [({"X": None}, INV), ({"hits": None}, INV), ({"M": 0}, INV), ({"K": 0}, INV), ({"ldx": K - 8}, INV), ({"thr": -1}, INV),
     ({"nO": -1}, INV), ({"nO": K + 1}, INV), ({"O": None}, INV), ({"X": P(1) + 2}, ALIGN), ({"ldx": K + 4}, ALIGN),
     ({"ws": None}, WS), ({"wsb": 16}, WS)])

run("quaff_select_outliers",
    dict(xi=P(1), K=K, nO=nO, O=P(2), ws=P(3), wsb=BIG, st=None),
    [({"xi": None}, INV), ({"K": 0}, INV), ({"nO": -1}, INV), ({"nO": K + 1}, INV), ({"O": None}, INV), ({"ws": None}, WS),
     ({"wsb": 16}, WS)])

run("quaff_lora_down",
    dict(X=P(1), ldx=K, M=M, K=K, A=P(2), r=r, T=P(3), status=None, ws=P(4), wsb=BIG, st=None),
    [({"M": -1}, INV), ({"K": 0}, INV), ({"r": 0}, INV), ({"X": None}, INV), ({"A": None}, INV), ({"T": None}, INV),
     ({"ldx": K - 8}, INV), ({"r": 12}, SHAPE), ({"r": 72}, SHAPE), ({"K": K - 4}, SHAPE), ({"X": P(1) + 2}, ALIGN),
     ({"T": P(3) + 2}, ALIGN), ({"ldx": K + 4}, ALIGN), ({"ws": None}, WS), ({"ws": P(4) + 4}, WS), ({"wsb": 64}, WS)])

run("quaff_qlinear_fwd",
    dict(M=M, K=K, N=N, Xq=P(1), ldxq=K, xqo=P(2), ldxo=nOp, nOp=nOp, dx=P(3), Wq=P(4), ldwq_main=K, dW=P(5), wqo=P(6), ldwq=nOp,
         dwo=P(7), X=P(8), ldx=K, A=P(9), B=P(10), r=r, scale=2.0, T=P(11), Y=P(12), ydt=Q.QUAFF_BF16, ldy=N, acc1=None, acc2=None,
         status=None, ws=P(13), wsb=BIG, st=None),
    [({"M": -1}, INV), ({"K": 0}, INV), ({"N": 0}, INV), ({"nOp": -32}, INV), ({"r": -8}, INV), ({"Xq": None}, INV), ({"dx": None}, INV),
     ({"Wq": None}, INV), ({"dW": None}, INV), ({"Y": None}, INV), ({"ldxq": K - 16}, INV), ({"ldwq_main": K - 16}, INV),
     ({"ldy": N - 8}, INV), ({"xqo": None}, INV), ({"wqo": None}, INV), ({"dwo": None}, INV), ({"ldxo": 16}, INV), ({"ldwq": 16}, INV),
     ({"B": None}, INV), ({"T": None}, INV), ({"A": None}, INV), ({"ldx": K - 8}, INV), ({"ydt": 7}, INV),
     ({"nOp": 48, "ldxo": 48, "ldwq": 48}, SHAPE), ({"r": 12}, SHAPE), ({"r": 72}, SHAPE), ({"N": N - 4, "ldy": N}, SHAPE),
     ({"Xq": P(1) + 8}, ALIGN), ({"Wq": P(4) + 8}, ALIGN), ({"ldxq": K + 8}, ALIGN), ({"ldwq_main": K + 8}, ALIGN),
     ({"xqo": P(2) + 8}, ALIGN), ({"wqo": P(6) + 8}, ALIGN), ({"ldxo": nOp + 8}, ALIGN), ({"ldwq": nOp + 8}, ALIGN),
     ({"T": P(11) + 2}, ALIGN), ({"B": P(10) + 2}, ALIGN), ({"X": P(8) + 2}, ALIGN), ({"ldx": K + 4}, ALIGN), ({"Y": P(12) + 2}, ALIGN),
     ({"ws": None}, WS), ({"ws": P(13) + 4}, WS), ({"wsb": 64}, WS)])

bwd = dict(M=M, K=K, N=N, dY=P(1), lddy=N, Wq=P(2), ldwq_main=K, dW=P(3), wqo=P(4), ldwq=nOp, dwo=P(5), nOp=nOp, O=P(6), nO=nO, s=P(7),
           X=P(8), ldx=K, T=P(9), A=P(10), B=P(11), r=r, scale=2.0, dX=P(12), lddx=K, dA=P(13), dB=P(14), acc=0, G=None)
bwd_cases = [({"M": -1}, INV), ({"K": 0}, INV), ({"N": 0}, INV), ({"nOp": -32}, INV), ({"nO": -1}, INV), ({"nO": nOp + 1}, INV),
             ({"r": -8}, INV), ({"dY": None}, INV), ({"lddy": N - 8}, INV), ({"Wq": None}, INV), ({"dW": None}, INV),
             ({"ldwq_main": K - 16}, INV), ({"wqo": None}, INV), ({"dwo": None}, INV), ({"ldwq": 16}, INV), ({"O": None}, INV),
             ({"s": None}, INV), ({"A": None}, INV), ({"B": None}, INV), ({"dA": None}, INV), ({"dB": None}, INV), ({"X": None}, INV),
             ({"T": None}, INV), ({"ldx": K - 8}, INV), ({"lddx": K - 8}, INV),
             ({"nOp": 48, "ldwq": 48}, SHAPE), ({"r": 12}, SHAPE), ({"r": 72}, SHAPE),
             ({"dY": P(1) + 2}, ALIGN), ({"lddy": N + 4}, ALIGN), ({"Wq": P(2) + 8}, ALIGN), ({"ldwq_main": K + 8}, ALIGN),
             ({"wqo": P(4) + 8}, ALIGN), ({"ldwq": nOp + 8}, ALIGN), ({"dX": P(12) + 2}, ALIGN), ({"lddx": K + 4}, ALIGN),
             ({"A": P(10) + 2}, ALIGN), ({"B": P(11) + 2}, ALIGN), ({"G": P(15) + 2}, ALIGN), ({"X": P(8) + 2}, ALIGN),
             ({"T": P(9) + 2}, ALIGN), ({"dA": P(13) + 4}, ALIGN), ({"dB": P(14) + 4}, ALIGN), ({"ldx": K + 4}, ALIGN),
             ({"dW": P(3) + 4}, ALIGN),
             ({"ws": None}, WS), ({"ws": P(16) + 4}, WS), ({"wsb": 64}, WS)]
tail = dict(status=None, ws=P(16), wsb=BIG, st=None)
run("quaff_qlinear_bwd", {**bwd, **tail},
    bwd_cases + [({"N": N - 4, "lddy": N}, SHAPE), ({"dwo": P(5) + 4}, ALIGN),
                 ({"K": 32776, "ldwq_main": 32784, "ldx": 32776, "lddx": 32776}, SHAPE)])
run("quaff_qlinear_bwd_int8", {**bwd, "dbg": None, **tail},
    bwd_cases + [({"dX": None}, INV), ({"N": N - 8, "lddy": N}, SHAPE), ({"N": 16400, "lddy": 16400}, SHAPE)])

run("quaff_quant_grad",
    dict(dY=P(1), lddy=N, M=M, N=N, dW=P(2), Zq=P(3), ldz=N, dz=P(4), st=None),
    [({"dY": None}, INV), ({"dW": None}, INV), ({"Zq": None}, INV), ({"dz": None}, INV), ({"M": -1}, INV), ({"N": 0}, INV),
     ({"lddy": N - 8}, INV), ({"ldz": N - 16}, INV), ({"N": N - 8}, SHAPE), ({"N": 16400, "lddy": 16400, "ldz": 16400}, SHAPE),
     ({"dY": P(1) + 2}, ALIGN), ({"Zq": P(3) + 8}, ALIGN), ({"dW": P(2) + 4}, ALIGN), ({"lddy": N + 4}, ALIGN), ({"ldz": N + 8}, ALIGN)])

# empty batches are valid and need no device at all
f = dict(M=0, K=K, N=N, Xq=P(1), ldxq=K, xqo=P(2), ldxo=nOp, nOp=nOp, dx=P(3), Wq=P(4), ldwq_main=K, dW=P(5), wqo=P(6), ldwq=nOp,
         dwo=P(7), X=P(8), ldx=K, A=P(9), B=P(10), r=r, scale=2.0, T=P(11), Y=P(12), ydt=Q.QUAFF_BF16, ldy=N, acc1=None, acc2=None,
         status=None, ws=P(13), wsb=BIG, st=None)
empty = [L.quaff_lora_down(P(1), K, 0, K, P(2), r, P(3), None, P(4), BIG, None),
         L.quaff_qlinear_fwd(*f.values()),
         L.quaff_quant_act(P(1), K, 0, K, P(2), nO, P(3), P(4), K, P(5), nOp, nOp, P(6), None),
         L.quaff_quant_grad(P(1), N, 0, N, P(2), P(3), N, P(4), None),
         # backward of an empty batch that accumulates (or wants no LoRA gradients) has nothing to store either
         L.quaff_qlinear_bwd(*{**bwd, "M": 0, "acc": 1, **tail}.values()),
         L.quaff_qlinear_bwd(*{**bwd, "M": 0, "dA": None, "dB": None, **tail}.values()),
         L.quaff_qlinear_bwd_int8(*{**bwd, "M": 0, "acc": 1, "dbg": None, **tail}.values())]
for which in range(8):                          # sizes of an empty batch are defined (and small)
    empty.append(0 if 0 <= Q.workspace_bytes(which, 0, K, N, nOp, r) < (1 << 24) else 1)
print(json.dumps({"bad": [list(map(str, b)) for b in bad], "empty": empty}))
'''


def test_every_entry_point_rejects_bad_arguments_with_the_documented_status():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, (r.stdout[-2000:], r.stderr[-2000:])
    out = json.loads(r.stdout.strip().splitlines()[-1])
    assert out["bad"] == [], out["bad"]
    assert out["empty"] == [0] * len(out["empty"])
