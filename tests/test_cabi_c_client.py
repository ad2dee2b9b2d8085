"""The boundary is a C ABI: a plain C11 program (gcc, no C++, no Python) includes include/quaff.h, links libquaff.so and
runs two steps of the path.  Without a GPU the program is compiled and linked; with one it runs and its output file is
compared with the CPU oracle."""
import os
import struct
import subprocess

import numpy as np
import pytest

from paper_2505_14742_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def _compile(tmp_path):
    lib = build.build_library()
    exe = str(tmp_path / "cabi_client")
    cmd = ["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-pedantic", "-O1",
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
           os.path.join(ROOT, "tests", "cabi_client", "client.c"), "-o", exe,
           lib, "-L", os.path.join(CUDA, "lib64"), "-lcudart",
           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(CUDA, "lib64")]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    return exe


def test_header_is_valid_c11_and_a_c_program_links(tmp_path):
    assert os.path.exists(_compile(tmp_path))


@pytest.mark.gpu
def test_c_program_runs_the_path_and_matches_the_oracle(tmp_path):
    import oracle
    from paper_2505_14742_b200 import synth
    exe = _compile(tmp_path)
    M, K, nO, gamma = 300, 3088, 33, 0.2
    nOp = 64
    rng = np.random.default_rng(4242)
    O = np.sort(rng.permutation(K)[:nO]).astype(np.int32)
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[:, O] *= rng.uniform(20, 100, nO).astype(np.float32)
    X = synth.f32_to_bf16_bits(x)
    wmax = (0.05 + 0.05 * rng.random(nO)).astype(np.float32)
    s0 = (1.0 + rng.random(nO)).astype(np.float32)
    fin, fout = str(tmp_path / "in.bin"), str(tmp_path / "out.bin")
    with open(fin, "wb") as f:
        f.write(struct.pack("<4if", M, K, nO, nOp, gamma))
        f.write(X.tobytes()); f.write(O.tobytes()); f.write(wmax.tobytes()); f.write(s0.tobytes())
    r = subprocess.run([exe, fin, fout], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    raw = open(fout, "rb").read()
    s_new = np.frombuffer(raw, np.float32, nO, 0)
    Xq = np.frombuffer(raw, np.int8, M * K, 4 * nO).reshape(M, K)
    xqo = np.frombuffer(raw, np.int8, M * nOp, 4 * nO + M * K).reshape(M, nOp)
    dx = np.frombuffer(raw, np.float32, M, 4 * nO + M * K + M * nOp)
    os_, _, _ = oracle.momentum_update(X, O, wmax, gamma, s0)
    oXq, oxqo, odx = oracle.quant_act(X, O, os_, nOp)
    assert np.array_equal(s_new, os_)
    assert np.array_equal(Xq, oXq) and np.array_equal(xqo, oxqo) and np.array_equal(dx, odx)
