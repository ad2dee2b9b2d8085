"""The C-ABI library loads without a GPU and exports every symbol that include/quaff.h declares."""
import ctypes
import os
import re

from paper_2505_14742_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "quaff.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(quaff_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(build.build_library())
    names = _declared()
    assert len(names) >= 8
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names():
    from paper_2505_14742_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    for n in binding.EXPORTS:
        if n not in ("quaff_status_string", "quaff_workspace_bytes"):
            assert callable(getattr(binding, n))


def test_status_strings_and_workspace_sizes_without_gpu():
    from paper_2505_14742_b200 import binding as Q
    assert Q.status_string(0) == "ok"
    assert "align" in Q.status_string(Q.QUAFF_ERR_ALIGNMENT)
    assert Q.workspace_bytes(Q.QUAFF_WS_MOMENTUM, 16, 64, 64, 32, 0) % 256 == 0
    small = Q.workspace_bytes(Q.QUAFF_WS_BWD, 256, 512, 512, 32, 8)
    big = Q.workspace_bytes(Q.QUAFF_WS_BWD, 2048, 3072, 9216, 32, 16)
    assert 0 < small < big


def test_host_only_paths_from_two_threads():
    """Workspace sizes, status strings and argument validation (which returns before any CUDA call) driven from two
    host threads at once give the same answers as from one."""
    import threading
    from paper_2505_14742_b200 import binding as Q
    L = Q.lib()
    shapes = [(256, 512, 512, 32, 8), (2048, 3072, 9216, 32, 16), (8192, 11008, 4096, 64, 64), (512, 2048, 4096, 128, 8)]
    want = [[Q.workspace_bytes(w, *sh) for w in range(8)] for sh in shapes]
    bad = []

    def worker():
        for _ in range(300):
            for sh, ref in zip(shapes, want):
                if [Q.workspace_bytes(w, *sh) for w in range(8)] != ref:
                    bad.append(sh)
            # null pointers / bad sizes: rejected on the host, no device needed
            if L.quaff_qlinear_bwd(16, 64, 64, None, 64, None, 64, None, None, 0, None, 0, None, 0, None, None, 0, None, None, None, 0,
                                   1.0, None, 0, None, None, 0, None, None, None, 0, None) != Q.QUAFF_ERR_INVALID_ARG:
                bad.append("bwd")
            if L.quaff_momentum_apply(None, None, 5000, 0.5, None, None, None) != Q.QUAFF_ERR_UNSUPPORTED_SHAPE:
                bad.append("apply")
            if Q.status_string(Q.QUAFF_ERR_TIMEOUT) != "device-side wait timed out":
                bad.append("str")

    ts = [threading.Thread(target=worker) for _ in range(2)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert not bad, bad[:3]
