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
