"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ones.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ones_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2108_03645_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_every_declared_symbol():
    from paper_2108_03645_b200 import binding
    assert sorted(binding._SIGNATURES) == _declared()


def test_calls_that_need_no_device():
    from paper_2108_03645_b200 import binding
    L = binding.lib()
    assert L.ones_workspace_bytes(0, 10) == 0 and L.ones_workspace_bytes(10, 0) == 0
    small, big = L.ones_workspace_bytes(16, 32), L.ones_workspace_bytes(2048, 65536)
    assert 0 < small < 1 << 20
    assert 2 * 65536 * 2048 * 4 <= big < 2 * 65536 * 2048 * 4 + (8 << 20)
    assert L.ones_strerror(0) == b"ok" and b"unknown" in L.ones_strerror(-99)
    assert L.ones_select_top_scratch_bytes(100, 0) == 0 and L.ones_select_top_scratch_bytes(100, 2) > 0
    # argument errors are reported before any CUDA call
    assert L.ones_create(None, None, 1, 1, 1, None, None, 0, None) == -1
    assert L.ones_evolve(None, 1, 0) == -1 and L.ones_destroy(None) == 0
