"""The C-ABI library loads and exports every symbol include/pivot.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2607_24593_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "pivot.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b([a-z_0-9]+)\s*\(", text)) - {"defined"})


def test_library_builds_and_exports_declared_symbols():
    lib = ctypes.CDLL(build.build())
    names = declared_symbols()
    assert "pivot_index_prefill" in names and "pivot_index_decode" in names and "dense_index" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_symbols():
    from paper_2607_24593_b200 import binding
    assert sorted(binding.SYMBOLS) == declared_symbols()
    s = binding.lib.pivot_status_str
    assert s(0) == b"ok" and b"workspace" in s(3)
    assert binding.pivot_workspace_bytes(2048, 512, 512, 256) > 0
    assert binding.pivot_workspace_bytes(0, 1, 1, 1) == 0
