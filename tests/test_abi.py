"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2505_13254_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "heterospec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hs_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    path = build.build()
    L = ctypes.CDLL(path)
    names = declared_symbols()
    assert set(binding.EXPORTS) == set(names)
    for n in names:
        assert hasattr(L, n), n


def test_status_strings_and_workspace_size_need_no_gpu():
    L = binding.lib()
    assert L.hs_status_string(0) == b"ok"
    assert L.hs_status_string(7) == b"malformed tree"
    assert 256 << 10 < binding.hs_workspace_bytes(1, 60, 128256, 32, 8) < 4 << 20     # counters + chunk partials only
    assert binding.hs_workspace_bytes(0, 60, 128256, 32, 8) == 0


def test_struct_sizes_match_the_header():
    # 7 floats + 10 ints; 14 / 11 pointers; attention descriptor with natural alignment
    assert ctypes.sizeof(binding._Policy) == 4 * 17
    assert ctypes.sizeof(binding._QuantOut) == 8 * 14
    assert ctypes.sizeof(binding._PrunedTree) == 8 * 11
    assert ctypes.sizeof(binding._TreeBatch) == 8 + 3 * 8
    assert ctypes.sizeof(binding._AttnDesc) == 9 * 4 + 4 + 2 * 8 + 2 * 8 + 8
    assert ctypes.sizeof(binding._AcceptOut) == 7 * 8 + 8
    assert ctypes.sizeof(binding._ExpandState) == 3 * 4 + 4 + 9 * 8
