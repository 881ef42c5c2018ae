"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2605_23764_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "moe_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_host_side_queries_work_without_a_gpu():
    build.build()
    assert binding.moe_strerror(0) == "ok" and "wait" in binding.moe_strerror(2)
    nbytes = binding.moe_workspace_bytes(256, 256, 8, 2, 0, 128, 0)
    assert nbytes > 256 * 2 * 256 * 2
    assert binding.moe_workspace_bytes(256, 250, 8, 2, 0, 128, 0) == 0  # d % 8 != 0 is rejected
    assert binding.moe_workspace_bytes(256, 256, 8, 9, 0, 128, 0) == 0  # k > E
    train = binding.moe_workspace_bytes(256, 256, 8, 2, 0, 128, binding.MOE_FLAG_SAVE_FOR_BWD)
    assert train > nbytes
