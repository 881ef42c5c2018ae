"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2605_23764_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        text = open(os.path.join(inc, f)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


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


def test_binding_refuses_undersized_tensors_before_the_call():
    """An undersized output would let a layout kernel write out of bounds on the device; the binding raises
    instead (checked before any device work, so this runs without a GPU)."""
    import pytest
    import torch
    T, E, k, S = 16, 4, 2, 1
    i32 = torch.int32
    ids = torch.zeros(T, k, dtype=i32)
    good = dict(counts=torch.zeros(E + S, dtype=i32), offsets=torch.zeros(E + S + 1, dtype=i32),
                row_of=torch.zeros(T * (k + S), dtype=i32), src_of=torch.zeros(T * (k + S), dtype=i32))
    for name in good:
        bad = dict(good)
        bad[name] = good[name][:-1].clone()
        with pytest.raises(binding.MoeError, match=name):
            binding.moe_layout_noalloc(ids, T, E, k, S, bad["counts"], bad["offsets"], bad["row_of"], bad["src_of"])
    with pytest.raises(binding.MoeError, match="topk_ids"):
        binding.moe_layout_noalloc(ids[:-1].clone(), T, E, k, S, *good.values())
    with pytest.raises(binding.MoeError, match="status2"):
        binding.moe_layout_noalloc(ids, T, E, k, S, *good.values(), status2=torch.zeros(1, dtype=i32))
    # calls on a context: the handle must be known, and sizes are checked against the context's shape
    import ctypes
    fake = ctypes.c_void_p(12345)
    with pytest.raises(binding.MoeError, match="unknown context"):
        binding.moe_layout(fake, ids, T)
    binding._CTX_SHAPE[fake.value] = (T, 64, E, k, S, 32, 0)
    try:
        with pytest.raises(binding.MoeError, match="row_of"):
            binding.moe_layout(fake, ids, T, row_of=torch.zeros(T * (k + S) - 1, dtype=i32))
        with pytest.raises(binding.MoeError, match="topk_w"):
            binding.moe_route(fake, torch.zeros(T, E), T, ids, torch.zeros(T * k - 1))
        with pytest.raises(binding.MoeError, match="W_down"):
            bf = torch.bfloat16
            binding.moe_ffn_fwd(fake, torch.zeros(T, 64, dtype=bf), ids, torch.zeros(T, k), torch.zeros(E + S, 64, 64, dtype=bf),
                                torch.zeros(E + S, 64, 31, dtype=bf), torch.zeros(T, 64, dtype=bf), T)
    finally:
        binding._CTX_SHAPE.pop(fake.value)
