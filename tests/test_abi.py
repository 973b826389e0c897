"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "subgen.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(subgen_[a-z_0-9]+)\s*\(", src)))


def test_header_symbols_are_exported():
    from paper_2402_06082_b200 import binding, build
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), "missing export " + n
    assert set(names) == set(binding.EXPORTS)


def test_invalid_configuration_is_rejected_on_the_host():
    from paper_2402_06082_b200 import binding
    L = binding.load()
    cfg = binding.SubgenConfig(1, 4, 3, 128, 0.5, 8, 64, 16, 0, binding.DTYPE_BF16, 0, 0, None, 0, None)
    assert L.subgen_workspace_bytes(ctypes.byref(cfg)) == 0          # H not a multiple of Hkv
    assert b"multiple" in L.subgen_last_error()
    cfg = binding.SubgenConfig(1, 4, 4, 96, 0.5, 8, 64, 16, 0, binding.DTYPE_BF16, 0, 0, None, 0, None)
    assert L.subgen_workspace_bytes(ctypes.byref(cfg)) == 0          # unsupported head dimension
    cfg = binding.SubgenConfig(2, 4, 4, 128, 0.5, 8, 64, 16, 0, binding.DTYPE_BF16, 128, 0, None, 0, None)
    n = L.subgen_workspace_bytes(ctypes.byref(cfg))
    assert n > 2 * 4 * 128 * (1 + 8) * 128 * 2                       # at least the cluster arrays


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    from paper_2402_06082_b200 import binding
    with pytest.raises(binding.SubgenError):
        binding.SubGen(1, 1, 64, 0.5, 4, 16, 8)
    L = binding.load()
    assert not L.subgen_create(1, 1, 64, 0.5, 4, 16, 8, 0)
    assert b"no usable CUDA device" in L.subgen_last_error()
