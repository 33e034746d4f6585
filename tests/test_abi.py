"""Host-side checks that need no GPU: the built library exports the declared C ABI."""
import ctypes
import os
import re

import pytest

from paper_2602_03203_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fkv_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_host_argument_checks_need_no_device():
    lib = binding.lib()
    cfg = binding.FkvConfig(36, 8, 4, 128, 1, 16, 16, 0, 8192, 0, 32768, 0)
    n = ctypes.c_size_t(0)
    assert lib.fkv_workspace_bytes(ctypes.byref(cfg), ctypes.byref(n)) == 0
    # Qwen3-4B shape at 32K: the pool alone holds 288 segments x 2048 pages x 9792 bytes.
    assert n.value > 288 * 2048 * 9792
    for field, bad in [("head_dim", 96), ("page_size", 32), ("scorer_hidden", 32), ("group_size", 9), ("budget", 0)]:
        c2 = binding.FkvConfig(36, 8, 4, 128, 1, 16, 16, 0, 8192, 0, 32768, 0)
        setattr(c2, field, bad)
        assert lib.fkv_workspace_bytes(ctypes.byref(c2), ctypes.byref(n)) == -1, field
    assert lib.fkv_workspace_bytes(None, ctypes.byref(n)) == -1
    assert lib.fkv_evict(None, 0, None) == -1 and lib.fkv_decode_attn(None, 0, None, None, ctypes.c_float(0), None) == -1


def test_no_cpu_path():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(RuntimeError):
        binding.Cache(1, 2, 4, 64, 1, 64, 128)
