"""The C-ABI shared library builds for sm_100a, loads on a machine without a GPU, and
exports every symbol include/mpt.h declares.  No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1710_03740_b200 import build, binding
    build.build()
    return binding.lib()


def test_header_symbols_are_exported(lib):
    from paper_1710_03740_b200 import binding
    text = open(os.path.join(ROOT, "include", "mpt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(mpt_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations parsed"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_host_side_validation(lib):
    from paper_1710_03740_b200 import binding
    assert "sm_100a" in binding.mpt_version()
    layers = [(256, 512, 1), (512, 10, 0)]
    n = binding.mpt_workspace_bytes(layers, 64, False)
    n_mom = binding.mpt_workspace_bytes(layers, 64, True)
    P = 256 * 512 + 512 * 10
    assert n >= P * 8 and n_mom >= n + P * 4
    # chain mismatch, ReLU on the last layer, empty list, null out-pointer
    with pytest.raises(binding.MptError) as e:
        binding.mpt_workspace_bytes([(256, 512, 1), (500, 10, 0)], 64, False)
    assert e.value.code == -2
    with pytest.raises(binding.MptError):
        binding.mpt_workspace_bytes([(256, 512, 1), (512, 10, 1)], 64, False)
    with pytest.raises(binding.MptError):
        binding.mpt_workspace_bytes(layers, 0, False)
    arr = binding._layer_array(layers)
    assert lib.mpt_workspace_bytes(arr, 2, 64, 0, None) == -1
    # mpt_create argument checks that fail before any CUDA call
    ctx = ctypes.c_void_p()
    assert lib.mpt_create(arr, 2, 1024.0, 0.01, 0.0, 64, None, 0, None, ctypes.byref(ctx)) == -1
    assert lib.mpt_create(arr, 2, 0.0, 0.01, 0.0, 64, ctypes.c_void_p(256), 1 << 30, None, ctypes.byref(ctx)) == -1
    assert lib.mpt_create(arr, 2, 1024.0, 0.01, 1.0, 64, ctypes.c_void_p(256), 1 << 30, None, ctypes.byref(ctx)) == -1
    assert lib.mpt_create(arr, 2, 1024.0, 0.01, 0.0, 64, ctypes.c_void_p(260), 1 << 30, None, ctypes.byref(ctx)) == -4
    assert lib.mpt_create(arr, 2, 1024.0, 0.01, 0.0, 64, ctypes.c_void_p(256), 16, None, ctypes.byref(ctx)) == -4
    # null context
    assert lib.mpt_forward(None, None, 1) == -1
    assert lib.mpt_step(None, None) == -1
    assert lib.mpt_last_error(None) == b"null context"
