"""The C-ABI library loads and exports what include/snn_conv.h declares.
No compute call is made here (no GPU is needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2110_09195_b200 import build
    build.build()
    from paper_2110_09195_b200 import binding
    return binding.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "snn_conv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(snn_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2110_09195_b200 import binding
    declared = _declared_symbols()
    assert "snn_conv_create" in declared and "snn_conv_forward" in declared and "snn_conv_destroy" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    assert sorted(binding.EXPORTED_SYMBOLS) == declared


def test_version_and_error_strings(lib):
    assert b"sm_100a" in lib.snn_version()
    assert lib.snn_last_error() is not None
    assert lib.snn_kernel_launches() >= 0


def test_argument_errors_need_no_gpu(lib):
    from paper_2110_09195_b200 import binding
    h = ctypes.c_void_p()
    assert lib.snn_conv_create(None, ctypes.byref(h)) == 1
    assert b"null descriptor" in lib.snn_last_error()
    assert lib.snn_conv_destroy(None) == 0
    assert lib.snn_conv_forward(None, None, 1, 8, 8, None, 0, 0, None) == 1
    # bad tau is rejected before any CUDA call
    import numpy as np
    with pytest.raises(binding.SnnError) as ei:
        binding.SnnConv(4, 4, 10, np.zeros(1024, np.uint16), np.zeros(64, np.uint8), np.ones(4, np.float32))
    assert ei.value.status == 1
    cb = np.zeros(32, np.uint16)
    cb[3] = 600
    with pytest.raises(binding.SnnError) as ei:
        binding.SnnConv(4, 4, 5, cb, np.zeros(64, np.uint8), np.ones(4, np.float32))
    assert ei.value.status == 1 and "9-bit" in str(ei.value)
    with pytest.raises(binding.SnnError) as ei:
        binding.SnnConv(4, 4, 5, np.zeros(32, np.uint16), np.zeros(64, np.uint8),
                        np.array([1, np.nan, 1, 1], np.float32))
    assert ei.value.status == 1
    with pytest.raises(binding.SnnError):
        binding.SnnConv(4, 4, 5, np.zeros(32, np.uint16), np.zeros(64, np.uint8), np.ones(4, np.float32), stride=3)


def test_no_device_is_a_loud_error(lib):
    import numpy as np
    import torch
    from paper_2110_09195_b200 import binding
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.SnnError) as ei:
        binding.SnnConv(4, 4, 5, np.zeros(32, np.uint16), np.zeros(64, np.uint8), np.ones(4, np.float32))
    assert ei.value.status == 3 and "no CPU path" in str(ei.value)


def test_product_does_not_touch_the_oracle():
    """The library, its binding and its build step never import or read oracle/."""
    pkg = os.path.join(ROOT, "paper_2110_09195_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2110_09195_b200" not in text and "libsnnconv" not in text
