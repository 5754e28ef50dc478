"""The C-ABI library builds, loads and exports every function `include/dbp.h` declares
(no compute calls here: this runs without a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "dbp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+char\s*\*\s*|unsigned\s+long\s+long\s+|long\s+long\s+|int\s+)(\w+)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_header_declares_the_boundary():
    names = _declared_functions()
    for must in ("nsd_quantize", "dithered_linear_backward", "dithered_conv_backward"):
        assert must in names
    assert len(names) >= 14


def test_library_exports_every_declared_symbol():
    from paper_2004_04729_b200 import build, binding
    lib = ctypes.CDLL(build.build())
    for name in _declared_functions():
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTED_SYMBOLS) == _declared_functions()


def test_host_side_argument_checks_need_no_gpu():
    from paper_2004_04729_b200 import binding
    lib = binding.load_library()
    assert lib.dbp_status_string(0) == b"ok"
    assert lib.dbp_status_string(-2) == b"unsupported configuration"
    b, o, v = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    assert lib.dbp_sparse_bytes(0, ctypes.byref(b), ctypes.byref(o), ctypes.byref(v)) == -1
    assert lib.dbp_sparse_bytes(1025, ctypes.byref(b), ctypes.byref(o), ctypes.byref(v)) == 0
    assert (b.value, o.value, v.value) == (2 * 32 * 4, 2 * 32 * 2, 2048)
    assert lib.dbp_destroy(None) == -1
    # per-layer seeds: output l of the SplitMix64 sequence started at the seed (published vector:
    # the first outputs for seed 0)
    assert lib.dbp_layer_seed(0, 0) == 0xE220A8397B1DCDAF
    assert lib.dbp_layer_seed(0, 1) == 0x6E789E6AA1B965F4
    assert lib.nsd_quantize(None, None, 0, 10, 0, 2.0, None, None) == -1
    # unsupported kernel size is refused before anything touches the device
    assert lib.dithered_conv_backward(None, None, None, None, 0, 1, 1, 1, 4, 4, 7, 1, 3, 0, 2.0,
                                      None, None, None, None, None, 0) == -2


def test_binding_refuses_to_run_without_cuda():
    import torch
    from paper_2004_04729_b200 import Context
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(RuntimeError):
        Context(0)
