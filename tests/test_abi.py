"""The C-ABI library loads on a machine without a GPU and exports what include/fdg.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2509_05679_b200 import build
    return build.build_lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fdg.h")).read()
    return sorted(set(re.findall(r"FDG_API[^;(]*?\b(fdg_\w+)\s*\(", text)))


def test_header_declares_the_three_core_entry_points():
    names = declared_symbols()
    for core in ("fdg_create", "fdg_step", "fdg_params"):
        assert core in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_covers_every_declared_symbol(libpath):
    from paper_2509_05679_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()
    binding.lib()


def test_create_without_a_device_reports_an_error_instead_of_falling_back(libpath):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2509_05679_b200 import binding, synth
    with pytest.raises(binding.FdgError):
        binding.Context(synth.mlp_layers([8, 4, 3]), [2], 1, 2, 0.1, dtype="fp32", in_shape=(1, 1, 8), num_classes=3)
    # straight through the C ABI: FDG_ERR_ARCH and a message, no crash
    L = binding.lib()
    layers = (binding.fdg_layer * 1)(binding.fdg_layer(0, 8, 3, 1, 1))
    opt = binding.fdg_options(0, 1, 1, 8, 3, 0, 0, 0, None)
    h = ctypes.c_void_p()
    st = L.fdg_create(layers, 1, None, 1, 1, 2, 0.1, ctypes.byref(opt), None, ctypes.byref(h))
    assert st == 4 and not h.value
    assert b"CUDA" in L.fdg_last_error(None)
