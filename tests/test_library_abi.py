"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2604_26881_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "faasmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = declared_functions()
    assert "moe_layer_forward" in names and "moe_route" in names and len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in faasmoe.h but not exported"
    assert sorted(binding.EXPORTS) == names, "binding and header disagree on the entry points"


def test_strerror_and_null_checks_need_no_gpu():
    lib = binding.load_library()
    assert binding.strerror(0) == "ok"
    assert "G" in binding.strerror(binding.MOE_ERR_G)
    # host-detectable argument errors return before any CUDA call
    assert lib.moe_create(None, None) == binding.MOE_ERR_NULL
    assert lib.moe_destroy(None) == binding.MOE_ERR_NULL
    assert lib.moe_layer_forward(None, 0, None, None, 1, 1, None, None) == binding.MOE_ERR_NULL
    assert lib.moe_launch_count(None) == -1
    bad = binding.MoeConfig(250, 8, 128, 2, 0, 1, 1, 8, 8, 1, 1e-6)
    ctx = ctypes.c_void_p()
    assert lib.moe_create(ctypes.byref(bad), ctypes.byref(ctx)) == binding.MOE_ERR_SHAPE
