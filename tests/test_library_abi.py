"""The C-ABI library loads and exports every symbol include/cake.h declares
(no compute calls: runs without a GPU)."""
import ctypes
import os
import re

from paper_2503_12491_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cake.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cake_[a-z0-9_]+)\s*\(", text)))


def test_header_and_binding_list_the_same_entry_points():
    assert declared_symbols() == sorted(binding.EXPORTS)


def test_library_builds_loads_and_exports_everything():
    path = build.build()
    lib = ctypes.CDLL(path)
    for name in declared_symbols():
        assert hasattr(lib, name), name
    lib.cake_strerror.restype = ctypes.c_char_p
    lib.cake_strerror.argtypes = [ctypes.c_int32]
    assert lib.cake_strerror(0) == b"ok"
    assert b"order" in lib.cake_strerror(-7)
    lib.cake_launch_count.restype = ctypes.c_int64
    assert lib.cake_launch_count() == 0


def test_config_struct_matches_header_layout():
    # 9 int32, 3 float, int64, int32 (+pad), int64, 2 int32, float (+pad)
    assert ctypes.sizeof(binding.CakeConfig) == 88
    assert binding.CakeConfig.total_budget.offset == 48
    assert binding.CakeConfig.max_total_tokens.offset == 64
    assert binding.CakeConfig.indicator_mode.offset == 72
    assert binding.CakeConfig.alloc_mode.offset == 76
    assert binding.CakeConfig.pyramid_slope.offset == 80


def test_argument_errors_need_no_gpu():
    lib = binding.load_library()
    assert lib.cake_create(None, None) == binding.CAKE_ERR_ARG
    h = ctypes.c_void_p()
    bad = binding.CakeConfig(4, 4, 3, 64, 16, 5, 0, 0, 0, 1.0, 1.0, 1.0, 512, 1, 512)   # 4 % 3 != 0
    assert lib.cake_create(ctypes.byref(bad), ctypes.byref(h)) == binding.CAKE_ERR_ARG
    small = binding.CakeConfig(4, 4, 4, 64, 16, 5, 0, 0, 0, 1.0, 1.0, 1.0, 63, 1, 512)  # B < L*S_w
    assert lib.cake_create(ctypes.byref(small), ctypes.byref(h)) == binding.CAKE_ERR_BUDGET
    even = binding.CakeConfig(4, 4, 4, 64, 16, 4, 0, 0, 0, 1.0, 1.0, 1.0, 512, 1, 512)  # even kernel
    assert lib.cake_create(ctypes.byref(even), ctypes.byref(h)) == binding.CAKE_ERR_ARG
    mode = binding.CakeConfig(4, 4, 4, 64, 16, 5, 0, 0, 0, 1.0, 1.0, 1.0, 512, 1, 512, 5)  # no such indicator
    assert lib.cake_create(ctypes.byref(mode), ctypes.byref(h)) == binding.CAKE_ERR_ARG
    alloc = binding.CakeConfig(4, 4, 4, 64, 16, 5, 0, 0, 0, 1.0, 1.0, 1.0, 512, 1, 512, 0, 3)  # no such allocation
    assert lib.cake_create(ctypes.byref(alloc), ctypes.byref(h)) == binding.CAKE_ERR_ARG
    slope = binding.CakeConfig(4, 4, 4, 64, 16, 5, 0, 0, 0, 1.0, 1.0, 1.0, 512, 1, 512, 0, 2, 1.5)
    assert lib.cake_create(ctypes.byref(slope), ctypes.byref(h)) == binding.CAKE_ERR_ARG
    assert lib.cake_begin(None, 0, None, None) == binding.CAKE_ERR_ARG
    assert lib.cake_allocate(None, 0, None) == binding.CAKE_ERR_ARG
