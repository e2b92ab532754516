"""The C-ABI library loads and exports every symbol include/gear.h declares (no compute calls, no GPU)."""
import ctypes
import os
import re

from paper_2403_05527_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gear_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    handle = ctypes.CDLL(path)
    names = declared_symbols()
    assert {"gear_compress", "gear_append_buffer", "gear_decode_attn", "gear_free"} <= set(names)
    for name in names:
        assert hasattr(handle, name), name
    assert set(names) == set(binding._SIGNATURES), set(names) ^ set(binding._SIGNATURES)


def test_config_struct_matches_header_size():
    # 11 x int32/float, int64, uint64, 2 x uint32 with natural alignment
    assert ctypes.sizeof(binding.GearConfig) == 72
    assert ctypes.sizeof(binding.GearBytes) == 64
    assert binding.strerror(0) == "ok" and "aligned" in binding.strerror(binding.GEAR_ERR_ALIGN)


def test_argument_errors_are_return_codes_without_a_gpu():
    lib = binding.lib()
    assert lib.gear_create(None, None) == binding.GEAR_ERR_ARG
    h = ctypes.c_void_p()
    bad = binding.make_config(1, 3, 2, 2, 64, 2.0, 64, 4, 4096)          # 3 query heads over 2 kv heads
    assert lib.gear_create(ctypes.byref(h), ctypes.byref(bad)) == binding.GEAR_ERR_SHAPE
    bad = binding.make_config(1, 1, 1, 3, 64, 2.0, 64, 4, 4096)          # 3-bit
    assert lib.gear_create(ctypes.byref(h), ctypes.byref(bad)) == binding.GEAR_ERR_ARG
    bad = binding.make_config(1, 1, 1, 2, 64, 2.0, 96, 4, 4096)          # buffer not a multiple of the group
    assert lib.gear_create(ctypes.byref(h), ctypes.byref(bad)) == binding.GEAR_ERR_SHAPE
    bad = binding.make_config(1, 1, 1, 2, 16, 10.0, 16, 4, 4096, head_dim=64)
    assert lib.gear_create(ctypes.byref(h), ctypes.byref(bad)) == binding.GEAR_ERR_SHAPE
    assert lib.gear_decode_attn(None, None, None, 0.0, None) == binding.GEAR_ERR_ARG
    assert lib.gear_append_buffer(None, None, None, None, None) == binding.GEAR_ERR_ARG
    lib.gear_free(None)
