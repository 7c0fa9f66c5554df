"""The C-ABI library loads without a GPU and exports every symbol the public headers declare."""
import ctypes
import os
import re

import pytest

from paper_2506_06266_b200 import binding, buildlib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    buildlib.build()
    return binding.load_library()


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"CART_API\s+[\w\s\*]+?\b(cart_\w+)\s*\(", text)
    return names


def test_headers_declare_the_expected_entry_points():
    names = declared_functions()
    for must in ("cart_register_cartridge", "cart_append_kv", "cart_decode_attention", "cart_compose"):
        assert must in names
    assert sorted(names) == sorted(binding.EXPORTS)


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name
        assert ctypes.cast(getattr(lib, name), ctypes.c_void_p).value


def test_status_strings(lib):
    assert binding.cart_status_string(0) == "CART_OK"
    assert binding.cart_status_string(binding.CART_ERR_TIMEOUT) == "CART_ERR_TIMEOUT"
    assert len({binding.cart_status_string(i) for i in range(10)}) == 10


def test_config_validation_needs_no_device(lib):
    good = binding.make_config(28, 24, 8, 64, 64)
    assert binding.cart_scratch_bytes(good) % 256 == 0
    bigger = binding.make_config(28, 24, 8, 256, 64)
    assert binding.cart_scratch_bytes(bigger) > binding.cart_scratch_bytes(good)
    for bad, status in [
        (binding.make_config(28, 24, 8, 64, 64, head_dim=64), binding.CART_ERR_SHAPE),
        (binding.make_config(28, 24, 7, 64, 64), binding.CART_ERR_SHAPE),
        (binding.make_config(28, 72, 8, 64, 64), binding.CART_ERR_SHAPE),       # group of 9 heads
        (binding.make_config(0, 24, 8, 64, 64), binding.CART_ERR_INVALID_ARG),
        (binding.make_config(28, 24, 8, 0, 64), binding.CART_ERR_INVALID_ARG),
    ]:
        with pytest.raises(binding.CartError) as ei:
            binding.cart_scratch_bytes(bad)
        assert ei.value.status == status


def test_create_rejects_bad_arena_before_touching_cuda(lib):
    cfg = binding.make_config(2, 8, 8, 4, 4, arena=None, arena_bytes=1 << 20)
    with pytest.raises(binding.CartError) as ei:
        binding.cart_create(cfg)
    assert ei.value.status == binding.CART_ERR_INVALID_ARG
    cfg = binding.make_config(2, 8, 8, 4, 4, arena=0x1000100, arena_bytes=1024)   # far too small
    with pytest.raises(binding.CartError) as ei:
        binding.cart_create(cfg)
    assert ei.value.status == binding.CART_ERR_OOM


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(ImportError):
        binding.load_library(str(tmp_path / "libcart.so"))
