"""CPU-only checks of the C-ABI library: it loads, exports what the headers declare, and rejects bad
arguments before touching the GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2502_16927_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared():
    names = []
    for header in ("bigmac.h", "bigmac_debug.h"):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(bigmac_[a-z_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"bigmac_layer_create", "bigmac_forward", "bigmac_backward", "bigmac_route"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert lib.bigmac_status_string(0) == b"ok"
    for code in range(-6, 0):
        assert lib.bigmac_status_string(code) not in (b"ok", b"unknown status")


@pytest.mark.parametrize("bad", [
    dict(k=9),                      # k > E
    dict(d=0), dict(r=-4), dict(E=0), dict(k=0),
    dict(dtype=7), dict(act=9), dict(flags=64),
])
def test_create_rejects_invalid_configs_without_a_gpu(lib, bad):
    base = dict(d=128, r=32, h=128, E=8, k=2, max_tokens=256, dtype=0, act=0, flags=0)
    base.update(bad)
    cfg = binding.bigmac_config_t(*[base[n] for n in ("d", "r", "h", "E", "k", "max_tokens", "dtype", "act", "flags")])
    handle = C.c_void_p()
    assert lib.bigmac_layer_create(C.byref(cfg), C.byref(handle)) == -1
    assert not handle.value


def test_create_rejects_unsupported_shapes(lib):
    for over in (dict(dtype=1, r=32), dict(dtype=0, d=6), dict(E=2048, k=1)):
        base = dict(d=128, r=64, h=128, E=8, k=2, max_tokens=256, dtype=0, act=0, flags=0)
        base.update(over)
        cfg = binding.bigmac_config_t(*[base[n] for n in ("d", "r", "h", "E", "k", "max_tokens", "dtype", "act", "flags")])
        handle = C.c_void_p()
        assert lib.bigmac_layer_create(C.byref(cfg), C.byref(handle)) == -2


def test_null_arguments(lib):
    handle = C.c_void_p()
    assert lib.bigmac_layer_create(None, C.byref(handle)) == -1
    assert lib.bigmac_layer_destroy(None) == -1
    assert lib.bigmac_forward(None, None, 0, None, None, None, None, None, 0, None) == -1
    assert lib.bigmac_backward(None, None, None, 0, None, None, None, None, 0, None, 0, None) == -1
    assert lib.bigmac_route(None, None, 0, None, None, None, 0, None) == -1


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2502_16927_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|import_module\(.oracle|libbigmac_oracle", text, re.M), f
