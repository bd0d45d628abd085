"""The C-ABI library loads on a machine without a GPU and exports every symbol zeda.h declares;
argument checks that need no device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def zeda():
    from paper_2605_18643_b200 import build
    build.build_library()
    from paper_2605_18643_b200 import zeda as z
    return z


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "zeda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zeda_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(zeda):
    names = declared_symbols()
    assert "zeda_moe_create" in names and "zeda_route" in names and "zeda_moe_forward" in names
    assert "zeda_moe_destroy" in names and len(names) >= 10
    for n in names:
        assert hasattr(zeda.lib, n), n
    assert sorted(zeda.EXPORTS) == names


def test_version_and_error_strings(zeda):
    assert "sm_100a" in zeda.version()
    assert isinstance(zeda.last_error(), str)


def test_workspace_size_and_config_checks(zeda):
    cfg = zeda.Config(2048, 768, 128, 64, 8, 8192, 0, 0, 0, 0)
    need = zeda.workspace_bytes(cfg)
    assert need % 256 == 0
    slots = 8192 * 8
    assert need > slots * (768 + 2048) * 2          # at least the two pair buffers
    assert need < 1 << 30
    small = zeda.Config(2048, 768, 128, 64, 8, 64, 0, 0, 0, 0)
    assert zeda.workspace_bytes(small) < need
    for bad in (zeda.Config(2040, 768, 128, 64, 8, 64, 0, 0, 0, 0),     # d % 64
                zeda.Config(2048, 768, 0, 64, 8, 64, 0, 0, 0, 0),        # no normal expert
                zeda.Config(2048, 768, 4, 2, 8, 64, 0, 0, 0, 0),         # K > candidates
                zeda.Config(2048, 768, 128, 64, 17, 64, 0, 0, 0, 0),     # K too large
                zeda.Config(2048, 768, 500, 64, 8, 64, 0, 0, 0, 0),      # too many candidates
                zeda.Config(2048, 768, 128, 64, 8, 0, 0, 0, 0, 0),       # max_tokens
                zeda.Config(2048, 768, 128, 64, 8, 64, 7, 0, 0, 0),      # gate mode
                zeda.Config(2048, 768, 128, 64, 8, 64, 0, 0, 0, 3)):     # unknown flag bits
        assert zeda.workspace_bytes(bad) == 0
        assert zeda.last_error() != ""


def test_create_rejects_bad_arguments_before_touching_a_device(zeda):
    cfg = zeda.Config(256, 128, 8, 4, 2, 64, 0, 0, 0, 0)
    h = ctypes.c_void_p()
    st = zeda.lib.zeda_moe_create(ctypes.byref(cfg), None, None, None, None, None, 0, ctypes.byref(h))
    assert st == zeda.ERR_INVALID_ARG and not h.value
    bad = zeda.Config(250, 128, 8, 4, 2, 64, 0, 0, 0, 0)
    st = zeda.lib.zeda_moe_create(ctypes.byref(bad), None, None, None, None, None, 0, ctypes.byref(h))
    assert st == zeda.ERR_UNSUPPORTED
    assert zeda.lib.zeda_moe_forward(None, None, 1, None, None) == zeda.ERR_INVALID_ARG
    assert zeda.lib.zeda_route(None, None, 1, None, None, None, None, None, None, None) == zeda.ERR_INVALID_ARG
    assert zeda.lib.zeda_moe_destroy(None) == zeda.OK


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_18643_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "zeda_oracle" not in text, f
    otext = open(os.path.join(ROOT, "oracle", "__init__.py")).read() + open(os.path.join(ROOT, "oracle", "zeda_oracle.c")).read()
    assert "paper_2605_18643_b200" not in otext and "libzeda.so" not in otext and "import torch" not in otext
