"""CPU checks of the C-ABI boundary: the library builds, loads and exports every symbol the
header declares; configuration validation and workspace sizing (host logic) need no GPU."""
import ctypes
import os
import re

import pytest

from paper_2604_07394_b200 import build as flux_build
from paper_2604_07394_b200 import flux

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    flux_build.build()
    return flux.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "flux_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(flux_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(flux.EXPORTS) == names


def test_version_and_error_string(lib):
    assert lib.flux_version().decode() == "0.1"
    assert isinstance(flux.last_error(), str)


def test_workspace_size_and_config_validation(lib):
    cfg = flux.make_config(32, 32, 8, 128, 4096, 8, 65792)
    n = flux.flux_workspace_size(cfg)
    assert 1 << 20 < n < 1 << 28
    bigger = flux.make_config(32, 32, 8, 128, 4096, 16, 65792)
    assert flux.flux_workspace_size(bigger) > n
    bad = [
        flux.make_config(32, 32, 8, 128, 4096, 8, 65792, head_dim=64),
        flux.make_config(32, 30, 8, 128, 4096, 8, 65792),          # Hq % Hkv != 0
        flux.make_config(32, 34, 2, 128, 4096, 8, 65792),          # more than 16 query heads per KV head
        flux.make_config(32, 32, 8, -1, 4096, 8, 65792),
        flux.make_config(32, 32, 8, 128, 0, 8, 65792),             # window must be >= 1
        flux.make_config(32, 32, 8, 128, 4096, 0, 65792),
        flux.make_config(32, 32, 8, 128, 4096, 8, 0),
        flux.make_config(32, 32, 8, 128, 4096, 8, 65792, kv_layout=7),
        flux.make_config(32, 32, 8, 128, 4096, 8, 65792, softmax_scale=float("nan")),
    ]
    codes = []
    for c in bad:
        with pytest.raises(flux.FluxError) as e:
            flux.flux_workspace_size(c)
        codes.append(e.value.code)
        assert flux.last_error() != ""
    assert codes[0] == flux.FLUX_E_UNSUPPORTED_SHAPE and codes[1] == flux.FLUX_E_UNSUPPORTED_SHAPE
    assert codes[3] == flux.FLUX_E_INVALID_ARG and codes[5] == flux.FLUX_E_CAPACITY


def test_null_arguments_are_rejected_without_a_device(lib):
    assert lib.flux_workspace_size(None, None) == flux.FLUX_E_INVALID_ARG
    assert lib.flux_plan_set_workspace(None, None, 0) == flux.FLUX_E_INVALID_ARG
    assert lib.flux_router_apply(None, None, None, 1, None, None) == flux.FLUX_E_INVALID_ARG
    assert lib.flux_attn_decode(None, 0, 1, None, None, None, None, None, None) == flux.FLUX_E_INVALID_ARG
    assert lib.flux_launch_count(None) == 0
    h = ctypes.c_void_p(123)
    cfg = flux.make_config(4, 8, 2, 64, 256, 1, 2048, head_dim=96)
    assert lib.flux_plan_create(ctypes.byref(cfg), ctypes.byref(h)) == flux.FLUX_E_UNSUPPORTED_SHAPE
    assert not h.value
