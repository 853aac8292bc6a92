"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and rejects bad
configurations on the host before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2609_13285_b200 import binding as gb
from paper_2609_13285_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    gbuild.build()
    return gb.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gva.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(g[vq]a_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert set(gb.EXPORTS) <= set(names)


def test_status_strings(lib):
    assert gb.status_string(0) == "ok"
    assert "page" in gb.status_string(gb.GVA_ERR_BAD_PAGE)
    assert gb.status_string(99) == "unknown status"


def _create(**kw):
    args = dict(H=16, G=4, d_v=64, d_c=64, d_r=16, page_size=64)
    args.update(kw)
    cfg = gb.GvaConfig(args["H"], args["G"], args["d_v"], args["d_c"], args["d_r"], args["page_size"],
                       args.get("cache_dtype", gb.GVA_BF16), args.get("kernel", 0), args.get("rope_base", 10000.0),
                       args.get("softmax_scale", 0.0), 0)
    h = ctypes.c_void_p()
    return gb.load().gva_create(ctypes.byref(h), ctypes.byref(cfg), 0), h


def test_create_rejects_bad_configs_on_the_host(lib):
    assert _create(H=0)[0] == gb.GVA_ERR_INVALID_ARG
    assert _create(H=16, G=3)[0] == gb.GVA_ERR_UNSUPPORTED           # H % G != 0
    assert _create(H=16, G=8)[0] == gb.GVA_ERR_UNSUPPORTED           # H / G != 4
    assert _create(d_v=96)[0] == gb.GVA_ERR_UNSUPPORTED
    assert _create(d_r=20)[0] == gb.GVA_ERR_UNSUPPORTED
    assert _create(d_v=128, d_r=24)[0] == gb.GVA_ERR_UNSUPPORTED
    assert _create(page_size=48)[0] == gb.GVA_ERR_UNSUPPORTED
    assert _create(cache_dtype=7)[0] == gb.GVA_ERR_INVALID_ARG
    assert _create(rope_base=0.5)[0] == gb.GVA_ERR_INVALID_ARG
    assert _create(kernel=gb.GVA_KERNEL_MMA, cache_dtype=gb.GVA_F32)[0] == gb.GVA_ERR_UNSUPPORTED
    assert lib.gva_create(None, None, 0) == gb.GVA_ERR_INVALID_ARG


def test_null_handle_calls_fail_cleanly(lib):
    assert lib.gva_destroy(None) == gb.GVA_ERR_INVALID_ARG
    assert lib.gva_decode_workspace_bytes(None, 1, 1, 0) == 0
    assert lib.gva_last_num_splits(None) == 0
    assert lib.gva_absorb_query(None, None, None, None, None, None, 1, None) == gb.GVA_ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(gb, "_lib", None)
    monkeypatch.setattr(gb, "LIB_PATH", "/nonexistent/libgva.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        gb.load()
