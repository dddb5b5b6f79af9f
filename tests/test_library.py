"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares; the binding's
structs match the header's layout."""
import ctypes as C
import os
import re

import pytest

from paper_2501_14183_b200 import binding as vd
from paper_2501_14183_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(vardrop_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return vd.load()


def test_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"vardrop_hash", "vardrop_select", "vardrop_attn_fwd", "vardrop_attn_bwd"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(vd.EXPORTS)


def test_status_strings_and_version(lib):
    assert lib.vardrop_version().decode().count(".") == 1
    texts = [lib.vardrop_status_string(i).decode() for i in range(7)]
    assert texts[0] == "ok" and len(set(texts)) == 7
    assert lib.vardrop_status_string(99).decode() == "unknown status"


def test_struct_layouts_match_header():
    assert C.sizeof(vd.HashCfg) == 28
    assert C.sizeof(vd.SelectCfg) == 40 and vd.SelectCfg.rate.offset == 16 and vd.SelectCfg.seed.offset == 24
    assert C.sizeof(vd.AttnCfg) == 48 and vd.AttnCfg.sB.offset == 24


def test_workspace_queries_need_no_gpu(lib):
    assert vd.vardrop_hash_workspace_bytes(vd.HashCfg(32, 321, 96, 3, 0, 0, 0)) >= 4
    s1 = vd.vardrop_select_workspace_bytes(vd.SelectCfg(1, 321, 0, 0.3, 1, 0))
    s2 = vd.vardrop_select_workspace_bytes(vd.SelectCfg(4, 321, 0, 0.3, 1, 0))
    assert 0 < s1 < s2
    assert vd.vardrop_select_workspace_bytes(vd.SelectCfg(1, 0, 0, 0.3, 1, 0)) == 0          # invalid config
    a = vd.vardrop_attn_workspace_bytes(vd.AttnCfg(32, 321, 8, 64, 0.0))
    assert a > 4 * 32 * 384 * 8 * 128
    assert vd.vardrop_attn_workspace_bytes(vd.AttnCfg(32, 321, 8, 128, 0.0)) == 0            # unsupported head dim


def test_host_side_validation_needs_no_gpu(lib):
    # argument checks run before any CUDA call: bad configs are rejected on a machine without a GPU too
    st = lib.vardrop_hash(None, C.byref(vd.HashCfg(2, 4, 8200, 3, 0, 0, 0)), None, None, None, None, 0, None)
    assert st == vd.ERR_UNSUPPORTED and b"above 8192" in lib.vardrop_last_error()
    st = lib.vardrop_hash(None, C.byref(vd.HashCfg(2, 4, 96, 3, 0, 0, 0)), None, None, None, None, 0, None)
    assert st == vd.ERR_INVALID_ARG and b"x is NULL" in lib.vardrop_last_error()
    st = lib.vardrop_attn_fwd(None, None, None, None, None, C.byref(vd.AttnCfg(1, 8, 1, 48, 0.0)), None, None, None, 0, None)
    assert st == vd.ERR_UNSUPPORTED
