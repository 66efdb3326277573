"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
function include/efim.h declares, and rejects bad arguments before launching."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2505_21889_b200 as efim
from paper_2505_21889_b200 import binding as B
from paper_2505_21889_b200 import build as efim_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    efim_build.build()


def _declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(efim_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    lib = efim.load_library()
    declared = _declared_functions()
    assert len(declared) >= 8
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"


def test_version_and_strerror():
    assert efim.efim_version() >= 100
    assert efim.efim_strerror(0) == "ok"
    assert "workspace" in efim.efim_strerror(4)


def test_rope_table_matches_definition():
    t = efim.efim_rope_table_build(10000.0, 8, 50)
    p, f = 37, 2
    assert abs(t[p, f] - np.cos(p * 10000.0 ** (-2 * f / 8))) < 1e-7
    assert abs(t[p, 4 + f] - np.sin(p * 10000.0 ** (-2 * f / 8))) < 1e-7
    with pytest.raises(efim.EfimError):
        efim.efim_rope_table_build(10000.0, 7, 4)


def _cache_desc(D=128, P=16, Hq=8, Hkv=2, k=0x10000, v=0x20000):
    return B._CacheDesc(k, v, 64, P, Hq, Hkv, D)


def test_bad_arguments_are_rejected_on_the_host():
    lib = efim.load_library()
    ok = _cache_desc()
    for bad, code in [(_cache_desc(D=96), 2), (_cache_desc(P=32), 2), (_cache_desc(Hq=7), 1),
                      (_cache_desc(k=0), 1), (_cache_desc(k=0x10008), 1)]:
        st = lib.efim_decode_attn(ctypes.byref(bad), 1, 0x1000, 16, 0x1000, 4, 0x1000, 0x1000, None, 0.0,
                                  None, 0, None, None)
        assert st == code
    # null inputs
    assert lib.efim_decode_attn(ctypes.byref(ok), 1, None, 16, 0x1000, 4, 0x1000, 0x1000, None, 0.0,
                                None, 0, None, None) == 1
    # max_ctx_len beyond what the block table can address
    assert lib.efim_decode_attn(ctypes.byref(ok), 1, 0x1000, 65, 0x1000, 4, 0x1000, 0x1000, None, 0.0,
                                None, 0, None, None) == 3
    # workspace too small (many chunks for a long context)
    assert lib.efim_decode_workspace_bytes(ctypes.byref(ok), 1, 1 << 16) > 0
    assert lib.efim_decode_attn(ctypes.byref(ok), 1, 0x1000, 1 << 16, 0x1000, 1 << 12, 0x1000, 0x1000, None, 0.0,
                                None, 0, None, None) == 4
    # prefill: host mirrors are validated (sum of new_len must equal total_new_tokens, lengths fit the table)
    c = np.array([10, 20], np.int32)
    n = np.array([3, 4], np.int32)
    bd = B._BatchDesc(2, 4, 8, 0x1000, 0x1000, 0x1000, 0x1000, c.ctypes.data, n.ctypes.data)
    assert lib.efim_append_prefill_attn(ctypes.byref(ok), ctypes.byref(bd), 0x1000, 0x1000, None, 0.0,
                                        None, 0, None, None) == 1
    bd.total_new_tokens = 7
    c[1] = 62
    assert lib.efim_append_prefill_attn(ctypes.byref(ok), ctypes.byref(bd), 0x1000, 0x1000, None, 0.0,
                                        None, 0, None, None) == 3
    c[1] = 20
    assert lib.efim_prefill_workspace_bytes(ctypes.byref(ok), ctypes.byref(bd)) > 0
    assert lib.efim_append_prefill_attn(ctypes.byref(ok), ctypes.byref(bd), 0x1000, 0x1000, None, 0.0,
                                        None, 0, None, None) == 4
    # empty batch is a no-op
    bd0 = B._BatchDesc(0, 4, 0, None, None, None, None, None, None)
    assert lib.efim_kv_append(ctypes.byref(ok), ctypes.byref(bd0), None, None, None, None, None, None) == 0
