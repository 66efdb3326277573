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
    # a (page, kv head) pair has to fit one 32-bit coordinate
    big = B._CacheDesc(0x10000, 0x20000, 1 << 28, 16, 8, 8, 128)
    assert lib.efim_decode_attn(ctypes.byref(big), 1, 0x1000, 16, 0x1000, 4, 0x1000, 0x1000, None, 0.0,
                                None, 0, None, None) == 2
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
    # the one-call turn: k and v come together or not at all; the self-test refuses long limits
    assert lib.efim_append_prefill_step(ctypes.byref(ok), ctypes.byref(bd), None, 0x1000, 0x1000, None, 0x1000, None,
                                        0.0, None, 0, 0, None, 0, None, None) == 1
    assert lib.efim_selftest_bounded_wait(10**9, 0x1000, None, None) == 1
    assert lib.efim_selftest_bounded_wait(1000, None, None, None) == 1
    # fragment spans: sizing call and argument checks
    lib.efim_fim_fragment_spans.restype = ctypes.c_int64
    lib.efim_fim_fragment_spans.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                            ctypes.c_void_p, ctypes.c_int64]
    assert lib.efim_fim_fragment_spans(1, 1000, 1, 200, None, 0) >= 6
    assert lib.efim_fim_fragment_spans(1, 1000, 0, 200, None, 0) == -1
    assert lib.efim_fim_fragment_spans(1, 10, 1, 200, None, 3) == -1
    # empty batch is a no-op
    bd0 = B._BatchDesc(0, 4, 0, None, None, None, None, None, None)
    assert lib.efim_kv_append(ctypes.byref(ok), ctypes.byref(bd0), None, None, None, None, None, None) == 0


def _batch_desc(cached, new, max_pages):
    c = np.asarray(cached, np.int32)
    n = np.asarray(new, np.int32)
    bd = B._BatchDesc(len(c), max_pages, int(n.sum()), 0x1000, 0x1000, 0x1000, 0x1000, c.ctypes.data, n.ctypes.data)
    bd._keep = (c, n)
    return bd


def test_prefill_planner_splits_few_long_items_and_not_many_short_ones():
    """Host planning of efim_append_prefill_attn, seen through its two queries: few long
    work items get their key range split (partials + a merge launch) when that is estimated to
    finish sooner; a nearly full wave and many items do not."""
    lib = efim.load_library()
    cache = _cache_desc(Hq=32, Hkv=8)
    # 2 sequences x 8 kv heads x 2 row tiles = 32 items of 65 key tiles cannot fill 148 SMs -> split
    few = _batch_desc([8192] * 2, [128] * 2, 600)
    assert lib.efim_prefill_launch_count(ctypes.byref(cache), ctypes.byref(few)) == 2
    ws_few = lib.efim_prefill_workspace_bytes(ctypes.byref(cache), ctypes.byref(few))
    rows = 2 * 128 * 32
    assert ws_few > rows * 128 * 4 * 2            # room for at least two fp32 partials per (token, head)
    # cfg4a-like: 128 such items nearly fill one wave; cutting them would only add a ragged wave and a merge
    wave = _batch_desc([8192] * 8, [128] * 8, 600)
    assert lib.efim_prefill_launch_count(ctypes.byref(cache), ctypes.byref(wave)) == 1
    # cfg4b-like: 3200 items -> one launch, workspace is just the work list
    many = _batch_desc([5120] * 8, [3200] * 8, 600)
    assert lib.efim_prefill_launch_count(ctypes.byref(cache), ctypes.byref(many)) == 1
    ws_many = lib.efim_prefill_workspace_bytes(ctypes.byref(cache), ctypes.byref(many))
    items = 8 * 8 * (3200 * 4 // 256)
    assert items * 32 <= ws_many < items * 32 + 4096
    # nothing new -> nothing to do
    none = _batch_desc([100, 200], [0, 0], 32)
    assert lib.efim_prefill_launch_count(ctypes.byref(cache), ctypes.byref(none)) == 0
    assert lib.efim_prefill_workspace_bytes(ctypes.byref(cache), ctypes.byref(none)) == 0


def test_decode_planner_chunks():
    lib = efim.load_library()
    cache = _cache_desc(Hq=32, Hkv=8)
    # large batch x long context: chunks of 2048 keys, merge needed
    assert lib.efim_decode_launch_count(ctypes.byref(cache), 256, 32832) == 2
    ws = lib.efim_decode_workspace_bytes(ctypes.byref(cache), 256, 32832)
    n_chunks = -(-32832 // 2048)
    assert ws >= 256 * 32 * n_chunks * 129 * 4
    # a context of one chunk needs neither workspace nor merge
    assert lib.efim_decode_launch_count(ctypes.byref(cache), 4096, 200) == 1
    assert lib.efim_decode_workspace_bytes(ctypes.byref(cache), 4096, 200) == 0


def test_prefill_plan_blob_sizes_and_errors():
    """efim_prefill_plan: the blob is a 256-byte head plus the work list and split sizes; a
    buffer that is too small is refused; a batch with nothing new still gets a valid (empty) plan."""
    lib = efim.load_library()
    lib.efim_prefill_plan_bytes.restype = ctypes.c_size_t
    cache = _cache_desc(Hq=32, Hkv=8)
    many = _batch_desc([5120] * 8, [3200] * 8, 600)
    n = lib.efim_prefill_plan_bytes(ctypes.byref(cache), ctypes.byref(many))
    items = 8 * 8 * (3200 * 4 // 256)
    assert 256 + items * 32 <= n < 256 + items * 32 + 1024
    buf = np.zeros(n, np.uint8)
    assert lib.efim_prefill_plan(ctypes.byref(cache), ctypes.byref(many), buf.ctypes.data, n) == 0
    assert bytes(buf[:4]) == b"EFIM" and buf[256:].any()
    assert lib.efim_prefill_plan(ctypes.byref(cache), ctypes.byref(many), buf.ctypes.data, n - 1) == 4
    assert lib.efim_prefill_plan(ctypes.byref(cache), ctypes.byref(many), None, n) == 1
    none = _batch_desc([100, 200], [0, 0], 32)
    assert lib.efim_prefill_plan_bytes(ctypes.byref(cache), ctypes.byref(none)) == 256
    assert lib.efim_prefill_plan(ctypes.byref(cache), ctypes.byref(none), buf.ctypes.data, 256) == 0


_ITEM = np.dtype([("seq", "i4"), ("kvh", "i2"), ("chunk", "i2"), ("row0", "i4"), ("tile_begin", "i4"),
                  ("tile_end", "i4"), ("cached", "i4"), ("new_len", "i4"), ("tok0", "i4")])


def _plan_items(lib, cache, batch):
    lib.efim_prefill_plan_bytes.restype = ctypes.c_size_t
    n = lib.efim_prefill_plan_bytes(ctypes.byref(cache), ctypes.byref(batch))
    buf = np.zeros(n, np.uint8)
    assert lib.efim_prefill_plan(ctypes.byref(cache), ctypes.byref(batch), buf.ctypes.data, n) == 0
    n_items = int(np.frombuffer(buf[:64].tobytes(), np.int32)[6])
    return np.frombuffer(buf[256:256 + 32 * n_items].tobytes(), _ITEM)


def test_prefill_work_list_covers_every_row_and_key_once_and_is_ordered_by_cost():
    """The work list of a ragged batch (a few waves of CTAs): every (sequence, kv head, block
    of 256 packed rows) appears with the whole key range its last row sees, cut into
    disjoint chunks if at all; items carry their sequence's lengths and first query row; and
    the launch order is costliest first, a tile of a two-tile item (more than 128 rows)
    weighing 2.1 and a tile of a one-tile item 0.9."""
    lib = efim.load_library()
    Hq, Hkv = 8, 2
    G = Hq // Hkv
    cache = _cache_desc(Hq=Hq, Hkv=Hkv)
    cached = [3000, 500, 7000, 40, 2222, 900, 5000, 64]
    new = [200, 17, 40, 130, 1, 64, 33, 90]
    items = _plan_items(lib, cache, _batch_desc(cached, new, 512))
    tok0 = np.concatenate([[0], np.cumsum(new)])
    seen = {}
    for it in items:
        s = int(it["seq"])
        assert (it["cached"], it["new_len"], it["tok0"]) == (cached[s], new[s], tok0[s])
        assert 0 <= it["kvh"] < Hkv and it["row0"] % 256 == 0 and it["row0"] < new[s] * G
        seen.setdefault((s, int(it["kvh"]), int(it["row0"])), []).append((int(it["tile_begin"]), int(it["tile_end"])))
    want = {(s, h, r0) for s in range(len(new)) for h in range(Hkv) for r0 in range(0, new[s] * G, 256)}
    assert set(seen) == want
    for (s, h, r0), ranges in seen.items():
        last_tok = (min(new[s] * G, r0 + 256) - 1) // G
        tiles = -(-(cached[s] + last_tok + 1) // 128)
        ranges.sort()
        assert ranges[0][0] == 0 and ranges[-1][1] == tiles
        assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))      # disjoint, no gap
    rows_here = np.minimum(items["new_len"] * G - items["row0"], 256)
    cost = (items["tile_end"] - items["tile_begin"]) * np.where(rows_here > 128, 21, 9)
    assert (np.diff(cost) <= 0).all()
