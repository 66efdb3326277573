"""Input generators: host and torch pool fills agree bit for bit; workloads have the stated shapes."""
import numpy as np
import pytest
import torch

from efim_synth import make_workload, pool_bits_np, pool_fill_torch, WORKLOAD_NAMES, bf16_bits_to_f32
from efim_synth.pool import K_POOL_ID, V_POOL_ID


def test_pool_fill_numpy_equals_torch_and_looks_standard_normal():
    n = 300_000
    t = torch.empty(n, dtype=torch.bfloat16)
    pool_fill_torch(t, seed=5, tensor_id=K_POOL_ID, chunk=70_001)
    got = t.view(torch.int16).numpy().view(np.uint16)
    want = pool_bits_np(5, K_POOL_ID, 0, n)
    assert np.array_equal(got, want)
    # index beyond 2^32 uses the high word
    a = pool_bits_np(5, V_POOL_ID, (1 << 33) + 7, 100)
    b = pool_bits_np(5, V_POOL_ID, 7, 100)
    assert not np.array_equal(a, b)
    x = bf16_bits_to_f32(want).astype(np.float64)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01 and np.abs(x).max() < 3.6


@pytest.mark.parametrize("name", WORKLOAD_NAMES)
def test_workload_shapes(name):
    w = make_workload(name, small=name not in ("cfg1",))
    B = w.batch
    assert w.block_table.shape[0] == B and w.q_indptr[-1] == w.total_new_tokens
    used = w.block_table[w.block_table >= 0]
    assert len(np.unique(used)) == len(used) and used.max() < w.num_pages      # drawn without replacement
    for s in range(B):
        need = -(-(int(w.cached_len[s]) + int(w.new_len[s]) + w.decode_steps) // w.page_size)
        assert np.all(w.block_table[s, :need] >= 0)
        if not name.startswith("cfg4"):          # the cfg4 variants share one table sized for the longest
            assert np.all(w.block_table[s, need:] == -1)
    q, k, v = w.new_qkv()
    assert q.shape == (w.total_new_tokens, w.num_q_heads, w.head_dim) and k.shape == v.shape
    w2 = make_workload(name, small=name not in ("cfg1",))
    assert np.array_equal(w2.block_table, w.block_table) and np.array_equal(w2.new_qkv()[0], q)


def test_full_size_length_ranges():
    w = make_workload("cfg2")
    assert w.batch == 16 and w.cached_len.min() >= 2048 and w.cached_len.max() <= 8192
    assert w.new_len.min() >= 32 and w.new_len.max() <= 256 and w.num_pages == 65536
    w = make_workload("cfg3")
    assert w.batch == 64 and w.decode_rows.sum() == 32 and np.all(w.new_len[w.decode_rows] == 1)
    w = make_workload("cfg4b")
    assert np.all(w.cached_len == 5120) and np.all(w.new_len == 3200)
    w = make_workload("cfg1")
    assert w.cached_len[0] == 240 and w.new_len[0] == 16 and w.decode_steps == 8


def test_compact_host_pool_matches_page_bits():
    w = make_workload("cfg5", small=True)
    kp, vp, bt, seqs = w.compact_host_pool([1, 3])
    pg = w.pages_of(3)
    assert np.array_equal(kp[bt[1, 0]], w.page_bits("k", pg[:1])[0])
    assert np.array_equal(vp[bt[1, len(pg) - 1]], w.page_bits("v", pg[-1:])[0])
