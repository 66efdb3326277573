"""GPU edge cases and device-side error reporting, through the C ABI: shared cached pages,
the last page id of the pool, optional arguments, the EFIM_DEV_* bits of every call (bad
page ids and positions are reported and skipped, never dereferenced), the one-call
append+prefill step against the two calls it replaces, and the bounded device wait."""
import numpy as np
import pytest
import torch

from efim_synth import make_workload
from oracle import efim_oracle as orc

pytestmark = pytest.mark.gpu

BAD_PAGE, BAD_POSITION, TIMEOUT = 0x1, 0x2, 0x4


def _mods():
    import paper_2505_21889_b200 as efim
    import tests.gpu_harness as H
    from tests.test_gpu_parity import _custom, _check_turn
    return efim, H, _custom, _check_turn


def test_two_sequences_read_the_same_cached_pages():
    """Cross-request reuse (Sec. 1): two requests with the same `<P>prefix<S>suffix<M>` share
    its pages for reading; each appends its own `inc` into pages of its own."""
    efim, H, _custom, _check_turn = _mods()
    w = _custom(8, 2, 128, [160, 160, 33], [37, 5, 20])
    w.block_table[1, :10] = w.block_table[0, :10]            # 160 cached tokens = 10 shared pages
    dw, ref = _check_turn(w)
    assert set(w.pages_of(0)[:10]) == set(w.pages_of(1)[:10])


def test_last_page_of_the_pool_is_addressable():
    efim, H, _custom, _check_turn = _mods()
    w = _custom(4, 4, 64, [40, 3], [30, 140])
    last = w.num_pages - 1
    # page 2 of sequence 1 holds cached and new tokens: give it the pool's last id (swapping
    # with wherever the seeded permutation had put that id, if anywhere)
    w.block_table[w.block_table == last] = w.block_table[1, 2]
    w.block_table[1, 2] = last
    _check_turn(w)


def test_kv_append_without_q_and_decode_without_lse_custom_scale():
    efim, H, _custom, _check_turn = _mods()
    w = _custom(8, 2, 128, [100, 17, 900], [40, 3, 1])
    a, b = H.DeviceWorkload(w), H.DeviceWorkload(w)
    a.gpu_kv_append()
    efim.efim_kv_append(b.cache, b.batch, b.rope, None, b.k_new, b.v_new, b.status)      # d_q = NULL
    torch.cuda.synchronize()
    assert int(b.status.item()) == 0
    assert torch.equal(a.k_pool.view(torch.int16), b.k_pool.view(torch.int16))
    assert torch.equal(a.v_pool.view(torch.int16), b.v_pool.view(torch.int16))
    assert torch.equal(b.q.view(torch.int16), H.bits_to_torch(b.q_bits).view(torch.int16))   # untouched
    # decode with d_lse = NULL and a caller-given scale, against the oracle
    kp, vp, bt, seqs = w.compact_host_pool()
    orc.kv_append(kp, vp, bt, w.cached_len, w.new_len, a.q_bits, a.k_bits, a.v_bits, w.rope_base)
    ctx = (w.cached_len + w.new_len).astype(np.int32)
    q = w._normal_bits(77, (3, 8, 128))
    o, _ = orc.decode_attention(q, kp, vp, bt, ctx, 8, sm_scale=0.05)
    out = torch.empty((3, 8, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(max(efim.efim_decode_workspace_bytes(a.cache, 3, int(ctx.max())), 256), dtype=torch.uint8,
                     device="cuda")
    efim.efim_decode_attn(a.cache, 3, torch.from_numpy(ctx).cuda(), int(ctx.max()), a.batch.d_block_table,
                          H.bits_to_torch(q), out, None, 0.05, ws, a.status)
    torch.cuda.synchronize()
    assert int(a.status.item()) == 0
    H.assert_attn_close(H.torch_to_bits(out), o, "decode, no lse, scale 0.05")


def test_kv_append_reports_bad_page_and_bad_position_and_skips_them():
    efim, H, _custom, _check_turn = _mods()
    w = _custom(4, 2, 64, [30, 64, 10], [40, 20, 5])
    dw = H.DeviceWorkload(w)
    # sequence 0's new tokens span pages 1..4; page 3 gets an id outside the pool, page 4 a negative one
    table = dw.batch.d_block_table.clone()
    table[0, 3] = w.num_pages + 9
    table[0, 4] = -7
    sentinel_k = dw.k_pool.clone()
    bad = efim.Batch(w.cached_len, w.new_len, table)
    efim.efim_kv_append(dw.cache, bad, dw.rope, dw.q, dw.k_new, dw.v_new, dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == BAD_PAGE
    kp, vp, bt, seqs = w.compact_host_pool()
    q_rot = orc.kv_append(kp, vp, bt, w.cached_len, w.new_len, dw.q_bits, dw.k_bits, dw.v_bits, w.rope_base)
    # the pages of the two bad entries were never written ...
    for pg in (int(w.block_table[0, 3]), int(w.block_table[0, 4])):
        assert torch.equal(dw.k_pool[pg].view(torch.int16), sentinel_k[pg].view(torch.int16))
    # ... every other page of every sequence holds what the oracle holds
    for s in range(3):
        pg = w.pages_of(s, int(w.cached_len[s] + w.new_len[s]))
        keep = [i for i in range(len(pg)) if not (s == 0 and i in (3, 4))]
        assert np.array_equal(dw.pages_from_device("v", pg[keep]), vp[bt[s, keep]])
        H.assert_rope_close(dw.pages_from_device("k", pg[keep]), kp[bt[s, keep]], "k pages")
    # tokens of the skipped pages keep their unrotated q; all others are rotated
    ind = w.q_indptr
    tok = np.arange(int(w.new_len[0]))
    skipped = ((30 + tok) // 16 >= 3)
    got_q = H.torch_to_bits(dw.q)
    assert np.array_equal(got_q[ind[0]:ind[1]][skipped], dw.q_bits[ind[0]:ind[1]][skipped])
    H.assert_rope_close(got_q[ind[0]:ind[1]][~skipped], q_rot[ind[0]:ind[1]][~skipped], "q of good tokens")
    H.assert_rope_close(got_q[ind[1]:], q_rot[ind[1]:], "q of other sequences")
    # a position beyond the rotary table: reported, the token is skipped
    dw2 = H.DeviceWorkload(w)
    short = efim.Rope(w.rope_base, w.head_dim, 80, False)            # sequence 1 reaches position 83
    before = dw2.k_pool.clone()
    efim.efim_kv_append(dw2.cache, dw2.batch, short, dw2.q, dw2.k_new, dw2.v_new, dw2.status)
    torch.cuda.synchronize()
    assert int(dw2.status.item()) == BAD_POSITION
    pg5 = int(w.block_table[1, 5])                                    # positions 80..83 live in page 5, slots 0..3
    assert torch.equal(dw2.k_pool[pg5].view(torch.int16), before[pg5].view(torch.int16))
    pg4 = int(w.block_table[1, 4])                                    # positions 64..79 were appended
    assert not torch.equal(dw2.k_pool[pg4].view(torch.int16), before[pg4].view(torch.int16))


@pytest.mark.parametrize("head_dim", [128, 64])
@pytest.mark.parametrize("bad_id", ["beyond_pool", "negative"])
def test_prefill_reports_bad_page_keeps_other_rows(bad_id, head_dim):
    """A block-table entry outside the pool among the pages a row sees: EFIM_DEV_BAD_PAGE,
    finite output everywhere, the sequences that do not see the entry are unaffected, and the
    sequence that does gets what the header promises: the page's 16 keys count as zero keys
    with zero values."""
    efim, H, _custom, _check_turn = _mods()
    w = _custom(8, 2, head_dim, [300, 200, 500], [140, 60, 9])
    dw = H.DeviceWorkload(w)
    dw.gpu_kv_append()
    table = dw.batch.d_block_table.clone()
    table[1, 6] = w.num_pages + 3 if bad_id == "beyond_pool" else -5   # a cached page of sequence 1
    bad = efim.Batch(w.cached_len, w.new_len, table)
    ws = torch.empty(max(efim.efim_prefill_workspace_bytes(dw.cache, bad), 256), dtype=torch.uint8, device="cuda")
    efim.efim_append_prefill_attn(dw.cache, bad, dw.q, dw.out, dw.lse, 0.0, ws, dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == BAD_PAGE
    assert torch.isfinite(dw.out.float()).all() and torch.isfinite(dw.lse).all()
    ref = dw.oracle_turn([0, 2])
    H.assert_attn_close(H.torch_to_bits(dw.out)[ref["rows"]], ref["o"], "rows that do not see the bad entry")
    H.assert_lse_close(dw.lse.cpu().numpy()[ref["rows"]], ref["lse"], "rows that do not see the bad entry")
    one = dw.oracle_turn([1])
    kp, vp = one["k_pool"].copy(), one["v_pool"].copy()
    kp[one["bt"][0, 6]] = 0                                   # bf16 bit pattern 0 = +0.0
    vp[one["bt"][0, 6]] = 0
    o, lse = orc.append_prefill_attention(one["q_rot"], kp, vp, one["bt"], one["cached"], one["new"], w.num_q_heads)
    H.assert_attn_close(H.torch_to_bits(dw.out)[one["rows"]], o, "rows that see the bad entry as zero keys")
    H.assert_lse_close(dw.lse.cpu().numpy()[one["rows"]], lse, "rows that see the bad entry as zero keys")


@pytest.mark.parametrize("static", [False, True])
def test_decode_length_beyond_the_planned_maximum_is_clamped_and_reported(static):
    """A device length above max_ctx_len (but inside the block table): clamped to what the
    chunks cover, EFIM_DEV_BAD_POSITION set, output finite, other rows exact, no access past
    the partials (several chunks, so the merge kernel runs)."""
    efim, H, _custom, _check_turn = _mods()
    Hq, Hkv, D = 8, 2, 128
    w = _custom(Hq, Hkv, D, [3000, 2500, 7000, 40], [0, 0, 0, 0], seed=21, extra=0)
    dw = H.DeviceWorkload(w)
    max_ctx = 3000                                           # what the caller claims
    assert efim.efim_decode_launch_count(dw.cache, 4, max_ctx) == 2
    true_len = np.array([3000, 2500, 40, 40], np.int32)
    lied_len = np.array([3000, 2500, 6900, 40], np.int32)   # row 2 exceeds max_ctx, within its table row
    q = w._normal_bits(9, (4, Hq, D))
    dq = H.bits_to_torch(q)

    def run(lens):
        out = torch.empty_like(dq)
        lse = torch.empty((4, Hq), dtype=torch.float32, device="cuda")
        dw.status.zero_()
        if static:
            efim.efim_decode_attn_static(dw.cache, 4, torch.from_numpy(lens).cuda(), max_ctx, dw.batch.d_block_table,
                                         dq, out, lse, 0.0, dw.status)
        else:
            nbytes = efim.efim_decode_workspace_bytes(dw.cache, 4, max_ctx)
            guard = 4096
            ws = torch.full((nbytes + guard,), 0x5A, dtype=torch.uint8, device="cuda")
            efim.efim_decode_attn(dw.cache, 4, torch.from_numpy(lens).cuda(), max_ctx, dw.batch.d_block_table, dq, out,
                                  lse, 0.0, ws[:nbytes], dw.status)
            torch.cuda.synchronize()
            assert bool((ws[nbytes:] == 0x5A).all()), "wrote past the workspace"
        torch.cuda.synchronize()
        return out, lse, int(dw.status.item())

    out0, lse0, st0 = run(true_len)
    assert st0 == 0
    out1, lse1, st1 = run(lied_len)
    assert st1 == BAD_POSITION
    assert torch.isfinite(out1.float()).all() and torch.isfinite(lse1).all()
    for r in (0, 1, 3):
        assert torch.equal(out0[r].view(torch.int16), out1[r].view(torch.int16)) and torch.equal(lse0[r], lse1[r])
    kp, vp, bt, seqs = w.compact_host_pool()
    o, lse = orc.decode_attention(q, kp, vp, bt, true_len, Hq)
    H.assert_attn_close(H.torch_to_bits(out0), o, "decode rows at their true lengths")


@pytest.mark.parametrize("name,interleaved,use_rope,planned", [
    ("cfg2", False, True, True), ("cfg3", False, True, False), ("cfg4a", True, True, True),
    ("cfg1", False, True, False), ("cfg1", True, False, True), ("cfg4b", False, True, True),
])
def test_step_call_equals_append_then_prefill(name, interleaved, use_rope, planned):
    """efim_append_prefill_step (k/v appended, q rotated as the attention kernel loads it)
    against efim_kv_append + efim_append_prefill_attn: out, lse and pools bit for bit; q is
    left as it came."""
    efim, H, _custom, _check_turn = _mods()
    w = make_workload(name, small=name != "cfg1")
    a = H.DeviceWorkload(w, interleaved=interleaved, use_rope=use_rope)
    b = H.DeviceWorkload(w, interleaved=interleaved, use_rope=use_rope)
    a.gpu_kv_append()
    a.gpu_prefill()
    ws = torch.empty(max(efim.efim_prefill_workspace_bytes(b.cache, b.batch), 256), dtype=torch.uint8, device="cuda")
    plan = efim.efim_prefill_plan(b.cache, b.batch) if planned else None
    efim.efim_append_prefill_step(b.cache, b.batch, b.rope, b.q, b.k_new, b.v_new, b.out, b.lse, 0.0, ws, b.status,
                                  plan=plan)
    torch.cuda.synchronize()
    assert int(a.status.item()) == 0 and int(b.status.item()) == 0
    assert torch.equal(a.out.view(torch.int16), b.out.view(torch.int16)) and torch.equal(a.lse, b.lse)
    assert torch.equal(a.k_pool.view(torch.int16), b.k_pool.view(torch.int16))
    assert torch.equal(a.v_pool.view(torch.int16), b.v_pool.view(torch.int16))
    assert torch.equal(b.q.view(torch.int16), H.bits_to_torch(b.q_bits).view(torch.int16))


def test_step_call_reports_a_position_beyond_the_rotary_table():
    efim, H, _custom, _check_turn = _mods()
    w = _custom(4, 2, 64, [30, 64], [40, 20])
    dw = H.DeviceWorkload(w)
    short = efim.Rope(w.rope_base, w.head_dim, 80, False)            # sequence 1 reaches position 83
    ws = torch.empty(max(efim.efim_prefill_workspace_bytes(dw.cache, dw.batch), 256), dtype=torch.uint8, device="cuda")
    efim.efim_append_prefill_step(dw.cache, dw.batch, short, dw.q, dw.k_new, dw.v_new, dw.out, dw.lse, 0.0, ws,
                                  dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == BAD_POSITION
    assert torch.isfinite(dw.out.float()).all()
    ref = dw.oracle_turn([0])
    H.assert_attn_close(H.torch_to_bits(dw.out)[ref["rows"]], ref["o"], "the sequence inside the table")


def test_many_single_tile_items_beside_long_row_blocks():
    """More items of at most 128 rows than two per SM, beside row blocks of 256: all rows
    against the oracle, and the same bits from run to run."""
    efim, H, _custom, _check_turn = _mods()
    rng = np.random.default_rng(77)
    B, Hq = 11, 32
    cached = rng.integers(0, 700, size=B).astype(np.int32)
    new = rng.integers(1, 129, size=B).astype(np.int32)
    new[3], cached[3] = 128, 256                  # a full tile on a tile edge
    new[5], cached[5] = 300, 90                   # two row blocks: 256 rows and 44 rows
    new[7], cached[7] = 1, 0                      # a lone first token
    w = _custom(Hq, Hq, 128, cached, new, seed=31)
    dw, ref = _check_turn(w)
    first = (H.torch_to_bits(dw.out).copy(), dw.lse.cpu().numpy().copy())
    dw.out.zero_()
    dw.lse.zero_()
    dw.gpu_prefill()
    torch.cuda.synchronize()
    assert np.array_equal(H.torch_to_bits(dw.out), first[0]) and np.array_equal(dw.lse.cpu().numpy(), first[1])


@pytest.mark.parametrize("Hq,Hkv,D,cached,new", [
    (28, 4, 128, [5000, 130, 0, 2047, 900], [1, 4, 3, 1, 2]),        # 7, 28, 21 rows; odd and even tile counts
    (8, 2, 128, [12000, 1, 127, 128, 255], [8, 8, 7, 1, 8]),         # 32 rows exactly; one key tile; tile edges
    (4, 4, 64, [3000, 40, 513], [32, 33, 31]),                       # 32 rows / 33 rows: both sides of the boundary
    (16, 2, 128, [700, 9000], [4, 5]),                               # 32 rows, and 40 rows (the 128-row shape)
    (32, 8, 128, [16000], [2]),                                      # one long sequence: cut into key chunks
])
def test_row_blocks_of_at_most_32_rows(Hq, Hkv, D, cached, new):
    """Items of at most 32 packed rows (one-token rows of a mixed batch, short `inc`s) run in
    the CTA shape that holds the rows once per 32-lane quarter and merges eight partial
    states per row: all rows against the oracle, with and without key chunks, at both head
    dims, next to items just above the boundary; and the one-call turn (q rotated on load)
    gives the same bits as the two calls."""
    efim, H, _custom, _check_turn = _mods()
    w = _custom(Hq, Hkv, D, cached, new, seed=53)
    dw, ref = _check_turn(w)
    two_call = (H.torch_to_bits(dw.out).copy(), dw.lse.cpu().numpy().copy())
    b = H.DeviceWorkload(w)
    ws = torch.empty(max(efim.efim_prefill_workspace_bytes(b.cache, b.batch), 256), dtype=torch.uint8, device="cuda")
    efim.efim_append_prefill_step(b.cache, b.batch, b.rope, b.q, b.k_new, b.v_new, b.out, b.lse, 0.0, ws, b.status)
    torch.cuda.synchronize()
    assert int(b.status.item()) == 0
    assert np.array_equal(H.torch_to_bits(b.out), two_call[0]) and np.array_equal(b.lse.cpu().numpy(), two_call[1])


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (4, 4, 64), (7, 1, 128)])
def test_decode_rows_of_very_different_lengths_in_a_few_chunks(Hq, Hkv, D):
    """A handful of chunks per row: rows that end in the first chunk (their later chunks have
    no keys), an empty row and rows that end on and just past a chunk edge, against the
    oracle; twice, for run-to-run identity."""
    efim, H, _custom, _check_turn = _mods()
    lens = np.array([1, 300, 0, 1500, 700, 1499, 256, 257], np.int32)
    w = _custom(Hq, Hkv, D, np.maximum(lens, 1), [0] * len(lens), seed=41, extra=0)
    dw = H.DeviceWorkload(w)
    B, max_ctx = len(lens), 1500
    assert efim.efim_decode_launch_count(dw.cache, B, max_ctx) == 2
    ws = torch.empty(efim.efim_decode_workspace_bytes(dw.cache, B, max_ctx), dtype=torch.uint8, device="cuda")
    kp, vp, bt, seqs = w.compact_host_pool()
    q = w._normal_bits(3, (B, Hq, D))
    o, lse = orc.decode_attention(q, kp, vp, bt, lens, Hq)
    dq = H.bits_to_torch(q)
    outs = []
    for _ in range(2):
        out = torch.full_like(dq, 9.0)
        lse_d = torch.full((B, Hq), 9.0, dtype=torch.float32, device="cuda")
        efim.efim_decode_attn(dw.cache, B, torch.from_numpy(lens).cuda(), max_ctx, dw.batch.d_block_table, dq, out, lse_d,
                              0.0, ws, dw.status)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        outs.append((out, lse_d))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16)) and torch.equal(outs[0][1], outs[1][1])
    out, lse_d = outs[0]
    assert torch.all(out[2] == 0) and torch.all(torch.isinf(lse_d[2]))
    keep = lens > 0
    H.assert_attn_close(H.torch_to_bits(out)[keep], o[keep], "decode, ragged rows")
    H.assert_lse_close(lse_d.cpu().numpy()[keep], lse[keep], "decode, ragged rows")


def test_garbage_beyond_the_context_and_odd_cached_values():
    """What a real cache holds: the slots of a sequence's last page beyond its context are
    uninitialised (here NaN and Inf patterns, in K and in V), and cached values include
    zeros of both signs, bf16 subnormals and entries several sigma out.  Neither the prefill
    nor the decode kernel may let the former leak into a result; the latter must be read
    exactly (the oracle gets the same bits)."""
    efim, H, _custom, _check_turn = _mods()
    w = _custom(8, 2, 128, [300, 77, 130], [40, 3, 129], seed=51, extra=2)
    odd = np.array([0x0000, 0x8000, 0x0001, 0x807F, 0x0040, 0x4100, 0xC120, 0x3F80], np.uint16)  # 0, -0, subnormals, 8, -10, 1
    real_page_bits = w.page_bits

    def page_bits(which, page_ids):
        out = real_page_bits(which, page_ids)
        flat = out.reshape(len(page_ids), -1)
        flat[:, 5::97] = odd[(np.arange(flat[:, 5::97].shape[1]) + (0 if which == "k" else 3)) % len(odd)]
        return out
    w.page_bits = page_bits
    dw = H.DeviceWorkload(w)
    used = np.array(sorted(set(w.block_table[w.block_table >= 0].tolist())), np.int64)
    idx = torch.as_tensor(used, device="cuda")
    dw.k_pool[idx] = H.bits_to_torch(page_bits("k", used))
    dw.v_pool[idx] = H.bits_to_torch(page_bits("v", used))
    nan_inf = torch.tensor([0x7FC0, 0x7F80, 0xFF80, 0x7FFF], dtype=torch.int32).to(torch.int16).cuda().view(torch.bfloat16)
    for sq in range(w.batch):
        L = int(w.cached_len[sq] + w.new_len[sq])
        pg, slot = int(w.block_table[sq, L // 16]), L % 16       # the page the context ends in, first slot beyond it
        for pool in (dw.k_pool, dw.v_pool):
            pool[pg, :, slot:, :] = nan_inf[torch.arange(pool[pg, :, slot:, :].numel(), device="cuda") % 4].view(
                pool[pg, :, slot:, :].shape)
    dw.gpu_kv_append()
    dw.gpu_prefill()
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0
    ref = dw.oracle_turn()
    H.assert_attn_close(H.torch_to_bits(dw.out), ref["o"], "prefill beside NaN slots")
    H.assert_lse_close(dw.lse.cpu().numpy(), ref["lse"], "prefill beside NaN slots")
    # decode over the same contexts (every key so far; the NaN slots lie just beyond)
    ctx = (w.cached_len + w.new_len).astype(np.int32)
    q = w._normal_bits(8, (w.batch, 8, 128))
    o, lse = orc.decode_attention(q, ref["k_pool"], ref["v_pool"], ref["bt"], ctx, 8)
    out = torch.empty((w.batch, 8, 128), dtype=torch.bfloat16, device="cuda")
    lse_d = torch.empty((w.batch, 8), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(efim.efim_decode_workspace_bytes(dw.cache, w.batch, int(ctx.max())), 256), dtype=torch.uint8,
                     device="cuda")
    efim.efim_decode_attn(dw.cache, w.batch, torch.from_numpy(ctx).cuda(), int(ctx.max()), dw.batch.d_block_table,
                          H.bits_to_torch(q), out, lse_d, 0.0, ws, dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0
    H.assert_attn_close(H.torch_to_bits(out), o, "decode beside NaN slots")
    H.assert_lse_close(lse_d.cpu().numpy(), lse, "decode beside NaN slots")


def test_planned_prefill_with_resident_lists_can_be_captured_in_a_graph():
    """With lists_resident = 1 the planned call copies nothing and only launches, so it can be
    recorded into a CUDA graph (a model's per-layer loop); the replay gives the same bits."""
    efim, H, _custom, _check_turn = _mods()
    w = make_workload("cfg3", small=True)
    dw = H.DeviceWorkload(w)
    dw.gpu_kv_append()
    plan = efim.efim_prefill_plan(dw.cache, dw.batch)
    ws = torch.empty(max(efim.efim_prefill_workspace_bytes(dw.cache, dw.batch), 256), dtype=torch.uint8, device="cuda")
    efim.efim_append_prefill_attn(dw.cache, dw.batch, dw.q, dw.out, dw.lse, 0.0, ws, dw.status, plan=plan)   # uploads the lists
    torch.cuda.synchronize()
    want_out, want_lse = dw.out.clone(), dw.lse.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            efim.efim_append_prefill_attn(dw.cache, dw.batch, dw.q, dw.out, dw.lse, 0.0, ws, dw.status, plan=plan,
                                          lists_resident=True, stream=side)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        dw.out.zero_()
        dw.lse.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        assert torch.equal(dw.out.view(torch.int16), want_out.view(torch.int16)) and torch.equal(dw.lse, want_lse)


def test_bounded_wait_expires_and_reports():
    """One warp waits on a barrier nothing completes, with nothing in flight: after the
    limit the kernel sets EFIM_DEV_TIMEOUT and ends normally; the context stays usable."""
    efim, H, _custom, _check_turn = _mods()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    limit_ns = 1_000_000                                     # 1 ms
    efim.efim_selftest_bounded_wait(limit_ns, status, waited)
    torch.cuda.synchronize()
    assert int(status.item()) == TIMEOUT
    # (the clock is read every 1024 polls, so the wait overshoots the limit by some polls' worth)
    assert limit_ns <= int(waited.item()) < 1_000_000_000
    with pytest.raises(efim.EfimError):
        efim.efim_selftest_bounded_wait(10_000_000_000, status, waited)      # limits above 0.1 s are refused
    # the context is intact: a real call still runs and is correct
    _check_turn(make_workload("cfg1"))
