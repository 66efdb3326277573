"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle on the
same seeded inputs.  Scatter/layout bit-exact; RoPE within one bf16 ulp; attention
outputs max abs <= 2e-2 and mean abs <= 2e-3 (bf16 operands, fp32 accumulation)."""
import numpy as np
import pytest
import torch

from efim_synth import make_workload
from oracle import efim_oracle as orc

pytestmark = pytest.mark.gpu


def _harness():
    import tests.gpu_harness as H
    return H


def _check_turn(w, seqs=None, interleaved=False, use_rope=True, sm_scale=None):
    H = _harness()
    dw = H.DeviceWorkload(w, interleaved=interleaved, use_rope=use_rope)
    dw.gpu_kv_append()
    dw.gpu_prefill(0.0 if sm_scale is None else sm_scale)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0
    ref = dw.oracle_turn(seqs, sm_scale)
    # --- cache contents of every page these sequences own
    for r, s in enumerate(ref["seqs"]):
        pg = w.pages_of(s)
        want_k = ref["k_pool"][ref["bt"][r, :len(pg)]]
        want_v = ref["v_pool"][ref["bt"][r, :len(pg)]]
        got_k = dw.pages_from_device("k", pg)
        got_v = dw.pages_from_device("v", pg)
        assert np.array_equal(got_v, want_v), "V pages must match bit for bit"
        if use_rope:
            H.assert_rope_close(got_k, want_k, "K pages")
            # slots not written this turn are untouched: exact
            C, N = int(w.cached_len[s]), int(w.new_len[s])
            tok = np.arange(len(pg) * w.page_size)
            old = (tok < C) | (tok >= C + N)
            gk = np.transpose(got_k, (0, 2, 1, 3)).reshape(len(tok), -1)
            wk = np.transpose(want_k, (0, 2, 1, 3)).reshape(len(tok), -1)
            assert np.array_equal(gk[old], wk[old])
        else:
            assert np.array_equal(got_k, want_k)
    # --- rotated q
    got_q = H.torch_to_bits(dw.q)[ref["rows"]]
    if use_rope:
        H.assert_rope_close(got_q, ref["q_rot"], "rotated q")
    else:
        assert np.array_equal(got_q, ref["q_rot"])
    # --- attention
    got_o = H.torch_to_bits(dw.out)[ref["rows"]]
    H.assert_attn_close(got_o, ref["o"], f"{w.name} append-prefill")
    got_lse = dw.lse.cpu().numpy()[ref["rows"]]
    H.assert_lse_close(got_lse, ref["lse"], f"{w.name} append-prefill")
    return dw, ref


def test_cfg1_turn_and_decode_steps():
    H = _harness()
    import paper_2505_21889_b200 as efim
    w = make_workload("cfg1")
    dw, ref = _check_turn(w)
    # 8 decode steps: append one token, attend over everything so far
    kp, vp, bt = ref["k_pool"], ref["v_pool"], ref["bt"]
    ctx = (w.cached_len + w.new_len).astype(np.int32)
    B = w.batch
    d_bt = dw.batch.d_block_table
    for step in range(w.decode_steps):
        q, k, v = w.decode_qkv(step)
        one = np.ones(B, np.int32)
        q_rot = orc.kv_append(kp, vp, bt, ctx, one, q, k, v, w.rope_base)
        ctx = ctx + 1
        o, lse = orc.decode_attention(q_rot, kp, vp, bt, ctx, w.num_q_heads)
        sb = efim.Batch(ctx - 1, one, d_bt)
        dq, dk, dv = H.bits_to_torch(q), H.bits_to_torch(k), H.bits_to_torch(v)
        efim.efim_kv_append(dw.cache, sb, dw.rope, dq, dk, dv, dw.status)
        d_ctx = torch.from_numpy(ctx).cuda()
        out = torch.empty_like(dq)
        lse_d = torch.empty((B, w.num_q_heads), dtype=torch.float32, device="cuda")
        nbytes = efim.efim_decode_workspace_bytes(dw.cache, B, int(ctx.max()))
        ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        efim.efim_decode_attn(dw.cache, B, d_ctx, int(ctx.max()), d_bt, dq, out, lse_d, 0.0, ws, dw.status)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        H.assert_rope_close(H.torch_to_bits(dq), q_rot, "decode q")
        H.assert_attn_close(H.torch_to_bits(out), o, f"cfg1 decode step {step}")
        H.assert_lse_close(lse_d.cpu().numpy(), lse, "decode")
    pg = w.pages_of(0)
    assert np.array_equal(dw.pages_from_device("v", pg), vp[bt[0, :len(pg)]])


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4a", "cfg4b", "cfg4b_3072"])
def test_small_configs_all_rows(name):
    _check_turn(make_workload(name, small=True))


@pytest.mark.parametrize("interleaved,use_rope", [(True, True), (False, False)])
def test_cfg1_rope_variants(interleaved, use_rope):
    _check_turn(make_workload("cfg1"), interleaved=interleaved, use_rope=use_rope)


def test_custom_scale():
    _check_turn(make_workload("cfg1"), sm_scale=0.2)


def _custom(Hq, Hkv, D, cached, new, seed=7, extra=3):
    from efim_synth.workloads import Workload, _block_table
    cached = np.asarray(cached, np.int32)
    new = np.asarray(new, np.int32)
    rng = np.random.default_rng([seed, 99])
    pages = int((-(-(cached + new + extra) // 16)).sum()) + 7
    bt = _block_table(rng, pages, cached + new + extra, 16)
    return Workload(f"custom{Hq}_{Hkv}_{D}", seed, Hq, Hkv, D, 16, pages, 10000.0, cached, new, bt, decode_steps=extra)


@pytest.mark.parametrize("Hq,Hkv,D,cached,new", [
    (4, 4, 64, [237], [16]),                 # cached length not page aligned
    (8, 2, 128, [0, 5, 300], [33, 1, 130]),  # nothing cached; one new token; spans tiles
    (7, 1, 128, [100, 17], [40, 3]),         # group of 7
    (14, 2, 64, [64, 0], [0, 50]),           # a sequence with no new tokens
    (6, 2, 128, [15, 16, 17], [17, 16, 15]), # around page edges
    (1, 1, 64, [1], [1]),
    (16, 1, 128, [50], [9]),                 # group of 16
])
def test_edge_shapes(Hq, Hkv, D, cached, new):
    _check_turn(_custom(Hq, Hkv, D, cached, new))


@pytest.mark.parametrize("name", ["cfg5"])
def test_decode_loop_small(name):
    H = _harness()
    import paper_2505_21889_b200 as efim
    w = make_workload(name, small=True)
    dw = H.DeviceWorkload(w)
    kp, vp, bt, seqs = w.compact_host_pool()
    ctx = w.cached_len.astype(np.int32).copy()
    B = w.batch
    d_bt = dw.batch.d_block_table
    max_ctx = int(ctx.max()) + w.decode_steps
    nbytes = efim.efim_decode_workspace_bytes(dw.cache, B, max_ctx)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    one = np.ones(B, np.int32)
    for step in range(w.decode_steps):
        q, k, v = w.decode_qkv(step)
        q_rot = orc.kv_append(kp, vp, bt, ctx, one, q, k, v, w.rope_base)
        sb = efim.Batch(ctx, one, d_bt)
        ctx = ctx + 1
        o, lse = orc.decode_attention(q_rot, kp, vp, bt, ctx, w.num_q_heads)
        dq, dk, dv = H.bits_to_torch(q), H.bits_to_torch(k), H.bits_to_torch(v)
        efim.efim_kv_append(dw.cache, sb, dw.rope, dq, dk, dv, dw.status)
        d_ctx = torch.from_numpy(ctx).cuda()
        out = torch.empty_like(dq)
        lse_d = torch.empty((B, w.num_q_heads), dtype=torch.float32, device="cuda")
        efim.efim_decode_attn(dw.cache, B, d_ctx, max_ctx, d_bt, dq, out, lse_d, 0.0, ws, dw.status)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        H.assert_attn_close(H.torch_to_bits(out), o, f"{name} decode step {step}")
        H.assert_lse_close(lse_d.cpu().numpy(), lse, "decode")


@pytest.mark.parametrize("Hq,Hkv,D", [(5, 1, 128), (12, 2, 128), (7, 1, 64), (28, 4, 128), (8, 1, 128), (16, 1, 128),
                                        (20, 2, 64)])
def test_decode_group_sizes_against_oracle(Hq, Hkv, D):
    """Groups of 5 to 8 query heads per kv head run in one CTA (two passes over the page in
    shared memory); larger groups are cut evenly.  Plain and fused steps against the oracle."""
    H = _harness()
    import paper_2505_21889_b200 as efim
    ctx0 = [1, 15, 16, 17, 333, 1200, 2100]
    w = _custom(Hq, Hkv, D, ctx0, [0] * len(ctx0), seed=Hq * 100 + D, extra=3)
    dw = H.DeviceWorkload(w)
    kp, vp, bt, seqs = w.compact_host_pool()
    ctx = np.array(ctx0, np.int32)
    B = w.batch
    max_ctx = int(ctx.max()) + 3
    ws = torch.empty(max(efim.efim_decode_workspace_bytes(dw.cache, B, max_ctx), 256), dtype=torch.uint8, device="cuda")
    one = np.ones(B, np.int32)
    for step in range(3):
        q, k, v = w.decode_qkv(step)
        q_rot = orc.kv_append(kp, vp, bt, ctx, one, q, k, v, w.rope_base)
        ctx = ctx + 1
        o, lse = orc.decode_attention(q_rot, kp, vp, bt, ctx, Hq)
        dq, dk, dv = H.bits_to_torch(q), H.bits_to_torch(k), H.bits_to_torch(v)
        out = torch.empty_like(dq)
        lse_d = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
        d_ctx = torch.from_numpy(ctx).cuda()
        if step == 1:                                  # the two-call form in the middle of the loop
            efim.efim_kv_append(dw.cache, efim.Batch(ctx - 1, one, dw.batch.d_block_table), dw.rope, dq, dk, dv, dw.status)
            efim.efim_decode_attn(dw.cache, B, d_ctx, max_ctx, dw.batch.d_block_table, dq, out, lse_d, 0.0, ws, dw.status)
        else:
            efim.efim_decode_step(dw.cache, B, d_ctx, max_ctx, dw.batch.d_block_table, dw.rope, dq, dk, dv, out, lse_d,
                                  0.0, ws, dw.status)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        H.assert_attn_close(H.torch_to_bits(out), o, f"G={Hq // Hkv} D={D} step {step}")
        H.assert_lse_close(lse_d.cpu().numpy(), lse, f"G={Hq // Hkv} D={D} step {step}")
    used = np.array(sorted(set(w.block_table[w.block_table >= 0].tolist())), np.int64)
    assert np.array_equal(dw.pages_from_device("v", used), vp)
    H.assert_rope_close(dw.pages_from_device("k", used), kp, "k pages after the loop")


def test_decode_one_long_row_many_chunks():
    """A lone long row is cut into more than 32 chunks (so that every SM gets work); the merge
    then takes more than one pass over the lanes for the chunks' lse values."""
    H = _harness()
    import paper_2505_21889_b200 as efim
    Hq, Hkv, D = 8, 2, 128
    w = _custom(Hq, Hkv, D, [12000, 40], [0, 0], seed=5, extra=2)
    dw = H.DeviceWorkload(w)
    kp, vp, bt, seqs = w.compact_host_pool()
    ctx = w.cached_len.astype(np.int32).copy()
    B = w.batch
    max_ctx = int(ctx.max()) + 2
    nbytes = efim.efim_decode_workspace_bytes(dw.cache, B, max_ctx)
    assert nbytes > 33 * B * Hq * D * 4, "expected more than 32 chunks"
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    one = np.ones(B, np.int32)
    for step in range(2):
        q, k, v = w.decode_qkv(step)
        q_rot = orc.kv_append(kp, vp, bt, ctx, one, q, k, v, w.rope_base)
        ctx = ctx + 1
        o, lse = orc.decode_attention(q_rot, kp, vp, bt, ctx, Hq)
        dq, dk, dv = H.bits_to_torch(q), H.bits_to_torch(k), H.bits_to_torch(v)
        out = torch.empty_like(dq)
        lse_d = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
        efim.efim_decode_step(dw.cache, B, torch.from_numpy(ctx).cuda(), max_ctx, dw.batch.d_block_table, dw.rope,
                              dq, dk, dv, out, lse_d, 0.0, ws, dw.status)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        H.assert_attn_close(H.torch_to_bits(out), o, f"long row, step {step}")
        H.assert_lse_close(lse_d.cpu().numpy(), lse, "decode")


def test_decode_zero_length_and_bad_page_flag():
    H = _harness()
    import paper_2505_21889_b200 as efim
    w = _custom(4, 2, 128, [40, 0, 90], [0, 0, 0])
    dw = H.DeviceWorkload(w)
    ctx = torch.tensor([40, 0, 90], dtype=torch.int32, device="cuda")
    q = H.bits_to_torch(w._normal_bits(5, (3, 4, 128)))
    out = torch.full_like(q, 7.0)
    lse = torch.zeros((3, 4), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(efim.efim_decode_workspace_bytes(dw.cache, 3, 96), 256), dtype=torch.uint8, device="cuda")
    efim.efim_decode_attn(dw.cache, 3, ctx, 96, dw.batch.d_block_table, q, out, lse, 0.0, ws, dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0
    assert torch.all(out[1] == 0) and torch.all(torch.isinf(lse[1])) and torch.all(lse[1] < 0)
    # a block-table id outside the pool is reported, not dereferenced
    bad = dw.batch.d_block_table.clone()
    bad[2, 1] = w.num_pages + 5
    efim.efim_decode_attn(dw.cache, 3, ctx, 96, bad, q, out, lse, 0.0, ws, dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) & 0x1
    assert torch.isfinite(out.float()).all()
    # a device length beyond what the block table addresses is clamped and reported
    dw.status.zero_()
    cap = dw.batch.d_block_table.shape[1] * 16
    too_long = torch.tensor([40, 0, cap + 100], dtype=torch.int32, device="cuda")
    efim.efim_decode_attn(dw.cache, 3, too_long, 96, dw.batch.d_block_table, q, out, lse, 0.0, ws, dw.status)
    torch.cuda.synchronize()
    assert int(dw.status.item()) & 0x2


def test_pages_outside_the_batch_are_untouched():
    H = _harness()
    w = make_workload("cfg2", small=True)
    dw = H.DeviceWorkload(w)
    used = set(w.block_table[w.block_table >= 0].tolist())
    free = np.array([p for p in range(w.num_pages) if p not in used][:200])
    before_k, before_v = dw.pages_from_device("k", free), dw.pages_from_device("v", free)
    assert np.array_equal(before_k, w.page_bits("k", free))      # device fill == host fill
    dw.gpu_kv_append()
    dw.gpu_prefill()
    torch.cuda.synchronize()
    assert np.array_equal(dw.pages_from_device("k", free), before_k)
    assert np.array_equal(dw.pages_from_device("v", free), before_v)


def test_run_to_run_bit_reproducible():
    H = _harness()
    w = make_workload("cfg3", small=True)
    outs = []
    for _ in range(2):
        dw = H.DeviceWorkload(w)
        dw.gpu_kv_append()
        dw.gpu_prefill()
        torch.cuda.synchronize()
        outs.append((H.torch_to_bits(dw.out), dw.lse.cpu().numpy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("T,Hq,Hkv,D,interleaved", [
    (1024, 4, 2, 128, False),     # four warps per token
    (1023, 6, 2, 64, True),       # eight warps per token, odd token count
    (4096, 4, 4, 64, False),      # two warps per token
    (5000, 3, 1, 128, True),      # two warps per token, heads not a multiple of the lanes' head stride
    (16384, 2, 1, 64, False),     # one warp per token
    (16391, 2, 2, 128, False),    # one warp per token, ragged last CTA
])
def test_kv_append_token_count_regimes(T, Hq, Hkv, D, interleaved):
    """efim_kv_append picks the number of warps per token from the token count; every
    variant must place and rotate exactly like the oracle (rows of three sequences,
    unaligned starts)."""
    H = _harness()
    import paper_2505_21889_b200 as efim
    new = [T // 3, T // 5, T - T // 3 - T // 5]
    w = _custom(Hq, Hkv, D, [13, 0, 255], new, seed=T, extra=0)
    dw = H.DeviceWorkload(w, interleaved=interleaved)
    dw.gpu_kv_append()
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0
    kp, vp, bt, seqs = w.compact_host_pool()
    q_rot = orc.kv_append(kp, vp, bt, w.cached_len, w.new_len, dw.q_bits, dw.k_bits, dw.v_bits, w.rope_base,
                          interleaved)
    used = np.array(sorted(set(w.block_table[w.block_table >= 0].tolist())), np.int64)
    assert np.array_equal(dw.pages_from_device("v", used), vp)            # placement and copy: bit-exact
    H.assert_rope_close(dw.pages_from_device("k", used), kp, "k pages")
    H.assert_rope_close(H.torch_to_bits(dw.q), q_rot, "q")


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4a"])
def test_planned_prefill_is_bit_identical_and_checks_its_plan(name):
    """efim_append_prefill_attn_planned with a plan made once (as for every layer of a model)
    gives the same bits as the call that plans inside; a plan for other lengths is refused."""
    H = _harness()
    import paper_2505_21889_b200 as efim
    w = make_workload(name, small=True)
    dw = H.DeviceWorkload(w)
    dw.gpu_kv_append()
    dw.gpu_prefill()
    torch.cuda.synchronize()
    want_out, want_lse = dw.out.clone(), dw.lse.clone()
    plan = efim.efim_prefill_plan(dw.cache, dw.batch)
    for resident in (False, True, True):                   # the same plan: uploaded once, then only launched
        dw.out.zero_()
        dw.lse.zero_()
        efim.efim_append_prefill_attn(dw.cache, dw.batch, dw.q, dw.out, dw.lse, 0.0, dw.ws, dw.status, plan=plan,
                                      lists_resident=resident)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        assert torch.equal(dw.out.view(torch.int16), want_out.view(torch.int16)) and torch.equal(dw.lse, want_lse)
    other = efim.Batch(w.cached_len + 1, w.new_len, dw.batch.d_block_table)
    with pytest.raises(efim.EfimError) as e:
        efim.efim_append_prefill_attn(dw.cache, other, dw.q, dw.out, dw.lse, 0.0, dw.ws, dw.status, plan=plan)
    assert e.value.code == 1
    with pytest.raises(efim.EfimError):                    # a truncated blob
        efim.efim_append_prefill_attn(dw.cache, dw.batch, dw.q, dw.out, dw.lse, 0.0, dw.ws, dw.status, plan=plan[:64])


@pytest.mark.parametrize("Hq,Hkv,D,interleaved,use_rope", [
    (8, 2, 128, False, True),     # group of 4: one pass over a page's keys
    (7, 1, 128, False, True),     # group of 7: two passes over the staged page, K/V fetched once
    (4, 4, 64, True, True),       # head_dim 64, interleaved pairing
    (6, 2, 64, False, False),     # no rotation
    (10, 2, 128, True, True),     # group of 5
    (16, 1, 64, False, True),     # group of 16: two CTAs of 8 heads share the new token's page
])
def test_fused_decode_step_equals_append_then_decode(Hq, Hkv, D, interleaved, use_rope):
    """efim_decode_step against efim_kv_append + efim_decode_attn on the same inputs, over
    several steps (page edges included): outputs, lse and the pools bit for bit; q untouched."""
    H = _harness()
    import paper_2505_21889_b200 as efim
    ctx0 = [15, 16, 31, 300, 1, 700]
    w = _custom(Hq, Hkv, D, ctx0, [0] * len(ctx0), seed=11, extra=6)
    a, b = H.DeviceWorkload(w, interleaved=interleaved, use_rope=use_rope), \
        H.DeviceWorkload(w, interleaved=interleaved, use_rope=use_rope)
    B = w.batch
    ctx = np.array(ctx0, np.int32)
    max_ctx = int(ctx.max()) + 6
    ws_a = torch.empty(max(efim.efim_decode_workspace_bytes(a.cache, B, max_ctx), 256), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty_like(ws_a)
    one = np.ones(B, np.int32)
    for step in range(6):
        q, k, v = w.decode_qkv(step)
        qa, ka, va = H.bits_to_torch(q), H.bits_to_torch(k), H.bits_to_torch(v)
        qb, kb, vb = qa.clone(), ka.clone(), va.clone()
        d_ctx = torch.from_numpy(ctx + 1).cuda()
        out_a, out_b = torch.empty_like(qa), torch.empty_like(qa)
        lse_a = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
        lse_b = torch.empty_like(lse_a)
        efim.efim_kv_append(a.cache, efim.Batch(ctx, one, a.batch.d_block_table), a.rope, qa, ka, va, a.status)
        efim.efim_decode_attn(a.cache, B, d_ctx, max_ctx, a.batch.d_block_table, qa, out_a, lse_a, 0.0, ws_a, a.status)
        efim.efim_decode_step(b.cache, B, d_ctx, max_ctx, b.batch.d_block_table, b.rope, qb, kb, vb, out_b, lse_b, 0.0,
                              ws_b, b.status)
        torch.cuda.synchronize()
        assert int(a.status.item()) == 0 and int(b.status.item()) == 0
        assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)) and torch.equal(lse_a, lse_b), step
        assert torch.equal(qb.view(torch.int16), H.bits_to_torch(q).view(torch.int16))      # q is read only
        ctx = ctx + 1
    assert torch.equal(a.k_pool.view(torch.int16), b.k_pool.view(torch.int16))
    assert torch.equal(a.v_pool.view(torch.int16), b.v_pool.view(torch.int16))
