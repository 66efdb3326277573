"""Parity at the full sizes of the five configs, in the launch configuration bench.py
times.  The GPU processes the whole batch; the oracle recomputes every row of cfg2, cfg3
and cfg4a, every row of one cfg4b sequence plus token windows of others, and 16 sequences
of cfg5 at decode steps 0, 31 and 63, from the same seeded bytes."""
import numpy as np
import pytest
import torch

import paper_2505_21889_b200 as efim
from efim_synth import make_workload
from oracle import efim_oracle as orc

pytestmark = pytest.mark.gpu


def _run_turn(w, seqs, windows=None):
    import tests.gpu_harness as H
    dw = H.DeviceWorkload(w)
    dw.gpu_kv_append()
    dw.gpu_prefill()
    torch.cuda.synchronize()
    assert int(dw.status.item()) == 0
    ref = dw.oracle_turn(seqs, windows=windows)
    for r, s in enumerate(ref["seqs"]):
        pg = w.pages_of(s, int(w.cached_len[s] + w.new_len[s]))
        assert np.array_equal(dw.pages_from_device("v", pg), ref["v_pool"][ref["bt"][r, :len(pg)]])
        H.assert_rope_close(dw.pages_from_device("k", pg), ref["k_pool"][ref["bt"][r, :len(pg)]], f"{w.name} K pages")
    H.assert_rope_close(H.torch_to_bits(dw.q)[ref["rows"]], ref["q_rot"], f"{w.name} q")
    H.assert_attn_close(H.torch_to_bits(dw.out)[ref["attn_rows"]], ref["o"], f"{w.name} full size")
    H.assert_lse_close(dw.lse.cpu().numpy()[ref["attn_rows"]], ref["lse"], f"{w.name} full size")
    # every output of the batch is finite (also the rows the oracle did not recompute)
    assert torch.isfinite(dw.out.float()).all()
    return dw, ref


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4a"])
def test_full_size_all_rows(name):
    """Every row of the batch against the oracle (cfg3: its 32 prefill rows and its 32
    one-token decode rows, all through the prefill call)."""
    _run_turn(make_workload(name), None)


def test_cfg4b_full_one_sequence_all_rows_and_windows_of_others():
    """The FIM-miss recompute: all 3,200 rows of one sequence, and of two other sequences the
    first, a middle (across a row-tile edge) and the last window of 48 tokens."""
    w = make_workload("cfg4b")
    _run_turn(w, [5])
    n = int(w.new_len[0])
    for first in (0, n // 2 - 24, n - 48):
        _run_turn(w, [0, 7], windows=[(first, 48), (first, 48)])


def test_cfg4b_3072_full_token_windows():
    w = make_workload("cfg4b_3072")
    n = int(w.new_len[2])
    for first in (0, n // 2 - 24, n - 48):
        _run_turn(w, [2], windows=[(first, 48)])


def test_cfg5_full_decode_steps_16_sequences():
    import tests.gpu_harness as H
    w = make_workload("cfg5")
    dw = H.DeviceWorkload(w)
    ctx_all = w.cached_len.astype(np.int32).copy()
    order = np.argsort(ctx_all)
    # shortest, longest and 14 spread over the length order
    seqs = sorted({int(order[0]), int(order[-1])} | {int(order[i]) for i in range(9, 256, 18)})
    assert len(seqs) >= 16
    kp, vp, bt, seqs = w.compact_host_pool(seqs)
    B = w.batch
    steps = w.decode_steps                       # all 64; the oracle checks steps 0, 31 and 63
    check = {0, 31, steps - 1}
    max_ctx = int(ctx_all.max()) + w.decode_steps
    ws = torch.empty(max(efim.efim_decode_workspace_bytes(dw.cache, B, max_ctx), 256), dtype=torch.uint8, device="cuda")
    one_all = np.ones(B, np.int32)
    one = np.ones(len(seqs), np.int32)
    ctx = ctx_all[seqs].copy()
    for step in range(steps):
        q, k, v = w.decode_qkv(step)
        q_rot = orc.kv_append(kp, vp, bt, ctx, one, q[seqs], k[seqs], v[seqs], w.rope_base)
        sb = efim.Batch(ctx_all, one_all, dw.batch.d_block_table)
        ctx_all = ctx_all + 1
        ctx = ctx + 1
        dq, dk, dv = H.bits_to_torch(q), H.bits_to_torch(k), H.bits_to_torch(v)
        efim.efim_kv_append(dw.cache, sb, dw.rope, dq, dk, dv, dw.status)
        out = torch.empty_like(dq)
        lse_d = torch.empty((B, w.num_q_heads), dtype=torch.float32, device="cuda")
        efim.efim_decode_attn(dw.cache, B, torch.from_numpy(ctx_all).cuda(), max_ctx, dw.batch.d_block_table, dq, out,
                              lse_d, 0.0, ws, dw.status)
        if step not in check:
            continue
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        o, lse = orc.decode_attention(q_rot, kp, vp, bt, ctx, w.num_q_heads)
        H.assert_attn_close(H.torch_to_bits(out)[seqs], o, f"cfg5 full decode step {step}")
        H.assert_lse_close(lse_d.cpu().numpy()[seqs], lse, "decode")
        assert torch.isfinite(out.float()).all()
        # the fused step on the same inputs (it stores the same k/v again): identical bits at full size
        out_f = torch.empty_like(out)
        lse_f = torch.empty_like(lse_d)
        efim.efim_decode_step(dw.cache, B, torch.from_numpy(ctx_all).cuda(), max_ctx, dw.batch.d_block_table, dw.rope,
                              H.bits_to_torch(q), dk, dv, out_f, lse_f, 0.0, ws, dw.status)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        assert torch.equal(out_f.view(torch.int16), out.view(torch.int16)) and torch.equal(lse_f, lse_d)
    for r, s in enumerate(seqs):
        pg = w.pages_of(s, int(ctx_all[s]))[-2:]
        want = vp[bt[r, len(w.pages_of(s, int(ctx_all[s]))) - 2: len(w.pages_of(s, int(ctx_all[s])))]]
        assert np.array_equal(dw.pages_from_device("v", pg), want)
