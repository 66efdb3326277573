"""End to end through the front end and the three GPU calls: a small multi-turn replay
whose every round is checked against the oracle's FULL recompute of the whole prompt
(no cache, no reuse).  This is the paper's central claim (Sec. 1) seen through the cache
manager: with the EFIM order the cached prefix and suffix pages give exactly what
recomputing them would."""
import numpy as np
import pytest
import torch

from efim_synth import infill_sessions, bf16_bits_to_f32
from oracle import efim_oracle as orc

pytestmark = pytest.mark.gpu

HQ, HKV, D, VOCAB, GEN = 4, 2, 64, 200, 6


def _full_recompute(layer_bits, prompt, gen):
    """Oracle: prefill of the whole prompt from position 0, then the decode steps."""
    q_tab, k_tab, v_tab = layer_bits
    L = len(prompt)
    pages = -(-(L + len(gen)) // 16)
    kp = np.zeros((pages, HKV, 16, D), np.uint16)
    vp = np.zeros_like(kp)
    bt = np.arange(pages, dtype=np.int32)[None, :]
    zero, n = np.zeros(1, np.int32), np.array([L], np.int32)
    q_rot = orc.kv_append(kp, vp, bt, zero, n, q_tab[prompt], k_tab[prompt], v_tab[prompt], 10000.0)
    o, _ = orc.append_prefill_attention(q_rot, kp, vp, bt, zero, n, HQ)
    od = None
    for s, g in enumerate(gen):
        ctx = np.array([L + s], np.int32)
        qd = orc.kv_append(kp, vp, bt, ctx, np.ones(1, np.int32), q_tab[[g]], k_tab[[g]], v_tab[[g]], 10000.0)
        od, _ = orc.decode_attention(qd, kp, vp, bt, ctx + 1, HQ)
    return o, od


@pytest.mark.parametrize("scheme,graph", [("efim", False), ("fim", False), ("efim", True)])
def test_replay_with_reuse_equals_full_recompute(scheme, graph):
    import tests.gpu_harness as H
    from paper_2505_21889_b200 import replay
    sessions = infill_sessions(5, users=3, rounds=3, vocab=VOCAB, prefix0=(60, 140), suffix0=(30, 80),
                               typed=(4, 20), gen=GEN)
    longest = max(len(t["prefix"]) + len(t["suffix"]) + 3 + GEN for u in sessions for t in u)
    layer = replay.Layer(5, VOCAB, HQ, HKV, D, pool_pages=256, max_position=longest + 1)
    seen = []

    def observe(r, group, prompts, cached, bt, out, dec_out):
        assert group == [0, 1, 2]
        out_bits, dec_bits = H.torch_to_bits(out), H.torch_to_bits(dec_out)
        row = 0
        for u, prompt in enumerate(prompts):
            o, od = _full_recompute(layer.bits, prompt, sessions[u][r]["gen"])
            n_new = len(prompt) - cached[u]
            H.assert_attn_close(out_bits[row:row + n_new], o[cached[u]:], f"{scheme} round {r} user {u} prefill")
            H.assert_attn_close(dec_bits[u:u + 1], od, f"{scheme} round {r} user {u} last decode step")
            row += n_new
            if r > 0 and scheme == "efim":      # prefix and suffix (and the specials) are cache hits
                t0 = sessions[u][0]
                assert cached[u] >= (len(t0["prefix"]) + len(t0["suffix"]) + 3) // 16 * 16
        seen.append(cached.copy())

    totals = replay.run_scheme(scheme, sessions, layer, 256, -(-longest // 16), observe, graph=graph)
    assert len(seen) == 3 and (seen[0] == 0).all() and totals["evictions"] == 0
    assert totals["computed_tokens"] + totals["hit_tokens"] == totals["prompt_tokens"]
    if scheme == "fim":                         # the suffix follows the changed prefix: never reusable
        for r in (1, 2):
            for u in range(3):
                assert seen[r][u] <= 1 + len(sessions[u][r - 1]["prefix"])


def test_reuse_rates_order_and_fall_with_a_small_pool():
    from paper_2505_21889_b200 import replay
    sessions = infill_sessions(6, users=4, rounds=4, vocab=VOCAB, prefix0=(200, 400), suffix0=(100, 200),
                               typed=(4, 20), gen=GEN)
    longest = max(len(t["prefix"]) + len(t["suffix"]) + 3 + GEN for u in sessions for t in u)
    mp = -(-longest // 16)
    layer = replay.Layer(6, VOCAB, HQ, HKV, D, pool_pages=1024, max_position=longest + 1)
    rate = {s: replay.run_scheme(s, sessions, layer, 1024, mp)["reuse_rate"] for s in replay.SCHEMES}
    assert rate["none"] == 0.0 < rate["fim"] < rate["efim"]
    # users served two at a time from a pool that holds little more than the running pair:
    # by a user's next turn its pages have been taken (Sec. 5.3: reuse falls as users outgrow memory)
    tight = replay.run_scheme("efim", sessions, layer, 2 * mp + 8, mp, batch_size=2)
    assert tight["evictions"] > 0 and tight["reuse_rate"] < rate["efim"]
