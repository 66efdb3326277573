"""Pins for the CPU oracle: every check here compares the oracle with something
other than itself - a closed form, a library routine on a special case, a dense
brute force with Python loops, hand-derived values (tests/golden), or an
identity the paper's reordering relies on (EFIM Sec. 1, Sec. 2.2 / Fig. 3)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import efim_oracle as orc
from efim_synth import f32_to_bf16_bits, bf16_bits_to_f32

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(rng, shape):
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


def _random_paged_case(rng, B, Hq, Hkv, D, P, cached, new, extra_pages=5):
    """Build pools + block table; cached part holds random bf16 'already rotated' data."""
    cached = np.asarray(cached, np.int32)
    new = np.asarray(new, np.int32)
    need = -(-(cached + new) // P)
    num_pages = int(need.sum()) + extra_pages
    perm = rng.permutation(num_pages)
    bt = np.full((B, int(need.max()) + 1), -1, np.int32)
    off = 0
    for s in range(B):
        bt[s, :need[s]] = perm[off:off + need[s]]
        off += need[s]
    k_pool = _bits(rng, (num_pages, Hkv, P, D))
    v_pool = _bits(rng, (num_pages, Hkv, P, D))
    T = int(new.sum())
    q, k, v = _bits(rng, (T, Hq, D)), _bits(rng, (T, Hkv, D)), _bits(rng, (T, Hkv, D))
    return k_pool, v_pool, bt, cached, new, q, k, v


# ---------------------------------------------------------------- bf16 rounding
def test_bf16_roundtrip_and_matches_torch_rne():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.f64_to_bf16(x.astype(np.float64))
    assert np.array_equal(got, want)
    assert np.array_equal(orc.f64_to_bf16(orc.bf16_to_f64(want)), want)
    assert np.array_equal(orc.bf16_to_f64(want), bf16_bits_to_f32(want).astype(np.float64))


def test_bf16_single_rounding_from_f64():
    # 1 + 2^-8 is the tie between 1.0 and 1+2^-7; adding 2^-30 must round UP.
    # Rounding through float32 first would land on the tie and give 1.0.
    x = np.array([1.0 + 2.0 ** -8 + 2.0 ** -30, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8,
                  -(1.0 + 2.0 ** -8 + 2.0 ** -30), 0.0, 2.0 ** -133, 2.0 ** -134, 1.5 * 2.0 ** -133])
    got = orc.bf16_to_f64(orc.f64_to_bf16(x))
    want = np.array([1.0 + 2.0 ** -7, 1.0, 1.0 + 2.0 ** -6, -(1.0 + 2.0 ** -7), 0.0,
                     2.0 ** -133, 0.0, 2.0 ** -132])
    assert np.array_equal(got, want)


# ---------------------------------------------------------------- RoPE
def test_rope_position_zero_is_identity_and_norm_preserved():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 3, 16))
    for inter in (False, True):
        assert np.array_equal(orc.rope_rotate_f64(x, np.zeros(5, int), 10000.0, inter), x)
        y = orc.rope_rotate_f64(x, np.array([1, 7, 100, 4095, 32767]), 10000.0, inter)
        assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=0, atol=1e-12)


def test_rope_d2_is_plane_rotation_by_p_radians():
    # D = 2: one frequency, theta_0 = base^0 = 1, so the vector turns by `pos` radians
    # counter-clockwise: (a + ib) * e^{i pos}.
    rng = np.random.default_rng(2)
    x = rng.standard_normal((6, 2, 2))
    pos = np.array([0, 1, 2, 3, 10, 1000])
    z = (x[..., 0] + 1j * x[..., 1]) * np.exp(1j * pos)[:, None]
    for inter in (False, True):       # with one pair both pairings coincide
        y = orc.rope_rotate_f64(x, pos, 12345.0, inter)
        assert np.allclose(y[..., 0], z.real, atol=1e-12) and np.allclose(y[..., 1], z.imag, atol=1e-12)


def test_rope_frequencies_follow_base_power():
    # a unit vector on pair f turns by pos * base^(-2f/D): read the angle back with atan2
    D, base, pos = 8, 10000.0, 3
    for f in range(D // 2):
        x = np.zeros((1, 1, D))
        x[0, 0, f] = 1.0
        y = orc.rope_rotate_f64(x, np.array([pos]), base)[0, 0]
        ang = math.atan2(y[f + D // 2], y[f])
        assert abs(ang - pos * base ** (-2.0 * f / D)) < 1e-12
        mask = np.ones(D, bool)
        mask[[f, f + D // 2]] = False
        assert np.all(y[mask] == 0.0)


def test_rope_relative_position_property():
    # <R_m q, R_n k> depends on m - n only: shift all positions by a constant.
    rng = np.random.default_rng(3)
    q = rng.standard_normal((4, 2, 32))
    k = rng.standard_normal((4, 2, 32))
    p = np.array([0, 5, 17, 40])
    for inter in (False, True):
        s0 = np.einsum("thd,uhd->htu", orc.rope_rotate_f64(q, p, 10000.0, inter),
                       orc.rope_rotate_f64(k, p, 10000.0, inter))
        s1 = np.einsum("thd,uhd->htu", orc.rope_rotate_f64(q, p + 1234, 10000.0, inter),
                       orc.rope_rotate_f64(k, p + 1234, 10000.0, inter))
        assert np.allclose(s0, s1, atol=1e-10)


def test_rope_interleaved_is_rotate_half_after_dim_permutation():
    rng = np.random.default_rng(4)
    D = 16
    x = rng.standard_normal((3, 2, D))
    p = np.array([3, 9, 200])
    perm = np.concatenate([np.arange(0, D, 2), np.arange(1, D, 2)])    # interleaved index of half-layout slot
    y_half = orc.rope_rotate_f64(x[..., perm], p, 500.0, False)
    y_int = orc.rope_rotate_f64(x, p, 500.0, True)
    assert np.allclose(y_int[..., perm], y_half, atol=1e-14)


def test_rope_rotate_half_matches_transformers_llama():
    # Library special case: the rotate-half convention of the Llama-family reference code.
    tf = pytest.importorskip("transformers.models.llama.modeling_llama")
    rng = np.random.default_rng(5)
    T, H, D, base = 7, 3, 32, 10000.0
    x = rng.standard_normal((T, H, D))
    pos = np.array([0, 1, 2, 50, 777, 4096, 30000])
    inv_freq = 1.0 / (base ** (torch.arange(0, D, 2, dtype=torch.float64) / D))
    freqs = torch.from_numpy(pos).to(torch.float64)[:, None] * inv_freq[None, :]
    emb = torch.cat([freqs, freqs], dim=-1)
    cos, sin = emb.cos()[None], emb.sin()[None]                # [1, T, D]
    xt = torch.from_numpy(x).permute(1, 0, 2)[None]            # [1, H, T, D]
    qe, _ = tf.apply_rotary_pos_emb(xt, xt, cos, sin)
    want = qe[0].permute(1, 0, 2).numpy()
    got = orc.rope_rotate_f64(x, pos, base, False)
    assert np.allclose(got, want, atol=1e-12)


def test_rope_bits_version_rounds_the_f64_result_once():
    rng = np.random.default_rng(6)
    xb = _bits(rng, (9, 2, 64))
    pos = np.arange(100, 109)
    want = torch.from_numpy(orc.rope_rotate_f64(orc.bf16_to_f64(xb), pos, 10000.0))
    # float64 -> bfloat16 in torch is a single RNE rounding
    want_bits = want.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.rope_rotate(xb, pos, 10000.0), want_bits)


# ---------------------------------------------------------------- paging
def test_paged_scatter_then_gather_is_identity_and_touches_nothing_else():
    rng = np.random.default_rng(7)
    B, Hkv, D, P = 3, 2, 8, 16
    cached = np.array([0, 5, 33], np.int32)
    new = np.array([17, 1, 40], np.int32)
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, B, 2, Hkv, D, P, cached, new)
    sentinel = k_pool.copy()
    orc.paged_write(k_pool, bt, cached, new, k)
    t = 0
    written = np.zeros(k_pool.shape[:1] + k_pool.shape[2:3], bool)      # [page, slot]
    for s in range(B):
        got = orc.paged_gather(k_pool, bt[s], int(cached[s] + new[s]))
        assert np.array_equal(got[cached[s]:], k[t:t + new[s]])
        assert np.array_equal(got[:cached[s]], orc.paged_gather(sentinel, bt[s], int(cached[s])))
        for i in range(new[s]):
            pos = cached[s] + i
            written[bt[s, pos // P], pos % P] = True
        t += new[s]
    untouched = ~written
    assert np.array_equal(np.transpose(k_pool, (0, 2, 1, 3))[untouched],
                          np.transpose(sentinel, (0, 2, 1, 3))[untouched])
    assert written.sum() == new.sum()


def test_paged_layout_formula():
    # element (page, head, slot, dim) of a flat pool: (((page*Hkv)+h)*P+slot)*D+d
    Hkv, P, D = 3, 16, 4
    pool = np.zeros((6, Hkv, P, D), np.uint16)
    bt = np.array([[4, 1, -1]], np.int32)
    rows = np.arange(1 * Hkv * D, dtype=np.uint16).reshape(1, Hkv, D) + 1
    orc.paged_write(pool, bt, np.array([21]), np.array([1]), rows)
    flat = pool.reshape(-1)
    for h in range(Hkv):
        for d in range(D):
            idx = (((1 * Hkv) + h) * P + (21 % P)) * D + d
            assert flat[idx] == rows[0, h, d]
    assert np.count_nonzero(flat) == Hkv * D


def test_attention_invariant_under_page_permutation():
    rng = np.random.default_rng(8)
    B, Hq, Hkv, D, P = 2, 4, 2, 16, 16
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, B, Hq, Hkv, D, P, [37, 20], [9, 30])
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o0, l0 = orc.append_prefill_attention(q, k_pool, v_pool, bt, cached, new, Hq)
    perm = rng.permutation(k_pool.shape[0])            # new id of old page p is perm[p]
    k2 = np.empty_like(k_pool)
    v2 = np.empty_like(v_pool)
    k2[perm] = k_pool
    v2[perm] = v_pool
    bt2 = np.where(bt >= 0, perm[np.maximum(bt, 0)], -1).astype(np.int32)
    o1, l1 = orc.append_prefill_attention(q, k2, v2, bt2, cached, new, Hq)
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)


# ---------------------------------------------------------------- attention: brute force + library
def _dense_brute_force(Q, K, V, C, scale, G):
    """Pure-Python dense causal attention on de-paged arrays; rows are new tokens.
    Q [N,Hq,D], K,V [L,Hkv,D] as nested float lists."""
    N, Hq, D = len(Q), len(Q[0]), len(Q[0][0])
    out = [[[0.0] * D for _ in range(Hq)] for _ in range(N)]
    lse = [[0.0] * Hq for _ in range(N)]
    for i in range(N):
        for h in range(Hq):
            kh = h // G
            scores = []
            for j in range(C + i + 1):
                acc = 0.0
                for d in range(D):
                    acc += Q[i][h][d] * K[j][kh][d]
                scores.append(acc * scale)
            tot = math.fsum(math.exp(sc) for sc in scores)
            for j, sc in enumerate(scores):
                w = math.exp(sc) / tot
                for d in range(D):
                    out[i][h][d] += w * V[j][kh][d]
            lse[i][h] = math.log(tot)
    return np.array(out), np.array(lse)


@pytest.mark.parametrize("B,Hq,Hkv,D,cached,new", [
    (1, 2, 2, 2, [0], [5]),
    (2, 4, 2, 8, [3, 18], [4, 2]),
    (3, 4, 1, 8, [17, 0, 31], [1, 20, 3]),
    (1, 3, 3, 64, [20], [13]),
])
def test_attention_matches_dense_brute_force(B, Hq, Hkv, D, cached, new):
    rng = np.random.default_rng(9)
    P = 16
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, B, Hq, Hkv, D, P, cached, new)
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o, lse = orc.append_prefill_attention(q, k_pool, v_pool, bt, cached, new, Hq)
    t = 0
    for s in range(B):
        L = int(cached[s] + new[s])
        # de-page by hand (not through the oracle's gather)
        Kd = np.stack([bf16_bits_to_f32(k_pool[bt[s, p // P], :, p % P, :]).astype(np.float64) for p in range(L)])
        Vd = np.stack([bf16_bits_to_f32(v_pool[bt[s, p // P], :, p % P, :]).astype(np.float64) for p in range(L)])
        Qd = bf16_bits_to_f32(q[t:t + new[s]]).astype(np.float64)
        ob, lb = _dense_brute_force(Qd.tolist(), Kd.tolist(), Vd.tolist(), int(cached[s]),
                                    1.0 / math.sqrt(D), Hq // Hkv)
        assert np.allclose(o[t:t + new[s]], ob, atol=1e-10, rtol=0)
        assert np.allclose(lse[t:t + new[s]], lb, atol=1e-10, rtol=0)
        t += new[s]


@pytest.mark.parametrize("C", [0, 11])
def test_attention_matches_torch_sdpa_fp64(C):
    # Library special case: C = 0 is plain causal self-attention (is_causal);
    # C > 0 uses an explicit boolean mask j <= C + i.  GQA via enable_gqa-free repeat.
    rng = np.random.default_rng(10)
    Hq, Hkv, D, P, N = 4, 2, 16, 16, 21
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, 1, Hq, Hkv, D, P, [C], [N])
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o, lse = orc.append_prefill_attention(q, k_pool, v_pool, bt, cached, new, Hq)
    L = C + N
    Kd = np.stack([bf16_bits_to_f32(k_pool[bt[0, p // P], :, p % P, :]) for p in range(L)]).astype(np.float64)
    Vd = np.stack([bf16_bits_to_f32(v_pool[bt[0, p // P], :, p % P, :]) for p in range(L)]).astype(np.float64)
    Qt = torch.from_numpy(bf16_bits_to_f32(q).astype(np.float64)).permute(1, 0, 2)[None]          # [1,Hq,N,D]
    Kt = torch.from_numpy(Kd).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]          # [1,Hq,L,D]
    Vt = torch.from_numpy(Vd).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]
    if C == 0:
        want = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, is_causal=True)
    else:
        mask = torch.arange(L)[None, :] <= (C + torch.arange(N))[:, None]
        want = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, attn_mask=mask)
    assert np.allclose(o, want[0].permute(1, 0, 2).numpy(), atol=1e-12)
    sc = (Qt @ Kt.transpose(-1, -2)) / math.sqrt(D)
    sc = sc.masked_fill(~(torch.arange(L)[None, :] <= (C + torch.arange(N))[:, None]), float("-inf"))
    want_lse = torch.logsumexp(sc, dim=-1)[0].permute(1, 0).numpy()
    assert np.allclose(lse, want_lse, atol=1e-12)


# ---------------------------------------------------------------- attention: closed forms
def _const_case(D=8, L=37, Hq=2, Hkv=1, P=16, C=30):
    rng = np.random.default_rng(11)
    return _random_paged_case(rng, 1, Hq, Hkv, D, P, [C], [L - C])


def test_single_key_returns_its_value():
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(np.random.default_rng(12), 1, 2, 2, 8, 16, [0], [1])
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o, lse = orc.append_prefill_attention(q, k_pool, v_pool, bt, cached, new, 2)
    assert np.array_equal(o[0], bf16_bits_to_f32(v[0]).astype(np.float64))
    want = (bf16_bits_to_f32(q[0]).astype(np.float64) * bf16_bits_to_f32(k[0]).astype(np.float64)).sum(-1) / math.sqrt(8)
    assert np.allclose(lse[0], want, atol=1e-14)


def test_constant_values_give_that_constant_and_weights_sum_to_one():
    k_pool, v_pool, bt, cached, new, q, k, v = _const_case()
    v_pool[:] = f32_to_bf16_bits(np.array([2.5], np.float32))[0]
    v[:] = v_pool.flat[0]
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o, _ = orc.append_prefill_attention(q, k_pool, v_pool, bt, cached, new, 2)
    assert np.allclose(o, 2.5, atol=1e-12, rtol=0)       # sum of weights == 1


def test_zero_query_gives_running_mean_and_lse_log_count():
    k_pool, v_pool, bt, cached, new, q, k, v = _const_case()
    q[:] = 0
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o, lse = orc.append_prefill_attention(q, k_pool, v_pool, bt, cached, new, 2)
    C, N, P = int(cached[0]), int(new[0]), 16
    Vd = np.stack([bf16_bits_to_f32(v_pool[bt[0, p // P], 0, p % P, :]) for p in range(C + N)]).astype(np.float64)
    for i in range(N):
        assert np.allclose(o[i, 0], Vd[:C + i + 1].mean(axis=0), atol=1e-12)
        assert np.allclose(o[i, 1], Vd[:C + i + 1].mean(axis=0), atol=1e-12)
        assert abs(lse[i, 0] - math.log(C + i + 1)) < 1e-12     # all scores equal (0): lse = 0 + log(count)


def test_dominant_key_selects_its_value_and_future_key_is_masked():
    # key at position 3 scores +40/sqrt(D)*... above everything: o ~ v_3 for rows that see it;
    # a dominant key placed at a FUTURE position must have no effect on earlier rows.
    D, P = 4, 16
    rng = np.random.default_rng(13)
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, 1, 1, 1, D, P, [4], [4])
    one = f32_to_bf16_bits(np.array([1.0], np.float32))[0]
    big = f32_to_bf16_bits(np.array([80.0], np.float32))[0]
    q[:] = 0
    q[:, 0, 0] = one                     # every query = e_0
    k_pool[:] = 0
    k[:] = 0
    k[2, 0, 0] = big                     # new token 2 (position 6) has key 80*e_0 -> score 40
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o, lse = orc.append_prefill_attention(q, k_pool, v_pool, bt, cached, new, 1)
    v6 = bf16_bits_to_f32(v[2, 0]).astype(np.float64)
    Vd = np.stack([bf16_bits_to_f32(v_pool[bt[0, p // P], 0, p % P, :]) for p in range(8)]).astype(np.float64)
    for i in (0, 1):                     # positions 4, 5 do not see position 6: plain running mean
        assert np.allclose(o[i, 0], Vd[:4 + i + 1].mean(axis=0), atol=1e-12)
    for i in (2, 3):                     # positions 6, 7 see it: weight of the rest ~ e^-40
        assert np.allclose(o[i, 0], v6, atol=1e-15 + 8 * math.exp(-40) * 4)
        assert abs(lse[i, 0] - 40.0) < 1e-12


def test_hand_derived_golden_example():
    # tests/golden/attention_d2_hand.txt: D=2, scale given, 3 keys, weights 1/7, 2/7, 4/7
    rows = [l.split("#")[0].split() for l in open(os.path.join(GOLDEN, "attention_d2_hand.txt"))]
    rows = [r for r in rows if r]
    vals = {r[0]: [float(x) for x in r[1:]] for r in rows}
    P = 16
    k_pool = np.zeros((2, 1, P, 2), np.uint16)
    v_pool = np.zeros((2, 1, P, 2), np.uint16)
    bt = np.array([[1, 0]], np.int32)
    kk = np.array(vals["k"], np.float32).reshape(3, 1, 2)
    vv = np.array(vals["v"], np.float32).reshape(3, 1, 2)
    qq = np.array(vals["q"], np.float32).reshape(1, 1, 2)
    # keys 0,1 cached, key 2 and the query are the appended token
    orc.paged_write(k_pool, bt, np.array([0]), np.array([3]), f32_to_bf16_bits(kk))
    orc.paged_write(v_pool, bt, np.array([0]), np.array([3]), f32_to_bf16_bits(vv))
    o, lse = orc.append_prefill_attention(f32_to_bf16_bits(qq), k_pool, v_pool, bt, np.array([2]), np.array([1]),
                                          1, sm_scale=vals["scale"][0])
    assert np.allclose(o[0, 0], vals["o"], atol=1e-6)          # file gives 7 significant digits
    assert abs(lse[0, 0] - vals["lse"][0]) < 1e-6


# ---------------------------------------------------------------- kv_append's position rule
def test_kv_append_from_an_empty_cache_starts_at_position_zero():
    """Sec. 1: `inc` follows `<P>prefix<S>suffix<M>`, so a token's position is its
    index in the reordered prompt and the first token of an empty cache has
    position 0 - where the rotation is the identity.  Token 0 must come back
    bit for bit and land in page block_table[s][0], slot 0; token 1 must not
    (it is turned by one radian on the fastest pair)."""
    rng = np.random.default_rng(30)
    B, Hq, Hkv, D, P = 2, 2, 2, 8, 16
    new = np.array([3, 18], np.int32)
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, B, Hq, Hkv, D, P, [0, 0], new)
    k_before = k_pool.copy()
    q_rot = orc.kv_append(k_pool, v_pool, bt, cached, new, q, k, v, 10000.0)
    t = 0
    for s in range(B):
        assert np.array_equal(q_rot[t], q[t])
        assert np.array_equal(k_pool[bt[s, 0], :, 0, :], k[t])
        assert np.array_equal(v_pool[bt[s, 0], :, 0, :], v[t])
        assert not np.array_equal(q_rot[t + 1], q[t + 1])
        assert not np.array_equal(k_pool[bt[s, 0], :, 1, :], k[t + 1])
        t += int(new[s])
    # the 18-token sequence spills into its second page at slots 0 and 1 only
    assert np.array_equal(k_pool[bt[1, 1], :, 2:, :], k_before[bt[1, 1], :, 2:, :])
    assert not np.array_equal(k_pool[bt[1, 1], :, :2, :], k_before[bt[1, 1], :, :2, :])


def test_kv_append_turns_token_i_by_cached_len_plus_i_radians():
    """D = 2 has the single frequency theta_0 = 1, so new token i of a sequence
    with C cached tokens is the input times e^{i(C+i)} as a complex number
    (computed here with cmath, not with the oracle's formula), rounded once to
    bf16.  An offset of one position turns by one more radian: far outside the
    rounding."""
    import cmath
    rng = np.random.default_rng(31)
    B, Hq, Hkv, D, P = 2, 3, 1, 2, 16
    C = np.array([37, 5], np.int32)
    N = np.array([4, 13], np.int32)
    k_pool, v_pool, bt, C, N, q, k, v = _random_paged_case(rng, B, Hq, Hkv, D, P, C, N)
    q_rot = orc.kv_append(k_pool, v_pool, bt, C, N, q, k, v, 777.0)
    qf, kf = bf16_bits_to_f32(q).astype(np.float64), bf16_bits_to_f32(k).astype(np.float64)
    t = 0
    for s in range(B):
        for i in range(int(N[s])):
            pos = int(C[s]) + i
            turn = cmath.exp(1j * pos)
            for h in range(Hq):
                z = complex(qf[t, h, 0], qf[t, h, 1]) * turn
                got = bf16_bits_to_f32(q_rot[t, h]).astype(np.float64)
                assert abs(got[0] - z.real) <= 2.0 ** -8 * abs(z.real) + 1e-30
                assert abs(got[1] - z.imag) <= 2.0 ** -8 * abs(z.imag) + 1e-30
            z = complex(kf[t, 0, 0], kf[t, 0, 1]) * turn
            got = bf16_bits_to_f32(k_pool[bt[s, pos // P], 0, pos % P]).astype(np.float64)
            assert abs(got[0] - z.real) <= 2.0 ** -8 * abs(z.real) + 1e-30
            assert abs(got[1] - z.imag) <= 2.0 ** -8 * abs(z.imag) + 1e-30
            assert np.array_equal(v_pool[bt[s, pos // P], 0, pos % P], v[t, 0])
            t += 1


# ---------------------------------------------------------------- the paper's invariants
def _full_turn(rng, B, Hq, Hkv, D, cached, new, base=10000.0, interleaved=False):
    P = 16
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, B, Hq, Hkv, D, P, cached, new)
    return k_pool, v_pool, bt, cached, new, q, k, v


def test_central_invariant_append_equals_rows_of_full_recompute():
    """EFIM Sec. 1: with prefix and suffix KV reused, attending only the `inc`
    tokens must give the rows [C, L) of a full causal prefill of the whole
    reordered prompt, and the cache after the append equals the cache of the
    full prefill."""
    rng = np.random.default_rng(14)
    B, Hq, Hkv, D, P = 2, 4, 2, 16, 16
    C = np.array([45, 16], np.int32)
    N = np.array([7, 19], np.int32)
    L = C + N
    need = -(-L // P)
    num_pages = int(need.sum()) + 3
    perm = rng.permutation(num_pages)
    bt = np.full((B, int(need.max())), -1, np.int32)
    off = 0
    for s in range(B):
        bt[s, :need[s]] = perm[off:off + need[s]]
        off += need[s]
    Tall = int(L.sum())
    q_all, k_all, v_all = _bits(rng, (Tall, Hq, D)), _bits(rng, (Tall, Hkv, D)), _bits(rng, (Tall, Hkv, D))
    zero = np.zeros(B, np.int32)
    # (a) full prefill of the whole prompt from an empty cache
    kA = np.zeros((num_pages, Hkv, P, D), np.uint16)
    vA = np.zeros_like(kA)
    qA = orc.kv_append(kA, vA, bt, zero, L, q_all, k_all, v_all, 10000.0)
    oA, lA = orc.append_prefill_attention(qA, kA, vA, bt, zero, L, Hq)
    # (b) turn 1 caches the first C tokens, turn 2 appends the last N
    kB = np.zeros_like(kA)
    vB = np.zeros_like(kA)
    starts = np.concatenate([[0], np.cumsum(L)])[:-1]
    idx_old = np.concatenate([np.arange(starts[s], starts[s] + C[s]) for s in range(B)])
    idx_new = np.concatenate([np.arange(starts[s] + C[s], starts[s] + L[s]) for s in range(B)])
    orc.kv_append(kB, vB, bt, zero, C, q_all[idx_old], k_all[idx_old], v_all[idx_old], 10000.0)
    qB = orc.kv_append(kB, vB, bt, C, N, q_all[idx_new], k_all[idx_new], v_all[idx_new], 10000.0)
    oB, lB = orc.append_prefill_attention(qB, kB, vB, bt, C, N, Hq)
    assert np.array_equal(kA, kB) and np.array_equal(vA, vB)
    assert np.allclose(oB, oA[idx_new], atol=1e-12, rtol=0)
    assert np.allclose(lB, lA[idx_new], atol=1e-12, rtol=0)
    # reuse levels none / prefix / prefix+suffix (Sec. 4.2) agree on shared rows
    a = 3
    C2, N2 = C + a, N - a
    keep = np.concatenate([np.arange(sum(N[:s]) + a, sum(N[:s + 1])) for s in range(B)])
    oC, lC = orc.append_prefill_attention(qB[keep], kB, vB, bt, C2, N2, Hq)
    assert np.allclose(oC, oB[keep], atol=1e-12, rtol=0)


def test_fim_order_would_invalidate_suffix_cache():
    """Sec. 1 / Fig. 3: in `<P>prefix+inc<S>suffix<M>` the suffix tokens move
    by len(inc) positions, so their rotated keys differ from the cached ones -
    the reuse EFIM gets is not available to the unreordered prompt."""
    rng = np.random.default_rng(15)
    suffix_k = _bits(rng, (12, 2, 32))
    prefix_len, inc = 40, 5
    cached = orc.rope_rotate(suffix_k, prefix_len + np.arange(12), 10000.0)
    shifted = orc.rope_rotate(suffix_k, prefix_len + inc + np.arange(12), 10000.0)
    assert np.mean(cached != shifted) > 0.5      # only the slowest frequencies survive bf16 rounding
    # while in EFIM order the suffix positions are unchanged by construction
    again = orc.rope_rotate(suffix_k, prefix_len + np.arange(12), 10000.0)
    assert np.array_equal(cached, again)


def test_split_kv_merge_is_exact_for_any_partition():
    rng = np.random.default_rng(16)
    D, L = 8, 50
    q = rng.standard_normal(D)
    K = rng.standard_normal((L, D))
    V = rng.standard_normal((L, D))
    sc = K @ q / math.sqrt(D)
    w = np.exp(sc - sc.max())
    o_full = (w[:, None] * V).sum(0) / w.sum()
    lse_full = sc.max() + math.log(w.sum())
    for cuts in ([0, 50], [0, 1, 50], [0, 16, 32, 48, 50], [0, 7, 7, 29, 50]):   # includes an empty chunk
        o_parts, l_parts = [], []
        for a, b in zip(cuts[:-1], cuts[1:]):
            if a == b:
                o_parts.append(np.zeros(D))
                l_parts.append(-np.inf)
                continue
            m = sc[a:b].max()
            ww = np.exp(sc[a:b] - m)
            o_parts.append((ww[:, None] * V[a:b]).sum(0) / ww.sum())
            l_parts.append(m + math.log(ww.sum()))
        o, lse = orc.merge_partials(np.array(o_parts), np.array(l_parts))
        assert np.allclose(o, o_full, atol=1e-12) and abs(lse - lse_full) < 1e-12


def test_decode_is_append_with_one_token():
    rng = np.random.default_rng(17)
    B, Hq, Hkv, D, P = 3, 4, 2, 8, 16
    ctx = np.array([1, 16, 45], np.int32)
    k_pool, v_pool, bt, cached, new, q, k, v = _random_paged_case(rng, B, Hq, Hkv, D, P, ctx - 1, [1, 1, 1])
    orc.paged_write(k_pool, bt, cached, new, k)
    orc.paged_write(v_pool, bt, cached, new, v)
    o, lse = orc.decode_attention(q, k_pool, v_pool, bt, ctx, Hq)
    for s in range(B):
        Kd = np.stack([bf16_bits_to_f32(k_pool[bt[s, p // P], :, p % P, :]) for p in range(ctx[s])]).astype(np.float64)
        Vd = np.stack([bf16_bits_to_f32(v_pool[bt[s, p // P], :, p % P, :]) for p in range(ctx[s])]).astype(np.float64)
        for h in range(Hq):
            sc = Kd[:, h // 2] @ bf16_bits_to_f32(q[s, h]).astype(np.float64) / math.sqrt(D)
            import scipy.special as sp
            w = sp.softmax(sc)
            assert np.allclose(o[s, h], w @ Vd[:, h // 2], atol=1e-12)
            assert abs(lse[s, h] - sp.logsumexp(sc)) < 1e-12


# ---------------------------------------------------------------- planted mistakes are caught
@pytest.mark.parametrize("mistake", ["sin_sign", "mask_off_by_one", "gqa_map", "no_scale", "position_off_by_one"])
def test_pins_catch_planted_mistakes(mistake, monkeypatch):
    """Plant a plausible bug in the oracle (CPU only) and check a pin fails."""
    if mistake == "sin_sign":
        real = np.sin
        monkeypatch.setattr(orc.np, "sin", lambda a: -real(a))
        with pytest.raises(AssertionError):
            test_rope_d2_is_plane_rotation_by_p_radians()
        monkeypatch.undo()
    elif mistake == "position_off_by_one":
        src = orc.rope_rotate
        def broken(x_bits, positions, base, interleaved=False):               # pos = C + i + 1
            return src(x_bits, np.asarray(positions) + 1, base, interleaved)
        monkeypatch.setattr(orc, "rope_rotate", broken)
        with pytest.raises(AssertionError):
            test_kv_append_from_an_empty_cache_starts_at_position_zero()
        with pytest.raises(AssertionError):
            test_kv_append_turns_token_i_by_cached_len_plus_i_radians()
    elif mistake == "mask_off_by_one":
        src = orc.append_prefill_attention
        def broken(q, kp, vp, bt, c, n, hq, sm_scale=None):
            return src(q, kp, vp, bt, np.asarray(c) - 1, n, hq, sm_scale)   # key C+i hidden
        monkeypatch.setattr(orc, "append_prefill_attention", broken)
        with pytest.raises((AssertionError, ValueError)):
            test_attention_matches_dense_brute_force(2, 4, 2, 8, [3, 18], [4, 2])
    elif mistake == "gqa_map":
        src = orc.append_prefill_attention
        def broken(q, kp, vp, bt, c, n, hq, sm_scale=None):
            return src(q[:, ::-1], kp, vp, bt, c, n, hq, sm_scale)            # heads mapped to wrong groups
        monkeypatch.setattr(orc, "append_prefill_attention", broken)
        with pytest.raises(AssertionError):
            test_attention_matches_dense_brute_force(2, 4, 2, 8, [3, 18], [4, 2])
    else:
        src = orc.append_prefill_attention
        def broken(q, kp, vp, bt, c, n, hq, sm_scale=None):
            return src(q, kp, vp, bt, c, n, hq, 1.0)
        monkeypatch.setattr(orc, "append_prefill_attention", broken)
        with pytest.raises(AssertionError):
            test_attention_matches_torch_sdpa_fp64(11)
