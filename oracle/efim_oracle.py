"""CPU oracle for the EFIM append-prefill / paged-decode path (TEST INFRASTRUCTURE).

This file is test infrastructure, not product code: only the tests, the smoke
check and the benchmark's CPU-baseline leg may call it.  It shares no code with
the CUDA library and imports nothing from it.

What it restates (EFIM paper, Sec. 1 and Sec. 2.2 / Fig. 3): the prompt is
reordered from `<P>prefix+inc<S>suffix<M>` to `<P>prefix<S>suffix<M>inc`, so
the keys/values of the first C = len(<P>prefix<S>suffix<M>) tokens are
unchanged between turns and stay in the KV cache; only the N tokens of `inc`
are new.  Per turn the model therefore (i) rotates the new tokens' q and k by
their positions C..C+N-1 and stores k, v in the cache, (ii) attends each new
token i over keys 0..C+i (causal, the paper makes "no architectural changes",
Sec. 3, so this is standard softmax attention), and (iii) decodes the middle
one token at a time over all keys so far.  The method reaches exactly the
result of the plain definition, so the oracle is that definition written out
in float64 from the bf16 input bits.

Readings where the paper is silent: softmax(q.k/sqrt(D)) with natural exp;
rotary pairing (f, f+D/2) ("rotate-half") or (2f, 2f+1) ("interleaved");
theta_f = base^(-2f/D); grouped-query map kv_head = q_head // (Hq/Hkv);
cache layout [page][kv_head][slot][dim] with token p of a sequence at page
block_table[p // P], slot p % P; rotated q and k are rounded to bf16
(nearest-even) before use, matching what the cache stores.

Pinned by tests/test_oracle_pins.py (closed forms, library special cases,
brute force on tiny inputs, the reuse invariant).  Numeric parity with the
paper itself: parity unpinned (the paper prints no values for this path).
"""
import numpy as np


# --------------------------------------------------------------------------
# bf16 <-> float64
# --------------------------------------------------------------------------
def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 to bfloat16, nearest with ties to even, in ONE rounding.

    bfloat16 has 8 significand bits (7 stored) and float32's exponent range.
    For |x| in [2^e, 2^(e+1)) the spacing is 2^(e-7) (2^-133 below 2^-126), so
    x is scaled to an integer grid, rounded with rint (ties to even) and scaled
    back; the result is exactly representable and the float32 cast is exact.
    """
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)                       # x = m * 2^e, 0.5 <= |m| < 1
    e = np.maximum(e - 1, -126)              # exponent of the leading bit, clamped at the subnormal edge
    ulp = np.ldexp(1.0, e - 7)
    r = np.rint(x / ulp) * ulp
    r = np.where(np.abs(r) >= 3.3895313892515355e38, np.copysign(np.inf, r), r)  # beyond max bf16 -> inf
    bits32 = r.astype(np.float32).view(np.uint32)
    return (bits32 >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# Rotary position embedding
# --------------------------------------------------------------------------
def rope_rotate_f64(x: np.ndarray, positions: np.ndarray, base: float,
                    interleaved: bool = False) -> np.ndarray:
    """Rotate head vectors by their token position, float64 in and out.

    x: float64 [T, H, D]; positions: int [T].  For frequency index
    f in [0, D/2): theta_f = base^(-2f/D), angle = pos * theta_f, and the pair
    (x_a, x_b) -> (x_a cos - x_b sin, x_b cos + x_a sin) with
    (a, b) = (f, f + D/2), or (2f, 2f+1) when `interleaved`.
    Position of a token = its index in the reordered prompt
    `<P>prefix<S>suffix<M>inc` (Sec. 1): inc[i] sits at C + i.
    """
    x = np.asarray(x, dtype=np.float64)
    T, H, D = x.shape
    half = D // 2
    f = np.arange(half, dtype=np.float64)
    theta = np.power(float(base), -2.0 * f / D)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * theta[None, :]     # [T, D/2]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    out = np.empty_like(x)
    if interleaved:
        xa, xb = x[..., 0::2], x[..., 1::2]
        out[..., 0::2] = xa * c - xb * s
        out[..., 1::2] = xb * c + xa * s
    else:
        xa, xb = x[..., :half], x[..., half:]
        out[..., :half] = xa * c - xb * s
        out[..., half:] = xb * c + xa * s
    return out


def rope_rotate(x_bits: np.ndarray, positions: np.ndarray, base: float,
                interleaved: bool = False) -> np.ndarray:
    """rope_rotate_f64 on bf16 bit patterns (uint16 [T, H, D]); the result is
    rounded once to bf16, which is what the cache stores and attention reads."""
    return f64_to_bf16(rope_rotate_f64(bf16_to_f64(x_bits), positions, base, interleaved))


# --------------------------------------------------------------------------
# Paged KV cache
# --------------------------------------------------------------------------
def paged_write(pool: np.ndarray, block_table: np.ndarray, start_pos: np.ndarray,
                count: np.ndarray, rows: np.ndarray) -> None:
    """Scatter token rows into a pool in place.

    pool: uint16 [num_pages, Hkv, P, D]; rows: uint16 [T, Hkv, D] packed
    sequence after sequence; sequence s contributes count[s] tokens that land
    at positions start_pos[s] .. start_pos[s]+count[s]-1, i.e. page
    block_table[s][pos // P], slot pos % P.  Nothing else is touched.
    """
    P = pool.shape[2]
    t = 0
    for s in range(len(count)):
        for i in range(int(count[s])):
            pos = int(start_pos[s]) + i
            page = int(block_table[s, pos // P])
            pool[page, :, pos % P, :] = rows[t]
            t += 1


def paged_gather(pool: np.ndarray, block_table_row: np.ndarray, length: int) -> np.ndarray:
    """Tokens [0, length) of one sequence, de-paged: uint16 [length, Hkv, D]."""
    P = pool.shape[2]
    n_pages = -(-length // P)
    pages = pool[np.asarray(block_table_row[:n_pages], dtype=np.int64)]      # [n, Hkv, P, D]
    tok = np.transpose(pages, (0, 2, 1, 3)).reshape(n_pages * P, pool.shape[1], pool.shape[3])
    return tok[:length]


def kv_append(k_pool, v_pool, block_table, cached_len, new_len, q_bits, k_bits, v_bits,
              rope_base, interleaved=False, use_rope=True):
    """One turn's cache update: rotate the new q and k, store k and v.

    Returns the rotated q (uint16 [T, Hq, D]); the pools are updated in place.
    Token i of sequence s has position cached_len[s] + i (the `inc` tokens
    follow `<P>prefix<S>suffix<M>`, Sec. 1).  v is stored unrotated.
    """
    pos = np.concatenate([np.arange(int(c), int(c) + int(n)) for c, n in zip(cached_len, new_len)]
                         + [np.zeros(0, dtype=np.int64)]).astype(np.int64)
    if use_rope:
        q_rot = rope_rotate(q_bits, pos, rope_base, interleaved) if q_bits is not None else None
        k_rot = rope_rotate(k_bits, pos, rope_base, interleaved)
    else:
        q_rot = None if q_bits is None else np.array(q_bits, dtype=np.uint16, copy=True)
        k_rot = np.asarray(k_bits, dtype=np.uint16)
    paged_write(k_pool, block_table, cached_len, new_len, k_rot)
    paged_write(v_pool, block_table, cached_len, new_len, np.asarray(v_bits, dtype=np.uint16))
    return q_rot


# --------------------------------------------------------------------------
# Attention
# --------------------------------------------------------------------------
def append_prefill_attention(q_rot_bits, k_pool, v_pool, block_table, cached_len, new_len,
                             num_q_heads, sm_scale=None):
    """Causal attention of the new tokens over cached + new keys.

    q_rot_bits: uint16 [T, Hq, D] (already rotated, packed by sequence); the
    pools must already hold the new tokens' k/v.  New token i of sequence s
    (position C+i) sees keys j <= C+i.  Returns (o float64 [T, Hq, D],
    lse float64 [T, Hq]) with lse = log sum_j exp(scale * q.k_j).
    """
    Hkv, D = k_pool.shape[1], k_pool.shape[3]
    G = num_q_heads // Hkv
    scale = 1.0 / np.sqrt(D) if sm_scale is None or sm_scale <= 0 else float(sm_scale)
    T = int(np.sum(new_len))
    o = np.zeros((T, num_q_heads, D), dtype=np.float64)
    lse = np.zeros((T, num_q_heads), dtype=np.float64)
    t0 = 0
    for s in range(len(new_len)):
        C, N = int(cached_len[s]), int(new_len[s])
        if N == 0:
            continue
        L = C + N
        K = bf16_to_f64(paged_gather(k_pool, block_table[s], L))        # [L, Hkv, D]
        V = bf16_to_f64(paged_gather(v_pool, block_table[s], L))
        Q = bf16_to_f64(q_rot_bits[t0:t0 + N])                          # [N, Hq, D]
        key_idx = np.arange(L)[None, :]
        visible = key_idx <= (C + np.arange(N))[:, None]                # [N, L]
        for h in range(num_q_heads):
            kh = h // G
            sc = scale * (Q[:, h, :] @ K[:, kh, :].T)                   # [N, L]
            sc = np.where(visible, sc, -np.inf)
            m = sc.max(axis=1, keepdims=True)
            w = np.exp(sc - m)
            z = w.sum(axis=1, keepdims=True)
            o[t0:t0 + N, h, :] = (w @ V[:, kh, :]) / z
            lse[t0:t0 + N, h] = (m + np.log(z))[:, 0]
        t0 += N
    return o, lse


def decode_attention(q_rot_bits, k_pool, v_pool, block_table, ctx_len, num_q_heads, sm_scale=None):
    """One decode step: one query token per sequence over keys [0, ctx_len[s]).

    q_rot_bits: uint16 [B, Hq, D].  ctx_len counts the token just appended.
    Same definition as append_prefill_attention with one new token; sequences
    with ctx_len 0 give o = 0, lse = -inf.
    """
    ctx_len = np.asarray(ctx_len)
    B = len(ctx_len)
    D = k_pool.shape[3]
    o = np.zeros((B, num_q_heads, D), dtype=np.float64)
    lse = np.full((B, num_q_heads), -np.inf, dtype=np.float64)
    for s in range(B):
        if int(ctx_len[s]) <= 0:
            continue
        os_, ls_ = append_prefill_attention(
            q_rot_bits[s:s + 1], k_pool, v_pool, block_table[s:s + 1],
            np.array([int(ctx_len[s]) - 1]), np.array([1]), num_q_heads, sm_scale)
        o[s], lse[s] = os_[0], ls_[0]
    return o, lse


def merge_partials(o_parts, lse_parts):
    """Combine attention results computed over disjoint key subsets.

    o_parts: float64 [S, ..., D]; lse_parts: float64 [S, ...].  With
    lse = log sum_c exp(lse_c), the whole-range output is
    sum_c exp(lse_c - lse) o_c; a subset with no keys has lse_c = -inf.
    """
    o_parts = np.asarray(o_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    m = lse_parts.max(axis=0)
    w = np.exp(lse_parts - m)
    z = w.sum(axis=0)
    o = (w[..., None] * np.where(np.isfinite(lse_parts)[..., None], o_parts, 0.0)).sum(axis=0) / z[..., None]
    return o, m + np.log(z)
