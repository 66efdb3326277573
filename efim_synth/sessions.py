"""Seeded multi-turn infilling sessions and per-token q/k/v tables (inputs only).

Shape of the paper's serving experiment (Sec. 4.2): `users` users, `rounds` rounds each;
a user's first request has a prefix and a suffix; every later request's prefix is the
previous prefix + the tokens generated for it + some newly typed tokens, the suffix
stays.  Defaults give an average input of about 2,355 tokens and 128 output tokens.

A "layer" without a model: token id t has fixed bf16 rows q_tab[t], k_tab[t], v_tab[t]
(N(0,1) draws), so equal tokens at equal positions have equal keys and values - which is
what makes a cached page reusable.  No attention or RoPE arithmetic lives here.
"""
import numpy as np

from .bf16 import f32_to_bf16_bits

TOK_P, TOK_S, TOK_M = 0, 1, 2          # special tokens; text tokens are 3 .. vocab-1


def token_tables(seed, vocab, num_q_heads, num_kv_heads, head_dim):
    """bf16 bit patterns: q_tab [vocab,Hq,D], k_tab [vocab,Hkv,D], v_tab [vocab,Hkv,D]."""
    def draw(tag, h):
        rng = np.random.default_rng([seed, tag])
        return f32_to_bf16_bits(rng.standard_normal((vocab, h, head_dim), dtype=np.float32))
    return draw(21, num_q_heads), draw(22, num_kv_heads), draw(23, num_kv_heads)


def infill_sessions(seed, users=16, rounds=5, vocab=4096, prefix0=(700, 1700), suffix0=(400, 1200),
                    typed=(8, 96), gen=128):
    """-> list over users of list over rounds of dict(prefix, suffix, gen) (lists of token ids)."""
    rng = np.random.default_rng([seed, 31])
    out = []
    for _ in range(users):
        prefix = rng.integers(3, vocab, int(rng.integers(prefix0[0], prefix0[1] + 1))).tolist()
        suffix = rng.integers(3, vocab, int(rng.integers(suffix0[0], suffix0[1] + 1))).tolist()
        turns = []
        for _ in range(rounds):
            g = rng.integers(3, vocab, gen).tolist()
            turns.append(dict(prefix=list(prefix), suffix=list(suffix), gen=g))
            prefix = prefix + g + rng.integers(3, vocab, int(rng.integers(typed[0], typed[1] + 1))).tolist()
        out.append(turns)
    return out
