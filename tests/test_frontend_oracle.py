"""Pins for the front-end oracle (prompt transformation of Sec. 3.1, cross-request KV
reuse of Sec. 1): hand-written layouts, format invariants, a brute-force
longest-common-prefix search, and the paper's claim that the EFIM order keeps the
suffix reusable where PSM does not."""
import os

import numpy as np
import pytest

from oracle import efim_frontend_oracle as fo

P_, S_, M_ = 901, 902, 903
FMT = {"PSM_NEW": fo.PSM_NEW, "EFIM": fo.EFIM, "PSM_SUFFIX": fo.PSM_SUFFIX, "PSM_SAME": fo.PSM_SAME,
       "PSM_RESET": fo.PSM_RESET, "PSM_REBASE": fo.PSM_REBASE}


def golden_turns():
    path = os.path.join(os.path.dirname(__file__), "golden", "efim_prompt_formats.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        pre, suf, fmt, prompt = [x.strip() for x in line.split("|")]
        yield [int(t) for t in pre.split()], [int(t) for t in suf.split()], FMT[fmt], [int(t) for t in prompt.split()]


def test_hand_written_prompt_layouts():
    pool = fo.SessionPool(P_, S_, M_)
    for prefix, suffix, fmt, prompt in golden_turns():
        got, got_fmt, inc_len = pool.transform(7, prefix, suffix)
        assert got == prompt and got_fmt == fmt
        assert inc_len == (len(prompt) - prompt.index(M_) - 1)


def _split(prompt):
    s, m = prompt.index(S_), prompt.index(M_)
    return prompt[1:s], prompt[s + 1:m], prompt[m + 1:]


def test_every_prompt_carries_exactly_the_request():
    """Whatever the format, the prompt holds the request's prefix (as common + inc) and suffix
    once each, between the three special tokens in P, S, M order."""
    rng = np.random.default_rng(0)
    pool = fo.SessionPool(P_, S_, M_)
    state = {}
    for _ in range(400):
        u = int(rng.integers(0, 5))
        prefix, suffix = state.get(u, ([], []))
        r = rng.random()
        if r < 0.6:
            prefix = prefix + rng.integers(0, 50, rng.integers(1, 9)).tolist()
        elif r < 0.8:
            suffix = rng.integers(0, 50, rng.integers(0, 9)).tolist()
        elif r < 0.9 and prefix:
            prefix = prefix[:rng.integers(0, len(prefix))] + [77]
        state[u] = (prefix, suffix)
        prompt, fmt, inc_len = pool.transform(u, prefix, suffix)
        assert prompt[0] == P_ and prompt.count(P_) == prompt.count(S_) == prompt.count(M_) == 1
        common, suf, inc = _split(prompt)
        assert common + inc == prefix and suf == suffix and len(inc) == inc_len
        assert (fmt == fo.EFIM) == (inc_len > 0)


def test_rebase_bounds_inc():
    pool = fo.SessionPool(P_, S_, M_, rebase_inc_tokens=4)
    pre = [1, 2, 3]
    assert pool.transform(0, pre, [9])[1] == fo.PSM_NEW
    assert pool.transform(0, pre + [4, 5], [9])[1:] == (fo.EFIM, 2)
    assert pool.transform(0, pre + [4, 5, 6, 7], [9])[1:] == (fo.EFIM, 4)
    prompt, fmt, n = pool.transform(0, pre + [4, 5, 6, 7, 8], [9])
    assert fmt == fo.PSM_REBASE and n == 0 and prompt == fo.psm_prompt(P_, S_, M_, pre + [4, 5, 6, 7, 8], [9])
    assert pool.transform(0, pre + [4, 5, 6, 7, 8, 10], [9])[1:] == (fo.EFIM, 1)


def _brute_force_cached_len(prompt, finished, P):
    """Longest run of full pages of `prompt` that is also the start of a finished sequence
    (only that sequence's full pages count), leaving at least one token to compute."""
    best = 0
    for seq in finished:
        lcp = 0
        while lcp < min(len(prompt), len(seq)) and prompt[lcp] == seq[lcp]:
            lcp += 1
        lcp = min(lcp, len(seq) // P * P)
        best = max(best, lcp // P * P)
    if best >= len(prompt):
        best -= P
    return best


@pytest.mark.parametrize("P", [4, 16])
def test_reuse_is_the_longest_common_page_prefix_when_nothing_is_evicted(P):
    rng = np.random.default_rng(1)
    cache = fo.PrefixCache(num_pages=100000, page_size=P)
    finished = []
    stems = [rng.integers(0, 9, 200).tolist() for _ in range(3)]
    for _ in range(120):
        stem = stems[int(rng.integers(0, 3))]
        prompt = stem[:int(rng.integers(1, 200))] + rng.integers(0, 9, int(rng.integers(0, 40))).tolist()
        h, cached, pages = cache.admit(prompt, reserve_tokens=8)
        assert cached == _brute_force_cached_len(prompt, finished, P)
        assert len(pages) == -(-(len(prompt) + 8) // P) and len(set(pages)) == len(pages)
        seq = prompt + rng.integers(0, 9, int(rng.integers(0, 9))).tolist()
        cache.finish(h, seq)
        finished.append(seq)


def test_lru_eviction_spares_pinned_pages_and_takes_the_oldest():
    cache = fo.PrefixCache(num_pages=6, page_size=2)
    a, b = [1, 2, 3, 4, 5], [6, 7, 8, 9, 5]
    h, c, pa = cache.admit(a)
    assert (c, pa) == (0, [0, 1, 2])
    cache.finish(h, a)                                  # pages 0,1 cached (blocks [1,2],[3,4]); page 2 freed
    h, c, pb = cache.admit(b)
    assert (c, pb) == (0, [2, 3, 4])                    # lowest free ids first
    cache.finish(h, b)                                  # pages 2,3 cached; 4 freed; free = {4, 5}
    h1, c1, p1 = cache.admit(a)                         # pins pages 0,1 (a's blocks), takes page 4 for the tail
    assert (c1, p1) == (4, [0, 1, 4])
    h2, c2, p2 = cache.admit([9, 9, 9, 9, 9, 9])        # needs 3 pages: free 5, then evicts b's pages, deepest first
    assert c2 == 0 and p2 == [5, 3, 2] and cache.evictions == 2
    with pytest.raises(fo.OutOfPages):                  # everything left is pinned
        cache.admit([8, 8, 8])
    cache.finish(h1, a)
    cache.finish(h2, [9] * 6)
    assert cache.admit(b)[1] == 0                       # b's pages are gone


def _session(order, rounds=5, prefix0=600, suffix0=300, inc=40, gen=16, P=16, seed=3):
    """One user, growing prefix, fixed suffix; returns the reuse rate over rounds 2.. ."""
    rng = np.random.default_rng(seed)
    pool = fo.SessionPool(P_, S_, M_)
    cache = fo.PrefixCache(100000, P)
    prefix = rng.integers(0, 800, prefix0).tolist()
    suffix = rng.integers(0, 800, suffix0).tolist()
    cached_total = prompt_total = 0
    for r in range(rounds):
        if order == "efim":
            prompt, _, _ = pool.transform(0, prefix, suffix)
        else:
            prompt = fo.psm_prompt(P_, S_, M_, prefix, suffix)
        h, cached, _ = cache.admit(prompt, gen)
        cache.finish(h, prompt + rng.integers(0, 800, gen).tolist())
        if r > 0:
            cached_total += cached
            prompt_total += len(prompt)
            if order == "efim":     # prefix and suffix KV are both reused (Sec. 1): all but inc and a page edge
                assert cached >= (1 + prefix0 + 1 + suffix0 + 1) // P * P
            else:                   # the suffix follows the changed prefix: only the old prefix can be reused
                assert cached <= 1 + len(prefix) - inc
        prefix = prefix + rng.integers(0, 800, inc).tolist()
    return cached_total / prompt_total


def test_efim_order_keeps_the_suffix_reusable_and_psm_does_not():
    assert _session("efim") > 0.85 > 0.70 > _session("psm")
