"""The library's host-side front end against its oracle, call by call, on seeded multi-user
sessions: prompts, formats, cached lengths, block tables, statistics and error returns
must be identical (integer work: bit-exact).  CPU only - the front end makes no CUDA call."""
import numpy as np
import pytest

import paper_2505_21889_b200 as efim
from oracle import efim_frontend_oracle as fo

P_, S_, M_ = 50001, 50002, 50003


def _drive(seed, users, turns, num_pages, page_size, rebase, max_pages=64):
    rng = np.random.default_rng(seed)
    fe = efim.Frontend(P_, S_, M_, num_pages, page_size, rebase)
    pool = fo.SessionPool(P_, S_, M_, rebase)
    cache = fo.PrefixCache(num_pages, page_size)
    state, open_reqs, formats = {}, [], set()
    for t in range(turns):
        u = int(rng.integers(0, users))
        prefix, suffix = state.get(u, (rng.integers(0, 30, int(rng.integers(20, 200))).tolist(),
                                       rng.integers(0, 30, int(rng.integers(0, 100))).tolist()))
        r = rng.random()
        if u in state:
            if r < 0.6:
                prefix = prefix + rng.integers(0, 30, int(rng.integers(1, 40))).tolist()
            elif r < 0.75:
                suffix = suffix + rng.integers(0, 30, int(rng.integers(1, 20))).tolist()
            elif r < 0.85:
                prefix = prefix[:int(rng.integers(1, len(prefix)))] + [31]
        state[u] = (prefix, suffix)
        want_prompt, want_fmt, want_inc = pool.transform(u, prefix, suffix)
        prompt, fmt, inc = fe.transform(u, prefix, suffix)
        assert prompt.tolist() == want_prompt and (fmt, inc) == (want_fmt, want_inc)
        formats.add(fmt)
        reserve = int(rng.integers(0, 24))
        row = np.zeros(max_pages, np.int32)
        try:
            wh, wcached, wpages = cache.admit(want_prompt, reserve)
        except fo.OutOfPages:
            with pytest.raises(efim.EfimError) as e:
                fe.admit(prompt, reserve, row)
            assert e.value.code == 4
            wh = None
        else:
            h, cached, npages = fe.admit(prompt, reserve, row)
            assert cached == wcached and row[:npages].tolist() == wpages and (row[npages:] == -1).all()
            gen = rng.integers(0, 30, int(rng.integers(0, reserve + 1))).tolist()
            open_reqs.append((h, wh, want_prompt + gen))
        # requests overlap: finish a random one now and then, all at the end
        while open_reqs and (rng.random() < 0.6 or len(open_reqs) > 3 or wh is None):
            h, wh2, seq = open_reqs.pop(int(rng.integers(0, len(open_reqs))))
            cache.finish(wh2, seq)
            fe.finish(h, seq)
            if wh is None:
                wh = 0
        s = fe.stats()
        assert (s["prompt_tokens"], s["hit_tokens"], s["evictions"], s["free_pages"]) == \
            (cache.prompt_tokens, cache.hit_tokens, cache.evictions, len(cache.free))
    fe.close()
    return formats, cache


def test_roomy_pool_matches_oracle_and_sees_every_format():
    formats, cache = _drive(seed=1, users=4, turns=300, num_pages=100000, page_size=16, rebase=0)
    assert {fo.PSM_NEW, fo.EFIM, fo.PSM_SUFFIX, fo.PSM_RESET} <= formats
    assert cache.evictions == 0 and cache.hit_tokens > 0


@pytest.mark.parametrize("seed,page_size,rebase", [(2, 16, 0), (3, 4, 50), (4, 8, 0)])
def test_tight_pool_matches_oracle_through_evictions_and_refusals(seed, page_size, rebase):
    formats, cache = _drive(seed=seed, users=6, turns=400, num_pages=2200 // page_size, page_size=page_size,
                            rebase=rebase, max_pages=1024 // page_size * 2)
    assert cache.evictions > 0
    if rebase:
        assert fo.PSM_REBASE in formats


def test_argument_errors():
    fe = efim.Frontend(1, 2, 3, 8, 4)
    row = np.zeros(2, np.int32)
    with pytest.raises(efim.EfimError) as e:          # 12 tokens need 3 pages, the row has 2
        fe.admit(np.arange(12, dtype=np.int32), 0, row)
    assert e.value.code == 3
    with pytest.raises(efim.EfimError) as e:          # unknown handle
        fe.finish(99, np.arange(4, dtype=np.int32))
    assert e.value.code == 1
    with pytest.raises(efim.EfimError):
        efim.Frontend(1, 2, 3, 0, 4)
