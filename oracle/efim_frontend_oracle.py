"""CPU oracle for the EFIM front end: prompt transformation and cross-request KV reuse.

TEST INFRASTRUCTURE ONLY: imported by tests/, by __graft_entry__.smoke() and by
bench.py's cpu_baseline leg; the product path (libefim.so) shares no code with it.

Two plain, slow, list-and-dict implementations:

* `SessionPool` - the prompt transformation of Sec. 3.1 (Fig. 7, steps 1-5): a
  per-user session remembers the prefix and suffix as they were laid out in the
  user's last prompt; a request whose prefix only grew is sent as
  `<P>common<S>suffix<M>inc` (the EFIM format of Sec. 1), everything else in the
  PSM format `<P>prefix<S>suffix<M>` (Sec. 2.1).
* `PrefixCache` - cross-request KV cache reuse as Sec. 1 states it: the KV of a
  prompt can be reused for exactly the tokens whose whole token prefix is identical
  to an earlier sequence's.  Reuse is per page of `page_size` tokens; pages of
  finished sequences stay cached until evicted, least recently used first.

Parity unpinned against the paper's numbers (it prints none for these steps); the
pins are the format definitions, hand-written examples and a brute-force
longest-common-prefix search (tests/test_frontend_oracle.py).
"""

# formats returned by SessionPool.transform
PSM_NEW = 0      # step 2: no session yet -> PSM, session created
EFIM = 1         # step 4: prefix grew -> common + suffix + inc
PSM_SUFFIX = 2   # step 5: prefix unchanged, suffix changed -> PSM (prefix KV still reusable)
PSM_SAME = 3     # the same request again -> PSM, identical to the last prompt
PSM_RESET = 4    # prefix no longer extends the session's (edited or shortened) -> PSM, session replaced
PSM_REBASE = 5   # inc would exceed the configured limit -> PSM with the whole prefix, session replaced


def psm_prompt(tok_p, tok_s, tok_m, prefix, suffix):
    """`<P>prefix<S>suffix<M>` (Sec. 1, Sec. 2.1)."""
    return [tok_p] + list(prefix) + [tok_s] + list(suffix) + [tok_m]


def efim_prompt(tok_p, tok_s, tok_m, common, suffix, inc):
    """`<P>prefix<S>suffix<M>inc` (Sec. 1): the increment of the prefix goes last."""
    return [tok_p] + list(common) + [tok_s] + list(suffix) + [tok_m] + list(inc)


class SessionPool:
    """Sec. 3.1, steps 1-5.  `rebase_inc_tokens` > 0 bounds `inc`: a longer increment is
    folded back into the prefix with one PSM prompt (0 = never; the paper has no bound)."""

    def __init__(self, tok_p, tok_s, tok_m, rebase_inc_tokens=0):
        self.tok = (tok_p, tok_s, tok_m)
        self.rebase = rebase_inc_tokens
        self.sessions = {}                      # user -> (prefix as laid out in the last prompt, suffix)

    def transform(self, user, prefix, suffix):
        """-> (prompt tokens, format, len(inc))."""
        prefix, suffix = list(prefix), list(suffix)
        if user not in self.sessions:                                     # steps 1, 2
            self.sessions[user] = (prefix, suffix)
            return psm_prompt(*self.tok, prefix, suffix), PSM_NEW, 0
        base, old_suffix = self.sessions[user]                            # step 3
        if len(prefix) > len(base) and prefix[:len(base)] == base:        # step 4
            inc = prefix[len(base):]
            if self.rebase > 0 and len(inc) > self.rebase:
                self.sessions[user] = (prefix, suffix)
                return psm_prompt(*self.tok, prefix, suffix), PSM_REBASE, 0
            self.sessions[user] = (base, suffix)
            return efim_prompt(*self.tok, base, suffix, inc), EFIM, len(inc)
        if prefix == base:                                                # step 5 (or a repeat)
            self.sessions[user] = (base, suffix)
            fmt = PSM_SAME if suffix == old_suffix else PSM_SUFFIX
            return psm_prompt(*self.tok, prefix, suffix), fmt, 0
        self.sessions[user] = (prefix, suffix)                            # prefix edited: start over
        return psm_prompt(*self.tok, prefix, suffix), PSM_RESET, 0


class OutOfPages(Exception):
    pass


class PrefixCache:
    """Page-granular cross-request KV reuse over a pool of `num_pages` pages.

    A cached page is identified by the whole token prefix up to and including its
    block.  admit() matches the longest run of cached full blocks at the start of the
    prompt (leaving at least one token to compute), pins them, and takes new pages for
    the rest plus `reserve_tokens` of decode room: the lowest-numbered never-used or
    freed page first, else the least recently used unpinned cached page (oldest use;
    among equals the deepest block).  finish() registers the full blocks of the
    finished sequence, frees duplicates, the partial last page and unused room.
    """

    def __init__(self, num_pages, page_size=16):
        self.P = page_size
        self.free = list(range(num_pages))       # kept sorted ascending
        self.by_prefix = {}                       # tuple(tokens[:(b+1)P]) -> page id
        self.page = {}                            # cached page id -> dict(prefix, ref, used)
        self.tick = 0
        self.requests = {}
        self.next_handle = 1
        self.prompt_tokens = 0
        self.hit_tokens = 0
        self.evictions = 0

    def _take_page(self):
        if self.free:
            return self.free.pop(0)
        cand = [(m["used"], -len(m["prefix"]), pid) for pid, m in self.page.items() if m["ref"] == 0]
        if not cand:
            raise OutOfPages()
        _, _, pid = min(cand)
        del self.by_prefix[self.page[pid]["prefix"]]
        del self.page[pid]
        self.evictions += 1
        return pid

    def admit(self, prompt, reserve_tokens=0):
        """-> (handle, cached_len, page ids covering len(prompt) + reserve_tokens tokens)."""
        prompt = list(prompt)
        P = self.P
        self.tick += 1
        matched = []
        for b in range(len(prompt) // P):
            pid = self.by_prefix.get(tuple(prompt[:(b + 1) * P]))
            if pid is None:
                break
            matched.append(pid)
        if matched and len(matched) * P >= len(prompt):
            matched.pop()                         # at least one token is computed
        for pid in matched:
            self.page[pid]["ref"] += 1
            self.page[pid]["used"] = self.tick
        need = -(-(len(prompt) + reserve_tokens) // P) - len(matched)
        fresh = []
        try:
            for _ in range(need):
                fresh.append(self._take_page())
        except OutOfPages:
            for pid in fresh:
                self._free(pid)
            for pid in matched:
                self.page[pid]["ref"] -= 1
            raise
        h = self.next_handle
        self.next_handle += 1
        self.requests[h] = (len(matched), matched + fresh)
        self.prompt_tokens += len(prompt)
        self.hit_tokens += len(matched) * P
        return h, len(matched) * P, matched + fresh

    def _free(self, pid):
        self.free.append(pid)
        self.free.sort()

    def finish(self, handle, tokens):
        """`tokens`: the whole sequence (prompt + generated) whose KV is now in the pages."""
        tokens = list(tokens)
        P = self.P
        n_matched, pages = self.requests.pop(handle)
        self.tick += 1
        for b, pid in enumerate(pages):
            if b < n_matched:
                self.page[pid]["ref"] -= 1
                self.page[pid]["used"] = self.tick
            elif (b + 1) * P <= len(tokens):
                key = tuple(tokens[:(b + 1) * P])
                if key in self.by_prefix:         # the same content was registered meanwhile
                    self.page[self.by_prefix[key]]["used"] = self.tick
                    self._free(pid)
                else:
                    self.by_prefix[key] = pid
                    self.page[pid] = dict(prefix=key, ref=0, used=self.tick)
            else:
                self._free(pid)

    def reuse_rate(self):
        return self.hit_tokens / self.prompt_tokens if self.prompt_tokens else 0.0
