"""Ragged multi-turn infilling workloads (shapes, lengths, block tables, draws).

After the EFIM reorder a turn's prompt is `<P>prefix<S>suffix<M>inc`: the
first `cached_len` tokens (prefix + suffix + the three special tokens) are
already in the paged KV cache, `new_len` tokens (`inc`) are new, and
`decode_steps` generated tokens follow.  A workload fixes, from one seed:
head counts, head_dim, page size, per-sequence cached/new lengths, a block
table that scatters every sequence's pages over a shared pool, and the bf16
draws for the new tokens' q/k/v.  The pool's prior contents come from
`pool.py` (a pure function of the element index).

Named workloads
  cfg1   1 seq, 4 q heads = 4 kv heads, D=64; cached 240 (160 prefix + 80
         suffix, specials counted inside), inc 16, 8 decode steps, 32 pages.
  cfg2   16 seqs, 32/32 heads, D=128; cached U[2048,8192], inc U[32,256];
         65,536-page pool.
  cfg3   64 seqs, 28/4 heads, D=128; 32 append-prefill rows (inc log-U[1,512]
         over cached log-U[1024,16384]) + 32 single-token decode rows over
         context log-U[1024,16384]; 131,072-page pool.
  cfg4a  8 seqs, 32/8 heads, D=128; cached 8192 (5120 prefix + 3072 suffix),
         inc 128 (the EFIM path).
  cfg4b  same pool/seed; cached 5120, new 3200 (inc 128 + suffix 3072: what
         the unreordered FIM prompt must recompute).  `cfg4b_3072` is the
         literal 3072-token variant.
  cfg5   256 seqs, 32/8 heads, D=128; context U[4096,32768], 64 decode steps
         (append 1 token, then decode attention).
`small=True` shrinks lengths/pool so a CPU oracle finishes in seconds while
still spanning several 128-token tiles and ragged tails.
"""
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

from .bf16 import f32_to_bf16_bits
from .pool import pool_bits_np, K_POOL_ID, V_POOL_ID

WORKLOAD_NAMES = ("cfg1", "cfg2", "cfg3", "cfg4a", "cfg4b", "cfg4b_3072", "cfg5")


@dataclass
class Workload:
    name: str
    seed: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_pages: int
    rope_base: float
    cached_len: np.ndarray          # int32 [B]
    new_len: np.ndarray             # int32 [B]
    block_table: np.ndarray         # int32 [B, max_pages_per_seq]; unused entries = -1
    decode_steps: int = 0
    decode_rows: Optional[np.ndarray] = None   # bool [B]: rows that are single-token decode (cfg3)
    meta: dict = field(default_factory=dict)

    # ---- derived sizes -------------------------------------------------
    @property
    def batch(self) -> int:
        return int(self.cached_len.shape[0])

    @property
    def q_indptr(self) -> np.ndarray:
        out = np.zeros(self.batch + 1, dtype=np.int32)
        np.cumsum(self.new_len, out=out[1:])
        return out

    @property
    def total_new_tokens(self) -> int:
        return int(self.new_len.sum())

    @property
    def max_pages_per_seq(self) -> int:
        return int(self.block_table.shape[1])

    def pool_shape(self):
        return (self.num_pages, self.num_kv_heads, self.page_size, self.head_dim)

    # ---- draws -----------------------------------------------------------
    def _normal_bits(self, tag: int, shape) -> np.ndarray:
        rng = np.random.default_rng([self.seed, tag])
        return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))

    def new_qkv(self):
        """bf16 bits of the new tokens' q [T,Hq,D], k [T,Hkv,D], v [T,Hkv,D]."""
        T = self.total_new_tokens
        return (self._normal_bits(11, (T, self.num_q_heads, self.head_dim)),
                self._normal_bits(12, (T, self.num_kv_heads, self.head_dim)),
                self._normal_bits(13, (T, self.num_kv_heads, self.head_dim)))

    def decode_qkv(self, step: int):
        """bf16 bits of decode step `step`: q [B,Hq,D], k [B,Hkv,D], v [B,Hkv,D]."""
        B = self.batch
        return (self._normal_bits(100 + 3 * step, (B, self.num_q_heads, self.head_dim)),
                self._normal_bits(101 + 3 * step, (B, self.num_kv_heads, self.head_dim)),
                self._normal_bits(102 + 3 * step, (B, self.num_kv_heads, self.head_dim)))

    # ---- pool contents -----------------------------------------------------
    def page_bits(self, which: str, page_ids) -> np.ndarray:
        """Prior contents of the given pages of the K ('k') or V ('v') pool:
        uint16 [len(page_ids), Hkv, P, D]."""
        tid = K_POOL_ID if which == "k" else V_POOL_ID
        per_page = self.num_kv_heads * self.page_size * self.head_dim
        out = np.empty((len(page_ids), per_page), dtype=np.uint16)
        for n, pg in enumerate(page_ids):
            out[n] = pool_bits_np(self.seed, tid, int(pg) * per_page, per_page)
        return out.reshape(len(page_ids), self.num_kv_heads, self.page_size, self.head_dim)

    def pages_of(self, s: int, upto_len: Optional[int] = None) -> np.ndarray:
        """Physical page ids of sequence s covering tokens [0, upto_len)."""
        if upto_len is None:
            upto_len = int(self.cached_len[s] + self.new_len[s] + self.decode_steps)
        n = -(-upto_len // self.page_size)
        return self.block_table[s, :n].copy()

    def compact_host_pool(self, seqs=None):
        """A dense host copy of just the pages the chosen sequences use.

        Returns (k_pool, v_pool, block_table, seqs) where the pools are uint16
        [n_used, Hkv, P, D], and block_table is this workload's table for those
        sequences with physical ids renumbered 0..n_used-1 (unused = -1).  Page
        renumbering does not change what any sequence sees.
        """
        if seqs is None:
            seqs = list(range(self.batch))
        used = []
        for s in seqs:
            used.extend(self.pages_of(s).tolist())
        used = np.array(sorted(set(used)), dtype=np.int64)
        remap = {int(p): i for i, p in enumerate(used)}
        bt = np.full((len(seqs), self.max_pages_per_seq), -1, dtype=np.int32)
        for r, s in enumerate(seqs):
            pg = self.pages_of(s)
            bt[r, :len(pg)] = [remap[int(p)] for p in pg]
        return self.page_bits("k", used), self.page_bits("v", used), bt, list(seqs)


def _uniform_int(rng, lo, hi, n):
    return rng.integers(lo, hi + 1, size=n).astype(np.int32)


def _log_uniform_int(rng, lo, hi, n):
    return np.rint(np.exp(rng.uniform(np.log(lo), np.log(hi), size=n))).astype(np.int32)


def _block_table(rng, num_pages, total_len, page_size):
    need = -(-total_len // page_size)
    B = len(total_len)
    if int(need.sum()) > num_pages:
        raise ValueError("pool too small for this workload")
    perm = rng.permutation(num_pages)[: int(need.sum())].astype(np.int32)
    bt = np.full((B, int(need.max())), -1, dtype=np.int32)
    off = 0
    for s in range(B):
        bt[s, : need[s]] = perm[off: off + need[s]]
        off += need[s]
    return bt


def make_workload(name: str, small: bool = False, seed: Optional[int] = None,
                  batch: Optional[int] = None) -> Workload:
    """`batch` overrides the number of sequences of cfg2/cfg5 (the pool shrinks or grows with it)."""
    if name not in WORKLOAD_NAMES:
        raise ValueError(f"unknown workload {name!r}; choose from {WORKLOAD_NAMES}")
    P = 16
    decode_rows = None
    meta = {}
    if name == "cfg1":
        sd = 0 if seed is None else seed
        Hq, Hkv, D, pages, steps = 4, 4, 64, 32, 8
        rng = np.random.default_rng([sd, 1])
        cached = np.array([240], np.int32)
        new = np.array([16], np.int32)
        meta = {"prefix": 160, "suffix": 80, "specials": 3}
    elif name == "cfg2":
        sd = 2 if seed is None else seed
        Hq, Hkv, D, steps = 32, 32, 128, 1
        rng = np.random.default_rng([sd, 1])
        if small:
            Hq = Hkv = 4
            pages = 2048
            cached = _uniform_int(rng, 200, 800, 6)
            new = _uniform_int(rng, 32, 256, 6)
        else:
            nb = 16 if batch is None else batch
            pages = 65536 * nb // 16
            cached = _uniform_int(rng, 2048, 8192, nb)
            new = _uniform_int(rng, 32, 256, nb)
    elif name == "cfg3":
        sd = 3 if seed is None else seed
        Hq, Hkv, D, steps = 28, 4, 128, 0
        rng = np.random.default_rng([sd, 1])
        if small:
            nb, pages, clo, chi, nhi = 8, 4096, 100, 1500, 200
        else:
            nb, pages, clo, chi, nhi = 64, 131072, 1024, 16384, 512
        h = nb // 2
        cached_p = _log_uniform_int(rng, clo, chi, h)
        new_p = _log_uniform_int(rng, 1, nhi, h)
        ctx_d = _log_uniform_int(rng, clo, chi, h)
        cached = np.concatenate([cached_p, ctx_d - 1]).astype(np.int32)
        new = np.concatenate([new_p, np.ones(h, np.int32)]).astype(np.int32)
        decode_rows = np.concatenate([np.zeros(h, bool), np.ones(h, bool)])
        order = rng.permutation(nb)          # a mixed batch, not two sorted halves
        cached, new, decode_rows = cached[order], new[order], decode_rows[order]
    elif name in ("cfg4a", "cfg4b", "cfg4b_3072"):
        sd = 4 if seed is None else seed
        Hq, Hkv, D, steps = 32, 8, 128, 0
        rng = np.random.default_rng([sd, 1])
        if small:
            Hq, Hkv = 8, 2
            nb, pages, prefix, suffix, inc = 2, 512, 320, 192, 40
        else:
            nb, pages, prefix, suffix, inc = 8, 8192, 5120, 3072, 128
        meta = {"prefix": prefix, "suffix": suffix, "inc": inc}
        if name == "cfg4a":
            cached = np.full(nb, prefix + suffix, np.int32)
            new = np.full(nb, inc, np.int32)
        elif name == "cfg4b":
            cached = np.full(nb, prefix, np.int32)
            new = np.full(nb, inc + suffix, np.int32)
        else:
            cached = np.full(nb, prefix, np.int32)
            new = np.full(nb, suffix, np.int32)
        # one block table for all three variants: sized for prefix+suffix+inc
        total = np.full(nb, prefix + suffix + inc, np.int32)
        bt = _block_table(rng, pages, total, P)
        return Workload(name, sd, Hq, Hkv, D, P, pages, 10000.0, cached, new, bt,
                        decode_steps=0, decode_rows=None, meta=meta)
    else:  # cfg5
        sd = 5 if seed is None else seed
        Hq, Hkv, D = 32, 8, 128
        rng = np.random.default_rng([sd, 1])
        if small:
            Hq, Hkv = 8, 2
            nb, pages, steps = 12, 4096, 4
            ctx = _uniform_int(rng, 300, 3000, nb)
        else:
            nb, steps = (256 if batch is None else batch), 64
            pages = 2112 * nb
            ctx = _uniform_int(rng, 4096, 32768, nb)
        # the decode loop: step t appends one token at position ctx+t
        cached = ctx.astype(np.int32)
        new = np.zeros(nb, np.int32)
    total = cached + new + steps
    bt = _block_table(rng, pages, total, P)
    return Workload(name, sd, Hq, Hkv, D, P, pages, 10000.0, cached, new, bt,
                    decode_steps=steps, decode_rows=decode_rows, meta=meta)
