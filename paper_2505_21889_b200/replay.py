"""Kernel-level replay of the paper's serving experiment (Sec. 4.2 "Inference speedup",
Sec. 5.2): users x rounds of multi-turn infilling through one layer's attention path,
under three schemes -

  none   PSM prompts, no cross-request KV reuse            (the paper's "Baseline")
  fim    PSM prompts + cross-request KV reuse               ("FIM": only the prefix is reusable)
  efim   Sec. 3.1 prompt transformation + the same reuse   ("EFIM": prefix and suffix reusable)

Every round batches the users' requests: the front end (efim_frontend_*) turns each request
into a prompt, a cached length and a block-table row; the tokens that are not cached go
through efim_kv_append + efim_append_prefill_attn, the generated tokens through
efim_decode_step (append fused with decode attention), one step per token.  A pool smaller than the users'
working set makes the front end evict and the reuse rate fall (Sec. 5.3, sensitivity to
the number of users).  Only the attention path of ONE layer is timed - no linear layers,
no sampling - so the ratios are those of this path, not of end-to-end serving.

    python -m paper_2505_21889_b200.replay --users 16 --rounds 5 --pool-pages 16384
"""
import argparse
import json

import numpy as np
import torch

from . import binding as efim
from efim_synth import token_tables, infill_sessions, TOK_P, TOK_S, TOK_M

SCHEMES = ("none", "fim", "efim")


class Layer:
    """Device copies of the per-token q/k/v tables, the page pools and the rotary table."""

    def __init__(self, seed, vocab, num_q_heads, num_kv_heads, head_dim, pool_pages, max_position, device="cuda"):
        def dev(bits):
            return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
        self.device = device
        self.bits = token_tables(seed, vocab, num_q_heads, num_kv_heads, head_dim)
        self.q_tab, self.k_tab, self.v_tab = (dev(b) for b in self.bits)
        shape = (pool_pages, num_kv_heads, 16, head_dim)
        self.k_pool = torch.zeros(shape, dtype=torch.bfloat16, device=device)
        self.v_pool = torch.zeros(shape, dtype=torch.bfloat16, device=device)
        self.cache = efim.Cache(self.k_pool, self.v_pool, num_q_heads)
        self.rope = efim.Rope(10000.0, head_dim, max_position, False, device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.num_q_heads, self.head_dim = num_q_heads, head_dim

    def qkv(self, token_ids):
        idx = torch.as_tensor(np.asarray(token_ids, np.int64), device=self.device)
        return self.q_tab[idx].contiguous(), self.k_tab[idx].contiguous(), self.v_tab[idx].contiguous()


def _timed(fn):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fn()
    e1.record()
    return e0, e1


def run_scheme(scheme, sessions, layer, pool_pages, max_pages_per_seq, observe=None, batch_size=None, graph=False,
               shuffle_seed=None):
    """Replays all rounds under one scheme; in every round the users are served in batches of
    `batch_size` (default: all at once).  `observe(round, users, prompts, cached, bt, out,
    dec_out)` is called after every batch (for tests).  With `graph` the decode steps of a
    batch (two or three small launches per token) are captured into one CUDA graph and
    replayed, which takes the host's launch pace out of the decode time.  `shuffle_seed` serves
    the users of a round in a seeded random order instead of 0, 1, 2, ... (closed-loop clients
    do not come back in lockstep; a fixed cyclic order is the worst case for LRU).  Returns totals."""
    assert scheme in SCHEMES
    n_users, rounds = len(sessions), len(sessions[0])
    batch_size = batch_size or n_users
    fe = efim.Frontend(TOK_P, TOK_S, TOK_M, pool_pages)
    events, totals = [], dict(prompt_tokens=0, computed_tokens=0, hit_tokens=0, evictions=0, decode_tokens=0)
    order_rng = np.random.default_rng([shuffle_seed, 41]) if shuffle_seed is not None else None
    orders = [order_rng.permutation(n_users).tolist() if order_rng is not None else list(range(n_users))
              for _ in range(rounds)]
    for r, first in ((r, f) for r in range(rounds) for f in range(0, n_users, batch_size)):
        group = orders[r][first:first + batch_size]
        users = len(group)
        if scheme == "none":                     # nothing survives from round to round
            totals["evictions"] += fe.stats()["evictions"]
            fe.close()
            fe = efim.Frontend(TOK_P, TOK_S, TOK_M, pool_pages)
        prompts, handles = [], []
        bt = np.full((users, max_pages_per_seq), -1, np.int32)
        cached = np.zeros(users, np.int32)
        for u in range(users):
            t = sessions[group[u]][r]
            if scheme == "efim":
                prompt, _, _ = fe.transform(group[u], t["prefix"], t["suffix"])
            else:
                prompt = np.array([TOK_P] + t["prefix"] + [TOK_S] + t["suffix"] + [TOK_M], np.int32)
            h, cached[u], _ = fe.admit(prompt, len(t["gen"]), bt[u])
            prompts.append(prompt)
            handles.append(h)
        plen = np.array([len(p) for p in prompts], np.int32)
        new = plen - cached
        d_bt = torch.from_numpy(bt).to(layer.device)
        # ---- append-prefill of the tokens that are not cached
        q, k, v = layer.qkv(np.concatenate([p[c:] for p, c in zip(prompts, cached)]))
        batch = efim.Batch(cached, new, d_bt, layer.device)
        out = torch.empty_like(q)
        ws = torch.empty(max(efim.efim_prefill_workspace_bytes(layer.cache, batch), 256), dtype=torch.uint8,
                         device=layer.device)
        events.append(("prefill",) + _timed(lambda: (
            efim.efim_kv_append(layer.cache, batch, layer.rope, q, k, v, layer.status),
            efim.efim_append_prefill_attn(layer.cache, batch, q, out, None, 0.0, ws, layer.status))))
        # ---- decode of the generated middle, one token per step
        steps = len(sessions[group[0]][r]["gen"])
        ctx = plen.copy()
        one = np.ones(users, np.int32)
        max_ctx = int(plen.max()) + steps
        dws = torch.empty(max(efim.efim_decode_workspace_bytes(layer.cache, users, max_ctx), 256), dtype=torch.uint8,
                          device=layer.device)
        # per-step inputs are laid out up front so that the loop below only enqueues kernels
        gen_ids = np.array([[sessions[g][r]["gen"][s] for g in group] for s in range(steps)]).reshape(-1)
        dq_all, dk_all, dv_all = (x.view(steps, users, *x.shape[1:]) for x in layer.qkv(gen_ids))
        dec_all = torch.empty_like(dq_all)
        d_ctx_all = torch.from_numpy(np.stack([ctx + s + 1 for s in range(steps)])).to(layer.device)

        def decode_loop():
            for s in range(steps):
                efim.efim_decode_step(layer.cache, users, d_ctx_all[s], max_ctx, d_bt, layer.rope, dq_all[s],
                                      dk_all[s], dv_all[s], dec_all[s], None, 0.0, dws, layer.status)
        if graph and steps > 0:
            g = torch.cuda.CUDAGraph()
            torch.cuda.synchronize()
            with torch.cuda.graph(g):
                decode_loop()
            # the first launch of a new graph also uploads it to the device (≈1 ms for these 256
            # nodes); a server captures once per batch shape, so that cost is kept out of the time.
            # The steps are idempotent: a replay writes the same K/V slots and outputs again.
            g.replay()
            torch.cuda.synchronize()
            events.append(("decode",) + _timed(g.replay))
        else:
            events.append(("decode",) + _timed(decode_loop))
        dec_out = dec_all[steps - 1] if steps > 0 else None
        torch.cuda.synchronize()
        if observe is not None:
            observe(r, group, prompts, cached.copy(), bt.copy(), out, dec_out)
        for u in range(users):
            fe.finish(handles[u], np.concatenate([prompts[u], np.array(sessions[group[u]][r]["gen"], np.int32)]))
        totals["prompt_tokens"] += int(plen.sum())
        totals["computed_tokens"] += int(new.sum())
        totals["hit_tokens"] += int(cached.sum())
        totals["decode_tokens"] += users * steps
    torch.cuda.synchronize()
    if int(layer.status.item()) != 0:
        raise RuntimeError(f"device status 0x{int(layer.status.item()):x}")
    totals["evictions"] += fe.stats()["evictions"]
    fe.close()
    totals["prefill_ms"] = sum(a.elapsed_time(b) for kind, a, b in events if kind == "prefill")
    totals["decode_ms"] = sum(a.elapsed_time(b) for kind, a, b in events if kind == "decode")
    totals["reuse_rate"] = totals["hit_tokens"] / totals["prompt_tokens"]
    return totals


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--users", type=int, default=16)
    ap.add_argument("--rounds", type=int, default=5)
    ap.add_argument("--gen", type=int, default=128)
    ap.add_argument("--pool-pages", type=int, default=16384)
    ap.add_argument("--batch-size", type=int, default=16, help="users served together (the rest wait their turn)")
    ap.add_argument("--heads", type=int, nargs=2, default=(32, 8), metavar=("HQ", "HKV"))
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--in-order", action="store_true", help="serve users 0, 1, 2, ... in every round (default: seeded random order)")
    ap.add_argument("--graph", action="store_true", help="replay each batch's decode steps as one CUDA graph")
    ap.add_argument("--schemes", nargs="+", default=list(SCHEMES), choices=SCHEMES)
    a = ap.parse_args()
    vocab = 4096
    sessions = infill_sessions(a.seed, a.users, a.rounds, vocab, gen=a.gen)
    longest = max(len(t["prefix"]) + len(t["suffix"]) + 3 + len(t["gen"]) for u in sessions for t in u)
    max_pages = -(-longest // 16)
    torch.cuda.set_device(0)
    layer = Layer(a.seed, vocab, a.heads[0], a.heads[1], 128, a.pool_pages, longest + 1)
    base = None
    for scheme in a.schemes:
        run_scheme(scheme, [u[:1] for u in sessions], layer, a.pool_pages, max_pages, batch_size=a.batch_size)   # warm-up
        t = run_scheme(scheme, sessions, layer, a.pool_pages, max_pages, batch_size=a.batch_size, graph=a.graph,
                       shuffle_seed=None if a.in_order else a.seed)
        t.update(scheme=scheme, users=a.users, rounds=a.rounds, pool_pages=a.pool_pages, batch_size=a.batch_size, graph=a.graph,
                 avg_input_tokens=t["prompt_tokens"] / (a.users * a.rounds), layer_ms=t["prefill_ms"] + t["decode_ms"])
        if scheme == "none":
            base = t["layer_ms"]
        if base:
            t["layer_time_vs_none"] = t["layer_ms"] / base
        print(json.dumps(t), flush=True)


if __name__ == "__main__":
    main()
