"""Shared plumbing for the GPU parity tests: put a seeded workload on the device,
run the C-ABI calls, and compute the oracle's answer for chosen sequences from the
same bytes.  Nothing here computes attention or RoPE itself."""
import numpy as np
import torch

import paper_2505_21889_b200 as efim
from efim_synth import pool_fill_torch, bf16_bits_to_f32
from efim_synth.pool import K_POOL_ID, V_POOL_ID
from oracle import efim_oracle as orc

# spec tolerances for bf16 attention outputs with fp32 accumulation
MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3
# lse: 1e-3 absolute.  The largest error seen over all cases, full sizes included, is 4.2e-4
# (rows with thousands of keys; the scores leave the tensor core with ~1e-4 of absolute error
# at |score| ~ 10), the decode kernel's fp32 FMA chains stay below 3e-5.
LSE_TOL = 1e-3


def bits_to_torch(bits: np.ndarray, device="cuda"):
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def torch_to_bits(t) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def ordered(bits: np.ndarray) -> np.ndarray:
    """Map bf16 bit patterns to integers ordered like the values (adjacent floats differ by 1)."""
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def assert_rope_close(got_bits, want_bits, what):
    """fp32 table + fp32 FMA against fp64-then-round.  The fp32 result carries an
    absolute error of a few 2^-24 * |input| (inputs are |x| < 8), so it either rounds
    to the same bf16 value, to a neighbour when the exact result sits within that
    error of a rounding tie, or - where a*cos and b*sin cancel and the result is
    tiny - differs by that absolute error although it spans several tiny ulps."""
    d = np.abs(ordered(got_bits) - ordered(want_bits))
    abs_err = np.abs(bf16_bits_to_f32(got_bits).astype(np.float64) - bf16_bits_to_f32(want_bits).astype(np.float64))
    bad = (d > 1) & (abs_err > 4e-6)
    assert not bad.any(), f"{what}: {int(bad.sum())} elements beyond one bf16 ulp and beyond fp32 rounding error"
    if d.size:
        assert (d == 0).mean() >= 0.99, f"{what}: only {(d == 0).mean():.4f} identical"


def assert_attn_close(got_bf16_bits, want_f64, what):
    got = bf16_bits_to_f32(got_bf16_bits).astype(np.float64)
    err = np.abs(got - want_f64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    print(f"out max abs err {err.max(initial=0):.3e} mean {err.mean() if err.size else 0.0:.3e}  [{what}]")
    assert err.max(initial=0) <= MAX_ABS_TOL, f"{what}: max abs err {err.max():.4g}"
    assert err.mean() <= MEAN_ABS_TOL, f"{what}: mean abs err {err.mean():.4g}"


def assert_lse_close(got, want, what):
    """|lse error| against the fp64 oracle; the figure is printed so a run with -rP shows the
    margin every case leaves."""
    err = float(np.abs(np.asarray(got, np.float64) - want).max(initial=0))
    print(f"lse max abs err {err:.3e}  [{what}]")
    assert err <= LSE_TOL, f"{what}: lse max abs err {err:.4g}"


class DeviceWorkload:
    """A workload resident on the GPU plus the oracle's view of selected sequences."""

    def __init__(self, w, interleaved=False, use_rope=True, device="cuda"):
        self.w = w
        self.device = device
        self.interleaved = interleaved
        self.k_pool = torch.empty(w.pool_shape(), dtype=torch.bfloat16, device=device)
        self.v_pool = torch.empty(w.pool_shape(), dtype=torch.bfloat16, device=device)
        pool_fill_torch(self.k_pool, w.seed, K_POOL_ID)
        pool_fill_torch(self.v_pool, w.seed, V_POOL_ID)
        self.cache = efim.Cache(self.k_pool, self.v_pool, w.num_q_heads)
        self.batch = efim.Batch(w.cached_len, w.new_len, w.block_table, device=device)
        max_pos = int((w.cached_len + w.new_len).max()) + w.decode_steps + 1
        self.rope = efim.Rope(w.rope_base, w.head_dim, max_pos, interleaved, device) if use_rope else None
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        q, k, v = w.new_qkv()
        self.q_bits, self.k_bits, self.v_bits = q, k, v
        self.q = bits_to_torch(q, device)
        self.k_new = bits_to_torch(k, device)
        self.v_new = bits_to_torch(v, device)
        self.out = torch.empty_like(self.q)
        self.lse = torch.empty(q.shape[:2], dtype=torch.float32, device=device)

    # ---- GPU path ---------------------------------------------------------
    def gpu_kv_append(self):
        efim.efim_kv_append(self.cache, self.batch, self.rope, self.q, self.k_new, self.v_new, self.status)

    def gpu_prefill(self, sm_scale=0.0):
        nbytes = efim.efim_prefill_workspace_bytes(self.cache, self.batch)
        self.ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device)
        efim.efim_append_prefill_attn(self.cache, self.batch, self.q, self.out, self.lse, sm_scale,
                                      self.ws, self.status)

    def pages_from_device(self, which, page_ids):
        pool = self.k_pool if which == "k" else self.v_pool
        idx = torch.as_tensor(np.asarray(page_ids, dtype=np.int64), device=self.device)
        return torch_to_bits(pool[idx])

    # ---- oracle on a subset of sequences ------------------------------------
    def oracle_turn(self, seqs=None, sm_scale=None, windows=None):
        """Run the oracle's kv_append + append_prefill_attention for `seqs`.
        Returns dict with rotated q bits, pools (compact), block table, o, lse, row index.
        `windows` = list of (first_token, count) per sequence restricts the attention rows
        to those new tokens (the cache update is still done for all of them); by the reuse
        identity this is the oracle called with cached_len + first_token."""
        w = self.w
        kp, vp, bt, seqs = w.compact_host_pool(seqs)
        ind = w.q_indptr
        rows = np.concatenate([np.arange(ind[s], ind[s + 1]) for s in seqs] + [np.zeros(0, np.int64)]).astype(np.int64)
        cached = w.cached_len[seqs]
        new = w.new_len[seqs]
        q_rot = orc.kv_append(kp, vp, bt, cached, new, self.q_bits[rows], self.k_bits[rows], self.v_bits[rows],
                              w.rope_base, self.interleaved, use_rope=self.rope is not None)
        attn_rows = rows
        if windows is None:
            o, lse = orc.append_prefill_attention(q_rot, kp, vp, bt, cached, new, w.num_q_heads, sm_scale)
        else:
            starts = np.concatenate([[0], np.cumsum(new)])[:-1]
            first = np.array([f for f, _ in windows], np.int64)
            cnt = np.array([min(c, int(n) - f) for (f, c), n in zip(windows, new)], np.int64)
            local = np.concatenate([np.arange(starts[i] + first[i], starts[i] + first[i] + cnt[i])
                                    for i in range(len(seqs))]).astype(np.int64)
            o, lse = orc.append_prefill_attention(q_rot[local], kp, vp, bt, cached + first, cnt, w.num_q_heads,
                                                  sm_scale)
            attn_rows = rows[local]
        return dict(q_rot=q_rot, k_pool=kp, v_pool=vp, bt=bt, seqs=seqs, rows=rows, o=o, lse=lse,
                    cached=cached, new=new, attn_rows=attn_rows)
