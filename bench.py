#!/usr/bin/env python
"""Benchmark of the EFIM per-turn GPU path on synthetic multi-turn infilling batches.

One "step" = one turn of one layer over one ragged batch:
    efim_kv_append(inc tokens: q and k rotated, k/v stored in the pages)
    -> efim_append_prefill_attn_planned (the work list is planned once per batch)
    -> efim_decode_step (kv_append of 1 generated token per sequence fused with decode attention)
`value` = new tokens (inc + generated) that went through the path per second, inputs
resident in HBM; `e2e` = the same with the step's q/k/v coming from pinned host
memory and the outputs copied back, copies inside the timed region (pipelined over
three streams: the copies of neighbouring steps run beside a step's kernels).
`configs` = every full-size workload (cfg2, cfg3, cfg4a, cfg4b, cfg5) timed the same way
for at least half a second each, with its roofline fractions against the measured and
the nominal peaks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

With N > 1 every rank (one per GPU; started by torchrun, or by this script itself when
it is run plainly with --gpus N) runs its own replica of the workload (its own pool and
seed); there is no exchange inside the path, so the job value is the sum of tokens over
the slowest rank's time (weak scaling).
"""
import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "append_prefill_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}      # datasheet figures (dense), context only
BASE_SEED = {"cfg1": 0, "cfg2": 2, "cfg3": 3, "cfg4a": 4, "cfg4b": 4, "cfg4b_3072": 4, "cfg5": 5}
CONFIG_BLOCK = ("cfg2", "cfg3", "cfg4a", "cfg4b", "cfg5")


# --------------------------------------------------------------------------- helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def recorded_traffic(workload, call):
    """DRAM bytes per launch of `call` on `workload` from the committed ncu summary, or
    None when there is none or the kernel source changed since it was taken."""
    import glob
    import hashlib
    for path in glob.glob(os.path.join(ROOT, "profiles", "dram_traffic_*.txt")):
        for line in open(path):
            if not line.startswith("traffic "):
                continue
            kv = dict(tok.split("=", 1) for tok in line.split()[1:])
            if kv.get("workload") != workload or kv.get("call") != call:
                continue
            src = os.path.join(ROOT, kv["source"])
            if os.path.exists(src) and hashlib.sha1(open(src, "rb").read()).hexdigest() == kv["sha1"]:
                return int(kv["dram_bytes"])
    return None


def workload_counts(w):
    """Algorithmic work of one step (unmasked pairs, each K/V byte once)."""
    C = w.cached_len.astype(np.int64)
    N = w.new_len.astype(np.int64)
    D, Hq, Hkv = w.head_dim, w.num_q_heads, w.num_kv_heads
    pairs = int((N * C + N * (N + 1) // 2).sum())
    L = C + N
    has_new = N > 0
    return {
        "new_tokens": int(N.sum()),
        "decode_tokens": int(w.batch) if w.decode_steps > 0 else 0,
        "prefill_flops": 4 * D * Hq * pairs,
        "prefill_kv_bytes": int(4 * D * Hkv * L[has_new].sum()),
        "decode_kv_bytes": int(4 * D * Hkv * (L + 1).sum()) if w.decode_steps > 0 else 0,
        "kv_append_bytes_per_token": 4 * D * (Hq + 2 * Hkv),
    }


def config_of(w, world):
    """The `config` object of a bench line: names the workload (both arms print the same)."""
    return {"workload": w.name, "batch": w.batch, "num_q_heads": w.num_q_heads, "num_kv_heads": w.num_kv_heads,
            "head_dim": w.head_dim, "page_size": w.page_size, "new_tokens": int(w.new_len.sum()),
            "decode_tokens": int(w.batch) if w.decode_steps > 0 else 0,
            "cached_tokens": int(w.cached_len.sum()), "pool_pages": w.num_pages,
            "l2": "256 MiB flush between steps; K/V read per step exceeds L2",
            "parallelism": f"replicas x{world}"}


class ClockSampler:
    """nvidia-smi clock/throttle samples while the timed regions run (read-only)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.samples = []          # (wall time, sm MHz, max MHz, power W, [reasons])

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm, mx = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            try:
                power = float(parts[2])
            except ValueError:
                power = None
            reasons = [nm for nm, val in zip(self.NAMES, parts[4:8]) if val.lower().startswith("active")]
            self.samples.append((time.time(), sm, mx, power, reasons))

    def wait_first(self, timeout=3.0):
        """nvidia-smi needs a moment to print its first line; a timed region that ends before it
        would go unsampled."""
        t0 = time.time()
        while self.proc is not None and not self.samples and time.time() - t0 < timeout:
            time.sleep(0.02)

    def window(self, t0, t1):
        """Summary of the samples taken between two wall-clock times."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        rows = [s for s in list(self.samples) if t0 <= s[0] <= t1]
        if not rows:                           # a region shorter than the sampling period: nearest sample
            rows = sorted(list(self.samples), key=lambda s: abs(s[0] - 0.5 * (t0 + t1)))[:1]
        reasons = sorted({r for s in rows for r in s[4]})
        power = [s[3] for s in rows if s[3] is not None]
        return {"sm_mhz": float(np.median([s[1] for s in rows])) if rows else None,
                "sm_max_mhz": float(max(s[2] for s in rows)) if rows else None,
                "power_w_max": max(power) if power else None,
                "samples": len(rows), "reasons": reasons}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()


def aggregate_over_ranks(local_ms, local_tokens, dist=None):
    """Job-level numbers: slowest rank's time, sum of the ranks' tokens."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms), float(local_tokens)
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=dev)
    n = torch.tensor([float(local_tokens)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


# --------------------------------------------------------------------------- starting the ranks
def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def relaunch_under_torchrun(argv, n):
    """`python bench.py --gpus N` run plainly: start the N ranks (one per GPU) the way a
    launcher would, pass the command line on, and return the launcher's exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_rank_selfcheck(args):
    """--selfcheck-ranks: the rank plumbing of the multi-GPU leg (rendezvous from the
    launcher's environment, max/sum reduction, rank 0 prints) on CPU with gloo and a stand-in
    measurement, so that it can be tested without GPUs."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if world > 1:
        dist.init_process_group("gloo")
    ms, tokens = aggregate_over_ranks(10.0 + 5.0 * rank, 1000 * (rank + 1), dist if world > 1 else None)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"selfcheck": "ranks", "n_gpus": world, "ms": ms, "tokens": tokens}))


# --------------------------------------------------------------------------- CPU oracle leg
class OracleSample:
    """The oracle's inputs for chosen sequences of a workload, staged once (not timed)."""

    def __init__(self, w, seqs):
        self.w = w
        self.kp, self.vp, self.bt, self.seqs = w.compact_host_pool(seqs)
        q, k, v = w.new_qkv()
        ind = w.q_indptr
        rows = np.concatenate([np.arange(ind[s], ind[s + 1]) for s in self.seqs] + [np.zeros(0, np.int64)]).astype(np.int64)
        self.q, self.k, self.v = q[rows], k[rows], v[rows]
        self.cached, self.new = w.cached_len[self.seqs], w.new_len[self.seqs]
        if w.decode_steps > 0:
            dq, dk, dv = w.decode_qkv(0)
            self.dq, self.dk, self.dv = dq[self.seqs], dk[self.seqs], dv[self.seqs]

    def step(self):
        """One step of the oracle; returns (seconds, tokens)."""
        from oracle import efim_oracle as orc
        w = self.w
        kp, vp = self.kp.copy(), self.vp.copy()                # the step updates the cache: fresh copy, not timed
        t0 = time.perf_counter()
        q_rot = orc.kv_append(kp, vp, self.bt, self.cached, self.new, self.q, self.k, self.v, w.rope_base)
        orc.append_prefill_attention(q_rot, kp, vp, self.bt, self.cached, self.new, w.num_q_heads)
        tokens = int(self.new.sum())
        if w.decode_steps > 0:
            ctx = (self.cached + self.new).astype(np.int32)
            one = np.ones(len(self.seqs), np.int32)
            q1 = orc.kv_append(kp, vp, self.bt, ctx, one, self.dq, self.dk, self.dv, w.rope_base)
            orc.decode_attention(q1, kp, vp, self.bt, ctx + 1, w.num_q_heads)
            tokens += len(self.seqs)
        return time.perf_counter() - t0, tokens

    def describe(self, tokens):
        every = len(self.seqs) == self.w.batch
        which = "all sequences" if every else f"sequences {self.seqs}"
        return f"{which} of {self.w.name} ({tokens} tokens per step, all heads)"


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def pick_sample(w, budget_flops=3.6e11):
    """Sequences of the workload, shortest first, until ~budget of oracle work."""
    C = w.cached_len.astype(np.int64)
    N = w.new_len.astype(np.int64)
    flops = 4 * w.head_dim * w.num_q_heads * (N * C + N * (N + 1) // 2 + C + N + 1)
    order = np.argsort(flops, kind="stable")
    chosen, tot = [], 0
    for s in order:
        if chosen and tot + flops[s] > budget_flops:
            break
        chosen.append(int(s))
        tot += int(flops[s])
    return sorted(chosen)


def oracle_cfg1_one_thread():
    """The whole of cfg1 (its turn and its 8 decode steps) through the oracle on one thread."""
    from efim_synth import make_workload
    from oracle import efim_oracle as orc
    w = make_workload("cfg1")
    kp, vp, bt, _ = w.compact_host_pool()
    q, k, v = w.new_qkv()

    def run():
        t0 = time.perf_counter()
        q_rot = orc.kv_append(kp, vp, bt, w.cached_len, w.new_len, q, k, v, w.rope_base)
        orc.append_prefill_attention(q_rot, kp, vp, bt, w.cached_len, w.new_len, w.num_q_heads)
        ctx = (w.cached_len + w.new_len).astype(np.int32)
        one = np.ones(w.batch, np.int32)
        for stp in range(w.decode_steps):
            dq, dk, dv = w.decode_qkv(stp)
            q1 = orc.kv_append(kp, vp, bt, ctx, one, dq, dk, dv, w.rope_base)
            ctx = ctx + 1
            orc.decode_attention(q1, kp, vp, bt, ctx, w.num_q_heads)
        return time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            run()
            sec = min(run() for _ in range(3))
        threads = 1
    except Exception:
        run()
        sec = min(run() for _ in range(3))
        threads = oracle_threads()
    tokens = int(w.new_len.sum()) + w.batch * w.decode_steps
    return {"workload": "cfg1", "seconds": sec, "tokens": tokens, "tokens_per_s": tokens / sec, "threads": threads,
            "what": "kv_append + append-prefill of 16 tokens over 240 cached, then 8 decode steps; best of 3"}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step (the same
    sequences the native arm's cpu_baseline leg takes)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from efim_synth import make_workload
    w = make_workload(args.workload, batch=args.batch)
    smp = OracleSample(w, pick_sample(w))
    for _ in range(args.warmup):
        smp.step()
    tot_s, tot_tok = 0.0, 0
    for _ in range(args.steps):
        s, tok = smp.step()
        tot_s += s
        tot_tok += tok
    value = tot_tok / tot_s
    sample = smp.describe(tot_tok // max(args.steps, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_s / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_of(w, max(args.gpus, 1)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- native leg
class TurnRunner:
    """A workload resident on the device and the calls of one step on it."""

    def __init__(self, w, dev, efim):
        import torch
        from efim_synth import pool_fill_torch
        from efim_synth.pool import K_POOL_ID, V_POOL_ID
        self.w, self.dev, self.efim, self.torch = w, dev, efim, torch
        self.cnt = workload_counts(w)
        B, Hq, D = w.batch, w.num_q_heads, w.head_dim
        self.has_decode = w.decode_steps > 0
        self.k_pool = torch.empty(w.pool_shape(), dtype=torch.bfloat16, device=dev)
        self.v_pool = torch.empty(w.pool_shape(), dtype=torch.bfloat16, device=dev)
        pool_fill_torch(self.k_pool, w.seed, K_POOL_ID)
        pool_fill_torch(self.v_pool, w.seed, V_POOL_ID)
        self.cache = efim.Cache(self.k_pool, self.v_pool, Hq)
        self.batch = efim.Batch(w.cached_len, w.new_len, w.block_table, device=dev)
        self.ctx_after = (w.cached_len + w.new_len).astype(np.int32)
        self.rope = efim.Rope(w.rope_base, D, int(self.ctx_after.max()) + w.decode_steps + 2, False, dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.bits = w.new_qkv()
        self.T = self.bits[0].shape[0]
        self.q0, self.k_new, self.v_new = (self.to_dev(x) for x in self.bits)
        self.q = self.q0.clone()                 # rotated in place by every step, restored between steps
        self.out = torch.empty_like(self.q)
        self.ws_p = torch.empty(max(efim.efim_prefill_workspace_bytes(self.cache, self.batch), 256),
                                dtype=torch.uint8, device=dev)
        # The work list depends on the batch's lengths only, not on the layer: planned once per
        # batch (as a model would, then run for every layer) and timed on its own.
        self.plan, self.plan_ms, self.uploaded = None, 0.0, False
        if self.T > 0:
            efim.efim_prefill_plan(self.cache, self.batch)
            t_plan = time.perf_counter()
            for _ in range(10):
                self.plan = efim.efim_prefill_plan(self.cache, self.batch)
            self.plan_ms = (time.perf_counter() - t_plan) / 10 * 1e3
        if self.has_decode:
            self.dbits = w.decode_qkv(0)
            self.dq, self.dk, self.dv = (self.to_dev(x) for x in self.dbits)     # read only (rotated on load)
            self.dout = torch.empty_like(self.dq)
            self.d_ctx = torch.from_numpy(self.ctx_after + 1).to(dev)
            self.max_ctx = int(self.ctx_after.max()) + w.decode_steps
            self.ws_d = torch.empty(max(efim.efim_decode_workspace_bytes(self.cache, B, self.max_ctx), 256),
                                    dtype=torch.uint8, device=dev)
        self.stream = torch.cuda.current_stream()

    def to_dev(self, bits):
        return self.torch.from_numpy(bits.view(np.int16)).to(self.dev).view(self.torch.bfloat16)

    def launches_per_step(self):
        n = 0
        if self.T > 0:
            n += 1 + self.efim.efim_prefill_launch_count(self.cache, self.batch)
        if self.has_decode:
            n += self.efim.efim_decode_launch_count(self.cache, self.w.batch, self.max_ctx)
        return n

    def step(self, marks=None, io=None):
        """The calls of one turn on the current stream; marks = 4 events or None;
        io = another set of input/output tensors (q, k, v, out, dq, dk, dv, dout) or None."""
        efim = self.efim
        q_, k_, v_, out_, dq_, dk_, dv_, dout_ = io if io else (
            self.q, self.k_new, self.v_new, self.out,
            *((self.dq, self.dk, self.dv, self.dout) if self.has_decode else (None,) * 4))
        if marks: marks[0].record(self.stream)
        if self.T > 0:
            efim.efim_kv_append(self.cache, self.batch, self.rope, q_, k_, v_, self.status)
        if marks: marks[1].record(self.stream)
        if self.T > 0:
            efim.efim_append_prefill_attn(self.cache, self.batch, q_, out_, None, 0.0, self.ws_p, self.status,
                                          plan=self.plan, lists_resident=self.uploaded)
            self.uploaded = True                 # the lists stay at the head of ws_p: uploaded once per batch
        if marks: marks[2].record(self.stream)
        if self.has_decode:
            # the generated token's kv_append is fused into the decode kernel
            efim.efim_decode_step(self.cache, self.w.batch, self.d_ctx, self.max_ctx, self.batch.d_block_table,
                                  self.rope, dq_, dk_, dv_, dout_, None, 0.0, self.ws_d, self.status)
        if marks: marks[3].record(self.stream)

    def restore(self, flush):
        """Between timed steps, outside the event pairs: the unrotated q back, L2 evicted."""
        if self.T > 0:
            self.q.copy_(self.q0)
        if flush is not None:
            flush.fill_(1)

    def check_status(self):
        st = int(self.status.item())
        if st != 0:
            raise RuntimeError(f"device status word {st:#x} after the run ({self.w.name})")


def frac_pair(achieved, measured_peak, nominal_peak):
    return {"achieved": achieved, "frac_of_measured": achieved / measured_peak, "frac_of_nominal": achieved / nominal_peak}


def call_records(cnt, seg_ms, peaks, has_decode, decode_tokens=None):
    """Per-call figures of one step from its mean segment times (ms): kv_append, append-prefill, decode."""
    t_app, t_pre, t_dec = seg_ms
    hbm, tc = peaks["hbm_gbs"], peaks["bf16_tflops"]
    rec = {}
    if cnt["new_tokens"] > 0:
        app_bytes = cnt["kv_append_bytes_per_token"] * cnt["new_tokens"]
        rec["kv_append"] = {"ms": t_app, "bytes": app_bytes, "bound": "hbm", "unit": "GB/s",
                            **frac_pair(app_bytes / t_app / 1e6, hbm, NOMINAL["hbm_gbs"]),
                            "note": "q read + rewritten in place, k and v read + written into the pages"}
        intensity = cnt["prefill_flops"] / max(cnt["prefill_kv_bytes"], 1)
        tflops = cnt["prefill_flops"] / t_pre / 1e9
        ceil_meas = min(tc, intensity * hbm / 1e3)
        ceil_nom = min(NOMINAL["bf16_tflops"], intensity * NOMINAL["hbm_gbs"] / 1e3)
        rec["append_prefill"] = {
            "ms": t_pre, "flops": cnt["prefill_flops"], "kv_bytes": cnt["prefill_kv_bytes"],
            "intensity_flop_per_byte": intensity, "bound": "tensor" if intensity * hbm / 1e3 >= tc else "hbm",
            "tflops": tflops, "kv_gbs": cnt["prefill_kv_bytes"] / t_pre / 1e6,
            "ceiling_tflops_measured": ceil_meas, "ceiling_tflops_nominal": ceil_nom,
            "frac_of_measured": tflops / ceil_meas, "frac_of_nominal": tflops / ceil_nom,
            "frac_of_measured_tensor_peak": tflops / tc, "frac_of_nominal_tensor_peak": tflops / NOMINAL["bf16_tflops"],
            "frac_of_measured_sustained_tensor_peak": tflops / peaks.get("bf16_tflops_sustained", tc),
            "note": "ceiling = min(tensor peak, intensity x HBM bandwidth)"}
    if has_decode:
        rec["decode_step"] = {"ms": t_dec, "bytes": cnt["decode_kv_bytes"], "bound": "hbm", "unit": "GB/s",
                              **frac_pair(cnt["decode_kv_bytes"] / t_dec / 1e6, hbm, NOMINAL["hbm_gbs"]),
                              "note": "kv_append of the generated token fused into the decode kernel"}
    return rec


def time_steps(torch, runner, flush, reps, warmup):
    """`reps` steps with an L2 flush before each; returns (per-step ms, mean segment ms, wall window)."""
    def ev():
        return torch.cuda.Event(enable_timing=True)
    for _ in range(warmup):
        runner.restore(flush)
        runner.step()
    torch.cuda.synchronize()
    marks = [[ev() for _ in range(4)] for _ in range(reps)]
    t0 = time.time()
    for i in range(reps):
        runner.restore(flush)                  # evict L2 between timed steps (outside the event pairs)
        runner.step(marks[i])
    torch.cuda.synchronize()
    t1 = time.time()
    seg = np.array([[m[j].elapsed_time(m[j + 1]) for j in range(3)] for m in marks])
    step_ms = np.array([m[0].elapsed_time(m[3]) for m in marks])
    return step_ms, seg.mean(axis=0), (t0, t1)


def measure_config(name, dev, efim, torch, flush, peaks, sampler, min_region_s=0.5):
    """One record of the `configs` block: a full-size workload timed for at least min_region_s."""
    from efim_synth import make_workload
    w = make_workload(name)
    r = TurnRunner(w, dev, efim)
    cnt = r.cnt
    if name == "cfg5":
        rec = measure_decode_loop(r, torch, peaks, sampler, min_region_s)
    else:
        probe, _, _ = time_steps(torch, r, flush, 5, 3)
        reps = int(min(max(20, np.ceil(min_region_s * 1e3 / max(float(probe.mean()), 1e-3))), 20000))
        step_ms, seg, window = time_steps(torch, r, flush, reps, 3)
        r.check_status()
        tokens = cnt["new_tokens"] + cnt["decode_tokens"]
        rec = {"workload": name, "reps": reps, "timed_region_s": float(step_ms.sum()) / 1e3,
               "ms_per_step": float(step_ms.mean()), "ms_per_step_min": float(step_ms.min()),
               "ms_per_step_median": float(np.median(step_ms)),
               "tokens_per_step": tokens, "tokens_per_s": tokens / (float(step_ms.mean()) / 1e3),
               "prefill_plan_host_ms": r.plan_ms, "gpu_launches_per_step": r.launches_per_step(),
               "calls": call_records(cnt, [float(x) for x in seg], peaks, r.has_decode),
               "l2": "256 MiB flush before every step", "clocks": sampler.window(*window)}
    rec["shape"] = {k: v for k, v in config_of(w, 1).items() if k not in ("l2", "parallelism", "workload")}
    del r
    torch.cuda.empty_cache()
    return rec


def measure_decode_loop(r, torch, peaks, sampler, min_region_s):
    """cfg5: the 64-step decode loop (each step appends one token per sequence, fused into the
    decode kernel, then attends over the grown context), timed whole and per step."""
    w, efim = r.w, r.efim
    B, steps = w.batch, w.decode_steps
    ctx0 = w.cached_len.astype(np.int32)
    d_ctx = [torch.from_numpy(ctx0 + t + 1).to(r.dev) for t in range(steps)]
    qkv = []
    for t in range(min(steps, 4)):             # four sets of draws, cycled: the values do not affect the time
        qkv.append(tuple(r.to_dev(x) for x in w.decode_qkv(t)))
    out = torch.empty_like(qkv[0][0])

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def loop(marks=None):
        for t in range(steps):
            q, k, v = qkv[t % len(qkv)]
            if marks: marks[t].record(r.stream)
            efim.efim_decode_step(r.cache, B, d_ctx[t], r.max_ctx, r.batch.d_block_table, r.rope, q, k, v, out, None,
                                  0.0, r.ws_d, r.status)
        if marks: marks[steps].record(r.stream)
    loop()
    torch.cuda.synchronize()
    probe = [ev() for _ in range(steps + 1)]
    loop(probe)
    torch.cuda.synchronize()
    loop_ms = probe[0].elapsed_time(probe[steps])
    n_loops = int(max(2, np.ceil(min_region_s * 1e3 / loop_ms)))
    all_marks = [[ev() for _ in range(steps + 1)] for _ in range(n_loops)]
    t0 = time.time()
    for m in all_marks:
        loop(m)
    torch.cuda.synchronize()
    t1 = time.time()
    r.check_status()
    whole = np.array([m[0].elapsed_time(m[steps]) for m in all_marks])
    per_step = np.array([[m[t].elapsed_time(m[t + 1]) for t in range(steps)] for m in all_marks])
    D, Hkv = w.head_dim, w.num_kv_heads
    bytes_per_step = np.array([int(4 * D * Hkv * (ctx0.astype(np.int64) + t + 1).sum()) for t in range(steps)])
    gbs = float(bytes_per_step.sum()) / (float(whole.mean()) / 1e3) / 1e9
    return {"workload": w.name, "reps": n_loops, "steps_per_loop": steps, "timed_region_s": float(whole.sum()) / 1e3,
            "loop_ms": float(whole.mean()), "loop_ms_min": float(whole.min()),
            "ms_per_step": float(per_step.mean()), "ms_per_step_min": float(per_step.min()),
            "ms_per_step_max": float(per_step.max()),
            "tokens_per_step": B, "tokens_per_s": B * steps / (float(whole.mean()) / 1e3),
            "gpu_launches_per_step": efim.efim_decode_launch_count(r.cache, B, r.max_ctx),
            "calls": {"decode_step": {"ms": float(per_step.mean()), "bytes": int(bytes_per_step.mean()), "bound": "hbm",
                                      "unit": "GB/s", **frac_pair(gbs, peaks["hbm_gbs"], NOMINAL["hbm_gbs"]),
                                      "note": "kv_append of the generated token fused into the decode kernel; "
                                              "plain launches, no CUDA graph"}},
            "l2": "none needed: 19.5 GB of K/V per step", "clocks": sampler.window(t0, t1)}


def run_native(args):
    import torch
    import paper_2505_21889_b200 as efim
    from paper_2505_21889_b200 import build as efim_build
    from efim_synth import make_workload

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        torch.cuda.set_device(0)
    dev = torch.device("cuda", torch.cuda.current_device())
    if not os.path.exists(efim.library_path()):
        efim_build.build()
    efim.load_library()                       # raises if the CUDA library is missing

    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()                           # before any warm-up: its first line takes a moment
    w = make_workload(args.workload, seed=BASE_SEED[args.workload] + 1000 * rank if rank else None, batch=args.batch)
    r = TurnRunner(w, dev, efim)
    cnt, has_decode = r.cnt, r.has_decode
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = r.stream

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # End to end: every step's q/k/v come from pinned host memory and its outputs go back to
    # pinned host memory.  The copies of step i+1 and i-1 run on their own streams beside the
    # kernels of step i (two sets of device and host buffers), as a serving loop would do it;
    # all of them lie inside the timed region.
    def pinned(bits):
        return torch.from_numpy(bits.view(np.int16)).pin_memory()
    h_ins = tuple(pinned(x) for x in r.bits) + (tuple(pinned(x) for x in r.dbits) if has_decode else ())
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    io_sets, h_outs = [], []
    for _ in range(2):
        d = (torch.empty_like(r.q), torch.empty_like(r.k_new), torch.empty_like(r.v_new), torch.empty_like(r.out))
        d += (torch.empty_like(r.dq), torch.empty_like(r.dk), torch.empty_like(r.dv), torch.empty_like(r.dout)) \
            if has_decode else (None,) * 4
        io_sets.append(d)
        h_outs.append((torch.empty(r.out.shape, dtype=torch.int16).pin_memory(),
                       torch.empty(r.dout.shape, dtype=torch.int16).pin_memory() if has_decode else None))

    def e2e_run(n):
        """n pipelined steps; returns (start, end) events that bracket all copies and kernels."""
        t0, t1 = ev(), ev()
        in_done = [None, None]
        comp_done = [None, None]
        out_done = [None, None]
        s_in.wait_stream(stream)
        s_out.wait_stream(stream)
        t0.record(stream)
        s_in.wait_event(t0)
        for i in range(n):
            b = i & 1
            io = io_sets[b]
            with torch.cuda.stream(s_in):
                if comp_done[b] is not None:
                    s_in.wait_event(comp_done[b])          # the kernels of step i-2 are done with these inputs
                dsts = (io[0], io[1], io[2]) + ((io[4], io[5], io[6]) if has_decode else ())
                for dst, src in zip(dsts, h_ins):
                    dst.copy_(src.view(torch.bfloat16), non_blocking=True)
                in_done[b] = ev(); in_done[b].record(s_in)
            stream.wait_event(in_done[b])
            if out_done[b] is not None:
                stream.wait_event(out_done[b])             # step i-2's outputs have left the device
            r.step(io=io)
            comp_done[b] = ev(); comp_done[b].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[b])
                h_outs[b][0].copy_(io[3].view(torch.int16), non_blocking=True)
                if has_decode:
                    h_outs[b][1].copy_(io[7].view(torch.int16), non_blocking=True)
                out_done[b] = ev(); out_done[b].record(s_out)
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)
        t1.record(stream)
        return t0, t1

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- device-resident timing: W warm-up steps, then exactly K timed steps
    warm = max(args.warmup, 3)
    for _ in range(warm):
        r.restore(flush)
        r.step()
    barrier()
    sampler.wait_first()
    marks = [[ev() for _ in range(4)] for _ in range(args.steps)]
    wall0 = time.time()
    for i in range(args.steps):
        r.restore(flush)                       # evict L2 between timed steps (outside the event pairs)
        r.step(marks[i])
    barrier()
    wall1 = time.time()
    seg = np.array([[m[j].elapsed_time(m[j + 1]) for j in range(3)] for m in marks])     # ms
    step_ms = np.array([m[0].elapsed_time(m[3]) for m in marks])
    local_ms = float(step_ms.sum())
    # ---------------- end to end (host buffers)
    e2e_run(3)
    barrier()
    e2e_t0, e2e_t1 = e2e_run(args.steps)
    barrier()
    wall2 = time.time()
    e2e_ms = float(e2e_t0.elapsed_time(e2e_t1))
    r.check_status()

    tokens_per_step = cnt["new_tokens"] + cnt["decode_tokens"]
    job_ms, job_tokens = aggregate_over_ranks(local_ms, tokens_per_step * args.steps, dist)
    job_e2e_ms, _ = aggregate_over_ranks(e2e_ms, 0, dist)
    if rank != 0:
        sampler.stop()
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    seg_mean = [float(x) for x in seg.mean(axis=0)]
    calls = call_records(cnt, seg_mean, peaks, has_decode)
    t_app, t_pre, t_dec = seg_mean
    breakdown = {
        "kv_append_ms": t_app, "kv_append_gbs": calls["kv_append"]["achieved"] if "kv_append" in calls else None,
        "prefill_plan_host_ms": r.plan_ms,     # once per batch, outside the step (amortised over a model's layers)
        "append_prefill_ms": t_pre,
        "append_prefill_tflops": calls["append_prefill"]["tflops"] if "append_prefill" in calls else None,
        "append_prefill_kv_gbs": calls["append_prefill"]["kv_gbs"] if "append_prefill" in calls else None,
        "decode_ms": t_dec, "decode_fused_append": True,
        "decode_kv_gbs": calls["decode_step"]["achieved"] if has_decode else None,
        "q_rotated_by": "efim_kv_append in place (prefill), the decode kernel on load (efim_decode_step)",
    }
    # dominant call of the step and the roofline that bounds it on this workload
    if t_pre >= t_dec:
        ap = calls["append_prefill"]
        if ap["bound"] == "tensor":
            roof = {"kernel": "efim_append_prefill_attn", "bound": "tensor", "achieved": ap["tflops"],
                    "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "algorithmic": cnt["prefill_flops"]}
        else:
            roof = {"kernel": "efim_append_prefill_attn", "bound": "hbm", "achieved": ap["kv_gbs"],
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "algorithmic": cnt["prefill_kv_bytes"]}
        roof["intensity_flop_per_byte"] = ap["intensity_flop_per_byte"]
    else:
        roof = {"kernel": "efim_decode_step", "bound": "hbm", "achieved": calls["decode_step"]["achieved"],
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "algorithmic": cnt["decode_kv_bytes"]}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["frac_of_nominal"] = roof["achieved"] / (NOMINAL["hbm_gbs"] if roof["bound"] == "hbm" else NOMINAL["bf16_tflops"])
    roof["peak_source"] = peaks["source"]
    roof["traffic"] = recorded_traffic(w.name if args.batch is None else None, roof["kernel"])
    roof["traffic_unit"] = "bytes/launch (ncu dram read+write)"

    h2d = sum(x.numel() for x in h_ins) * 2
    d2h = r.out.numel() * 2 + (r.dout.numel() * 2 if has_decode else 0)
    line = {
        "metric": METRIC, "value": job_tokens / (job_ms / 1e3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warm, "ms_per_step": job_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": config_of(w, world),
        "clocks": sampler.window(wall0, wall1),
        "e2e": {"value": job_tokens / (job_e2e_ms / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "overlap": "copies of steps i+1 and i-1 on their own streams beside the kernels of step i",
                "clocks": sampler.window(wall1, wall2)},
        "gpu_launches": r.launches_per_step() * args.steps,
        "breakdown": breakdown,
        "roofline": roof,
    }
    # free the headline workload before the other full-size ones come in
    del io_sets, h_outs
    launch_note = r.launches_per_step()
    del r
    torch.cuda.empty_cache()

    # ---------------- every full-size config, >= 0.5 s each (rank 0, N = 1 only)
    if world == 1 and not args.no_configs:
        cfgs = {}
        for name in CONFIG_BLOCK:
            cfgs[name] = measure_config(name, dev, efim, torch, flush, peaks, sampler)
        a, b = cfgs["cfg4a"], cfgs["cfg4b"]
        cfgs["cfg4_reuse_vs_recompute"] = {
            "efim_append_ms": a["ms_per_step"], "fim_miss_ms": b["ms_per_step"],
            "time_ratio": b["ms_per_step"] / a["ms_per_step"],
            "attention_time_ratio": b["calls"]["append_prefill"]["ms"] / a["calls"]["append_prefill"]["ms"],
            "algorithmic_attention_work_ratio": b["calls"]["append_prefill"]["flops"] / a["calls"]["append_prefill"]["flops"],
            "token_ratio": b["tokens_per_step"] / a["tokens_per_step"],
            "what": "cfg4a = 128 inc tokens over 8192 cached (EFIM order); cfg4b = 3200 tokens recomputed over "
                    "5120 cached (FIM order misses the suffix); same kernels, same seed"}
        line["configs"] = cfgs
    sampler.stop()

    # ---------------- CPU oracle on a bounded sample (rank 0, N = 1 only)
    if world == 1 and not args.no_cpu_baseline:
        smp = OracleSample(w, pick_sample(w))
        s, tok = smp.step()
        line["cpu_baseline"] = {"value": tok / s, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                "sample": smp.describe(tok) + f", {s:.1f} s",
                                "cfg1_one_thread": oracle_cfg1_one_thread()}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(BASE_SEED))
    ap.add_argument("--batch", type=int, default=None, help="override the sequence count of cfg2/cfg5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="headline workload only")
    ap.add_argument("--selfcheck-ranks", action="store_true",
                    help="run only the rank plumbing (gloo, CPU, stand-in measurement)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # run plainly with --gpus N: start the N ranks here
        sys.exit(relaunch_under_torchrun(sys.argv[1:], args.gpus))
    if args.selfcheck_ranks:
        run_rank_selfcheck(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
