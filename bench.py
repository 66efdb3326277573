#!/usr/bin/env python
"""Benchmark of the EFIM per-turn GPU path on synthetic multi-turn infilling batches.

One "step" = one turn of one layer over one ragged batch:
    efim_kv_append(inc tokens) -> efim_append_prefill_attn (planned once per batch)
    -> efim_decode_step (kv_append of 1 generated token per sequence fused with decode attention)
`value` = new tokens (inc + generated) that went through the path per second, inputs
resident in HBM; `e2e` = the same with the step's q/k/v coming from pinned host
memory and the outputs copied back, copies inside the timed region (pipelined over
three streams: the copies of neighbouring steps run beside a step's kernels).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

With N > 1 (torchrun, one rank per GPU) every rank runs its own replica of the
workload (its own pool and seed); there is no exchange inside the path, so the
job value is the sum of tokens over the slowest rank's time (weak scaling).
"""
import argparse
import json
import os
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


class ClockSampler:
    """nvidia-smi clock/throttle samples while the timed region runs (read-only)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


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


# --------------------------------------------------------------------------- CPU oracle leg
def oracle_sample_step(w, seqs, q_bits, k_bits, v_bits, dq, dk, dv):
    """One step of the oracle on the chosen sequences; returns (seconds, tokens)."""
    from oracle import efim_oracle as orc
    kp, vp, bt, seqs = w.compact_host_pool(seqs)           # input staging, not timed
    ind = w.q_indptr
    rows = np.concatenate([np.arange(ind[s], ind[s + 1]) for s in seqs]).astype(np.int64)
    cached, new = w.cached_len[seqs], w.new_len[seqs]
    t0 = time.perf_counter()
    q_rot = orc.kv_append(kp, vp, bt, cached, new, q_bits[rows], k_bits[rows], v_bits[rows], w.rope_base)
    orc.append_prefill_attention(q_rot, kp, vp, bt, cached, new, w.num_q_heads)
    tokens = int(new.sum())
    if w.decode_steps > 0:
        ctx = (cached + new).astype(np.int32)
        one = np.ones(len(seqs), np.int32)
        q1 = orc.kv_append(kp, vp, bt, ctx, one, dq[seqs], dk[seqs], dv[seqs], w.rope_base)
        orc.decode_attention(q1, kp, vp, bt, ctx + 1, w.num_q_heads)
        tokens += len(seqs)
    return time.perf_counter() - t0, tokens


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


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from efim_synth import make_workload
    w = make_workload(args.workload, batch=args.batch)
    q, k, v = w.new_qkv()
    dq, dk, dv = w.decode_qkv(0) if w.decode_steps > 0 else (None, None, None)
    seqs = pick_sample(w, 6e9)
    for _ in range(args.warmup):
        oracle_sample_step(w, seqs, q, k, v, dq, dk, dv)
    tot_s, tot_tok = 0.0, 0
    for _ in range(args.steps):
        s, tok = oracle_sample_step(w, seqs, q, k, v, dq, dk, dv)
        tot_s += s
        tot_tok += tok
    value = tot_tok / tot_s
    sample = f"sequences {seqs} of {w.name} ({tot_tok // max(args.steps, 1)} tokens per step), all heads"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_s / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- native leg
def run_native(args):
    import torch
    import paper_2505_21889_b200 as efim
    from paper_2505_21889_b200 import build as efim_build
    from efim_synth import make_workload, pool_fill_torch
    from efim_synth.pool import K_POOL_ID, V_POOL_ID

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

    base_seed = {"cfg1": 0, "cfg2": 2, "cfg3": 3, "cfg4a": 4, "cfg4b": 4, "cfg4b_3072": 4, "cfg5": 5}[args.workload]
    w = make_workload(args.workload, seed=base_seed + 1000 * rank if rank else None, batch=args.batch)
    cnt = workload_counts(w)
    B, Hq, Hkv, D = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    has_decode = w.decode_steps > 0

    def to_dev(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    k_pool = torch.empty(w.pool_shape(), dtype=torch.bfloat16, device=dev)
    v_pool = torch.empty(w.pool_shape(), dtype=torch.bfloat16, device=dev)
    pool_fill_torch(k_pool, w.seed, K_POOL_ID)
    pool_fill_torch(v_pool, w.seed, V_POOL_ID)
    cache = efim.Cache(k_pool, v_pool, Hq)
    batch = efim.Batch(w.cached_len, w.new_len, w.block_table, device=dev)
    ctx_after = (w.cached_len + w.new_len).astype(np.int32)
    max_pos = int(ctx_after.max()) + 2
    rope = efim.Rope(w.rope_base, D, max_pos, False, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    qb, kb, vb = w.new_qkv()
    T = qb.shape[0]
    # pinned host copies (the e2e leg reads these) and device-resident inputs
    h_q = torch.from_numpy(qb.view(np.int16)).pin_memory()
    h_k = torch.from_numpy(kb.view(np.int16)).pin_memory()
    h_v = torch.from_numpy(vb.view(np.int16)).pin_memory()
    q0, k_new, v_new = to_dev(qb), to_dev(kb), to_dev(vb)
    q = q0.clone()
    out = torch.empty_like(q)
    h_out = torch.empty(out.shape, dtype=torch.int16).pin_memory()
    ws_p = torch.empty(max(efim.efim_prefill_workspace_bytes(cache, batch), 256), dtype=torch.uint8, device=dev)
    # The work list depends on the batch's lengths only, not on the layer: planned once per
    # batch (as a model would, then run for every layer) and timed on its own.
    plan = None
    uploaded = [False]
    plan_ms = 0.0
    if T > 0:
        efim.efim_prefill_plan(cache, batch)
        t_plan = time.perf_counter()
        for _ in range(10):
            plan = efim.efim_prefill_plan(cache, batch)
        plan_ms = (time.perf_counter() - t_plan) / 10 * 1e3
    if has_decode:
        dqb, dkb, dvb = w.decode_qkv(0)
        h_dq = torch.from_numpy(dqb.view(np.int16)).pin_memory()
        h_dk = torch.from_numpy(dkb.view(np.int16)).pin_memory()
        h_dv = torch.from_numpy(dvb.view(np.int16)).pin_memory()
        dq0, dk, dv = to_dev(dqb), to_dev(dkb), to_dev(dvb)
        dq = dq0.clone()
        dout = torch.empty_like(dq)
        h_dout = torch.empty(dout.shape, dtype=torch.int16).pin_memory()
        dec_batch = efim.Batch(ctx_after, np.ones(B, np.int32), batch.d_block_table, device=dev)
        d_ctx = torch.from_numpy(ctx_after + 1).to(dev)
        max_ctx = int(ctx_after.max()) + 1
        dec_ws_bytes = efim.efim_decode_workspace_bytes(cache, B, max_ctx)
        ws_d = torch.empty(max(dec_ws_bytes, 256), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(marks=None, io=None):
        """The four calls of one turn on the current stream; marks = 5 events or None;
        io = another set of input/output tensors (q, k, v, out, dq, dk, dv, dout) or None."""
        q_, k_, v_, out_, dq_, dk_, dv_, dout_ = io if io else (
            q, k_new, v_new, out, *((dq, dk, dv, dout) if has_decode else (None,) * 4))
        if marks: marks[0].record(stream)
        efim.efim_kv_append(cache, batch, rope, q_, k_, v_, status)
        if marks: marks[1].record(stream)
        efim.efim_append_prefill_attn(cache, batch, q_, out_, None, 0.0, ws_p, status, plan=plan,
                                      lists_resident=uploaded[0])
        uploaded[0] = True                       # the lists stay at the head of ws_p: uploaded once per batch
        if marks: marks[2].record(stream)
        if marks: marks[3].record(stream)
        if has_decode:
            # the generated token's kv_append is fused into the decode kernel
            efim.efim_decode_step(cache, B, d_ctx, max_ctx, batch.d_block_table, rope, dq_, dk_, dv_, dout_, None, 0.0,
                                  ws_d, status)
        if marks: marks[4].record(stream)

    def reset_inputs():
        q.copy_(q0)
        if has_decode:
            dq.copy_(dq0)
        flush.fill_(1)                         # evict L2 between timed steps

    # End to end: every step's q/k/v come from pinned host memory and its outputs go back to
    # pinned host memory.  The copies of step i+1 and i-1 run on their own streams beside the
    # kernels of step i (two sets of device and host buffers), as a serving loop would do it;
    # all of them lie inside the timed region.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    io_sets, h_outs = [], []
    for _ in range(2):
        d = (torch.empty_like(q), torch.empty_like(k_new), torch.empty_like(v_new), torch.empty_like(out))
        d += (torch.empty_like(dq), torch.empty_like(dk), torch.empty_like(dv), torch.empty_like(dout)) \
            if has_decode else (None,) * 4
        io_sets.append(d)
        h_outs.append((torch.empty(out.shape, dtype=torch.int16).pin_memory(),
                       torch.empty(dout.shape, dtype=torch.int16).pin_memory() if has_decode else None))
    h_ins = (h_q, h_k, h_v) + ((h_dq, h_dk, h_dv) if has_decode else ())

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
                for dst, src in zip((io[0], io[1], io[2], io[4], io[5], io[6]), h_ins):
                    dst.copy_(src.view(torch.bfloat16), non_blocking=True)
                in_done[b] = ev(); in_done[b].record(s_in)
            stream.wait_event(in_done[b])
            if out_done[b] is not None:
                stream.wait_event(out_done[b])             # step i-2's outputs have left the device
            step(io=io)
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

    # launches of our kernels per step, as the library plans them
    launches = 1 + efim.efim_prefill_launch_count(cache, batch)
    if has_decode:
        launches += efim.efim_decode_launch_count(cache, B, max_ctx)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- device-resident timing
    for _ in range(max(args.warmup, 3)):
        reset_inputs()
        step()
    barrier()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    marks = [[ev() for _ in range(5)] for _ in range(args.steps)]
    for i in range(args.steps):
        reset_inputs()
        step(marks[i])
    barrier()
    seg = np.array([[m[j].elapsed_time(m[j + 1]) for j in range(4)] for m in marks])     # ms
    step_ms = np.array([m[0].elapsed_time(m[4]) for m in marks])
    local_ms = float(step_ms.sum())
    # ---------------- end to end (host buffers)
    e2e_run(3)
    barrier()
    e2e_t0, e2e_t1 = e2e_run(args.steps)
    barrier()
    clocks = sampler.stop()
    e2e_ms = float(e2e_t0.elapsed_time(e2e_t1))
    if int(status.item()) != 0:
        raise RuntimeError(f"device status word {int(status.item()):#x} after the run")

    tokens_per_step = cnt["new_tokens"] + cnt["decode_tokens"]
    job_ms, job_tokens = aggregate_over_ranks(local_ms, tokens_per_step * args.steps, dist)
    job_e2e_ms, _ = aggregate_over_ranks(e2e_ms, 0, dist)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    t_app, t_pre, t_app1, t_dec = [float(x) for x in seg.mean(axis=0)]
    kv_bytes = cnt["kv_append_bytes_per_token"] * cnt["new_tokens"]
    breakdown = {
        "kv_append_ms": t_app, "kv_append_gbs": kv_bytes / t_app / 1e6,
        "prefill_plan_host_ms": plan_ms,       # once per batch, outside the step (amortised over a model's layers)
        "append_prefill_ms": t_pre, "append_prefill_tflops": cnt["prefill_flops"] / t_pre / 1e9,
        "append_prefill_kv_gbs": cnt["prefill_kv_bytes"] / t_pre / 1e6,
        "decode_kv_append_ms": t_app1, "decode_ms": t_dec, "decode_fused_append": True,
        "decode_kv_gbs": (cnt["decode_kv_bytes"] / t_dec / 1e6) if has_decode else None,
    }
    # dominant call of the step and the roofline that bounds it on this workload
    intensity = cnt["prefill_flops"] / max(cnt["prefill_kv_bytes"], 1)
    ridge = peaks["bf16_tflops"] * 1e3 / peaks["hbm_gbs"]
    if t_pre >= t_dec:
        if intensity >= ridge:
            roof = {"kernel": "efim_append_prefill_attn", "bound": "tensor",
                    "achieved": breakdown["append_prefill_tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
        else:
            roof = {"kernel": "efim_append_prefill_attn", "bound": "hbm",
                    "achieved": breakdown["append_prefill_kv_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"kernel": "efim_decode_step", "bound": "hbm", "achieved": breakdown["decode_kv_gbs"],
                "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["peak_source"] = peaks["source"]
    roof["traffic"] = recorded_traffic(w.name if args.batch is None else None, roof["kernel"])
    roof["traffic_unit"] = "bytes/launch (ncu dram read+write)"
    roof["algorithmic"] = cnt["prefill_kv_bytes"] if roof["kernel"] == "efim_append_prefill_attn" and roof["bound"] == "hbm" \
        else (cnt["prefill_flops"] if roof["kernel"] == "efim_append_prefill_attn" else cnt["decode_kv_bytes"])
    roof["intensity_flop_per_byte"] = intensity

    # ---------------- CPU oracle on a bounded sample (rank 0, N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        seqs = pick_sample(w)
        dq_b = w.decode_qkv(0) if has_decode else (None, None, None)
        s, tok = oracle_sample_step(w, seqs, qb, kb, vb, *dq_b)
        cpu = {"value": tok / s, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": f"sequences {seqs} of {w.name} ({tok} tokens, all heads), {s:.1f} s"}

    h2d = (h_q.numel() + h_k.numel() + h_v.numel()) * 2
    d2h = h_out.numel() * 2
    if has_decode:
        h2d += (h_dq.numel() + h_dk.numel() + h_dv.numel()) * 2
        d2h += h_dout.numel() * 2
    line = {
        "metric": METRIC, "value": job_tokens / (job_ms / 1e3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": job_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": w.name, "batch": B, "num_q_heads": Hq, "num_kv_heads": Hkv, "head_dim": D,
                   "page_size": w.page_size, "new_tokens": cnt["new_tokens"], "decode_tokens": cnt["decode_tokens"],
                   "cached_tokens": int(w.cached_len.sum()), "pool_pages": w.num_pages,
                   "l2": "256 MiB flush between steps; K/V read per step exceeds L2",
                   "parallelism": f"replicas x{world}"},
        "clocks": clocks,
        "e2e": {"value": job_tokens / (job_e2e_ms / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "overlap": "copies of steps i+1 and i-1 on their own streams beside the kernels of step i"},
        "gpu_launches": launches * args.steps,
        "breakdown": breakdown,
        "roofline": roof,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--batch", type=int, default=None, help="override the sequence count of cfg2/cfg5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
