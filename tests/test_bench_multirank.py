"""The multi-GPU leg of bench.py shards by replica with no exchange on the data path;
what ranks do share is the timing reduction.  Checked here with two gloo ranks on CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, tokens = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000 * (rank + 1), dist)
    out[rank] = (ms, tokens)
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_over_two_ranks():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
    for rank in range(world):
        ms, tokens = out[rank]
        assert ms == 15.0            # the slowest rank's time
        assert tokens == 3000.0      # all ranks' tokens


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7) == (3.5, 7.0)


def test_workload_counts_match_definitions():
    sys.path.insert(0, ROOT)
    import bench
    from efim_synth import make_workload
    w = make_workload("cfg4a")
    c = bench.workload_counts(w)
    assert c["new_tokens"] == 8 * 128
    pairs = 8 * (128 * 8192 + 128 * 129 // 2)
    assert c["prefill_flops"] == 4 * 128 * 32 * pairs
    assert c["prefill_kv_bytes"] == 4 * 128 * 8 * 8 * (8192 + 128)
    assert c["kv_append_bytes_per_token"] == 4 * 128 * (32 + 16)


def test_plain_run_with_gpus_2_starts_two_ranks():
    """`python bench.py --gpus 2` without a launcher starts the two ranks itself; with
    --selfcheck-ranks they run the rank plumbing on CPU (gloo) with a stand-in measurement."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selfcheck-ranks"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                       # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["ms"] == 15.0 and out["tokens"] == 3000.0


def test_reference_arm_prints_the_contract_line_on_the_native_config():
    import json
    import subprocess
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    out = json.loads([ln for ln in res.stdout.splitlines() if ln.startswith("{")][-1])
    import bench
    from efim_synth import make_workload
    assert out["impl"] == "reference" and out["config"] == bench.config_of(make_workload("cfg1"), 1)
    assert out["e2e"]["value"] == out["value"] and out["cpu_baseline"]["kind"] == "oracle"
    assert out["steps"] == 2 and out["warmup"] == 1 and out["gpu_launches"] == 0
