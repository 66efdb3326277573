"""efim_decode_attn_static: the decode entry point for callers that may not allocate
device memory (no cudaMalloc once the KV pool owns the GPU, or code that is only ever
handed input/output pointers).  It runs the same plan and kernels as efim_decode_attn, so
it must give the same bits as that call with a caller workspace (and agree with the CPU
oracle), also when called repeatedly, since every call reuses the same fixed array inside
the library and finds the previous call's partials in it; and the caching allocator must
not see it.
Collected last on purpose (file name), so a failure here cannot hide other tests."""
import numpy as np
import pytest
import torch

import paper_2505_21889_b200 as efim
from efim_synth import make_workload
from oracle import efim_oracle as orc

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_twice():
    import tests.gpu_harness as H
    w = make_workload("cfg5", small=True)
    dw = H.DeviceWorkload(w)
    B = w.batch
    ctx_a = w.cached_len.astype(np.int32)
    max_ctx = int(ctx_a.max()) + 8
    need = efim.efim_decode_workspace_bytes(dw.cache, B, max_ctx)
    assert 0 < need <= efim.efim_decode_static_scratch_bytes()      # the case really uses the scratch array
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    kp, vp, bt, _ = w.compact_host_pool()
    # two calls in a row with different queries and lengths: the second one meets the
    # first one's partials in the shared array
    for call, ctx in enumerate([ctx_a, np.maximum(ctx_a - 7 * np.arange(B, dtype=np.int32), 1)]):
        q = H.bits_to_torch(w.decode_qkv(call)[0])
        d_ctx = torch.from_numpy(np.ascontiguousarray(ctx)).cuda()
        want = torch.empty_like(q)
        want_lse = torch.empty((B, w.num_q_heads), dtype=torch.float32, device="cuda")
        efim.efim_decode_attn(dw.cache, B, d_ctx, max_ctx, dw.batch.d_block_table, q, want, want_lse, 0.0, ws,
                              dw.status)
        got = torch.full_like(q, float("nan"))
        got_lse = torch.full_like(want_lse, float("nan"))
        torch.cuda.synchronize()
        # cumulative counts of allocations the caching allocator has served and of segments it
        # has taken from the driver (frees, e.g. by the garbage collector, do not move them)
        def allocations():
            st = torch.cuda.memory_stats()
            return st["allocation.all.allocated"], st["segment.all.allocated"]
        before = allocations()
        efim.efim_decode_attn_static(dw.cache, B, d_ctx, max_ctx, dw.batch.d_block_table, q, got, got_lse, 0.0,
                                     dw.status)
        torch.cuda.synchronize()
        assert allocations() == before
        assert int(dw.status.item()) == 0
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)) and torch.equal(got_lse, want_lse)
        o, lse = orc.decode_attention(H.torch_to_bits(q), kp, vp, bt, ctx, w.num_q_heads)
        H.assert_attn_close(H.torch_to_bits(got), o, f"static decode, call {call}")
        H.assert_lse_close(got_lse.cpu().numpy(), lse, f"static decode, call {call}")


def test_static_scratch_rejects_oversized_requests():
    import tests.gpu_harness as H
    w = make_workload("cfg5", small=True)
    dw = H.DeviceWorkload(w)
    rows, big_ctx = 512, 20000                    # 10 chunks of partials per (row, head): more than 8 MiB holds
    table = torch.zeros((rows, big_ctx // 16), dtype=torch.int32, device="cuda")
    assert efim.efim_decode_workspace_bytes(dw.cache, rows, big_ctx) > efim.efim_decode_static_scratch_bytes()
    d_ctx = torch.ones(rows, dtype=torch.int32, device="cuda")
    q = torch.zeros((rows, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(efim.EfimError) as e:
        efim.efim_decode_attn_static(dw.cache, rows, d_ctx, big_ctx, table, q, torch.empty_like(q))
    assert e.value.code == 4
