"""efim_decode_attn_static: the decode entry point for callers that may not allocate
device memory (no cudaMalloc once the KV pool owns the GPU, or code that is only ever
handed input/output pointers).  It must give exactly what efim_decode_attn gives with
a caller workspace, also when called repeatedly, since every call reuses the same
fixed array inside the library and finds the previous call's partials in it.
Collected last on purpose (file name), so a failure here cannot hide other tests."""
import numpy as np
import pytest
import torch

import paper_2505_21889_b200 as efim
from efim_synth import make_workload

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
        efim.efim_decode_attn_static(dw.cache, B, d_ctx, max_ctx, dw.batch.d_block_table, q, got, got_lse, 0.0,
                                     dw.status)
        torch.cuda.synchronize()
        assert int(dw.status.item()) == 0
        g = got.float().cpu().numpy().astype(np.float64)
        wv = want.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert np.abs(g - wv).max() <= H.MAX_ABS_TOL and np.abs(g - wv).mean() <= H.MEAN_ABS_TOL
        assert np.abs(got_lse.cpu().numpy() - want_lse.cpu().numpy()).max() <= H.LSE_TOL


def test_static_scratch_rejects_oversized_requests():
    import tests.gpu_harness as H
    w = make_workload("cfg5", small=True)
    dw = H.DeviceWorkload(w)
    rows = 4096                                   # far more (row, head, chunk) partials than 8 MiB holds
    big_ctx = dw.batch.d_block_table.shape[1] * 16
    assert efim.efim_decode_workspace_bytes(dw.cache, rows, big_ctx) > efim.efim_decode_static_scratch_bytes()
    d_ctx = torch.ones(rows, dtype=torch.int32, device="cuda")
    q = torch.zeros((rows, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(efim.EfimError) as e:
        efim.efim_decode_attn_static(dw.cache, rows, d_ctx, big_ctx, dw.batch.d_block_table, q, torch.empty_like(q))
    assert e.value.code == 4
