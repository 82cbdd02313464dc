"""kvswap_decode_step (all layers of one decode step in one call: each layer scored one layer ahead
of its attention, its TopK merged with the previous layer's split-K combine, the low-rank queries
of the layer after it formed in the same launch) gives exactly what the per-layer calls give.  The
per-layer calls themselves are checked against the oracle in test_gpu_parity.py."""
import pytest
import torch

from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import device_workload as DW
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _step_buffers(dw):
    wl, s = dw.wl, dw.shape
    L, B = wl.layers, wl.batch
    out = torch.full((L, B, wl.n_q_heads, wl.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((L, B, wl.n_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    idx = torch.full((L, B, s.n_scopes, wl.top_k), -7, dtype=torch.int32, device="cuda")
    nsel = torch.full((L, B, s.n_scopes), -7, dtype=torch.int32, device="cuda")
    return out, lse, idx, nsel


def _run_case(wl, meta_heads, scope, lookahead=0):
    dw = DW.build(wl, 1 if meta_heads == "joint" else wl.n_kv_heads, scope, walk_steps=1, reserve_bytes=1 << 30)
    assert dw.layers_resident == wl.layers
    ws = rt.alloc_workspace(dw.shape)
    for l in range(wl.layers):
        kv.kvswap_project_keys(dw.shape, dw.K[l], dw.proj[l], dw.meta[l], 0, wl.n_ctx, ws)
    q = dw.q_walk[0]

    # layer by layer through the three public calls
    out_a, lse_a, idx_a, nsel_a = _step_buffers(dw)
    for l in range(wl.layers):
        kv.kvswap_score_select(dw.shape, q[l], dw.proj[l], dw.meta[l], idx_a[l], nsel_a[l], None, ws)
        kv.kvswap_sparse_decode(dw.shape, q[l], dw.K[l], dw.V[l], idx_a[l], nsel_a[l], out_a[l], lse_a[l], ws)
    torch.cuda.synchronize()
    assert kv.kvswap_read_device_status(ws) == 0

    # the whole step in one call
    ws.fill_(0xFF)
    kv.kvswap_workspace_init(ws)
    out_b, lse_b, idx_b, nsel_b = _step_buffers(dw)
    kv.kvswap_decode_step(dw.shape, dw.layer_tables(lookahead), q, out_b, lse_b, idx_b, nsel_b, ws)
    torch.cuda.synchronize()
    assert kv.kvswap_read_device_status(ws) == 0
    assert torch.equal(nsel_a, nsel_b)
    assert torch.equal(idx_a, idx_b)
    assert not torch.isnan(out_b).any()
    assert torch.equal(out_a, out_b)
    assert torch.equal(lse_a, lse_b)

    # the same step with queries and outputs in host memory
    out_c, _, idx_c, nsel_c = _step_buffers(dw)
    q_host = q.cpu().pin_memory()
    out_host = torch.full(out_c.shape, float("nan"), dtype=torch.float32).pin_memory()
    q_dev = torch.zeros_like(q)
    kv.kvswap_decode_step_host(dw.shape, dw.layer_tables(lookahead), q_host, out_host, q_dev, out_c, idx_c, nsel_c, ws)
    torch.cuda.synchronize()
    assert torch.equal(idx_a, idx_c)
    assert torch.equal(out_a.cpu(), out_host)

    # repeated steps
    for _ in range(3):
        kv.kvswap_decode_step(dw.shape, dw.layer_tables(lookahead), q, out_b, lse_b, idx_b, nsel_b, ws)
    torch.cuda.synchronize()
    assert torch.equal(idx_a, idx_b) and torch.equal(out_a, out_b)
    assert kv.kvswap_read_device_status(ws) == 0


def test_single_layer_step():
    wl = W.CONFIGS[2].reduced("cfg2-one", n_ctx=2048 + 7, top_k=32, calib_rows=1024)
    _run_case(wl, "joint", W.SCOPE_KV_HEAD)


def test_decode_step_on_a_side_stream():
    wl = W.CONFIGS[3].reduced("cfg3-side", layers=3, batch=2, n_ctx=2048, top_k=20, calib_rows=1024)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        _run_case(wl, "joint", W.SCOPE_KV_HEAD)


@pytest.mark.parametrize("meta_heads", ["joint", "per_head"])
@pytest.mark.parametrize("scope", [W.SCOPE_KV_HEAD, W.SCOPE_ALL_HEADS])
def test_decode_step_equals_layer_by_layer_calls(meta_heads, scope):
    wl = W.CONFIGS[4].reduced("cfg4-step", layers=5, batch=2, n_ctx=4096 + 11, top_k=24, calib_rows=1024)
    _run_case(wl, meta_heads, scope)


@pytest.mark.parametrize("lookahead", [1, 2, 5, 1000])
def test_decode_step_over_many_layers(lookahead):
    """70 thin layers: the two streams hand over 140 times within one step."""
    wl = W.CONFIGS[3].reduced("cfg3-deep", layers=70, batch=1, n_ctx=1024 + 3, top_k=16, calib_rows=1024,
                              n_q_heads=8, n_kv_heads=2)
    _run_case(wl, "joint", W.SCOPE_KV_HEAD, lookahead)


@pytest.mark.parametrize("meta_heads", ["joint", "per_head"])
def test_decode_step_head_dim_64(meta_heads):
    """d = 64: the merged combine + TopK launch merges 14 rows of partials per CTA, and the low-rank
    queries formed a layer ahead take two 32-channel pieces per head."""
    wl = W.CONFIGS[4].reduced("cfg4-d64", layers=4, batch=3, n_ctx=4096 + 19, top_k=40, calib_rows=1024, head_dim=64)
    _run_case(wl, meta_heads, W.SCOPE_KV_HEAD)


@pytest.mark.parametrize("meta_heads", ["joint", "per_head"])
def test_decode_steps_back_to_back_with_alternating_queries(meta_heads):
    """Steps enqueued without a pause, alternating between two query sets: inside a step the TopK of a
    layer does not wait for the gather before it, the scorer reads queries that the launch before it
    formed, and consecutive steps reuse the same workspace buffers -- every step must still give what
    the per-layer calls give for its queries."""
    wl = W.CONFIGS[5].reduced("cfg5-soak", layers=6, batch=2, n_ctx=16384 + 5, top_k=96, calib_rows=1024, walk_steps=2)
    dw = DW.build(wl, 1 if meta_heads == "joint" else wl.n_kv_heads, W.SCOPE_KV_HEAD, reserve_bytes=1 << 30)
    ws = rt.alloc_workspace(dw.shape)
    for l in range(wl.layers):
        kv.kvswap_project_keys(dw.shape, dw.K[l], dw.proj[l], dw.meta[l], 0, wl.n_ctx, ws)
    refs = []
    for w in range(2):
        out, lse, idx, nsel = _step_buffers(dw)
        q = dw.q_walk[w]
        for l in range(wl.layers):
            kv.kvswap_score_select(dw.shape, q[l], dw.proj[l], dw.meta[l], idx[l], nsel[l], None, ws)
            kv.kvswap_sparse_decode(dw.shape, q[l], dw.K[l], dw.V[l], idx[l], nsel[l], out[l], lse[l], ws)
        refs.append((out, lse, idx, nsel))
    torch.cuda.synchronize()
    assert not torch.equal(refs[0][2], refs[1][2])          # the two query sets select differently
    layers = dw.layer_tables(1)
    bufs = [_step_buffers(dw) for _ in range(4)]
    bad = torch.zeros((), dtype=torch.int64, device="cuda")
    for i in range(120):
        out, lse, idx, nsel = bufs[i % 4]
        kv.kvswap_decode_step(dw.shape, layers, dw.q_walk[i % 2], out, lse, idx, nsel, ws)
        if i % 4 == 3:                                       # four steps back to back, then all four are checked
            for j in range(4):
                got, want = bufs[j], refs[j % 2]
                differs = torch.zeros((), dtype=torch.bool, device="cuda")
                for g, r in zip(got, want):
                    differs |= (g != r).any()
                bad += differs.to(torch.int64)
    torch.cuda.synchronize()
    assert int(bad) == 0
    assert kv.kvswap_read_device_status(ws) == 0


def test_decode_step_fp32_wide_rank_per_head():
    """fp32 everywhere, rank 128 per-head metadata, batch 64 (generic kernels on both streams)."""
    wl = W.CONFIGS[1].reduced("cfg1-wide", layers=6, batch=64, n_ctx=512, rank=128, head_dim=128, n_q_heads=32,
                              n_kv_heads=8, top_k=8, calib_rows=1536)
    _run_case(wl, "per_head", W.SCOPE_KV_HEAD)


def test_decode_step_can_be_captured_in_a_cuda_graph():
    """After a warm-up call (which creates the internal stream and events) the step records into a
    CUDA graph -- the internal stream forks from and joins the capturing stream -- and replays give
    the results of the stream-ordered call."""
    wl = W.CONFIGS[3].reduced("cfg3-graph", layers=4, batch=2, n_ctx=4096 + 5, top_k=32, calib_rows=1024)
    dw = DW.build(wl, 1, W.SCOPE_KV_HEAD, walk_steps=1, reserve_bytes=1 << 30)
    ws = rt.alloc_workspace(dw.shape)
    for l in range(wl.layers):
        kv.kvswap_project_keys(dw.shape, dw.K[l], dw.proj[l], dw.meta[l], 0, wl.n_ctx, ws)
    q = dw.q_walk[0]
    out, lse, idx, nsel = _step_buffers(dw)
    layers = dw.layer_tables()
    kv.kvswap_decode_step(dw.shape, layers, q, out, lse, idx, nsel, ws)
    torch.cuda.synchronize()
    want = (out.clone(), lse.clone(), idx.clone(), nsel.clone())
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        kv.kvswap_decode_step(dw.shape, layers, q, out, lse, idx, nsel, ws, stream=side)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            kv.kvswap_decode_step(dw.shape, layers, q, out, lse, idx, nsel, ws, stream=side)
    torch.cuda.synchronize()
    for t in (out, lse):
        t.fill_(float("nan"))
    idx.fill_(-7)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert kv.kvswap_read_device_status(ws) == 0
    for got, ref in zip((out, lse, idx, nsel), want):
        assert torch.equal(got, ref)
