"""GPU parity at the full benchmark sizes (configs 3, 4 and 5, one layer each, drawn on the
device exactly as bench.py draws them and launched through the same calls): the oracle cannot
redo a whole layer in seconds, so it recomputes sampled units -- one whole sequence per
configuration, every KV head and every query head of it -- element by element.

Each call is checked on its own inputs: the oracle scores the metadata the GPU produced, and the
attention check feeds both sides the oracle's selection for the sampled sequence."""
import numpy as np
import pytest
import torch

from oracle import kvswap_oracle as O
from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import device_workload as DW
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W
from parity_util import META_NAME, OUT_ATOL, OUT_ATOL_TIGHT, check_scores, check_selection, project_tolerance

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,meta_heads", [(5, "joint"), (4, "joint"), (3, "per_head")])
def test_full_size_layer_sampled_sequence(cfg, meta_heads):
    wl = W.CONFIGS[cfg].reduced(f"cfg{cfg}-one-layer", layers=1, walk_steps=1)
    mh = 1 if meta_heads == "joint" else wl.n_kv_heads
    dw = DW.build(wl, mh, W.SCOPE_KV_HEAD)
    shape = dw.shape
    ws = rt.alloc_workspace(shape)
    K, V, proj, meta, q = dw.K[0], dw.V[0], dw.proj[0], dw.meta[0], dw.q_walk[0, 0]
    b = wl.batch // 2                                            # the sampled sequence

    # ---- kvswap_project_keys: every metadata row of the sampled sequence ---------------------------
    kv.kvswap_project_keys(shape, K, proj, meta, 0, wl.n_ctx, ws)
    torch.cuda.synchronize()
    Kb, Vb = rt.to_host_f32(K[b:b + 1]), rt.to_host_f32(V[b:b + 1])
    qb, projh = rt.to_host_f32(q[b:b + 1]), proj.cpu().numpy()
    meta_gpu = rt.to_host_f32(meta[b:b + 1])
    meta_or = O.project_keys(Kb, projh, mh, META_NAME[wl.meta_dtype])
    err = np.abs(meta_gpu.astype(np.float64) - meta_or.astype(np.float64))
    assert np.all(err <= project_tolerance(Kb, projh, mh, meta_or, wl.meta_dtype)), f"metadata error {err.max():.3e}"
    assert np.mean(meta_gpu != meta_or.astype(np.float32)) < 0.02

    # ---- kvswap_score_select on the GPU's metadata --------------------------------------------------
    S, M = shape.n_scopes, wl.top_k
    idx = torch.empty((wl.batch, S, M), dtype=torch.int32, device="cuda")
    nsel = torch.empty((wl.batch, S), dtype=torch.int32, device="cuda")
    scores = torch.empty((wl.batch, S, shape.n_groups), dtype=torch.float32, device="cuda")
    kv.kvswap_score_select(shape, q, proj, meta, idx, nsel, scores, ws)
    torch.cuda.synchronize()
    q_lr = O.lowrank_query(qb, projh)
    s = O.head_scores(q_lr, meta_gpu, wl.n_kv_heads)
    R = O.pool(O.aggregate(s, wl.n_kv_heads, "kv_head"), wl.group_size)
    absdot = O.aggregate(O.head_scores(np.abs(q_lr), np.abs(meta_gpu.astype(np.float64)), wl.n_kv_heads),
                         wl.n_kv_heads, "kv_head").max(axis=2)
    check_scores(R, scores[b:b + 1].cpu().numpy(), absdot)
    check_selection(R, idx[b:b + 1].cpu().numpy(), nsel[b:b + 1].cpu().numpy(), M)

    # ---- kvswap_sparse_decode: the sampled sequence attends the oracle's selection ----------------------
    idx_o = O.select(R, M)
    idx[b:b + 1] = torch.from_numpy(idx_o.astype(np.int32)).cuda()
    out = torch.empty((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device="cuda")
    lse = torch.empty((wl.batch, wl.n_q_heads), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    # as the benchmark launches it: selection settled before the call; twice, so that the second
    # launch overlaps the first one's tail
    settled = shape.with_flags(kv.KVSWAP_INPUTS_SETTLED)
    out2, lse2 = torch.empty_like(out), torch.empty_like(lse)
    kv.kvswap_sparse_decode(settled, q, K, V, idx, nsel, out2, lse2, ws)
    kv.kvswap_sparse_decode(settled, q, K, V, idx, nsel, out, lse, ws)
    torch.cuda.synchronize()
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
    out_o, lse_o = O.attend(qb, Kb, Vb, idx_o, wl.group_size, "kv_head")
    eo = np.abs(out[b:b + 1].cpu().numpy() - out_o).max()
    el = np.abs(lse[b:b + 1].cpu().numpy() - lse_o).max()
    assert eo <= OUT_ATOL[wl.kv_dtype] and el <= OUT_ATOL[wl.kv_dtype], (eo, el)
    assert eo <= OUT_ATOL_TIGHT[wl.kv_dtype] and el <= OUT_ATOL_TIGHT[wl.kv_dtype], (eo, el)
    assert np.all(np.isfinite(out.cpu().numpy()))                 # every other sequence ran too
    assert kv.kvswap_read_device_status(ws) == 0


@pytest.mark.parametrize("cfg,lookahead", [(5, 0), (5, 1), (4, 0)])
def test_full_size_decode_step_equals_the_per_layer_calls(cfg, lookahead):
    """The call the benchmark times, at its shapes (six layers of the configuration): predictor and
    attention on two streams, settled launches, waits joined per two layers -- and exactly the
    results of the per-layer calls, which the test above ties to the oracle."""
    L = 6
    wl = W.CONFIGS[cfg].reduced(f"cfg{cfg}-six-layers", layers=L, walk_steps=2)
    dw = DW.build(wl, 1, W.SCOPE_KV_HEAD)
    assert dw.layers_resident == L
    shape = dw.shape
    ws = rt.alloc_workspace(shape)
    for l in range(L):
        kv.kvswap_project_keys(shape, dw.K[l], dw.proj[l], dw.meta[l], 0, wl.n_ctx, ws)
    B, S, M = wl.batch, shape.n_scopes, wl.top_k
    mk = lambda: (torch.full((L, B, wl.n_q_heads, wl.head_dim), float("nan"), device="cuda"),
                  torch.full((L, B, wl.n_q_heads), float("nan"), device="cuda"),
                  torch.full((L, B, S, M), -7, dtype=torch.int32, device="cuda"),
                  torch.full((L, B, S), -7, dtype=torch.int32, device="cuda"))
    layers = dw.layer_tables(lookahead)
    for step in range(2):
        q = dw.q_walk[step]
        out_a, lse_a, idx_a, nsel_a = mk()
        for l in range(L):
            kv.kvswap_score_select(shape, q[l], dw.proj[l], dw.meta[l], idx_a[l], nsel_a[l], None, ws)
            kv.kvswap_sparse_decode(shape, q[l], dw.K[l], dw.V[l], idx_a[l], nsel_a[l], out_a[l], lse_a[l], ws)
        out_b, lse_b, idx_b, nsel_b = mk()
        kv.kvswap_decode_step(shape, layers, q, out_b, lse_b, idx_b, nsel_b, ws)
        kv.kvswap_decode_step(shape, layers, q, out_b, lse_b, idx_b, nsel_b, ws)      # back to back, as in the bench
        torch.cuda.synchronize()
        assert kv.kvswap_read_device_status(ws) == 0
        assert torch.equal(idx_a, idx_b) and torch.equal(nsel_a, nsel_b)
        assert torch.equal(out_a, out_b) and torch.equal(lse_a, lse_b)
