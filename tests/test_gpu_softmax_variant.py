"""KVSWAP_SCORE_SOFTMAX (per-head softmax over the context before the head sum) against the oracle.

Tolerance.  The GPU forms each logit in fp32 (relative error ~ sqrt(r) 2^-24) and exponentiates it;
an absolute logit error e becomes a relative weight error e ln 2, so with base-2 logits of
magnitude up to ~60 the weights carry up to ~3e-5 relative error where the raw-logit predictor
carries 1e-5.  Group scores are therefore compared to 1e-4 relative (+1e-7), and the selection's
tie band is 1e-4 of the threshold score instead of 1e-5."""
import numpy as np
import pytest
import torch

from oracle import kvswap_oracle as O
from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W
from parity_util import META_NAME, SCOPE_NAME, DeviceLayer, check_selection
from test_gpu_parity import EDGE

pytestmark = pytest.mark.gpu

KV, ALL = W.SCOPE_KV_HEAD, W.SCOPE_ALL_HEADS


def _check(wl, meta_heads, scope):
    li = W.make_layer(wl, 0, meta_heads)
    dl = DeviceLayer(li, scope)
    dl.poison()
    meta_or = O.project_keys(li.K, li.proj, meta_heads, META_NAME[wl.meta_dtype])
    dl.set_meta(meta_or)
    shape = dl.shape.with_flags(kv.KVSWAP_SCORE_SOFTMAX)
    kv.kvswap_score_select(shape, dl.q, dl.proj, dl.meta, dl.idx, dl.nsel, dl.scores, dl.ws)
    torch.cuda.synchronize()
    idx_o, R = O.score_select(li.q, li.proj, meta_or, wl.group_size, wl.top_k, SCOPE_NAME[scope], head_softmax=True)
    NG = R.shape[2]
    Rg = dl.scores.cpu().numpy().reshape(-1)[:R.size].reshape(R.shape)
    assert np.all(np.isfinite(Rg)) and (Rg.size == 0 or Rg.min() >= 0.0)
    assert np.all(np.abs(Rg - R) <= 1e-4 * R + 1e-7), float(np.abs(Rg - R).max())
    idx, nsel = dl.idx.cpu().numpy(), dl.nsel.cpu().numpy()
    check_selection(R, idx, nsel, wl.top_k, select_band=1e-4)
    Mp = min(wl.top_k, NG)
    assert np.array_equal(idx[:, :, :Mp], O.select(Rg.astype(np.float64), wl.top_k))    # top-M' of its own scores
    # the variant feeds the same attention: the step's second call is unchanged
    idx2 = torch.full_like(dl.idx, -7)
    kv.kvswap_score_select(shape, dl.q, dl.proj, dl.meta, idx2, dl.nsel, None, dl.ws)  # scores in the workspace
    torch.cuda.synchronize()
    assert torch.equal(idx2, dl.idx)
    assert kv.kvswap_read_device_status(dl.ws) == 0


@pytest.mark.parametrize("meta_heads", ["joint", "per_head"])
@pytest.mark.parametrize("scope", [KV, ALL])
def test_softmax_variant_config1_and_config2(meta_heads, scope):
    for wl in (W.CONFIGS[1], W.CONFIGS[2].reduced("cfg2-soft", n_ctx=4096 + 5)):
        _check(wl, 1 if meta_heads == "joint" else wl.n_kv_heads, scope)


@pytest.mark.parametrize("cfg", [3, 4, 5])
def test_softmax_variant_reduced_configs(cfg):
    wl = W.REDUCED[cfg]
    _check(wl, 1, KV)
    _check(wl, wl.n_kv_heads, KV)


@pytest.mark.parametrize("name", ["group_size_odd", "group_size_twelve", "context_shorter_than_a_group", "ragged_tail",
                                  "gqa_ratio_three", "many_kv_heads", "top_k_covers_everything", "rank_24_fp32",
                                  "bf16_rank_128", "f16meta_group_32", "f16meta_twelve_scopes", "bf16_gqa_ratio_8",
                                  "several_tiles", "exactly_one_group"])
def test_softmax_variant_edge_cases(name):
    wl = EDGE[name]
    _check(wl, 1, KV)
    _check(wl, wl.n_kv_heads, ALL)


def test_softmax_variant_in_the_decode_step():
    """The flag reaches the predictor inside kvswap_decode_step: same selections as the per-layer call."""
    from paper_2511_11907_b200 import device_workload as DW
    wl = W.CONFIGS[3].reduced("cfg3-soft-step", layers=3, batch=2, n_ctx=2048 + 3, top_k=24, calib_rows=1024)
    dw = DW.build(wl, 1, KV, walk_steps=1, reserve_bytes=1 << 30)
    shape = dw.shape.with_flags(kv.KVSWAP_SCORE_SOFTMAX)
    ws = rt.alloc_workspace(shape)
    L, B, S, M = wl.layers, wl.batch, shape.n_scopes, wl.top_k
    for l in range(L):
        kv.kvswap_project_keys(shape, dw.K[l], dw.proj[l], dw.meta[l], 0, wl.n_ctx, ws)
    q = dw.q_walk[0]
    idx_a = torch.full((L, B, S, M), -7, dtype=torch.int32, device="cuda")
    nsel_a = torch.full((L, B, S), -7, dtype=torch.int32, device="cuda")
    for l in range(L):
        kv.kvswap_score_select(shape, q[l], dw.proj[l], dw.meta[l], idx_a[l], nsel_a[l], None, ws)
    idx_raw = torch.full_like(idx_a, -7)
    kv.kvswap_score_select(dw.shape, q[0], dw.proj[0], dw.meta[0], idx_raw[0], nsel_a[0], None, ws)
    out = torch.empty((L, B, wl.n_q_heads, wl.head_dim), device="cuda")
    idx_b, nsel_b = torch.full_like(idx_a, -7), torch.full_like(nsel_a, -7)
    kv.kvswap_decode_step(shape, dw.layer_tables(), q, out, None, idx_b, nsel_b, ws)
    torch.cuda.synchronize()
    assert torch.equal(idx_a, idx_b) and torch.isfinite(out).all()
    assert not torch.equal(idx_raw[0], idx_a[0])              # and it is a different predictor


def _tc(**kw):
    """A workload on the tensor-core path of the variant: joint fp16 metadata, r = 32, H_q <= 32."""
    base = dict(layers=1, batch=2, n_ctx=8 * 150 + 5, n_q_heads=8, n_kv_heads=2, head_dim=128, rank=32, group_size=8,
                top_k=20, kv_dtype=W.BF16, meta_dtype=W.F16, q_dtype=W.BF16, calib_rows=512)
    base.update(kw)
    return W.Workload("soft-tc", 1, **base)


@pytest.mark.parametrize("name,wl,scope", [
    ("one_head_per_scope", _tc(n_q_heads=8, n_kv_heads=8), KV),
    ("two_heads_per_scope", _tc(n_q_heads=16, n_kv_heads=8), KV),
    ("eight_heads_per_scope", _tc(n_q_heads=32, n_kv_heads=4), KV),
    ("sixteen_heads_per_scope", _tc(n_q_heads=32, n_kv_heads=2), KV),
    ("thirty_two_heads_per_scope", _tc(n_q_heads=32, n_kv_heads=1), KV),
    ("five_heads_per_scope", _tc(n_q_heads=10, n_kv_heads=2), KV),
    ("three_heads_all_heads_scope", _tc(n_q_heads=24, n_kv_heads=8), ALL),
    ("group_of_one", _tc(group_size=1, n_ctx=900, top_k=64), KV),
    ("group_of_two", _tc(group_size=2, n_ctx=2 * 601 + 1, top_k=33), KV),
    ("group_of_four_five_heads", _tc(group_size=4, n_q_heads=10, n_kv_heads=2, n_ctx=4 * 300 + 3), KV),
    ("group_of_sixteen", _tc(group_size=16, n_ctx=16 * 90 + 9, top_k=11), KV),
    ("group_of_twelve", _tc(group_size=12, n_ctx=12 * 100 + 7, top_k=11), KV),
    ("several_chunks", _tc(batch=1, n_ctx=8 * 700 + 3, top_k=100), KV),
    ("one_group_only", _tc(n_ctx=8, top_k=4), KV),
], ids=lambda x: x if isinstance(x, str) else None)
def test_softmax_variant_tensor_core_shapes(name, wl, scope):
    _check(wl, 1, scope)
