"""8-bit metadata (KVSWAP_E4M3, the reading of "the precision of the compact cache can be traded",
Sec. 4.1 / 4.2): kvswap_project_keys against the oracle's E4M3 rounding of the exact product, and
kvswap_score_select over the stored bytes against the oracle's predictor on the same stored values
(scores, selection comparator), on every path that writes or reads the format."""
import numpy as np
import pytest
import torch

from oracle import kvswap_oracle as O
from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W
from parity_util import SCOPE_NAME, check_scores, check_selection

pytestmark = pytest.mark.gpu

TABLE = O.e4m3_decode_table()
# position of every finite code in the ascending order of values (-0 and +0 share a position)
_finite = [c for c in range(256) if not np.isnan(TABLE[c])]
_order = sorted(_finite, key=lambda c: (TABLE[c], 0))
RANK = {}
for pos, c in enumerate(sorted(set(TABLE[_finite]))):
    for code in _finite:
        if TABLE[code] == c:
            RANK[code] = pos


def _setup(wl, meta_heads, scope, meta_exp):
    li = W.make_layer(wl, 0, meta_heads)
    shape = rt.shape_for(wl, meta_heads, scope).with_flags(kv.KVSWAP_META_EXP(meta_exp))
    K = rt.to_device(li.K_raw, wl.kv_dtype)
    q = rt.to_device(li.q_raw, wl.q_dtype)
    proj = torch.from_numpy(np.ascontiguousarray(li.proj, dtype=np.float32)).cuda()
    ws = rt.alloc_workspace(shape)
    meta = torch.zeros((wl.batch, meta_heads, wl.n_ctx, wl.rank), dtype=torch.uint8, device="cuda")
    return li, shape, K, q, proj, ws, meta


def _check_codes(codes_gpu, codes_or):
    same = codes_gpu == codes_or
    zero = (np.isin(codes_gpu, (0x00, 0x80))) & (np.isin(codes_or, (0x00, 0x80)))
    ok = same | zero
    assert ok.mean() >= 0.97, f"only {ok.mean():.4f} of the bytes equal the oracle's"
    # the GPU rounds an fp32 sum, the oracle the exact one: where they differ they are neighbours
    bad = np.flatnonzero(~ok.ravel())
    for g, o in zip(codes_gpu.ravel()[bad], codes_or.ravel()[bad]):
        assert abs(RANK[int(g)] - RANK[int(o)]) == 1, (hex(g), hex(o))


CASES = [
    # name, workload, meta_heads, meta_exp
    ("bf16-d128-joint", W.CONFIGS[2].reduced("p8a", n_ctx=1024 + 5, top_k=16, calib_rows=512, meta_dtype=W.E4M3), 1, 2),
    ("bf16-d128-per-head", W.CONFIGS[2].reduced("p8b", n_ctx=512, top_k=16, calib_rows=512, meta_dtype=W.E4M3), 8, 0),
    ("fp32-d64", W.CONFIGS[1].reduced("p8c", n_ctx=300, top_k=8, rank=32, meta_dtype=W.E4M3), 1, 1),
    ("saturating", W.CONFIGS[2].reduced("p8d", n_ctx=256, top_k=8, calib_rows=512, meta_dtype=W.E4M3), 1, -7),
]


@pytest.mark.parametrize("name,wl,meta_heads,meta_exp", CASES, ids=[c[0] for c in CASES])
def test_project_keys_e4m3_against_the_oracle(name, wl, meta_heads, meta_exp):
    li, shape, K, q, proj, ws, meta = _setup(wl, meta_heads, W.SCOPE_KV_HEAD, meta_exp)
    kv.kvswap_project_keys(shape, K, proj, meta, 0, wl.n_ctx, ws)
    torch.cuda.synchronize()
    exact = O.project_keys(li.K, li.proj, meta_heads, "f64")
    _, codes_or = O.e4m3_round(np.ldexp(exact, -meta_exp))
    _check_codes(meta.cpu().numpy(), codes_or)
    if name == "saturating":
        assert (np.abs(TABLE[codes_or]) == 448).any(), "the case is meant to saturate"
    # a short range (a flushed group) takes another kernel: rebuild the last group only
    meta2 = meta.clone()
    G = wl.group_size
    n1 = (wl.n_ctx // G) * G
    meta2[:, :, n1 - G:n1] = 0
    kv.kvswap_project_keys(shape, K, proj, meta2, n1 - G, n1, ws)
    torch.cuda.synchronize()
    _check_codes(meta2.cpu().numpy()[:, :, n1 - G:n1], codes_or[:, :, n1 - G:n1])
    assert torch.equal(meta2[:, :, :n1 - G], meta[:, :, :n1 - G])
    # and without a workspace (no tensor-memory path)
    meta3 = torch.zeros_like(meta)
    kv.kvswap_project_keys(shape, K, proj, meta3, 0, wl.n_ctx, None)
    torch.cuda.synchronize()
    _check_codes(meta3.cpu().numpy(), codes_or)


SEL_CASES = [
    ("G8-joint-kv", dict(group_size=8, n_ctx=4096 + 3, top_k=40), 1, W.SCOPE_KV_HEAD),
    ("G8-joint-all", dict(group_size=8, n_ctx=2048, top_k=40), 1, W.SCOPE_ALL_HEADS),
    ("G8-per-head", dict(group_size=8, n_ctx=2048 + 7, top_k=24), 8, W.SCOPE_KV_HEAD),
    ("G1", dict(group_size=1, n_ctx=777, top_k=50), 1, W.SCOPE_KV_HEAD),
    ("G4", dict(group_size=4, n_ctx=1000 + 2, top_k=30), 1, W.SCOPE_KV_HEAD),
    ("G16", dict(group_size=16, n_ctx=4096 + 40, top_k=20), 1, W.SCOPE_KV_HEAD),
    ("G32", dict(group_size=32, n_ctx=8192 + 31, top_k=10), 1, W.SCOPE_KV_HEAD),
    ("long-row", dict(group_size=8, n_ctx=8 * 9000 + 1, top_k=300), 1, W.SCOPE_KV_HEAD),
]


@pytest.mark.parametrize("name,over,meta_heads,scope", SEL_CASES, ids=[c[0] for c in SEL_CASES])
def test_score_select_over_e4m3_metadata(name, over, meta_heads, scope):
    wl = W.CONFIGS[2].reduced("s8-" + name, batch=2, calib_rows=512, meta_dtype=W.E4M3, **over)
    meta_exp = 1
    li, shape, K, q, proj, ws, meta = _setup(wl, meta_heads, scope, meta_exp)
    kv.kvswap_project_keys(shape, K, proj, meta, 0, wl.n_ctx, ws)
    S, NG = shape.n_scopes, wl.n_ctx // wl.group_size
    idx = torch.full((wl.batch, S, wl.top_k), -7, dtype=torch.int32, device="cuda")
    nsel = torch.full((wl.batch, S), -7, dtype=torch.int32, device="cuda")
    scores = torch.full((wl.batch, S, NG), float("nan"), dtype=torch.float32, device="cuda")
    kv.kvswap_score_select(shape, q, proj, meta, idx, nsel, scores, ws)
    torch.cuda.synchronize()
    assert kv.kvswap_read_device_status(ws) == 0
    stored = TABLE[meta.cpu().numpy()]                                   # the values the GPU wrote, decoded
    idx_or, R = O.score_select(li.q, li.proj, stored, wl.group_size, wl.top_k, SCOPE_NAME[scope], meta_exp=meta_exp)
    q_lr = O.lowrank_query(li.q, li.proj)
    Tabs = O.aggregate(O.head_scores(np.abs(q_lr), np.abs(stored) * 2.0 ** meta_exp, wl.n_kv_heads), wl.n_kv_heads,
                       SCOPE_NAME[scope])
    check_scores(R, scores.cpu().numpy(), Tabs.max(axis=2))
    check_selection(R, idx.cpu().numpy(), nsel.cpu().numpy(), wl.top_k)
    # without the score buffer (scores in the workspace) the selection is the same
    idx2 = torch.full_like(idx, -7)
    kv.kvswap_score_select(shape, q, proj, meta, idx2, nsel, None, ws)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2)


def test_decode_step_with_e4m3_metadata_equals_layer_by_layer_calls():
    from paper_2511_11907_b200 import device_workload as DW
    wl = W.CONFIGS[3].reduced("s8-step", layers=4, batch=2, n_ctx=4096 + 5, top_k=32, calib_rows=512, meta_dtype=W.E4M3)
    dw = DW.build(wl, 1, W.SCOPE_KV_HEAD)
    shape = dw.shape.with_flags(kv.KVSWAP_META_EXP(1))
    ws = rt.alloc_workspace(shape)
    L = wl.layers
    for l in range(L):
        kv.kvswap_project_keys(shape, dw.K[l], dw.proj[l], dw.meta[l], 0, wl.n_ctx, ws)
    S, M = shape.n_scopes, wl.top_k
    q = dw.q_walk[0]
    idx_a = torch.empty((L, wl.batch, S, M), dtype=torch.int32, device="cuda")
    nsel_a = torch.empty((L, wl.batch, S), dtype=torch.int32, device="cuda")
    out_a = torch.empty((L, wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device="cuda")
    idx_b, nsel_b, out_b = torch.empty_like(idx_a), torch.empty_like(nsel_a), torch.empty_like(out_a)
    for l in range(L):
        kv.kvswap_score_select(shape, q[l], dw.proj[l], dw.meta[l], idx_a[l], nsel_a[l], None, ws)
        kv.kvswap_sparse_decode(shape, q[l], dw.K[l], dw.V[l], idx_a[l], nsel_a[l], out_a[l], None, ws)
    kv.kvswap_decode_step(shape, dw.layer_tables(), q, out_b, None, idx_b, nsel_b, ws, None)
    torch.cuda.synchronize()
    assert torch.equal(idx_a, idx_b) and torch.equal(nsel_a, nsel_b) and torch.equal(out_a, out_b)
