"""The C++/OpenMP twin of the oracle (oracle/kvswap_oracle_omp.cpp, used to time the CPU baseline)
against the numpy oracle, which stays the parity authority: equal selections, group scores and
attention outputs to 1e-12, on config 1, a reduced config 2 and the awkward shapes (ragged tail,
rho = 3, per-head metadata, all-heads scope, M above the group count, an empty selection)."""
import numpy as np
import pytest

from oracle import kvswap_oracle as O
from oracle import omp_twin as T
from paper_2511_11907_b200 import workloads as W


def _layer(wl, meta_heads):
    li = W.make_layer(wl, 0, meta_heads)
    meta = O.project_keys(li.K, li.proj, meta_heads, "f16" if wl.meta_dtype == W.F16 else "f32")
    return li, meta


CASES = [
    ("config1", W.CONFIGS[1], 1, "kv_head"),
    ("config2-reduced", W.CONFIGS[2].reduced("c2r", n_ctx=4096 + 5, top_k=64, calib_rows=1024), 1, "kv_head"),
    ("per-head", W.CONFIGS[2].reduced("c2p", n_ctx=1024 + 3, top_k=16, calib_rows=512), 8, "kv_head"),
    ("all-heads", W.CONFIGS[2].reduced("c2a", n_ctx=1024, top_k=16, calib_rows=512), 1, "all_heads"),
    ("rho3-G16", W.CONFIGS[4].reduced("c4r", layers=1, batch=2, n_ctx=2048 + 9, top_k=8, calib_rows=512), 1, "kv_head"),
    ("M-above-NG", W.CONFIGS[1].reduced("c1m", n_ctx=64 + 3, top_k=1000), 1, "kv_head"),
]


@pytest.mark.parametrize("name,wl,meta_heads,scope", CASES, ids=[c[0] for c in CASES])
def test_twin_matches_the_numpy_oracle(name, wl, meta_heads, scope):
    li, meta = _layer(wl, meta_heads)
    idx_ref, R_ref = O.score_select(li.q, li.proj, meta, wl.group_size, wl.top_k, scope)
    idx, R = T.score_select(li.q, li.proj, meta, wl.group_size, wl.top_k, scope)
    assert idx.shape == idx_ref.shape and np.array_equal(idx, idx_ref)
    assert np.abs(R - R_ref).max() <= 1e-12 * max(1.0, np.abs(R_ref).max())
    out_ref, lse_ref = O.attend(li.q, li.K, li.V, idx_ref, wl.group_size, scope)
    out, lse = T.attend(li.q, li.K, li.V, idx_ref, wl.group_size, scope)
    assert np.abs(out - out_ref).max() <= 1e-12
    assert np.abs(lse - lse_ref).max() <= 1e-12


def test_twin_empty_selection_attends_the_tail_only():
    wl = W.CONFIGS[1].reduced("c1e", n_ctx=256 + 3)
    li, _ = _layer(wl, 1)
    S = wl.n_kv_heads
    none = np.empty((wl.batch, S, 0), dtype=np.int32)
    out_ref, lse_ref = O.attend(li.q, li.K, li.V, none, wl.group_size, "kv_head")
    out, lse = T.attend(li.q, li.K, li.V, none, wl.group_size, "kv_head")
    assert np.abs(out - out_ref).max() <= 1e-12 and np.abs(lse - lse_ref).max() <= 1e-12


def test_twin_resolves_ties_to_the_lower_index():
    """Duplicate metadata rows give exactly equal group scores: the twin must break the tie as O6 does."""
    rng = np.random.default_rng(3)
    B, Hq, Hkv, d, r, G, N = 1, 4, 2, 16, 8, 2, 64
    q = rng.standard_normal((B, Hq, d)).astype(np.float32)
    proj = rng.standard_normal((Hkv, d, r)).astype(np.float32)
    meta = rng.standard_normal((B, 1, N, r)).astype(np.float32)
    meta[:, :, 20:40] = meta[:, :, 0:20]                    # groups 10..19 repeat groups 0..9
    for M in (3, 7, 16):
        idx_ref, _ = O.score_select(q, proj, meta, G, M, "kv_head")
        idx, _ = T.score_select(q, proj, meta, G, M, "kv_head")
        assert np.array_equal(idx, idx_ref)


def test_twin_uses_threads():
    assert T.threads() >= 1
