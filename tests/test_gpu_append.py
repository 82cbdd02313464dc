"""kvswap_append_kv against the oracle (Sec. 4.4.1): a context grows token by token inside a K/V
store with spare rows; the rolling-buffer tail is attended at once, a completed group is flushed
into the compact cache, and the predictor and the attention over the grown context match the
oracle's at every checked length."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import kvswap_oracle as O
from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W
from parity_util import (META_NAME, OUT_ATOL_TIGHT, SCOPE_NAME, check_scores, check_selection, oracle_score_parts,
                         project_tolerance)

pytestmark = pytest.mark.gpu

KV, ALL = W.SCOPE_KV_HEAD, W.SCOPE_ALL_HEADS
_TD = {W.F32: torch.float32, W.BF16: torch.bfloat16, W.F16: torch.float16}


def _prefix(li, n):
    """The layer's inputs cut to the first n tokens."""
    return dataclasses.replace(li, wl=li.wl.reduced("prefix", n_ctx=n), K=li.K[:, :, :n], V=li.V[:, :, :n],
                               K_raw=li.K_raw[:, :, :n], V_raw=li.V_raw[:, :, :n])


def _grow_and_check(wl, n0, meta_heads, scope, check_at):
    """wl.n_ctx is the capacity and the final length; the device store starts with n0 tokens."""
    li = W.make_layer(wl, 0, meta_heads)
    B, Hkv, Nf, d, r, G = wl.batch, wl.n_kv_heads, wl.n_ctx, wl.head_dim, wl.rank, wl.group_size
    K_all, V_all = rt.to_device(li.K_raw, wl.kv_dtype), rt.to_device(li.V_raw, wl.kv_dtype)
    q = rt.to_device(li.q_raw, wl.q_dtype)
    proj = torch.from_numpy(np.ascontiguousarray(li.proj, dtype=np.float32)).cuda()
    K = torch.full_like(K_all, float("nan"))
    V = torch.full_like(V_all, float("nan"))
    K[:, :, :n0], V[:, :, :n0] = K_all[:, :, :n0], V_all[:, :, :n0]
    meta = torch.full((B, meta_heads, Nf, r), float("nan"), dtype=_TD[wl.meta_dtype], device="cuda")
    strides = dict(kv_strides=(Hkv * Nf * d, Nf * d, d), meta_strides=(meta_heads * Nf * r, Nf * r, r))

    def shape_at(n):
        return rt.shape_for(wl, meta_heads, scope, n_ctx=n, **strides)

    ws = rt.alloc_workspace(shape_at(Nf))
    if n0 >= G:                                              # prefill: the complete groups of the first n0 tokens
        kv.kvswap_project_keys(shape_at(n0), K, proj, meta, 0, n0 // G * G, ws)
    idx, nsel = rt.alloc_selection(shape_at(Nf))
    out, lse = rt.alloc_output(shape_at(Nf))
    S = shape_at(Nf).n_scopes
    scores = torch.empty((B, S, Nf // G), dtype=torch.float32, device="cuda")

    # The oracle's append (O8) is stepped beside the device, token by token, from the same start.
    K_o, V_o = li.K[:, :, :n0].copy(), li.V[:, :, :n0].copy()
    meta_o = O.project_keys(K_o[:, :, :n0 // G * G], li.proj, meta_heads, META_NAME[wl.meta_dtype])
    tol = project_tolerance(li.K, li.proj, meta_heads, O.project_keys(li.K, li.proj, meta_heads, META_NAME[wl.meta_dtype]),
                            wl.meta_dtype)
    for n in range(n0, Nf):
        flushed = kv.kvswap_append_kv(shape_at(n), K_all[:, :, n].contiguous(), V_all[:, :, n].contiguous(), K, V,
                                      proj, meta)
        K_o, V_o, meta_o, flushed_o = O.append_kv(K_o, V_o, meta_o, li.K[:, :, n], li.V[:, :, n], li.proj, G,
                                                  META_NAME[wl.meta_dtype])
        assert flushed == flushed_o
        n1 = n + 1
        if n1 not in check_at:
            continue
        torch.cuda.synchronize()
        # ---- the store and the compact cache against the oracle's ---------------------------------------
        assert K_o.shape[2] == n1 and meta_o.shape[2] == n1 // G * G
        assert np.array_equal(rt.to_host_f32(K[:, :, :n1]), K_o.astype(np.float32))
        assert np.array_equal(rt.to_host_f32(V[:, :, :n1]), V_o.astype(np.float32))
        assert torch.isnan(K[:, :, n1:].float()).all() and torch.isnan(V[:, :, n1:].float()).all()   # nothing beyond
        ng = n1 // G
        meta_gpu = rt.to_host_f32(meta)
        assert np.all(np.isfinite(meta_gpu[:, :, :ng * G]))
        err = np.abs(meta_gpu[:, :, :ng * G].astype(np.float64) - meta_o.astype(np.float64))
        assert np.all(err <= tol[:, :, :ng * G]), f"compact cache error {err.max():.3e}"
        assert np.isnan(meta_gpu[:, :, ng * G:]).all()                  # rows of the open group are not built
        # ---- predictor and attention over the grown context ------------------------------------------
        cur = _prefix(li, n1)
        sh = shape_at(n1)
        if ng == 0:
            continue
        meta_vals = meta_gpu[:, :, :n1].copy()
        meta_vals[:, :, ng * G:] = 0.0                                  # never read: rows of no group
        R, absdot = oracle_score_parts(cur, meta_vals, scope)
        kv.kvswap_score_select(sh, q, proj, meta, idx, nsel, scores, ws)
        torch.cuda.synchronize()
        Rg = scores.cpu().numpy().reshape(-1)[:B * S * ng].reshape(B, S, ng)      # the call's [B, S, NG] is dense
        check_scores(R, Rg, absdot)
        check_selection(R, idx.cpu().numpy(), nsel.cpu().numpy(), wl.top_k)
        idx_o = O.select(R, wl.top_k)
        full = np.full((B, S, wl.top_k), -1, dtype=np.int32)
        full[:, :, :idx_o.shape[2]] = idx_o
        idx.copy_(torch.from_numpy(full))
        nsel.fill_(idx_o.shape[2])
        kv.kvswap_sparse_decode(sh, q, K, V, idx, nsel, out, lse, ws)
        torch.cuda.synchronize()
        out_o, lse_o = O.attend(cur.q, cur.K, cur.V, idx_o, G, SCOPE_NAME[scope])
        eo, el = np.abs(out.cpu().numpy() - out_o).max(), np.abs(lse.cpu().numpy() - lse_o).max()
        assert eo <= OUT_ATOL_TIGHT[wl.kv_dtype] and el <= OUT_ATOL_TIGHT[wl.kv_dtype], (n1, eo, el)
        assert kv.kvswap_read_device_status(ws) == 0


@pytest.mark.parametrize("meta_heads", ["joint", "per_head"])
def test_growing_context_fp32(meta_heads):
    wl = W.CONFIGS[1].reduced("cfg1-grow", batch=2, n_ctx=4 * 40 + 3, top_k=12)              # G = 4
    mh = 1 if meta_heads == "joint" else wl.n_kv_heads
    _grow_and_check(wl, 4 * 30 + 1, mh, KV, check_at={122, 123, 124, 125, 128, 140, 163})


@pytest.mark.parametrize("meta_heads,scope", [("joint", KV), ("per_head", KV), ("joint", ALL)])
def test_growing_context_bf16(meta_heads, scope):
    wl = W.REDUCED[5].reduced("cfg5-grow", n_ctx=8 * 70 + 5, top_k=24)                        # G = 8
    mh = 1 if meta_heads == "joint" else wl.n_kv_heads
    n0 = 8 * 64 + 3
    _grow_and_check(wl, n0, mh, scope, check_at={n0 + 1, 8 * 65 - 1, 8 * 65, 8 * 65 + 1, 8 * 67, 8 * 70 + 5})


def test_growing_context_group_of_sixteen():
    wl = W.REDUCED[4].reduced("cfg4-grow", n_ctx=16 * 20 + 9, top_k=8)                        # G = 16, rho = 3
    _grow_and_check(wl, 16 * 17 + 15, 1, KV, check_at={16 * 18, 16 * 18 + 1, 16 * 19, 16 * 20 + 9})


def test_context_shorter_than_one_group_at_the_start():
    wl = W.CONFIGS[1].reduced("cfg1-short", batch=1, n_ctx=11, top_k=4)                       # G = 4
    _grow_and_check(wl, 1, 1, KV, check_at={2, 3, 4, 5, 8, 11})


def test_append_step_over_many_layers_equals_per_layer_appends():
    """35 layers (two launches of the row copy), three tokens, the last one completing a group."""
    wl = W.CONFIGS[3].reduced("cfg3-thin", layers=35, batch=2, n_ctx=8 * 5, n_q_heads=8, n_kv_heads=2, calib_rows=256)
    L, B, Hkv, d, r, G = wl.layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.rank, wl.group_size
    cap, n0 = wl.n_ctx, 8 * 4 + 5
    gen = torch.Generator(device="cuda").manual_seed(3)
    mk = lambda *shape: torch.randn(shape, generator=gen, device="cuda").to(torch.bfloat16)
    Ka, Va = [mk(B, Hkv, cap, d) for _ in range(L)], [mk(B, Hkv, cap, d) for _ in range(L)]
    Kb, Vb = [t.clone() for t in Ka], [t.clone() for t in Va]
    proj = [torch.randn((Hkv, d, r), generator=gen, device="cuda") for _ in range(L)]
    meta_a = [torch.full((B, 1, cap, r), float("nan"), dtype=torch.float16, device="cuda") for _ in range(L)]
    meta_b = [t.clone() for t in meta_a]
    strides = dict(kv_strides=(Hkv * cap * d, cap * d, d), meta_strides=(cap * r, cap * r, r))
    tables = kv.make_layers(Kb, Vb, meta_b, proj)
    for n in range(n0, n0 + 3):
        sh = rt.shape_for(wl, 1, KV, n_ctx=n, **strides)
        k_new, v_new = mk(L, B, Hkv, d), mk(L, B, Hkv, d)
        flushed_a = [kv.kvswap_append_kv(sh, k_new[l], v_new[l], Ka[l], Va[l], proj[l], meta_a[l]) for l in range(L)]
        flushed_b = kv.kvswap_append_step(sh, tables, k_new, v_new)
        assert all(f == flushed_b for f in flushed_a) and flushed_b == ((n + 1) % G == 0)
    torch.cuda.synchronize()
    for l in range(L):
        assert torch.equal(Ka[l], Kb[l]) and torch.equal(Va[l], Vb[l])
        assert torch.equal(meta_a[l].view(torch.int16), meta_b[l].view(torch.int16))
        assert torch.isfinite(meta_b[l][:, :, 8 * 4:8 * 5].float()).all() and torch.isnan(meta_b[l][:, :, :8 * 4].float()).all()


def test_append_refuses_a_store_without_room():
    wl = W.CONFIGS[1].reduced("cfg1-full", batch=1, n_ctx=64)
    B, Hkv, N, d, r = wl.batch, wl.n_kv_heads, wl.n_ctx, wl.head_dim, wl.rank
    K = torch.zeros((B, Hkv, N, d), device="cuda")
    meta = torch.zeros((B, 1, N, r), device="cuda")
    row = torch.zeros((B, Hkv, d), device="cuda")
    proj = torch.zeros((Hkv, d, r), device="cuda")
    dense = rt.shape_for(wl, 1, KV)
    with pytest.raises(kv.KVSwapError) as e:                 # dense strides: capacity unknown
        kv.kvswap_append_kv(dense, row, row, K, K, proj, meta)
    assert e.value.status == 2
    full = rt.shape_for(wl, 1, KV, kv_strides=(Hkv * N * d, N * d, d), meta_strides=(N * r, N * r, r))
    with pytest.raises(kv.KVSwapError) as e:                 # capacity N, context already N
        kv.kvswap_append_kv(full, row, row, K, K, proj, meta)
    assert e.value.status == 2
    torch.cuda.synchronize()
    assert float(K.abs().sum()) == 0.0
