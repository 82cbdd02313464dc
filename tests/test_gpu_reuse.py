"""Reuse buffer (Sec. 4.4.2) on the GPU against the oracle: slot assignment, miss lists and the
slot table bit for bit over walks of overlapping selections; attention served from the reuse
buffer, filled from a slow tier in pinned host memory, against attention over the whole store."""
import numpy as np
import pytest
import torch

from oracle import kvswap_oracle as O
from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W
from parity_util import OUT_ATOL_TIGHT, SCOPE_NAME

pytestmark = pytest.mark.gpu

KV, ALL = W.SCOPE_KV_HEAD, W.SCOPE_ALL_HEADS


class DeviceReuse:
    """State and outputs of kvswap_reuse_lookup for one layer."""

    def __init__(self, shape, n_slots, max_groups):
        self.shape, self.C, self.max_groups = shape, n_slots, max_groups
        B, S, M = shape.batch, shape.n_scopes, shape.top_k
        n = kv.kvswap_reuse_state_bytes(shape, n_slots, max_groups)
        assert n == 4 * B * S * (1 + n_slots + max_groups)
        self.state = torch.full((n // 4,), 12345, dtype=torch.int32, device="cuda")
        kv.kvswap_reuse_init(shape, n_slots, max_groups, self.state)
        self.slot_idx = torch.full((B, S, M), -9, dtype=torch.int32, device="cuda")
        self.miss_group = torch.full((B, S, M), -9, dtype=torch.int32, device="cuda")
        self.miss_slot = torch.full((B, S, M), -9, dtype=torch.int32, device="cuda")
        self.n_miss = torch.full((B, S), -9, dtype=torch.int32, device="cuda")

    def lookup(self, idx, nsel, shape=None):
        kv.kvswap_reuse_lookup(shape or self.shape, self.C, self.max_groups, idx, nsel, self.state, self.slot_idx,
                               self.miss_group, self.miss_slot, self.n_miss)

    def tables(self):
        B, S = self.shape.batch, self.shape.n_scopes
        st = self.state.cpu().numpy()
        P = B * S
        head = st[:P].reshape(B, S)
        slot_group = st[P:P + P * self.C].reshape(B, S, self.C)
        group_slot = st[P + P * self.C:].reshape(B, S, self.max_groups)
        return head, slot_group, group_slot


def _walk(rng, NG, M, prev, keep=0.7, ragged=True):
    """A step's selection: keeps ~70 % of the previous one, distinct, sometimes short or with holes."""
    if prev is None:
        cur = rng.choice(NG, size=M, replace=False)
    else:
        pool = np.setdiff1d(np.arange(NG), prev)
        fresh = rng.choice(pool, size=M, replace=False)
        cur = np.where(rng.random(M) < keep, prev, fresh)
        _, first = np.unique(cur, return_index=True)
        cur = cur[np.sort(first)]
        if len(cur) < M:
            extra = np.setdiff1d(np.arange(NG), cur)
            cur = np.concatenate([cur, rng.choice(extra, size=M - len(cur), replace=False)])
    n_sel = M
    lst = cur.astype(np.int32).copy()
    if ragged:
        r = rng.random()
        if r < 0.15:
            n_sel = int(rng.integers(0, M + 1))
        elif r < 0.3:
            lst[rng.integers(0, M)] = -1                   # "no group"
        elif r < 0.4:
            lst[rng.integers(0, M)] = NG + 3               # beyond the context
    return cur, lst, n_sel


@pytest.mark.parametrize("n_slots,M,NG", [(12, 12, 60), (20, 12, 60), (64, 40, 500), (1500, 1030, 5000)])
def test_lookup_follows_the_oracle_over_a_walk(n_slots, M, NG):
    G, B = 4, 2
    wl = W.CONFIGS[1].reduced("reuse", batch=B, n_ctx=G * NG + 2, top_k=M)
    shape = rt.shape_for(wl, 1, KV)
    S = shape.n_scopes
    dr = DeviceReuse(shape, n_slots, NG)
    rng = np.random.default_rng(n_slots + M)
    tables = [[([-1] * n_slots, 0) for _ in range(S)] for _ in range(B)]
    prev = [[None] * S for _ in range(B)]
    hits = total = 0
    for step in range(25 if M > 100 else 60):
        idx = np.full((B, S, M), -1, dtype=np.int32)
        nsel = np.zeros((B, S), dtype=np.int32)
        for b in range(B):
            for s in range(S):
                prev[b][s], idx[b, s], nsel[b, s] = _walk(rng, NG, M, prev[b][s])
        dr.lookup(torch.from_numpy(idx).cuda(), torch.from_numpy(nsel).cuda())
        torch.cuda.synchronize()
        slot_idx, mg, ms, nm = (t.cpu().numpy() for t in (dr.slot_idx, dr.miss_group, dr.miss_slot, dr.n_miss))
        head, slot_group, group_slot = dr.tables()
        for b in range(B):
            for s in range(S):
                lst = [int(j) if (i < nsel[b, s] and 0 <= j < NG) else -1 for i, j in enumerate(idx[b, s])]
                slots, loads, table, hd = O.reuse_step(*tables[b][s], lst)
                tables[b][s] = (table, hd)
                assert slot_idx[b, s].tolist() == slots
                assert nm[b, s] == len(loads)
                assert list(zip(mg[b, s, :len(loads)].tolist(), ms[b, s, :len(loads)].tolist())) == loads
                assert np.all(mg[b, s, len(loads):] == -1) and np.all(ms[b, s, len(loads):] == -1)
                assert slot_group[b, s].tolist() == table and head[b, s] == hd
                inverse = np.full(NG, -1)
                for c, g in enumerate(table):
                    if g >= 0:
                        inverse[g] = c
                assert np.array_equal(group_slot[b, s], inverse)
                n_valid = sum(1 for j in lst if j >= 0)
                hits += n_valid - len(loads)
                total += n_valid
    assert 0.3 < hits / total < 0.9                        # the walk keeps ~70 %: most steps mostly hit


def test_lookup_with_repeated_and_unordered_entries():
    """Lists as kvswap_sparse_decode accepts them: unsorted, with groups listed twice or three times."""
    G, B, NG, M, C = 4, 2, 80, 24, 24
    wl = W.CONFIGS[1].reduced("reuse-dup", batch=B, n_ctx=G * NG + 1, top_k=M)
    shape = rt.shape_for(wl, 1, KV)
    S = shape.n_scopes
    dr = DeviceReuse(shape, C, NG)
    rng = np.random.default_rng(77)
    tables = [[([-1] * C, 0) for _ in range(S)] for _ in range(B)]
    for step in range(40):
        idx = rng.integers(0, 30 + step, size=(B, S, M)).astype(np.int32)      # many repeats, drifting range
        idx = np.minimum(idx, NG - 1)
        nsel = np.full((B, S), M, dtype=np.int32)
        dr.lookup(torch.from_numpy(idx).cuda(), torch.from_numpy(nsel).cuda())
        torch.cuda.synchronize()
        slot_idx, mg, ms, nm = (t.cpu().numpy() for t in (dr.slot_idx, dr.miss_group, dr.miss_slot, dr.n_miss))
        head, slot_group, group_slot = dr.tables()
        for b in range(B):
            for s in range(S):
                slots, loads, table, hd = O.reuse_step(*tables[b][s], idx[b, s].tolist())
                tables[b][s] = (table, hd)
                assert slot_idx[b, s].tolist() == slots and nm[b, s] == len(loads)
                assert list(zip(mg[b, s, :len(loads)].tolist(), ms[b, s, :len(loads)].tolist())) == loads
                assert slot_group[b, s].tolist() == table and head[b, s] == hd
                assert np.all(group_slot[b, s] >= -1)                          # no claim marks left behind
                inverse = np.full(NG, -1)
                for c, g in enumerate(table):
                    if g >= 0:
                        inverse[g] = c
                assert np.array_equal(group_slot[b, s], inverse)


def _tiered_attention_case(wl, meta_heads, scope, n_slots, steps):
    li = W.make_layer(wl, 0, meta_heads)
    shape = rt.shape_for(wl, meta_heads, scope)
    B, Hkv, N, d, G, M = wl.batch, wl.n_kv_heads, wl.n_ctx, wl.head_dim, wl.group_size, wl.top_k
    NG, S = N // G, shape.n_scopes
    K, V = rt.to_device(li.K_raw, wl.kv_dtype), rt.to_device(li.V_raw, wl.kv_dtype)
    K_slow, V_slow = K.cpu().pin_memory(), V.cpu().pin_memory()          # the slow tier: host memory
    proj = torch.from_numpy(np.ascontiguousarray(li.proj, dtype=np.float32)).cuda()
    ws, meta = rt.alloc_workspace(shape), rt.alloc_meta(shape)
    kv.kvswap_project_keys(shape, K, proj, meta, 0, N, ws)
    idx, nsel = rt.alloc_selection(shape)
    out_ref, lse_ref = rt.alloc_output(shape)
    out, lse = rt.alloc_output(shape)
    R = (n_slots + 1) * G
    K_reuse = torch.full((B, Hkv, R, d), float("nan"), dtype=K.dtype, device="cuda")
    V_reuse = torch.full((B, Hkv, R, d), float("nan"), dtype=K.dtype, device="cuda")
    tail = N % G
    K_reuse[:, :, n_slots * G:n_slots * G + tail] = K[:, :, NG * G:]        # the rolling buffer stays in fast memory
    V_reuse[:, :, n_slots * G:n_slots * G + tail] = V[:, :, NG * G:]
    shape_r = kv.reuse_attention_shape(shape, n_slots)
    ws_r = rt.alloc_workspace(shape_r)
    dr = DeviceReuse(shape, n_slots, NG)
    qs = li.q_walk_raw if li.q_walk_raw is not None else np.stack([li.q_raw] * steps)
    rates = []
    for t in range(steps):
        q = rt.to_device(qs[t % len(qs)], wl.q_dtype)
        kv.kvswap_score_select(shape, q, proj, meta, idx, nsel, None, ws)
        kv.kvswap_sparse_decode(shape, q, K, V, idx, nsel, out_ref, lse_ref, ws)          # everything in HBM
        dr.lookup(idx, nsel)
        kv.kvswap_reuse_fill(shape, n_slots, K_slow, V_slow, K_reuse, V_reuse, dr.miss_group, dr.miss_slot, dr.n_miss)
        kv.kvswap_sparse_decode(shape_r, q, K_reuse, V_reuse, dr.slot_idx, nsel, out, lse, ws_r)
        torch.cuda.synchronize()
        assert kv.kvswap_read_device_status(ws_r) == 0
        # the slots hold the selected groups' rows
        idx_h, slot_h = idx.cpu().numpy(), dr.slot_idx.cpu().numpy()
        for b in range(B):
            for s in range(S):
                heads = [s] if scope == KV else range(Hkv)
                for i in (0, M // 2, M - 1):
                    j, c = int(idx_h[b, s, i]), int(slot_h[b, s, i])
                    assert 0 <= c < n_slots
                    for g in heads:
                        assert torch.equal(K_reuse[b, g, c * G:(c + 1) * G], K[b, g, j * G:(j + 1) * G])
                        assert torch.equal(V_reuse[b, g, c * G:(c + 1) * G], V[b, g, j * G:(j + 1) * G])
        # same tokens in the same order: the two attentions agree to rounding of the split merge
        tol = OUT_ATOL_TIGHT[wl.kv_dtype]
        assert (out - out_ref).abs().max().item() <= tol and (lse - lse_ref).abs().max().item() <= tol
        if t == steps - 1:                                                # and with the oracle
            qv = li.q_walk[t % len(qs)] if li.q_walk is not None else li.q
            out_o, _ = O.attend(qv, li.K, li.V, idx_h, G, SCOPE_NAME[scope])
            assert np.abs(out.cpu().numpy() - out_o).max() <= tol
        rates.append(1.0 - dr.n_miss.sum().item() / (B * S * min(M, NG)))
    assert rates[0] == 0.0
    return rates


def test_attention_from_the_reuse_buffer_bf16_random_walk():
    wl = W.REDUCED[5].reduced("cfg5-reuse", n_ctx=8192 + 5)               # walk of 8 correlated queries
    rates = _tiered_attention_case(wl, 1, KV, n_slots=96, steps=8)
    assert min(rates[1:]) > 0.3                                             # consecutive steps overlap


def test_attention_from_the_reuse_buffer_all_heads_scope_fp32():
    wl = W.CONFIGS[1].reduced("cfg1-reuse", batch=2, n_ctx=2048 + 3)
    _tiered_attention_case(wl, 1, ALL, n_slots=wl.top_k, steps=3)           # n_slots == M: every slot serves the step


def test_attention_from_the_reuse_buffer_group_of_sixteen():
    wl = W.REDUCED[4].reduced("cfg4-reuse", n_ctx=4096 + 9)
    _tiered_attention_case(wl, 1, KV, n_slots=40, steps=3)


@pytest.mark.parametrize("lookahead", [0, 1])
def test_tiered_decode_step_matches_the_step_over_the_full_store(lookahead):
    """Four layers, slow tier in pinned host memory, three consecutive steps (the reuse buffers carry
    over): outputs agree with kvswap_decode_step over the HBM-resident stores, selections are
    identical, every slot list points at slots holding the selected groups."""
    from paper_2511_11907_b200 import device_workload as DW
    wl = W.REDUCED[5].reduced("cfg5-tiered", layers=4, n_ctx=4096 + 3, top_k=48, walk_steps=3)
    dw = DW.build(wl, 1, KV, walk_steps=3, reserve_bytes=1 << 30)
    shape, L = dw.shape, wl.layers
    B, Hkv, N, d, G, M = wl.batch, wl.n_kv_heads, wl.n_ctx, wl.head_dim, wl.group_size, wl.top_k
    NG, S, C = N // G, shape.n_scopes, 80
    ws = rt.alloc_workspace(shape)
    for l in range(L):
        kv.kvswap_project_keys(shape, dw.K[l], dw.proj[l], dw.meta[l], 0, N, ws)
    K_slow = [k.cpu().pin_memory() for k in dw.K]
    V_slow = [v.cpu().pin_memory() for v in dw.V]
    R = (C + 1) * G
    K_r = [torch.full((B, Hkv, R, d), float("nan"), dtype=dw.K[0].dtype, device="cuda") for _ in range(L)]
    V_r = [torch.full((B, Hkv, R, d), float("nan"), dtype=dw.K[0].dtype, device="cuda") for _ in range(L)]
    for l in range(L):
        K_r[l][:, :, C * G:C * G + N % G] = dw.K[l][:, :, NG * G:]
        V_r[l][:, :, C * G:C * G + N % G] = dw.V[l][:, :, NG * G:]
    n_state = kv.kvswap_reuse_state_bytes(shape, C, NG) // 4
    state = [torch.empty(n_state, dtype=torch.int32, device="cuda") for _ in range(L)]
    for l in range(L):
        kv.kvswap_reuse_init(shape, C, NG, state[l])
    slot_idx = torch.full((L, B, S, M), -9, dtype=torch.int32, device="cuda")
    miss_group, miss_slot = torch.full_like(slot_idx, -9), torch.full_like(slot_idx, -9)
    n_miss = torch.full((L, B, S), -9, dtype=torch.int32, device="cuda")
    tiers = kv.make_tiers(C, NG, K_slow, V_slow, K_r, V_r, state, slot_idx, miss_group, miss_slot, n_miss)
    layers_hbm = dw.layer_tables(lookahead)
    layers_tiered = kv.make_layers(K_r, V_r, dw.meta, dw.proj, lookahead)
    ws_t = torch.empty(kv.kvswap_tiered_workspace_bytes(shape, C), dtype=torch.uint8, device="cuda")
    kv.kvswap_workspace_init(ws_t)
    mk = lambda: (torch.full((L, B, wl.n_q_heads, d), float("nan"), device="cuda"),
                  torch.full((L, B, wl.n_q_heads), float("nan"), device="cuda"),
                  torch.full((L, B, S, M), -7, dtype=torch.int32, device="cuda"),
                  torch.full((L, B, S), -7, dtype=torch.int32, device="cuda"))
    missed = []
    for t in range(3):
        q = dw.q_walk[t]
        out_a, lse_a, idx_a, nsel_a = mk()
        kv.kvswap_decode_step(shape, layers_hbm, q, out_a, lse_a, idx_a, nsel_a, ws)
        out_b, lse_b, idx_b, nsel_b = mk()
        kv.kvswap_decode_step_tiered(shape, layers_tiered, tiers, q, out_b, lse_b, idx_b, nsel_b, ws_t)
        torch.cuda.synchronize()
        assert kv.kvswap_read_device_status(ws_t) == 0
        assert torch.equal(idx_a, idx_b) and torch.equal(nsel_a, nsel_b)
        tol = OUT_ATOL_TIGHT[wl.kv_dtype]
        assert (out_a - out_b).abs().max().item() <= tol and (lse_a - lse_b).abs().max().item() <= tol
        sl, ix = slot_idx.cpu().numpy(), idx_b.cpu().numpy()
        assert sl.min() >= 0 and sl.max() < C
        for l in range(L):
            for b in range(B):
                for s in range(S):
                    assert len(set(sl[l, b, s].tolist())) == M                   # no slot serves two groups
                    for i in (0, M - 1):
                        j, c = int(ix[l, b, s, i]), int(sl[l, b, s, i])
                        assert torch.equal(K_r[l][b, s, c * G:(c + 1) * G], dw.K[l][b, s, j * G:(j + 1) * G])
        missed.append(int(n_miss.sum().item()))
    assert missed[0] == L * B * S * M and missed[1] < missed[0] and missed[2] < missed[0]


def test_tiered_growing_context_matches_the_hbm_resident_one():
    """Three layers; the context grows over two group boundaries.  Side A keeps everything in HBM
    (kvswap_append_step + kvswap_decode_step); side B keeps the full cache in pinned host memory
    (kvswap_append_step_tiered + kvswap_decode_step_tiered).  Same selections, same attention, and
    the slow tier ends up holding the appended rows of every completed group."""
    from paper_2511_11907_b200 import device_workload as DW
    cap = 2048 + 24
    wl = W.REDUCED[5].reduced("cfg5-tiered-grow", layers=3, n_ctx=cap, top_k=40, walk_steps=2)
    dw = DW.build(wl, 1, KV, walk_steps=2, reserve_bytes=1 << 30)
    L, B, Hkv, d, r, G, M = wl.layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.rank, wl.group_size, wl.top_k
    n0, steps, C = 2048 + 3, 19, 64
    strides = dict(kv_strides=(Hkv * cap * d, cap * d, d), meta_strides=(cap * r, cap * r, r))
    shape_at = lambda n: rt.shape_for(wl, 1, KV, n_ctx=n, **strides)
    S, NGcap = shape_at(cap).n_scopes, cap // G
    ws = rt.alloc_workspace(shape_at(cap))
    gen = torch.Generator(device="cuda").manual_seed(9)
    new_k = torch.randn((steps, L, B, Hkv, d), generator=gen, device="cuda").to(torch.bfloat16)
    new_v = torch.randn((steps, L, B, Hkv, d), generator=gen, device="cuda").to(torch.bfloat16)
    # side A: HBM stores (rows >= n0 poisoned), side B: slow tier in host memory + reuse stores
    for l in range(L):
        dw.K[l][:, :, n0:] = float("nan")
        dw.V[l][:, :, n0:] = float("nan")
    meta_a = [torch.full((B, 1, cap, r), float("nan"), dtype=torch.float16, device="cuda") for _ in range(L)]
    meta_b = [m.clone() for m in meta_a]
    for l in range(L):
        kv.kvswap_project_keys(shape_at(n0), dw.K[l], dw.proj[l], meta_a[l], 0, n0 // G * G, ws)
        meta_b[l].copy_(meta_a[l])
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
    K_slow, V_slow = [pin(k) for k in dw.K], [pin(v) for v in dw.V]
    R = (C + 1) * G
    K_r = [torch.full((B, Hkv, R, d), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(L)]
    V_r = [torch.full((B, Hkv, R, d), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(L)]
    for l in range(L):                                                   # the open group starts in the rolling rows
        K_r[l][:, :, C * G:C * G + n0 % G] = dw.K[l][:, :, n0 // G * G:n0]
        V_r[l][:, :, C * G:C * G + n0 % G] = dw.V[l][:, :, n0 // G * G:n0]
    state = [torch.empty(kv.kvswap_reuse_state_bytes(shape_at(cap), C, NGcap) // 4, dtype=torch.int32, device="cuda")
             for _ in range(L)]
    for l in range(L):
        kv.kvswap_reuse_init(shape_at(cap), C, NGcap, state[l])
    slot_idx = torch.empty((L, B, S, M), dtype=torch.int32, device="cuda")
    mg, ms = torch.empty_like(slot_idx), torch.empty_like(slot_idx)
    nm = torch.empty((L, B, S), dtype=torch.int32, device="cuda")
    tiers = kv.make_tiers(C, NGcap, K_slow, V_slow, K_r, V_r, state, slot_idx, mg, ms, nm)
    layers_a = kv.make_layers(dw.K, dw.V, meta_a, dw.proj)
    layers_b = kv.make_layers(K_r, V_r, meta_b, dw.proj)
    ws_t = torch.empty(kv.kvswap_tiered_workspace_bytes(shape_at(cap), C), dtype=torch.uint8, device="cuda")
    kv.kvswap_workspace_init(ws_t)
    mk = lambda: (torch.full((L, B, wl.n_q_heads, d), float("nan"), device="cuda"),
                  torch.full((L, B, S, M), -7, dtype=torch.int32, device="cuda"),
                  torch.full((L, B, S), -7, dtype=torch.int32, device="cuda"))
    flushes = 0
    for t in range(steps):
        n = n0 + t
        fa = kv.kvswap_append_step(shape_at(n), layers_a, new_k[t], new_v[t])
        fb = kv.kvswap_append_step_tiered(shape_at(n), layers_b, tiers, new_k[t], new_v[t])
        assert fa == fb == ((n + 1) % G == 0)
        flushes += fb
        q = dw.q_walk[t % 2]
        out_a, idx_a, nsel_a = mk()
        out_b, idx_b, nsel_b = mk()
        kv.kvswap_decode_step(shape_at(n + 1), layers_a, q, out_a, None, idx_a, nsel_a, ws)
        kv.kvswap_decode_step_tiered(shape_at(n + 1), layers_b, tiers, q, out_b, None, idx_b, nsel_b, ws_t)
        torch.cuda.synchronize()
        assert torch.equal(idx_a, idx_b) and torch.equal(nsel_a, nsel_b)
        assert not torch.isnan(out_b).any()
        assert (out_a - out_b).abs().max().item() <= OUT_ATOL_TIGHT[wl.kv_dtype]
    assert flushes == 2
    n_end = n0 + steps
    done = n_end // G * G                                                # rows of complete groups
    for l in range(L):
        assert torch.equal(K_slow[l][:, :, :done], dw.K[l][:, :, :done].cpu())
        assert torch.equal(V_slow[l][:, :, :done], dw.V[l][:, :, :done].cpu())
        assert torch.isnan(K_slow[l][:, :, done:].float()).all()         # the open group is not in the slow tier
        assert torch.equal(meta_a[l][:, :, :done].view(torch.int16), meta_b[l][:, :, :done].view(torch.int16))
        assert torch.equal(K_r[l][:, :, C * G:C * G + n_end % G], dw.K[l][:, :, done:n_end])
