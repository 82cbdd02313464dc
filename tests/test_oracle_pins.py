"""Pins for the CPU oracle: each oracle step is checked against something other than itself --
exact rational arithmetic, hand-worked examples (tests/golden/), closed forms, dense brute
force written independently with scalar loops, and special cases that reduce to a library
routine.  No GPU, no CUDA library."""
import itertools
import math
import os
import struct
from fractions import Fraction

import numpy as np
import pytest

from oracle import kvswap_oracle as O
from paper_2511_11907_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [float(v) for v in vals]
    return out


def _dyadic(rng, shape, bits=4, span=4):
    """Random values k / 2^bits in [-span, span]: exactly representable everywhere."""
    return rng.integers(-span * 2 ** bits, span * 2 ** bits + 1, size=shape).astype(np.float64) / 2 ** bits


def _half_bits_of_fraction(x: Fraction) -> int:
    """Nearest-even binary16 of an exact rational, via Python's own IEEE half packing."""
    # float(Fraction) is correctly rounded to double; values used here need < 53 bits, so exact.
    return struct.unpack("<H", struct.pack("<e", float(x)))[0]


# ------------------------------------------------------------------------------------------
# O1  project_keys
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("meta_heads", [1, 3])
def test_project_keys_exact_rational(meta_heads):
    rng = np.random.default_rng(5)
    B, Hkv, N, d, r = 2, 3, 5, 4, 3
    K = _dyadic(rng, (B, Hkv, N, d), bits=5)
    A = _dyadic(rng, (Hkv, d, r), bits=6, span=1)
    got = O.project_keys(K, A, meta_heads, "f16").view(np.uint16)
    for b in range(B):
        for n in range(N):
            for j in range(r):
                per_head = [sum(Fraction(K[b, g, n, c]) * Fraction(A[g, c, j]) for c in range(d))
                            for g in range(Hkv)]
                if meta_heads == 1:
                    assert got[b, 0, n, j] == _half_bits_of_fraction(sum(per_head))
                else:
                    for g in range(Hkv):
                        assert got[b, g, n, j] == _half_bits_of_fraction(per_head[g])


def test_project_keys_f16_rounds_ties_to_even():
    # 2049 is halfway between the binary16 neighbours 2048 and 2050 -> 2048; 2051 -> 2052.
    K = np.array([[[[2049.0], [2051.0]]]])            # B=1, H=1, N=2, d=1
    A = np.ones((1, 1, 1))
    m = O.project_keys(K, A, 1, "f16").astype(np.float64).ravel()
    assert m.tolist() == [2048.0, 2052.0]


def test_project_keys_flatten_is_head_major():
    # Joint adapter whose only non-zero row is (head 1, channel 2): metadata must pick K[:,1,:,2].
    rng = np.random.default_rng(0)
    K = _dyadic(rng, (1, 3, 6, 4))
    A = np.zeros((3, 4, 2))
    A[1, 2, 0] = 1.0
    A[2, 0, 1] = -2.0
    m = O.project_keys(K, A, 1, "f64")
    assert np.array_equal(m[0, 0, :, 0], K[0, 1, :, 2])
    assert np.array_equal(m[0, 0, :, 1], -2.0 * K[0, 2, :, 0])


# ------------------------------------------------------------------------------------------
# O2..O6 on the hand-worked example
# ------------------------------------------------------------------------------------------
def test_eq1_hand_worked_example():
    g = _read_golden("eq1_selection_example.txt")
    A = np.array(g["A"]).reshape(1, 2, 2)
    q = np.array(g["q"]).reshape(1, 2, 2)
    K = np.array(g["K"]).reshape(1, 1, 8, 2)
    meta = O.project_keys(K, A, 1, "f64")
    assert meta.ravel().tolist() == g["K_lr"]
    q_lr = O.lowrank_query(q, A)
    assert q_lr.ravel().tolist() == [1, 1, 0, 2]
    s = O.head_scores(q_lr, meta, 1)
    assert s[0, 0].tolist() == g["head0"] and s[0, 1].tolist() == g["head1"]
    T = O.aggregate(s, 1, "kv_head")
    assert T[0, 0].tolist() == g["T"]
    assert O.aggregate(s, 1, "all_heads")[0, 0].tolist() == g["T"]
    R = O.pool(T, 2)
    assert R[0, 0].tolist() == g["R"]
    for M in (1, 2, 3, 4):
        assert O.select(R, M)[0, 0].tolist() == [int(v) for v in g[f"top{M}"]]
    assert O.select(R, 9)[0, 0].tolist() == [0, 1, 2, 3]          # M > NG clamps
    idx, R2 = O.score_select(q, A, meta, 2, 2)
    assert idx[0, 0].tolist() == [0, 3] and R2[0, 0].tolist() == g["R"]


def test_sum_over_heads_comes_before_group_max():
    # head scores (two tokens, one group): head0 = (3, 0), head1 = (0, 2).
    # sum-then-max = max(3, 2) = 3; max-then-sum would give 5.
    s = np.array([[[3.0, 0.0], [0.0, 2.0]]])
    assert O.pool(O.aggregate(s, 1, "kv_head"), 2)[0, 0, 0] == 3.0


def test_scopes_partition_the_heads():
    rng = np.random.default_rng(3)
    s = _dyadic(rng, (2, 6, 7))                          # H_q = 6, H_kv = 3 -> rho = 2
    T = O.aggregate(s, 3, "kv_head")
    for g in range(3):
        assert np.array_equal(T[:, g], s[:, 2 * g] + s[:, 2 * g + 1])   # consecutive heads share a KV head
    assert np.array_equal(O.aggregate(s, 3, "all_heads")[:, 0], T.sum(axis=1))


def test_pool_drops_incomplete_tail_group():
    T = np.arange(11, dtype=np.float64).reshape(1, 1, 11) * np.array([1, -1] * 5 + [1])
    R = O.pool(T, 4)                                      # tokens 8..10 are the rolling-buffer tail
    assert R.shape == (1, 1, 2)
    assert R[0, 0].tolist() == [max(T[0, 0, :4]), max(T[0, 0, 4:8])]


# ------------------------------------------------------------------------------------------
# Eq. 1 special cases
# ------------------------------------------------------------------------------------------
def _exact_scores_loops(q, K, rho):
    """sum over the rho query heads of KV head g of q_h . k_{g,n}, by scalar loops."""
    B, Hq, d = q.shape
    Hkv, N = K.shape[1], K.shape[2]
    T = np.zeros((B, Hkv, N))
    for b in range(B):
        for h in range(Hq):
            g = h // rho
            for n in range(N):
                acc = 0.0
                for c in range(d):
                    acc += q[b, h, c] * K[b, g, n, c]
                T[b, g, n] += acc
    return T


@pytest.mark.parametrize("layout", ["joint", "per_head"])
def test_identity_projection_gives_exact_qk_ranking(layout):
    rng = np.random.default_rng(11)
    B, Hq, Hkv, N, d, G, M = 2, 6, 2, 24, 4, 3, 3
    q = _dyadic(rng, (B, Hq, d))
    K = _dyadic(rng, (B, Hkv, N, d))
    if layout == "joint":
        proj = np.eye(Hkv * d).reshape(Hkv, d, Hkv * d)      # A = I, A_g = its row block g
        meta = O.project_keys(K, proj, 1, "f64")
    else:
        proj = np.stack([np.eye(d)] * Hkv)
        meta = O.project_keys(K, proj, Hkv, "f64")
    T = O.aggregate(O.head_scores(O.lowrank_query(q, proj), meta, Hkv), Hkv, "kv_head")
    T_exact = _exact_scores_loops(q, K, Hq // Hkv)
    assert np.array_equal(T, T_exact)                        # dyadic inputs: exact in float64
    idx, R = O.score_select(q, proj, meta, G, M)
    for b in range(B):
        for g in range(Hkv):
            Rg = [max(T_exact[b, g, j * G:(j + 1) * G]) for j in range(N // G)]
            want = sorted(sorted(range(N // G), key=lambda j: (-Rg[j], j))[:M])
            assert idx[b, g].tolist() == want
    T_all = O.aggregate(O.head_scores(O.lowrank_query(q, proj), meta, Hkv), Hkv, "all_heads")
    assert np.array_equal(T_all[:, 0], T_exact.sum(axis=1))


@pytest.mark.parametrize("meta_heads", [1, 2])
def test_rank_r_keys_are_recovered_exactly(meta_heads):
    """Eckart-Young: if the keys have rank <= r and A comes from their own SVD, then
    K_lr A^T = Flatten(K) and the low-rank scores equal the exact ones."""
    rng = np.random.default_rng(21)
    B, Hq, Hkv, N, d, r = 1, 4, 2, 40, 8, 3
    if meta_heads == 1:
        flat = rng.standard_normal((N, r)) @ rng.standard_normal((r, Hkv * d))
        K = flat.reshape(N, Hkv, d).transpose(1, 0, 2)[None]
    else:
        K = np.stack([rng.standard_normal((N, r)) @ rng.standard_normal((r, d)) for _ in range(Hkv)])[None]
    calib = K[0].transpose(1, 0, 2)                           # [rows, H_kv, d]
    proj = W.adapter_from_calibration(calib, Hkv, d, r, meta_heads, dtype=np.float64)
    q = rng.standard_normal((B, Hq, d))
    meta = O.project_keys(K, proj, meta_heads, "f64")
    T = O.aggregate(O.head_scores(O.lowrank_query(q, proj), meta, Hkv), Hkv, "kv_head")
    T_exact = _exact_scores_loops(q, K, Hq // Hkv)
    np.testing.assert_allclose(T, T_exact, rtol=0, atol=1e-10)
    idx, _ = O.score_select(q, proj, meta, 4, 3)
    for g in range(Hkv):
        Rg = T_exact[0, g].reshape(-1, 4).max(axis=1)
        assert set(idx[0, g].tolist()) == set(np.argsort(-Rg, kind="stable")[:3].tolist())


def test_scores_invariant_under_rotation_of_adapter_and_selection_under_query_scale():
    rng = np.random.default_rng(8)
    B, Hq, Hkv, N, d, r = 2, 4, 2, 32, 8, 4
    q, K = rng.standard_normal((B, Hq, d)), rng.standard_normal((B, Hkv, N, d))
    A = rng.standard_normal((Hkv, d, r))
    Rot, _ = np.linalg.qr(rng.standard_normal((r, r)))
    AR = A @ Rot
    T1 = O.aggregate(O.head_scores(O.lowrank_query(q, A), O.project_keys(K, A, 1, "f64"), Hkv), Hkv, "kv_head")
    T2 = O.aggregate(O.head_scores(O.lowrank_query(q, AR), O.project_keys(K, AR, 1, "f64"), Hkv), Hkv, "kv_head")
    np.testing.assert_allclose(T1, T2, rtol=0, atol=1e-11)
    meta = O.project_keys(K, A, 1, "f16")
    i1, _ = O.score_select(q, A, meta, 4, 3)
    i2, _ = O.score_select(3.5 * q, A, meta, 4, 3)
    assert np.array_equal(i1, i2)


def test_presummed_lowrank_query_equals_sum_of_head_scores():
    # Linearity used by a fused scorer: (sum_h q_h A_g(h)) . K_lr[n] == sum_h (q_h A_g(h)) . K_lr[n]
    rng = np.random.default_rng(9)
    B, Hq, Hkv, N, d, r = 1, 6, 2, 16, 4, 3
    q, A = rng.standard_normal((B, Hq, d)), rng.standard_normal((Hkv, d, r))
    meta = rng.standard_normal((B, 1, N, r))
    q_lr = O.lowrank_query(q, A)
    T = O.aggregate(O.head_scores(q_lr, meta, Hkv), Hkv, "kv_head")
    u = q_lr.reshape(B, Hkv, Hq // Hkv, r).sum(axis=2)
    np.testing.assert_allclose(np.einsum("bsr,bnr->bsn", u, meta[:, 0]), T, rtol=0, atol=1e-12)


def test_per_head_metadata_uses_its_own_head():
    rng = np.random.default_rng(10)
    q, A = _dyadic(rng, (1, 4, 3)), _dyadic(rng, (2, 3, 2))
    meta = _dyadic(rng, (1, 2, 5, 2))
    s = O.head_scores(O.lowrank_query(q, A), meta, 2)
    for h in range(4):
        g = h // 2
        want = [float((q[0, h] @ A[g]) @ meta[0, g, n]) for n in range(5)]
        assert s[0, h].tolist() == want


# ------------------------------------------------------------------------------------------
# O6  select
# ------------------------------------------------------------------------------------------
def test_select_g1_reduces_to_stable_argsort():
    rng = np.random.default_rng(2)
    T = rng.standard_normal((2, 3, 50))
    T[0, 0, 7] = T[0, 0, 30]                                   # a tie
    R = O.pool(T, 1)
    idx = O.select(R, 9)
    for b, s in itertools.product(range(2), range(3)):
        assert idx[b, s].tolist() == sorted(np.argsort(-T[b, s], kind="stable")[:9].tolist())


def test_select_ties_resolve_to_lower_index():
    R = np.array([[[1.0, 5.0, 5.0, 0.0, 5.0, 5.0]]])
    assert O.select(R, 1)[0, 0].tolist() == [1]
    assert O.select(R, 2)[0, 0].tolist() == [1, 2]
    assert O.select(R, 3)[0, 0].tolist() == [1, 2, 4]
    assert O.select(R, 5)[0, 0].tolist() == [0, 1, 2, 4, 5]


def test_select_brute_force_enumeration():
    """On tiny inputs the selected set must maximise (sum of scores, then lexicographically
    smallest index set) over all subsets of size M."""
    rng = np.random.default_rng(4)
    for trial in range(20):
        NG, M = int(rng.integers(2, 9)), int(rng.integers(1, 5))
        R = rng.integers(-3, 4, size=(1, 1, NG)).astype(np.float64)      # many ties
        got = O.select(R, M)[0, 0].tolist()
        Mp = min(M, NG)
        best = max(itertools.combinations(range(NG), Mp),
                   key=lambda c: (sum(R[0, 0, j] for j in c), [-j for j in c]))
        assert got == list(best)


def test_single_head_identity_reduces_to_plain_topk_of_qk():
    rng = np.random.default_rng(6)
    N, d, M = 64, 8, 5
    q, K = rng.standard_normal((1, 1, d)), rng.standard_normal((1, 1, N, d))
    proj = np.eye(d)[None]
    idx, _ = O.score_select(q, proj, O.project_keys(K, proj, 1, "f64"), 1, M)
    want = np.argpartition(-(K[0, 0] @ q[0, 0]), M)[:M]
    assert set(idx[0, 0].tolist()) == set(want.tolist())


# ------------------------------------------------------------------------------------------
# O7  attend
# ------------------------------------------------------------------------------------------
def _dense_attention_loops(q, K, V, rho, tokens_of):
    """Textbook softmax attention with scalar loops; tokens_of(b, h) lists the attended tokens."""
    B, Hq, d = q.shape
    out = np.zeros((B, Hq, d))
    lse = np.zeros((B, Hq))
    for b in range(B):
        for h in range(Hq):
            g = h // rho
            toks = tokens_of(b, h)
            logit = [sum(q[b, h, c] * K[b, g, n, c] for c in range(d)) / math.sqrt(d) for n in toks]
            z = sum(math.exp(x) for x in logit)
            lse[b, h] = math.log(z)
            for x, n in zip(logit, toks):
                for c in range(d):
                    out[b, h, c] += math.exp(x) / z * V[b, g, n, c]
    return out, lse


def test_attention_closed_form_example():
    g = _read_golden("attention_closed_form.txt")
    q = np.array(g["q"]).reshape(1, 1, 4)
    K = np.zeros((1, 1, 3, 4))
    K[0, 0, 1, 0] = math.log(2.0)
    K[0, 0, 2, 0] = -2000.0
    V = np.array([g["v0"], g["v1"], [1e6, 1e6, 1e6, 1e6]]).reshape(1, 1, 3, 4)
    out, lse = O.attend(q, K, V, np.array([[[0, 1]]]), 1)
    np.testing.assert_allclose(out[0, 0], g["out"], rtol=0, atol=1e-14)
    assert abs(lse[0, 0] - math.log(g["lse_is_log"][0])) < 1e-14
    out3, lse3 = O.attend(q, K, V, np.array([[[0, 1, 2]]]), 1)        # exp(-2000) == 0
    np.testing.assert_allclose(out3, out, rtol=0, atol=1e-14)
    assert abs(lse3[0, 0] - lse[0, 0]) < 1e-14


@pytest.mark.parametrize("scope", ["kv_head", "all_heads"])
def test_all_groups_selected_equals_dense_attention(scope):
    rng = np.random.default_rng(12)
    B, Hq, Hkv, N, d, G = 2, 6, 2, 23, 4, 4                   # 5 groups + 3 tail tokens
    q, K, V = (rng.standard_normal(s) for s in [(B, Hq, d), (B, Hkv, N, d), (B, Hkv, N, d)])
    S = Hkv if scope == "kv_head" else 1
    idx = np.tile(np.arange(N // G, dtype=np.int32), (B, S, 1))
    out, lse = O.attend(q, K, V, idx, G, scope)
    want, want_lse = _dense_attention_loops(q, K, V, Hq // Hkv, lambda b, h: range(N))
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, rtol=0, atol=1e-12)


def test_sparse_attention_equals_dense_attention_over_the_selected_tokens():
    rng = np.random.default_rng(13)
    B, Hq, Hkv, N, d, G = 2, 4, 2, 26, 4, 3                   # 8 groups + 2 tail tokens
    q, K, V = (rng.standard_normal(s) for s in [(B, Hq, d), (B, Hkv, N, d), (B, Hkv, N, d)])
    idx = np.array([[[0, 5, 7], [2, 3, 6]], [[1, 2, 3], [0, 4, 7]]], dtype=np.int32)

    def toks(b, h):
        g = h // 2
        return [j * G + t for j in idx[b, g] for t in range(G)] + [24, 25]

    want, want_lse = _dense_attention_loops(q, K, V, 2, toks)
    out, lse = O.attend(q, K, V, idx, G, "kv_head")
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, rtol=0, atol=1e-12)
    # all_heads scope: every head uses row 0 of the index list
    out_a, _ = O.attend(q, K, V, idx[:, :1], G, "all_heads")
    want_a, _ = _dense_attention_loops(q, K, V, 2, lambda b, h: [j * G + t for j in idx[b, 0] for t in range(G)] + [24, 25])
    np.testing.assert_allclose(out_a, want_a, rtol=0, atol=1e-12)


def test_empty_selection_attends_only_the_tail():
    rng = np.random.default_rng(14)
    q, K, V = (rng.standard_normal(s) for s in [(1, 2, 4), (1, 1, 7, 4), (1, 1, 7, 4)])
    out, _ = O.attend(q, K, V, np.zeros((1, 1, 0), dtype=np.int32), 4)     # tokens 4..6
    want, _ = _dense_attention_loops(q, K, V, 2, lambda b, h: [4, 5, 6])
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)


def test_attention_invariants():
    rng = np.random.default_rng(15)
    B, Hq, Hkv, N, d, G = 1, 4, 2, 40, 8, 4
    q, K, V = (rng.standard_normal(s) for s in [(B, Hq, d), (B, Hkv, N, d), (B, Hkv, N, d)])
    idx = np.array([[[1, 4, 8], [0, 2, 9]]], dtype=np.int32)
    out, lse, probs = O.attend(q, K, V, idx, G, return_probs=True)
    for (b, h), (tokens, p) in probs.items():
        assert abs(p.sum() - 1.0) < 1e-12 and (p > 0).all()
        rows = V[b, h // 2, tokens]
        assert (out[b, h] <= rows.max(axis=0) + 1e-12).all() and (out[b, h] >= rows.min(axis=0) - 1e-12).all()
    # permuting whole groups of K and V together, with the index list following, changes nothing
    perm = rng.permutation(N // G)
    inv = np.argsort(perm)                                    # group j moves to slot inv[j]
    Kp = K.reshape(B, Hkv, N // G, G, d)[:, :, perm].reshape(B, Hkv, N, d)
    Vp = V.reshape(B, Hkv, N // G, G, d)[:, :, perm].reshape(B, Hkv, N, d)
    idx_p = np.sort(inv[idx], axis=-1).astype(np.int32)
    out_p, lse_p = O.attend(q, Kp, Vp, idx_p, G)
    np.testing.assert_allclose(out_p, out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse_p, lse, rtol=0, atol=1e-12)
    # softmax shift invariance: adding c*q/|q|^2*sqrt(d) to every key shifts all logits by c
    h = 0
    shift = 3.0 * q[0, h] / (q[0, h] @ q[0, h]) * math.sqrt(d)
    K2 = K.copy()
    K2[0, 0] += shift
    out2, lse2 = O.attend(q, K2, V, idx, G)
    np.testing.assert_allclose(out2[0, h], out[0, h], rtol=0, atol=1e-11)
    assert abs(lse2[0, h] - lse[0, h] - 3.0) < 1e-11


# ------------------------------------------------------------------------------------------
# Planted mistakes: the pins above must notice a wrong oracle (mistakes are planted on the CPU)
# ------------------------------------------------------------------------------------------
def test_pins_detect_planted_mistakes(monkeypatch):
    def fails(test, *a):
        try:
            test(*a)
        except AssertionError:
            return True
        return False

    real_lowrank, real_pool, real_select, real_attend = O.lowrank_query, O.pool, O.select, O.attend

    # wrong query-head -> KV-head map (h % H_kv instead of floor(h / rho))
    def bad_lowrank(q, proj):
        q64, A = q.astype(np.float64), proj.astype(np.float64)
        return np.stack([q64[:, h] @ A[h % A.shape[0]] for h in range(q64.shape[1])], axis=1)
    monkeypatch.setattr(O, "lowrank_query", bad_lowrank)
    assert fails(test_identity_projection_gives_exact_qk_ranking, "joint")
    monkeypatch.setattr(O, "lowrank_query", real_lowrank)

    # group mean instead of group max
    monkeypatch.setattr(O, "pool", lambda T, G: real_pool(T, G) * 0 + T[:, :, :T.shape[2] // G * G]
                        .reshape(T.shape[0], T.shape[1], -1, G).mean(axis=3))
    assert fails(test_eq1_hand_worked_example)
    monkeypatch.setattr(O, "pool", real_pool)

    # ties to the higher index
    def bad_select(R, M):
        return np.sort(np.argsort(-R[:, :, ::-1], axis=-1, kind="stable")[:, :, :min(M, R.shape[2])] * -1
                       + R.shape[2] - 1, axis=-1).astype(np.int32)
    monkeypatch.setattr(O, "select", bad_select)
    assert fails(test_select_ties_resolve_to_lower_index)
    monkeypatch.setattr(O, "select", real_select)

    # missing 1/sqrt(d)
    def bad_attend(q, K, V, idx, G, scope="kv_head", return_probs=False):
        return real_attend(q * math.sqrt(q.shape[-1]), K, V, idx, G, scope, return_probs)
    monkeypatch.setattr(O, "attend", bad_attend)
    assert fails(test_attention_closed_form_example)
    monkeypatch.setattr(O, "attend", real_attend)

    # tail forgotten
    def no_tail(q, K, V, idx, G, scope="kv_head", return_probs=False):
        N = K.shape[2] // G * G
        return real_attend(q, K[:, :, :N], V[:, :, :N], idx, G, scope, return_probs)
    monkeypatch.setattr(O, "attend", no_tail)
    assert fails(test_sparse_attention_equals_dense_attention_over_the_selected_tokens)
    monkeypatch.setattr(O, "attend", real_attend)


# ------------------------------------------------------------------------------------------
# O8  rolling-buffer append and group flush (Sec. 4.4.1)
# ------------------------------------------------------------------------------------------
def _grow(K0, V0, k_rows, v_rows, proj, G, meta_heads, meta_dtype="f64"):
    """Start from a context of K0.shape[2] tokens and append k_rows[t], v_rows[t] one by one."""
    N0 = K0.shape[2]
    meta = O.project_keys(K0[:, :, :N0 // G * G], proj, meta_heads, meta_dtype)
    K, V, flushes = K0, V0, []
    for t in range(len(k_rows)):
        K, V, meta, fl = O.append_kv(K, V, meta, k_rows[t], v_rows[t], proj, G, meta_dtype)
        flushes.append(fl)
    return K, V, meta, flushes


def test_append_hand_worked_example():
    """G = 2, one head, d = r = 2, identity adapter: the compact cache is the K rows of the complete
    groups, written out by hand."""
    K0 = np.array([[[[1., 2.], [3., 4.], [5., 6.]]]])              # N = 3: one group + one buffered token
    V0 = -K0
    proj = np.eye(2)[None]
    new_k = [np.array([[[7., 8.]]]), np.array([[[9., 10.]]]), np.array([[[11., 12.]]])]
    new_v = [-k for k in new_k]
    K, V, meta, flushes = _grow(K0, V0, new_k, new_v, proj, 2, 1)
    assert flushes == [True, False, True]                           # N+1 = 4, 5, 6
    assert np.array_equal(K[0, 0], [[1, 2], [3, 4], [5, 6], [7, 8], [9, 10], [11, 12]])
    assert np.array_equal(V, -K)
    assert np.array_equal(meta[0, 0], [[1, 2], [3, 4], [5, 6], [7, 8], [9, 10], [11, 12]])
    K, V, meta, fl = O.append_kv(K, V, meta, np.array([[[13., 14.]]]), np.array([[[0., 0.]]]), proj, 2, "f64")
    assert not fl and meta.shape[2] == 6 and K.shape[2] == 7        # token 6 waits in the rolling buffer


@pytest.mark.parametrize("meta_heads", [1, 3])
@pytest.mark.parametrize("G,N0,steps", [(4, 9, 11), (3, 6, 7), (1, 2, 3), (5, 1, 9)])
def test_incremental_compact_cache_equals_compressing_the_grown_context(meta_heads, G, N0, steps):
    """Row independence of O1: growing token by token gives the compact cache of the grown
    context, cut at its last complete group; flushes happen exactly when a group completes."""
    rng = np.random.default_rng(5)
    B, Hkv, d, r = 2, 3, 4, 2
    K0, V0 = _dyadic(rng, (B, Hkv, N0, d)), _dyadic(rng, (B, Hkv, N0, d))
    proj = _dyadic(rng, (Hkv, d, r))
    k_rows, v_rows = _dyadic(rng, (steps, B, Hkv, d)), _dyadic(rng, (steps, B, Hkv, d))
    K, V, meta, flushes = _grow(K0, V0, k_rows, v_rows, proj, G, meta_heads)
    N = N0 + steps
    assert K.shape[2] == N and np.array_equal(K[:, :, N0:], np.moveaxis(k_rows, 0, 2))
    assert np.array_equal(V[:, :, N0:], np.moveaxis(v_rows, 0, 2))
    assert flushes == [(N0 + t + 1) % G == 0 for t in range(steps)]
    want = O.project_keys(K[:, :, :N // G * G], proj, meta_heads, "f64")
    assert meta.shape == want.shape and np.array_equal(meta, want)


def test_appended_token_is_attended_at_once_and_ranked_only_after_its_group_completes():
    """The rolling buffer lets a new entry take part in attention immediately (a key aligned with
    the query and far larger than all others takes all the weight), while the predictor sees it
    only once its group has been flushed."""
    rng = np.random.default_rng(11)
    B, Hq, Hkv, d, r, G, N0 = 1, 2, 1, 4, 4, 4, 8                   # two complete groups
    K0, V0 = _dyadic(rng, (B, Hkv, N0, d)), _dyadic(rng, (B, Hkv, N0, d))
    proj = np.eye(d)[None]
    q = np.zeros((B, Hq, d)); q[:, :, 0] = 1.0
    hot_k = np.zeros((B, Hkv, d)); hot_k[:, :, 0] = 400.0
    hot_v = np.full((B, Hkv, d), 7.0)
    meta = O.project_keys(K0, proj, 1, "f64")
    K, V, meta, fl = O.append_kv(K0, V0, meta, hot_k, hot_v, proj, G, "f64")
    assert not fl
    out, _ = O.attend(q, K, V, np.zeros((B, 1, 0), dtype=np.int32), G)        # nothing selected: tail only
    assert np.allclose(out, 7.0, atol=1e-12)
    idx, R = O.score_select(q, proj, meta, G, 1)
    assert R.shape[2] == 2                                           # the new token is in no group yet
    for t in range(3):                                               # three cold tokens complete group 2
        K, V, meta, fl = O.append_kv(K, V, meta, np.zeros((B, Hkv, d)), np.zeros((B, Hkv, d)), proj, G, "f64")
    assert fl
    idx, R = O.score_select(q, proj, meta, G, 1)
    assert R.shape[2] == 3 and idx[0, 0, 0] == 2 and R[0, 0, 2] == pytest.approx(2 * 400.0)


def test_planted_mistakes_in_append_are_caught(monkeypatch):
    real = O.append_kv

    def fails(test, *args):
        try:
            test(*args)
        except AssertionError:
            return True
        except ValueError:
            return True
        return False

    def flush_one_late(K, V, meta, k_new, v_new, proj, G, meta_dtype="f16"):   # tests N % G, not (N+1) % G
        K2, V2, m2, fl = real(K, V, meta, k_new, v_new, proj, G, meta_dtype)
        if fl:
            return K2, V2, meta, False
        if K.shape[2] % G == 0 and K.shape[2] // G * G > meta.shape[2]:
            rows = O.project_keys(K[:, :, K.shape[2] - G:], proj, meta.shape[1], meta_dtype)
            return K2, V2, np.concatenate([meta, rows], axis=2), True
        return K2, V2, meta, False
    monkeypatch.setattr(O, "append_kv", flush_one_late)
    assert fails(test_append_hand_worked_example)

    def wrong_rows(K, V, meta, k_new, v_new, proj, G, meta_dtype="f16"):       # compresses the G rows before the new one
        K2, V2, m2, fl = real(K, V, meta, k_new, v_new, proj, G, meta_dtype)
        if fl:
            N = K.shape[2]
            rows = O.project_keys(K2[:, :, N - G:N], proj, meta.shape[1], meta_dtype)
            m2 = np.concatenate([meta, rows], axis=2)
        return K2, V2, m2, fl
    monkeypatch.setattr(O, "append_kv", wrong_rows)
    assert fails(test_incremental_compact_cache_equals_compressing_the_grown_context, 1, 4, 9, 11)

    def v_gets_k(K, V, meta, k_new, v_new, proj, G, meta_dtype="f16"):
        return real(K, V, meta, k_new, k_new, proj, G, meta_dtype)
    monkeypatch.setattr(O, "append_kv", v_gets_k)
    assert fails(test_appended_token_is_attended_at_once_and_ranked_only_after_its_group_completes)
    monkeypatch.setattr(O, "append_kv", real)


# ------------------------------------------------------------------------------------------
# O9  reuse buffer (Sec. 4.4.2)
# ------------------------------------------------------------------------------------------
def test_reuse_buffer_hand_worked_fifo_trace():
    """Four slots; every table below was written out by hand from the FIFO rule."""
    table, head = [-1, -1, -1, -1], 0
    slots, loads, table, head = O.reuse_step(table, head, [5, 9, 2])
    assert (slots, loads, table, head) == ([0, 1, 2], [(5, 0), (9, 1), (2, 2)], [5, 9, 2, -1], 3)
    slots, loads, table, head = O.reuse_step(table, head, [2, 7, 9])            # 2 and 9 hit, 7 takes the empty slot
    assert (slots, loads, table, head) == ([2, 3, 1], [(7, 3)], [5, 9, 2, 7], 0)
    slots, loads, table, head = O.reuse_step(table, head, [9, 4, 6])            # 5 is oldest; slot 1 (9) serves this step
    assert (slots, loads, table, head) == ([1, 0, 2], [(4, 0), (6, 2)], [4, 9, 6, 7], 3)
    slots, loads, table, head = O.reuse_step(table, head, [-1, 7, 3, -1])       # no-group entries; 7 hits at the head
    assert (slots, loads, table, head) == ([-1, 3, 0, -1], [(3, 0)], [3, 9, 6, 7], 1)
    slots, loads, table, head = O.reuse_step(table, head, [])
    assert (slots, loads, table, head) == ([], [], [3, 9, 6, 7], 1)
    slots, loads, table, head = O.reuse_step(table, head, [9])                  # a hit does not renew the slot's age
    assert (slots, loads, table, head) == ([1], [], [3, 9, 6, 7], 1)
    slots, loads, table, head = O.reuse_step(table, head, [8])                  # FIFO, not LRU: 9 goes although just used
    assert (slots, loads, table, head) == ([1], [(8, 1)], [3, 8, 6, 7], 2)


def test_reuse_buffer_against_a_queue_model_when_nothing_is_passed_over():
    """With steps whose groups are all new (no hit can sit at the head) the buffer is a plain
    FIFO queue of the last C loaded groups: compare with collections.deque."""
    import collections
    rng = np.random.default_rng(2)
    C = 7
    table, head = [-1] * C, 0
    queue = collections.deque(maxlen=C)
    fresh = iter(rng.permutation(1000))
    for _ in range(40):
        step = [int(next(fresh)) for _ in range(int(rng.integers(0, C + 1)))]
        slots, loads, table, head = O.reuse_step(table, head, step)
        queue.extend(step)
        assert [g for g, _ in loads] == step and sorted(g for g in table if g >= 0) == sorted(queue)
        assert [table[c] for c in slots] == step


def test_reuse_buffer_invariants_on_random_walks():
    """Random overlapping selections: every selected group is served by a slot that holds it, hits
    keep their slot and cost no load, loads = misses, slots are never shared, and the buffer
    only ever holds groups that were selected at some step."""
    rng = np.random.default_rng(4)
    C, NG, M = 12, 40, 8
    table, head = [-1] * C, 0
    prev = rng.choice(NG, size=M, replace=False)
    ever = set()
    for _ in range(200):
        keep = rng.random(M) < 0.7
        pool = np.setdiff1d(np.arange(NG), prev)
        cur = np.where(keep, prev, rng.choice(pool, size=M, replace=False))
        cur = np.array(list(dict.fromkeys(cur.tolist())))               # distinct, order kept
        before = {g: c for c, g in enumerate(table) if g >= 0}
        slots, loads, table, head = O.reuse_step(table, head, cur)
        ever |= set(cur.tolist())
        assert [table[c] for c in slots] == cur.tolist() and len(set(slots)) == len(slots)
        hits = [g for g in cur.tolist() if g in before]
        assert all(slots[cur.tolist().index(g)] == before[g] for g in hits)
        assert sorted(g for g, _ in loads) == sorted(set(cur.tolist()) - set(before))
        held = [g for g in table if g >= 0]
        assert len(set(held)) == len(held) and set(held) <= ever and 0 <= head < C
        prev = cur if len(cur) == M else rng.choice(NG, size=M, replace=False)


def test_reuse_buffer_rejects_what_it_cannot_serve():
    with pytest.raises(ValueError):
        O.reuse_step([-1, -1], 0, [1, 2, 3])


def test_reuse_buffer_serves_a_group_listed_twice_from_one_slot():
    """Worked by hand: 4 is loaded once, by its first entry; 9 (a hit) keeps its slot for both entries."""
    slots, loads, table, head = O.reuse_step([5, 9, -1], 2, [4, 9, 4, 9, 7])
    assert (slots, loads, table, head) == ([2, 1, 2, 1, 0], [(4, 2), (7, 0)], [7, 9, 4], 1)


def test_planted_mistakes_in_the_reuse_buffer_are_caught(monkeypatch):
    real = O.reuse_step

    def fails(test):
        try:
            test()
        except (AssertionError, KeyError, ValueError):
            return True
        return False

    def evicts_a_hit(slot_group, head, selected):                     # does not pass over busy slots
        table = [int(x) for x in slot_group]
        C = len(table)
        slots, loads = [], []
        for j in selected:
            if j < 0:
                slots.append(-1)
            elif j in table:
                slots.append(table.index(j))
            else:
                table[head] = int(j); slots.append(head); loads.append((int(j), head)); head = (head + 1) % C
        return slots, loads, table, head
    monkeypatch.setattr(O, "reuse_step", evicts_a_hit)
    assert fails(test_reuse_buffer_hand_worked_fifo_trace)
    assert fails(test_reuse_buffer_invariants_on_random_walks)

    def lru_instead_of_fifo(slot_group, head, selected):              # a hit renews the slot's age
        slots, loads, table, head2 = real(slot_group, head, selected)
        hit_slots = [c for c, j in zip(slots, selected) if j >= 0 and (int(j), c) not in loads]
        if hit_slots and not loads:
            head2 = (max(hit_slots) + 1) % len(table)
        return slots, loads, table, head2
    monkeypatch.setattr(O, "reuse_step", lru_instead_of_fifo)
    assert fails(test_reuse_buffer_hand_worked_fifo_trace)
    monkeypatch.setattr(O, "reuse_step", real)


# ------------------------------------------------------------------------------------------
# O3'  per-head softmax over the context (predictor variant)
# ------------------------------------------------------------------------------------------
def test_head_softmax_closed_form_and_normalisation():
    """d = 4, logits 0, 2 ln 2, 2 ln 3 (so logit / sqrt(d) = 0, ln 2, ln 3): weights 1/6, 2/6, 3/6; the
    token of the open group (N = 4, G = 3) gets none, whatever its logit."""
    s = np.array([[[0.0, 2 * math.log(2), 2 * math.log(3), 50.0]]])
    p = O.softmax_over_context(s, 4, 3)
    assert np.allclose(p[0, 0], [1 / 6, 2 / 6, 3 / 6, 0.0], atol=1e-15)
    rng = np.random.default_rng(8)
    s = rng.normal(size=(2, 5, 23)) * 30
    p = O.softmax_over_context(s, 64, 4)
    assert np.allclose(p[:, :, :20].sum(axis=2), 1.0, atol=1e-12) and np.all(p[:, :, 20:] == 0)
    assert np.allclose(O.softmax_over_context(s + 1234.5, 64, 4), p, atol=1e-12)      # shift invariance
    import scipy.special
    assert np.allclose(p[:, :, :20], scipy.special.softmax(s[:, :, :20] / 8.0, axis=2), atol=1e-14)


def test_head_softmax_changes_the_ranking_only_across_heads():
    """One head: softmax is monotone, so the selection equals the raw-logit selection.  Two heads: a
    sharply peaked head outvotes a nearly flat one, which the raw sum does not show -- an example,
    worked by hand, where the two readings select different groups."""
    rng = np.random.default_rng(3)
    proj = np.eye(4)[None]
    meta = _dyadic(rng, (1, 1, 24, 4))
    q1 = _dyadic(rng, (1, 1, 4))
    a, _ = O.score_select(q1, proj, meta, 2, 3)
    b, _ = O.score_select(q1, proj, meta, 2, 3, head_softmax=True)
    assert np.array_equal(a, b)
    # d = 4 (scale 1/2), G = 1, M = 1; head 0 sees logits (8, 0, 0, 0), head 1 sees (0, 10, 9.75, 9.75)
    meta = np.zeros((1, 1, 4, 4))
    meta[0, 0, :, 0] = [8, 0, 0, 0]
    meta[0, 0, :, 1] = [0, 10, 9.75, 9.75]
    q2 = np.zeros((1, 2, 4)); q2[0, 0, 0] = 1.0; q2[0, 1, 1] = 1.0
    raw, R_raw = O.score_select(q2, proj, meta, 1, 1)
    assert np.array_equal(R_raw[0, 0], [8, 10, 9.75, 9.75]) and raw[0, 0, 0] == 1
    soft, R_soft = O.score_select(q2, proj, meta, 1, 1, head_softmax=True)
    z0 = math.exp(4) + 3
    z1 = 1 + math.exp(5) + 2 * math.exp(4.875)
    want = [math.exp(4) / z0 + 1 / z1, 1 / z0 + math.exp(5) / z1, 1 / z0 + math.exp(4.875) / z1,
            1 / z0 + math.exp(4.875) / z1]
    assert np.allclose(R_soft[0, 0], want, atol=1e-14) and soft[0, 0, 0] == 0


# ------------------------------------------------------------------------------------------
# 8-bit metadata: the E4M3 storage format (reading of "precision can be traded", Sec. 4.1 / 4.2)
# ------------------------------------------------------------------------------------------
def _e4m3_golden():
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "e4m3_format.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                bits, val = line.split()
                rows.append((int(bits.replace(".", ""), 2), float(val)))
    return rows


def test_e4m3_table_matches_the_published_format_and_torch():
    table = O.e4m3_decode_table()
    for code, val in _e4m3_golden():
        if np.isnan(val):
            assert np.isnan(table[code])
        else:
            assert table[code] == val and np.signbit(table[code]) == np.signbit(val), (code, val)
    import torch
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(table), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(table[ok], ref[ok])


def _nearest_by_brute_force(x):
    """Nearest finite table entry of the same sign; of two equally near the one with the even code."""
    table = O.e4m3_decode_table()
    best = None
    for code in range(256):
        v = table[code]
        if np.isnan(v) or (code >= 128) != bool(np.signbit(x)):
            continue
        key = (abs(v - x), code & 1)
        if best is None or key < best[0]:
            best = (key, code)
    return best[1]


def test_e4m3_round_is_nearest_with_ties_to_even_and_saturates():
    # hand-worked: halfway cases go to the even mantissa; beyond 448 everything saturates
    cases = {1.0625: 1.0, 1.1875: 1.25, -1.0625: -1.0, 2.0 ** -10: 0.0, 3 * 2.0 ** -10: 2.0 ** -8,
             460.0: 448.0, 464.0: 448.0, 1000.0: 448.0, -1e9: -448.0, 0.0: 0.0, 0.0146484375: 0.0146484375 + 2.0 ** -10,
             15.5: 16.0, 0.99: 1.0, 447.9: 448.0, 2.0 ** -6 - 2.0 ** -10: 2.0 ** -6}
    # (0.0146484375 = 7.5 * 2^-9 lies halfway between the largest subnormal 7 * 2^-9 and the smallest
    # normal 8 * 2^-9: it goes to the even one, 8 * 2^-9 = 2^-6)
    for x, want in cases.items():
        v, code = O.e4m3_round(np.array([x]))
        assert v[0] == want, (x, v[0], want)
        assert O.e4m3_decode_table()[code[0]] == want
    rng = np.random.default_rng(5)
    xs = np.concatenate([rng.standard_normal(400) * s for s in (1e-3, 0.02, 1.0, 30.0, 300.0)])
    xs = np.concatenate([xs, np.array([(k + 0.5) * 2.0 ** -9 for k in range(16)])])      # subnormal halfway points
    v, code = O.e4m3_round(xs)
    for x, c in zip(xs, code):
        assert c == _nearest_by_brute_force(np.clip(x, -448, 448)), x
    # an independent library conversion agrees wherever it is defined (it has no saturation)
    import torch
    inside = np.abs(xs) < 464
    ref = torch.from_numpy(xs[inside]).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    nz = v[inside] != 0                                                              # the sign of a rounded zero is free
    assert np.array_equal(code[inside][nz], ref[nz])


def test_e4m3_planted_rounding_mistakes_are_caught(monkeypatch):
    xs = np.array([1.0625, 1.1875, 3 * 2.0 ** -10, 0.99])
    good = O.e4m3_round(xs)[0]
    monkeypatch.setattr(np, "rint", lambda a: np.floor(a + 0.5))          # halves away from zero
    assert not np.array_equal(O.e4m3_round(xs)[0], good)
    monkeypatch.setattr(np, "rint", np.floor)                             # truncation
    assert not np.array_equal(O.e4m3_round(xs)[0], good)


def test_project_keys_e4m3_rounds_the_exact_product_once():
    rng = np.random.default_rng(11)
    B, Hkv, N, d, r = 1, 2, 6, 4, 4
    K = (rng.integers(-8, 9, size=(B, Hkv, N, d)) / 4.0).astype(np.float32)       # dyadic: exact in every type
    proj = (rng.integers(-8, 9, size=(Hkv, d, r)) / 8.0).astype(np.float32)
    for meta_heads in (1, Hkv):
        for e in (0, 2, -1):
            meta = O.project_keys(K, proj, meta_heads, "e4m3", meta_exp=e)
            table = O.e4m3_decode_table()
            for m in range(meta_heads):
                for n in range(N):
                    for j in range(r):
                        heads = range(Hkv) if meta_heads == 1 else [m]
                        exact = sum(Fraction(float(K[0, g, n, c])) * Fraction(float(proj[g, c, j])) for g in heads for c in range(d))
                        exact = float(exact / Fraction(2) ** e)
                        assert meta[0, m, n, j] == table[_nearest_by_brute_force(exact)] or (meta[0, m, n, j] == 0 and table[_nearest_by_brute_force(exact)] == 0)


def test_score_select_undoes_the_power_of_two_of_8bit_metadata():
    """Scores of meta * 2^e stored as (meta, e) equal the scores of meta * 2^e passed directly; the
    selection does not depend on e as long as nothing saturates."""
    wl = W.CONFIGS[1].reduced("e4m3-sel", n_ctx=256, top_k=8)
    li = W.make_layer(wl, 0, 1)
    meta8 = O.project_keys(li.K, li.proj, 1, "e4m3", meta_exp=-2)
    idx_a, R_a = O.score_select(li.q, li.proj, meta8, wl.group_size, wl.top_k, meta_exp=-2)
    idx_b, R_b = O.score_select(li.q, li.proj, (meta8.astype(np.float64) * 0.25), wl.group_size, wl.top_k)
    assert np.array_equal(idx_a, idx_b) and np.allclose(R_a, R_b, rtol=0, atol=0)
    # and the 8-bit cache still ranks like the fp16 one on most groups (reported, not a pin of quality)
    meta16 = O.project_keys(li.K, li.proj, 1, "f32")
    idx_c, _ = O.score_select(li.q, li.proj, meta16, wl.group_size, wl.top_k)
    assert len(set(idx_a[0, 0]) & set(idx_c[0, 0])) >= wl.top_k // 2
