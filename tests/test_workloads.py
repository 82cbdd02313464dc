"""Host-side checks of the seeded input generators (no method arithmetic in them)."""
import numpy as np
import torch

from paper_2511_11907_b200 import workloads as W


def test_bf16_rounding_matches_torch_and_is_nearest_even():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(10000) * 10 ** rng.uniform(-3, 3, 10000)).astype(np.float32)
    bits = W.bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    # 1 + 2^-8 is halfway between bf16 neighbours 1 and 1 + 2^-7 -> even mantissa (1.0)
    assert W.bf16_values(W.bf16_bits(np.array([1 + 2 ** -8, 1 + 3 * 2 ** -8], np.float32))).tolist() == [1.0, 1 + 2 ** -6]
    assert np.array_equal(W.bf16_values(bits), W.bf16_values(W.bf16_bits(W.bf16_values(bits))))


def test_layers_are_deterministic_and_distinct():
    wl = W.CONFIGS[1]
    a, b = W.make_layer(wl, 0), W.make_layer(wl, 0)
    assert np.array_equal(a.K, b.K) and np.array_equal(a.proj, b.proj) and np.array_equal(a.q, b.q)
    c = W.make_layer(wl.reduced("x", layers=2), 1)
    assert not np.array_equal(a.K, c.K)


def test_adapter_columns_are_orthonormal_for_both_layouts():
    wl = W.CONFIGS[1]
    j = W.make_layer(wl, 0, meta_heads=1).proj.astype(np.float64)
    A = j.reshape(wl.n_kv_heads * wl.head_dim, wl.rank)
    np.testing.assert_allclose(A.T @ A, np.eye(wl.rank), atol=1e-6)
    p = W.make_layer(wl, 0, meta_heads=wl.n_kv_heads).proj.astype(np.float64)
    for g in range(wl.n_kv_heads):
        np.testing.assert_allclose(p[g].T @ p[g], np.eye(wl.rank), atol=1e-6)


def test_heavy_tokens_have_cosine_0p8_with_the_mean_query_and_outliers_are_scaled():
    wl = W.CONFIGS[4].reduced("t", batch=1, n_ctx=2048, calib_rows=1024)
    li = W.make_layer(wl, 0)
    rho = wl.rho
    och = W._outlier_channels(wl, W.layer_seed(wl, 0))
    for g in range(wl.n_kv_heads):
        qm = li.q[0, g * rho:(g + 1) * rho].astype(np.float64).mean(axis=0)
        k = li.K[0, g, li.heavy_pos[0]].astype(np.float64).copy()
        k[:, och[g]] /= wl.outlier_scale                     # undo the outlier scaling
        cos = (k @ qm) / np.linalg.norm(k, axis=1) / np.linalg.norm(qm)
        assert np.all(np.abs(cos - 0.8) < 0.02)              # bf16 rounding only
        mask = np.ones(wl.head_dim, bool)
        mask[och[g]] = False
        plain = np.setdiff1d(np.arange(wl.n_ctx), li.heavy_pos[0])
        assert li.K[0, g][plain][:, och[g]].std() > 8.0 and abs(li.K[0, g][plain][:, mask].std() - 1.0) < 0.05
    assert abs(li.V.std() - 1.0) < 0.05                      # V untouched


def test_random_walk_queries_are_correlated():
    wl = W.REDUCED[5]
    li = W.make_layer(wl, 0)
    assert li.q_walk.shape == (wl.walk_steps, wl.batch, wl.n_q_heads, wl.head_dim)
    a, b = li.q_walk[0].ravel().astype(np.float64), li.q_walk[1].ravel().astype(np.float64)
    assert abs(np.corrcoef(a, b)[0, 1] - 0.95) < 0.02
    assert np.array_equal(li.q_walk[0], li.q)


def test_generated_arrays_are_c_contiguous():
    li = W.make_layer(W.CONFIGS[1], 0, meta_heads=1)
    for a in (li.K, li.V, li.q, li.K_raw, li.V_raw, li.q_raw, li.proj):
        assert a.flags["C_CONTIGUOUS"]
