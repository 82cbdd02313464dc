"""Seeded random shapes inside the supported ranges, each run through the three calls against the
oracle exactly as the hand-picked cases are (run_layer_parity): dtypes, head counts, GQA ratios,
group sizes (powers of two and not), ranks, context lengths with and without a ragged tail, M
below and above the number of groups, both metadata layouts and both scopes."""
import numpy as np
import pytest

from paper_2511_11907_b200 import workloads as W
from test_gpu_parity import run_layer_parity

pytestmark = pytest.mark.gpu

KV, ALL = W.SCOPE_KV_HEAD, W.SCOPE_ALL_HEADS


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    kind = rng.choice(["f32", "bf16", "f16", "bf16_q32", "f16_q32"])
    kv_dtype = {"f32": W.F32, "bf16": W.BF16, "f16": W.F16, "bf16_q32": W.BF16, "f16_q32": W.F16}[kind]
    q_dtype = W.F32 if kind in ("f32", "bf16_q32", "f16_q32") else kv_dtype
    meta_dtype = W.F32 if (kind == "f32" and rng.random() < 0.7) else W.F16
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 4, 8]))
    rho = int(rng.choice([1, 2, 3, 4, 6, 8]))
    r = int(rng.choice([8, 16, 24, 32, 32, 32, 48, 64]))
    r = min(r, d)                                             # a per-head adapter has at most d columns
    G = int(rng.choice([1, 2, 3, 4, 4, 8, 8, 16, 5, 12, 32]))
    groups = int(rng.integers(1, 400))
    N = G * groups + int(rng.integers(0, G))
    M = int(rng.choice([1, 3, 16, 50, groups, groups + 7, max(1, groups // 2)]))
    B = int(rng.choice([1, 2, 3]))
    wl = W.Workload(f"fuzz{seed}", 1, 1, B, N, Hkv * rho, Hkv, d, r, G, M, kv_dtype, meta_dtype, q_dtype,
                    calib_rows=max(512, 2 * Hkv * d if rng.random() < 0.2 else 512),
                    heavy_frac=float(rng.choice([0.0, 0.0, 0.02])))
    meta_heads = 1 if rng.random() < 0.6 else Hkv
    scope = KV if rng.random() < 0.7 else ALL
    return wl, meta_heads, scope


@pytest.mark.parametrize("seed", range(48))
def test_random_shape(seed):
    wl, meta_heads, scope = _draw(seed)
    li = W.make_layer(wl, 0, meta_heads)
    run_layer_parity(li, scope)


def _draw16(seed):
    """A 16-bit or fp32 workload small enough for a multi-layer or multi-step check."""
    rng = np.random.default_rng(5000 + seed)
    bf = rng.random() < 0.7
    kv_dtype = W.BF16 if bf else W.F32
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4]))
    rho = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([2, 4, 8, 16, 3]))
    groups = int(rng.integers(20, 160))
    M = int(rng.integers(1, groups))
    return rng, dict(batch=int(rng.choice([1, 2])), n_q_heads=Hkv * rho, n_kv_heads=Hkv, head_dim=d,
                     rank=int(rng.choice([16, 32])), group_size=G, top_k=M, kv_dtype=kv_dtype,
                     meta_dtype=W.F16 if bf else W.F32, q_dtype=kv_dtype, calib_rows=512), groups


@pytest.mark.parametrize("seed", range(10))
def test_random_decode_step(seed):
    from test_gpu_decode_step import _run_case
    rng, kw, groups = _draw16(seed)
    G = kw["group_size"]
    wl = W.Workload(f"fuzz-step{seed}", 3, int(rng.integers(1, 9)), n_ctx=G * groups + int(rng.integers(0, G)), **kw)
    _run_case(wl, "joint" if rng.random() < 0.6 else "per_head", KV if rng.random() < 0.7 else ALL,
              lookahead=int(rng.choice([0, 1, 2, 3])))


@pytest.mark.parametrize("seed", range(8))
def test_random_growing_context(seed):
    from test_gpu_append import _grow_and_check
    rng, kw, groups = _draw16(100 + seed)
    G = kw["group_size"]
    steps = int(rng.integers(G, 3 * G + 2))
    n0 = G * groups + int(rng.integers(0, G))
    wl = W.Workload(f"fuzz-grow{seed}", 1, 1, n_ctx=n0 + steps, **kw)
    check_at = set(int(x) for x in rng.choice(np.arange(n0 + 1, n0 + steps + 1), size=min(5, steps), replace=False))
    check_at.add(n0 + steps)
    mh = 1 if rng.random() < 0.6 else kw["n_kv_heads"]
    _grow_and_check(wl, n0, mh, KV if rng.random() < 0.7 else ALL, check_at)


@pytest.mark.parametrize("seed", range(6))
def test_random_reuse_buffer_attention(seed):
    from test_gpu_reuse import _tiered_attention_case
    rng, kw, groups = _draw16(200 + seed)
    G, M = kw["group_size"], kw["top_k"]
    wl = W.Workload(f"fuzz-reuse{seed}", 5, 1, n_ctx=G * groups + int(rng.integers(0, G)), walk_steps=4, **kw)
    _tiered_attention_case(wl, 1, KV if rng.random() < 0.7 else ALL, n_slots=M + int(rng.integers(0, M + 3)), steps=4)
