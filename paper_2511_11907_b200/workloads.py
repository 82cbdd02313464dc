"""Seeded synthetic inputs for the KVSwap decode hot path.

This module only *draws inputs*: keys, values, queries, calibration keys and the
low-rank adapter obtained from them.  It contains none of the method's arithmetic
(no metadata projection, no scoring, no selection, no attention), so that the CPU
oracle and the CUDA library can both be fed from it without sharing any of the
code under test.

The synthetic tensors stand in for the language models and datasets of the paper's
evaluation (Sec. 5.1): they take the models' shapes (GQA head counts, head_dim 128,
16-bit KV entries of 512 B per head, Sec. 3.2 footnote) and the structure the
method relies on -- a small set of dominant tokens (Sec. 3.2, App. A.2) and
step-to-step overlap of the selected groups (Sec. 4.4.2).

The adapter ``proj`` follows Sec. 4.2: the top-r right singular vectors of a
flattened calibration K cache, computed offline.  It is an *input* of the library.

Everything is numpy on the host.  16-bit values are produced by rounding fp32
draws to nearest-even and are carried both as raw ``uint16`` bit patterns (what the
GPU receives) and as the exactly up-cast ``float32`` values (what the oracle
receives), so both sides see identical numbers.
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Optional

import numpy as np

BASE_SEED = 20251111

# dtype tags (same integer values as the C enum kvswap_dtype)
F32, BF16, F16 = 0, 1, 2
E4M3 = 3          # 8-bit metadata only
# scope tags (same integer values as the C enum kvswap_scope)
SCOPE_KV_HEAD, SCOPE_ALL_HEADS = 0, 1


# --------------------------------------------------------------------------------------
# 16-bit storage helpers (bit manipulation only)
# --------------------------------------------------------------------------------------
def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest-even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_values(bits: np.ndarray) -> np.ndarray:
    """Exact fp32 value of bfloat16 bit patterns."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f16_bits(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x).astype(np.float16).view(np.uint16)


def f16_values(bits: np.ndarray) -> np.ndarray:
    return bits.view(np.float16).astype(np.float32)


def store(x: np.ndarray, dtype: int):
    """Round ``x`` to storage type ``dtype``; returns (raw array for the GPU, fp32 values)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == F32:
        return x, x
    if dtype == BF16:
        b = bf16_bits(x)
        return b, bf16_values(b)
    if dtype == F16:
        b = f16_bits(x)
        return b, f16_values(b)
    raise ValueError(f"unknown dtype tag {dtype}")


def rng_for(seed: int, name: str) -> np.random.Generator:
    """Independent sub-stream per (seed, tensor name)."""
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, zlib.crc32(name.encode())])))


# --------------------------------------------------------------------------------------
# Workload description
# --------------------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Workload:
    """One of the benchmark configurations (or a reduced copy of one for fast tests)."""
    name: str
    config: int            # 1..5, used in the seed
    layers: int            # L
    batch: int             # B
    n_ctx: int             # N
    n_q_heads: int         # H_q
    n_kv_heads: int        # H_kv
    head_dim: int          # d
    rank: int              # r
    group_size: int        # G
    top_k: int             # M
    kv_dtype: int
    meta_dtype: int
    q_dtype: int
    calib_rows: int
    heavy_frac: float = 0.0      # fraction of positions with planted query-aligned keys
    outlier_channels: int = 0    # channels per KV head whose K entries are scaled
    outlier_scale: float = 10.0
    walk_steps: int = 1          # >1: random-walk queries over consecutive decode steps
    walk_corr: float = 0.95

    @property
    def rho(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_groups(self) -> int:
        return self.n_ctx // self.group_size

    def reduced(self, name: str, **kw) -> "Workload":
        return dataclasses.replace(self, name=name, **kw)


CONFIGS = {
    1: Workload("cfg1", 1, 1, 1, 2048, 8, 2, 64, 16, 4, 32, F32, F32, F32, 4096),
    2: Workload("cfg2", 2, 1, 1, 16384, 32, 8, 128, 32, 8, 256, BF16, F16, BF16, 8192, heavy_frac=0.01),
    3: Workload("cfg3", 3, 36, 8, 32768, 32, 8, 128, 32, 8, 400, BF16, F16, BF16, 8192),
    4: Workload("cfg4", 4, 28, 16, 65536, 24, 8, 128, 32, 16, 256, BF16, F16, BF16, 8192,
                heavy_frac=0.005, outlier_channels=4),
    5: Workload("cfg5", 5, 36, 4, 131072, 32, 8, 128, 32, 8, 1024, BF16, F16, BF16, 8192, walk_steps=64),
}


@dataclasses.dataclass
class LayerInputs:
    """Inputs of one layer.  ``*_raw`` go to the GPU; the fp32 arrays hold the same values."""
    wl: Workload
    layer: int
    meta_heads: int                 # 1 (joint adapter) or H_kv (one adapter per KV head)
    K: np.ndarray                   # [B, H_kv, N, d] fp32 values as stored
    V: np.ndarray
    q: np.ndarray                   # [B, H_q, d]
    K_raw: np.ndarray
    V_raw: np.ndarray
    q_raw: np.ndarray
    proj: np.ndarray                # [H_kv, d, r] fp32
    heavy_pos: Optional[np.ndarray] = None   # [B, n_heavy] planted positions
    q_walk: Optional[np.ndarray] = None      # [steps, B, H_q, d] fp32 values as stored
    q_walk_raw: Optional[np.ndarray] = None


# --------------------------------------------------------------------------------------
# Adapter from a calibration set (offline step of Sec. 4.2; fixture, not product code)
# --------------------------------------------------------------------------------------
def _fix_signs(vecs: np.ndarray) -> np.ndarray:
    """Make each column's largest-magnitude entry positive (determinism only)."""
    piv = np.argmax(np.abs(vecs), axis=0)
    sgn = np.sign(vecs[piv, np.arange(vecs.shape[1])])
    sgn[sgn == 0] = 1.0
    return vecs * sgn


def adapter_from_calibration(calib: np.ndarray, n_kv_heads: int, head_dim: int, rank: int,
                             meta_heads: int, dtype=np.float32) -> np.ndarray:
    """Top-``rank`` right singular vectors of the calibration keys, as ``[H_kv, d, r]`` fp32.

    ``calib`` is ``[rows, H_kv, d]``.  Joint adapter (meta_heads == 1): one SVD of the
    ``rows x (H_kv*d)`` flattened matrix, head-major columns, split into row blocks A_g.
    Per-head adapters (meta_heads == H_kv): one SVD of ``rows x d`` per head.
    No centering; singular values in decreasing order.
    """
    rows = calib.shape[0]
    c64 = calib.astype(np.float64)
    if meta_heads == 1:
        flat = c64.reshape(rows, n_kv_heads * head_dim)
        _, _, vt = np.linalg.svd(flat, full_matrices=False)
        a = _fix_signs(vt[:rank].T)                       # [(H_kv*d), r]
        return np.ascontiguousarray(a.reshape(n_kv_heads, head_dim, rank), dtype=dtype)
    out = np.empty((n_kv_heads, head_dim, rank), dtype=dtype)
    for g in range(n_kv_heads):
        _, _, vt = np.linalg.svd(c64[:, g, :], full_matrices=False)
        out[g] = _fix_signs(vt[:rank].T).astype(dtype)
    return out


def _outlier_channels(wl: Workload, seed: int) -> Optional[np.ndarray]:
    if wl.outlier_channels == 0:
        return None
    r = rng_for(seed, "outlier")
    return np.stack([r.choice(wl.head_dim, size=wl.outlier_channels, replace=False)
                     for _ in range(wl.n_kv_heads)])      # [H_kv, n_out]


def layer_seed(wl: Workload, layer: int) -> int:
    return BASE_SEED + 1000 * wl.config + layer


def make_layer(wl: Workload, layer: int = 0, meta_heads: int = 1) -> LayerInputs:
    """Draw all inputs of one layer of ``wl`` on the host."""
    seed = layer_seed(wl, layer)
    B, Hq, Hkv, N, d = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.n_ctx, wl.head_dim
    rho = wl.rho
    K = rng_for(seed, "K").standard_normal((B, Hkv, N, d), dtype=np.float32)
    V = rng_for(seed, "V").standard_normal((B, Hkv, N, d), dtype=np.float32)
    q = rng_for(seed, "q").standard_normal((B, Hq, d), dtype=np.float32)
    calib = rng_for(seed, "cal").standard_normal((wl.calib_rows, Hkv, d), dtype=np.float32)

    q_raw, q_vals = store(q, wl.q_dtype)

    heavy_pos = None
    if wl.heavy_frac > 0.0:
        n_heavy = int(round(wl.heavy_frac * N))
        hr = rng_for(seed, "heavy")
        heavy_pos = np.stack([np.sort(hr.choice(N, size=n_heavy, replace=False)) for _ in range(B)])
        for b in range(B):
            for g in range(Hkv):
                qm = q_vals[b, g * rho:(g + 1) * rho].astype(np.float64).mean(axis=0)
                qhat = qm / np.linalg.norm(qm)
                noise = hr.standard_normal((n_heavy, d))
                noise -= np.outer(noise @ qhat, qhat)
                noise /= np.linalg.norm(noise, axis=1, keepdims=True)
                K[b, g, heavy_pos[b]] = (np.sqrt(d) * (0.8 * qhat[None, :] + 0.6 * noise)).astype(np.float32)

    och = _outlier_channels(wl, seed)
    if och is not None:
        for g in range(Hkv):
            K[:, g, :, och[g]] *= np.float32(wl.outlier_scale)
            calib[:, g, och[g]] *= np.float32(wl.outlier_scale)

    K_raw, K_vals = store(K, wl.kv_dtype)
    V_raw, V_vals = store(V, wl.kv_dtype)
    proj = adapter_from_calibration(calib, Hkv, d, wl.rank, meta_heads)

    q_walk = q_walk_raw = None
    if wl.walk_steps > 1:
        wr = rng_for(seed, "walk")
        steps = [q.copy()]
        c = np.float32(wl.walk_corr)
        s = np.float32(np.sqrt(1.0 - wl.walk_corr ** 2))
        for _ in range(wl.walk_steps - 1):
            steps.append(c * steps[-1] + s * wr.standard_normal(q.shape, dtype=np.float32))
        q_walk_raw, q_walk = store(np.stack(steps), wl.q_dtype)

    return LayerInputs(wl=wl, layer=layer, meta_heads=meta_heads, K=K_vals, V=V_vals, q=q_vals,
                       K_raw=K_raw, V_raw=V_raw, q_raw=q_raw, proj=proj, heavy_pos=heavy_pos,
                       q_walk=q_walk, q_walk_raw=q_walk_raw)


# Reduced copies: same structure, sizes the fp64 oracle finishes in seconds, still several
# kernel tiles long and with a ragged tail (N not a multiple of G) where noted.
REDUCED = {
    3: CONFIGS[3].reduced("cfg3-small", layers=2, batch=2, n_ctx=4096 + 5, top_k=50, calib_rows=2048),
    4: CONFIGS[4].reduced("cfg4-small", layers=2, batch=2, n_ctx=8192 + 11, top_k=32, calib_rows=2048),
    5: CONFIGS[5].reduced("cfg5-small", layers=1, batch=2, n_ctx=8192, top_k=64, calib_rows=2048,
                          walk_steps=8),
}
