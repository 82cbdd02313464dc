"""Full-size synthetic workloads drawn directly in GPU memory (inputs only, no method arithmetic).

Same recipe as ``workloads.make_layer`` -- N(0,1) keys/values/queries per layer from
``seed = 20251111 + 1000*config + layer``, optional outlier channels and planted query-aligned
"heavy" keys, an adapter from the right singular vectors of a calibration set, random-walk
queries over consecutive decode steps -- but generated with ``torch.Generator(device="cuda")``
so that the 40-120 GB KV stores of the large configurations never pass through the host.
The adapter uses the eigenvectors of the calibration Gram matrix (the right singular vectors
of the calibration set) computed in float64 on the device.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import torch

from . import binding as kv
from . import runtime as rt
from . import workloads as W

_TD = {W.F32: torch.float32, W.BF16: torch.bfloat16, W.F16: torch.float16, W.E4M3: torch.float8_e4m3fn}


def _gen(seed: int, salt: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed * 131 + salt)
    return g


def adapter_on_device(calib: torch.Tensor, rank: int, meta_heads: int) -> torch.Tensor:
    """calib [rows, H_kv, d] fp32 -> proj [H_kv, d, r] fp32 (top-r right singular vectors)."""
    rows, Hkv, d = calib.shape

    def top_vectors(mat):                                  # mat [rows, D]
        m = mat.to(torch.float64)
        evals, evecs = torch.linalg.eigh(m.T @ m)
        v = evecs[:, torch.argsort(evals, descending=True)[:rank]]     # [D, r]
        piv = v.abs().argmax(dim=0)
        sgn = torch.sign(v[piv, torch.arange(rank, device=v.device)])
        sgn[sgn == 0] = 1
        return v * sgn

    if meta_heads == 1:
        a = top_vectors(calib.reshape(rows, Hkv * d))
        return a.reshape(Hkv, d, rank).to(torch.float32).contiguous()
    return torch.stack([top_vectors(calib[:, g]) for g in range(Hkv)]).to(torch.float32).contiguous()


@dataclasses.dataclass
class DeviceWorkload:
    wl: W.Workload
    shape: kv.kvswap_shape
    K: List[torch.Tensor]
    V: List[torch.Tensor]
    proj: List[torch.Tensor]
    meta: List[torch.Tensor]
    q_walk: torch.Tensor                 # [steps, L, B, H_q, d] q_dtype
    layers_resident: int                 # distinct K/V buffers (== L unless memory forced sharing)
    heavy_pos: Optional[List[torch.Tensor]] = None

    def layer_tables(self, max_lookahead: int = 0) -> kv.kvswap_layers:
        return kv.make_layers(self.K, self.V, self.meta, self.proj, max_lookahead)


def build(wl: W.Workload, meta_heads: int = 1, scope: int = W.SCOPE_KV_HEAD, device="cuda", rank_offset: int = 0,
          walk_steps: Optional[int] = None, reserve_bytes: int = 8 << 30) -> DeviceWorkload:
    """Draw the whole workload on ``device``.  Metadata buffers are allocated, not filled
    (kvswap_project_keys fills them).  If the K/V stores of all L layers do not fit in the free
    memory, fewer distinct buffers are drawn and layers share them round-robin; the number
    actually resident is returned in ``layers_resident`` and must be reported."""
    dev = torch.device(device)
    shape = rt.shape_for(wl, meta_heads, scope)
    B, Hq, Hkv, N, d, L = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.n_ctx, wl.head_dim, wl.layers
    rho = wl.rho
    kv_bytes = 2 * B * Hkv * N * d * torch.empty((), dtype=_TD[wl.kv_dtype]).element_size()
    meta_bytes = B * meta_heads * N * wl.rank * torch.empty((), dtype=_TD[wl.meta_dtype]).element_size()
    free, _ = torch.cuda.mem_get_info(dev)
    fit = int((free - reserve_bytes - L * meta_bytes) // kv_bytes)
    resident = max(1, min(L, fit))
    steps = walk_steps if walk_steps is not None else max(1, wl.walk_steps)

    K, V, proj, meta, heavy = [], [], [], [], []
    q_walk = torch.empty((steps, L, B, Hq, d), dtype=_TD[wl.q_dtype], device=dev)
    for l in range(L):
        seed = W.layer_seed(wl, l) + 7919 * rank_offset
        q0 = torch.randn((B, Hq, d), generator=_gen(seed, 3, dev), device=dev)
        qs = [q0]
        gw = _gen(seed, 4, dev)
        c, s = wl.walk_corr, (1.0 - wl.walk_corr ** 2) ** 0.5
        for _ in range(steps - 1):
            qs.append(c * qs[-1] + s * torch.randn((B, Hq, d), generator=gw, device=dev))
        q_walk[:, l] = torch.stack(qs).to(_TD[wl.q_dtype])

        calib = torch.randn((wl.calib_rows, Hkv, d), generator=_gen(seed, 5, dev), device=dev)
        och = None
        if wl.outlier_channels:
            go = _gen(seed, 6, dev)
            och = torch.stack([torch.randperm(d, generator=go, device=dev)[:wl.outlier_channels] for _ in range(Hkv)])
            for g in range(Hkv):
                calib[:, g, och[g]] *= wl.outlier_scale
        proj.append(adapter_on_device(calib, wl.rank, meta_heads))
        del calib

        if l < resident:
            Kl = torch.empty((B, Hkv, N, d), dtype=_TD[wl.kv_dtype], device=dev)
            Vl = torch.empty((B, Hkv, N, d), dtype=_TD[wl.kv_dtype], device=dev)
            gk, gv = _gen(seed, 1, dev), _gen(seed, 2, dev)
            for b in range(B):                                      # per sequence: bounded temporaries
                Kl[b] = torch.randn((Hkv, N, d), generator=gk, device=dev).to(_TD[wl.kv_dtype])
                Vl[b] = torch.randn((Hkv, N, d), generator=gv, device=dev).to(_TD[wl.kv_dtype])
            if wl.heavy_frac > 0:
                gh = _gen(seed, 7, dev)
                n_heavy = int(round(wl.heavy_frac * N))
                qv = q_walk[0, l].to(torch.float32)                  # stored query values
                pos_l = []
                for b in range(B):
                    pos = torch.randperm(N, generator=gh, device=dev)[:n_heavy].sort().values
                    pos_l.append(pos)
                    for g in range(Hkv):
                        qhat = qv[b, g * rho:(g + 1) * rho].mean(dim=0)
                        qhat = qhat / qhat.norm()
                        noise = torch.randn((n_heavy, d), generator=gh, device=dev)
                        noise -= torch.outer(noise @ qhat, qhat)
                        noise /= noise.norm(dim=1, keepdim=True)
                        Kl[b, g, pos] = ((d ** 0.5) * (0.8 * qhat[None] + 0.6 * noise)).to(_TD[wl.kv_dtype])
                heavy.append(torch.stack(pos_l))
            if och is not None:
                for g in range(Hkv):
                    Kl[:, g, :, och[g]] = (Kl[:, g, :, och[g]].to(torch.float32) * wl.outlier_scale).to(_TD[wl.kv_dtype])
            K.append(Kl)
            V.append(Vl)
        else:
            K.append(K[l % resident])
            V.append(V[l % resident])
        meta.append(torch.empty((B, meta_heads, N, wl.rank), dtype=_TD[wl.meta_dtype], device=dev))
    return DeviceWorkload(wl=wl, shape=shape, K=K, V=V, proj=proj, meta=meta, q_walk=q_walk,
                          layers_resident=resident, heavy_pos=heavy or None)
