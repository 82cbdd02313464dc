"""Small conveniences around the binding: shapes from workloads, host->device marshalling and
buffer allocation.  torch is used for device memory and streams only."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as kv
from . import workloads as W

_TORCH_DTYPE = {W.F32: torch.float32, W.BF16: torch.bfloat16, W.F16: torch.float16, W.E4M3: torch.float8_e4m3fn}


def shape_for(wl: W.Workload, meta_heads: int = 1, scope: int = W.SCOPE_KV_HEAD, **override) -> kv.kvswap_shape:
    args = dict(batch=wl.batch, n_ctx=wl.n_ctx, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                head_dim=wl.head_dim, rank=wl.rank, meta_heads=meta_heads, group_size=wl.group_size,
                top_k=wl.top_k, kv_dtype=wl.kv_dtype, meta_dtype=wl.meta_dtype, q_dtype=wl.q_dtype, scope=scope)
    args.update(override)
    return kv.make_shape(**args)


def to_device(raw: np.ndarray, dtype: int, device="cuda") -> torch.Tensor:
    """Raw storage array from the generators (fp32 values or uint16 bit patterns) -> device tensor."""
    if dtype == W.F32:
        return torch.from_numpy(np.ascontiguousarray(raw, dtype=np.float32)).to(device)
    t = torch.from_numpy(np.ascontiguousarray(raw).view(np.int16)).to(device)
    return t.view(_TORCH_DTYPE[dtype])


def to_host_f32(t: torch.Tensor) -> np.ndarray:
    """Exact fp32 values of a device tensor of any storage type."""
    return t.detach().to(torch.float32).cpu().numpy()


def alloc_workspace(shape: kv.kvswap_shape, device="cuda") -> torch.Tensor:
    n = kv.kvswap_workspace_bytes(shape)
    if n == 0:
        raise kv.KVSwapError(kv.kvswap_validate_shape(shape), "kvswap_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    kv.kvswap_workspace_init(ws)
    return ws


def alloc_meta(shape: kv.kvswap_shape, device="cuda") -> torch.Tensor:
    return torch.empty((shape.batch, shape.meta_heads, shape.n_ctx, shape.rank),
                       dtype=_TORCH_DTYPE[shape.meta_dtype], device=device)


def alloc_selection(shape: kv.kvswap_shape, device="cuda"):
    S = shape.n_scopes
    idx = torch.empty((shape.batch, S, shape.top_k), dtype=torch.int32, device=device)
    nsel = torch.empty((shape.batch, S), dtype=torch.int32, device=device)
    return idx, nsel


def alloc_output(shape: kv.kvswap_shape, device="cuda"):
    out = torch.empty((shape.batch, shape.n_q_heads, shape.head_dim), dtype=torch.float32, device=device)
    lse = torch.empty((shape.batch, shape.n_q_heads), dtype=torch.float32, device=device)
    return out, lse
