"""kvswap_sparse_decode_static -- the entry point for callers that may not allocate device
memory (a server whose memory manager owns the whole GPU, code inside a framework's enqueue
callback) and so cannot pass a workspace: its split-K partials sit in a buffer built into the
library.

Checked here, through the C ABI: its output equals that of kvswap_sparse_decode (which gets a
caller-allocated workspace) on two calls in a row with different inputs, so stale partials of
the first call cannot leak into the second; the device memory in use is the same before and
after a call (the property in its name); and a problem too large for the built-in buffer is
refused with its own status code before any pointer is looked at.  The file name sorts last so
that a run stopping at the first failure has already run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W
from parity_util import OUT_ATOL_TIGHT, DeviceLayer

pytestmark = pytest.mark.gpu


def _reference(dl):
    """The existing entry point, with a caller-provided workspace."""
    out, lse = rt.alloc_output(dl.shape)
    kv.kvswap_sparse_decode(dl.shape, dl.q, dl.K, dl.V, dl.idx, dl.nsel, out, lse, dl.ws)
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy()


def _static(dl):
    out, lse = rt.alloc_output(dl.shape)
    out.fill_(float("nan"))
    lse.fill_(float("nan"))
    kv.kvswap_sparse_decode_static(dl.shape, dl.q, dl.K, dl.V, dl.idx, dl.nsel, out, lse)
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy()


def test_static_scratch_entry_matches_workspace_entry_on_two_calls_in_a_row():
    wl = W.REDUCED[3]                                   # bf16 K/V, 2 sequences, ragged tail
    li = W.make_layer(wl, 0, 1)
    dl = DeviceLayer(li, W.SCOPE_KV_HEAD)
    rng = np.random.default_rng(7)
    tol = OUT_ATOL_TIGHT[wl.kv_dtype]
    for call in range(2):
        # a different selection and a different query on each call
        sel = np.stack([np.stack([np.sort(rng.choice(wl.n_groups, size=wl.top_k, replace=False))
                                  for _ in range(wl.n_kv_heads)]) for _ in range(wl.batch)]).astype(np.int32)
        dl.set_selection(sel)
        dl.q = torch.randn(dl.q.shape, device="cuda").to(dl.q.dtype)
        want_out, want_lse = _reference(dl)
        got_out, got_lse = _static(dl)
        assert np.all(np.isfinite(got_out)) and np.all(np.isfinite(got_lse))
        assert np.abs(got_out - want_out).max() <= tol, f"call {call}"
        assert np.abs(got_lse - want_lse).max() <= tol, f"call {call}"


def test_static_scratch_entry_leaves_device_memory_as_it_found_it():
    wl = W.REDUCED[3]
    li = W.make_layer(wl, 0, 1)
    dl = DeviceLayer(li, W.SCOPE_KV_HEAD)
    out, lse = rt.alloc_output(dl.shape)
    call = lambda: kv.kvswap_sparse_decode_static(dl.shape, dl.q, dl.K, dl.V, dl.idx, dl.nsel, out, lse)
    call()                                              # the first call on a device looks up the buffer's address
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    torch0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "the driver reports a different amount of free device memory after the calls"
    assert torch.cuda.memory_allocated() == torch0 and torch.cuda.memory_reserved() == reserved0


def test_static_scratch_entry_refuses_problems_beyond_its_buffer():
    # 2048 sequences x 32 heads x 130 floats of partials = 34 MB > the 8 MiB built-in buffer.
    shape = kv.make_shape(batch=2048, n_ctx=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, rank=32,
                          meta_heads=1, group_size=8, top_k=64, kv_dtype=W.BF16, meta_dtype=W.F16, q_dtype=W.BF16)
    assert kv.kvswap_validate_shape(shape) == 0
    lib = kv.load()
    lib.kvswap_sparse_decode_static.restype = ctypes.c_int
    lib.kvswap_sparse_decode_static.argtypes = [ctypes.POINTER(kv.kvswap_shape)] + [ctypes.c_void_p] * 8
    # the size check precedes every pointer check, so no pointer is needed to see the refusal
    status = lib.kvswap_sparse_decode_static(ctypes.byref(shape), None, None, None, None, None, None, None, None)
    assert status == 9
    assert "static" in kv.status_string(status)
