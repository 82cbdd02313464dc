"""ctypes binding of libkvswap.so: argument marshalling only.

Every function has the name and argument order of its C entry point (include/kvswap.h).
Tensors are torch CUDA tensors; the binding passes ``data_ptr()`` and the current CUDA stream
and raises ``KVSwapError`` on a non-zero status.  There is no fallback: if the shared library
is missing or cannot be loaded, importing a function from here raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkvswap.so")

KVSWAP_F32, KVSWAP_BF16, KVSWAP_F16, KVSWAP_E4M3 = 0, 1, 2, 3
KVSWAP_SCOPE_KV_HEAD, KVSWAP_SCOPE_ALL_HEADS = 0, 1
KVSWAP_INPUTS_SETTLED = 1      # kvswap_shape.flags
KVSWAP_SCORE_SOFTMAX = 2
KVSWAP_CHECK_INDICES = 4


def KVSWAP_META_EXP(e: int) -> int:
    """kvswap_shape.flags bits of the power of two 8-bit metadata is stored with."""
    return (int(e) & 0xff) << 8


class KVSwapError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class kvswap_shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch", "n_ctx", "n_q_heads", "n_kv_heads", "head_dim", "rank", "meta_heads", "group_size",
        "top_k", "kv_dtype", "meta_dtype", "q_dtype", "scope", "flags")] + [(n, ctypes.c_int64) for n in (
        "kv_stride_b", "kv_stride_h", "kv_stride_n", "meta_stride_b", "meta_stride_h", "meta_stride_n")]

    def with_flags(self, flags: int) -> "kvswap_shape":
        """A copy of the shape with `flags` set."""
        other = kvswap_shape.from_buffer_copy(self)
        other.flags = int(flags)
        return other

    @property
    def n_scopes(self) -> int:
        return self.n_kv_heads if self.scope == KVSWAP_SCOPE_KV_HEAD else 1

    @property
    def n_groups(self) -> int:
        return self.n_ctx // self.group_size


_lib = None


def load() -> ctypes.CDLL:
    """Load libkvswap.so (once).  Raises if it has not been built: there is no CPU fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} not found: build it with `python -m paper_2511_11907_b200.build` "
            "(the kvswap hot path has no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    P, V, I32, SZ = ctypes.POINTER(kvswap_shape), ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.kvswap_workspace_bytes.restype = SZ
    lib.kvswap_workspace_bytes.argtypes = [P]
    lib.kvswap_validate_shape.restype = ctypes.c_int
    lib.kvswap_validate_shape.argtypes = [P]
    lib.kvswap_project_keys.restype = ctypes.c_int
    lib.kvswap_project_keys.argtypes = [P, V, V, V, I32, I32, V, SZ, V]
    lib.kvswap_append_kv.restype = ctypes.c_int
    lib.kvswap_append_kv.argtypes = [P, V, V, V, V, V, V, ctypes.POINTER(ctypes.c_int32), V]
    lib.kvswap_reuse_state_bytes.restype = ctypes.c_size_t
    lib.kvswap_reuse_state_bytes.argtypes = [P, I32, I32]
    lib.kvswap_reuse_init.restype = ctypes.c_int
    lib.kvswap_reuse_init.argtypes = [P, I32, I32, V, SZ, V]
    lib.kvswap_reuse_lookup.restype = ctypes.c_int
    lib.kvswap_reuse_lookup.argtypes = [P, I32, I32, V, V, V, SZ, V, V, V, V, V]
    lib.kvswap_reuse_fill.restype = ctypes.c_int
    lib.kvswap_reuse_fill.argtypes = [P, I32, V, V, V, V, V, V, V, V]
    lib.kvswap_score_select.restype = ctypes.c_int
    lib.kvswap_score_select.argtypes = [P, V, V, V, V, V, V, V, SZ, V]
    lib.kvswap_sparse_decode.restype = ctypes.c_int
    lib.kvswap_sparse_decode.argtypes = [P, V, V, V, V, V, V, V, V, SZ, V]
    lib.kvswap_status_string.restype = ctypes.c_char_p
    lib.kvswap_status_string.argtypes = [ctypes.c_int]
    lib.kvswap_version.restype = ctypes.c_int
    lib.kvswap_version.argtypes = []
    lib.kvswap_workspace_init.restype = ctypes.c_int
    lib.kvswap_workspace_init.argtypes = [V, SZ, V]
    lib.kvswap_read_device_status.restype = ctypes.c_int
    lib.kvswap_read_device_status.argtypes = [V, V]
    lib.kvswap_read_probe.restype = ctypes.c_int
    lib.kvswap_read_probe.argtypes = [V, SZ, V, V]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().kvswap_status_string(int(status)).decode()


def make_shape(*, batch, n_ctx, n_q_heads, n_kv_heads, head_dim, rank, meta_heads, group_size, top_k,
               kv_dtype, meta_dtype, q_dtype, scope=KVSWAP_SCOPE_KV_HEAD, kv_strides=(0, 0, 0),
               meta_strides=(0, 0, 0), flags=0) -> kvswap_shape:
    return kvswap_shape(batch, n_ctx, n_q_heads, n_kv_heads, head_dim, rank, meta_heads, group_size, top_k,
                        kv_dtype, meta_dtype, q_dtype, scope, flags, *kv_strides, *meta_strides)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return getattr(stream, "cuda_stream", stream) or None


def _check(status: int, where: str) -> None:
    if status != 0:
        raise KVSwapError(status, where)


def kvswap_workspace_bytes(shape: kvswap_shape) -> int:
    return int(load().kvswap_workspace_bytes(ctypes.byref(shape)))


def kvswap_validate_shape(shape: kvswap_shape) -> int:
    return int(load().kvswap_validate_shape(ctypes.byref(shape)))


def kvswap_project_keys(shape, K, proj, meta_out, n_begin, n_end, ws, stream=None) -> None:
    _check(load().kvswap_project_keys(ctypes.byref(shape), _ptr(K), _ptr(proj), _ptr(meta_out), int(n_begin),
                                      int(n_end), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                      _stream(stream)), "kvswap_project_keys")


def kvswap_append_kv(shape: kvswap_shape, k_new, v_new, K, V, proj, meta, stream=None) -> bool:
    """Appends one token's entries at row shape.n_ctx; True if that completed (and flushed) a group."""
    flushed = ctypes.c_int32(0)
    _check(load().kvswap_append_kv(ctypes.byref(shape), _ptr(k_new), _ptr(v_new), _ptr(K), _ptr(V), _ptr(proj),
                                   _ptr(meta), ctypes.byref(flushed), _stream(stream)), "kvswap_append_kv")
    return bool(flushed.value)


def kvswap_reuse_state_bytes(shape: kvswap_shape, n_slots: int, max_groups: int) -> int:
    return int(load().kvswap_reuse_state_bytes(ctypes.byref(shape), n_slots, max_groups))


def kvswap_reuse_init(shape, n_slots, max_groups, state, stream=None) -> None:
    _check(load().kvswap_reuse_init(ctypes.byref(shape), n_slots, max_groups, _ptr(state),
                                    state.numel() * state.element_size(), _stream(stream)), "kvswap_reuse_init")


def kvswap_reuse_lookup(shape, n_slots, max_groups, group_idx, n_selected, state, slot_idx, miss_group, miss_slot,
                        n_miss, stream=None) -> None:
    _check(load().kvswap_reuse_lookup(ctypes.byref(shape), n_slots, max_groups, _ptr(group_idx), _ptr(n_selected),
                                      _ptr(state), state.numel() * state.element_size(), _ptr(slot_idx),
                                      _ptr(miss_group), _ptr(miss_slot), _ptr(n_miss), _stream(stream)),
           "kvswap_reuse_lookup")


def kvswap_reuse_fill(shape, n_slots, K_slow, V_slow, K_reuse, V_reuse, miss_group, miss_slot, n_miss,
                      stream=None) -> None:
    """K_slow / V_slow may be CUDA tensors or pinned CPU tensors (read by the GPU in place)."""
    _check(load().kvswap_reuse_fill(ctypes.byref(shape), n_slots, _ptr(K_slow), _ptr(V_slow), _ptr(K_reuse),
                                    _ptr(V_reuse), _ptr(miss_group), _ptr(miss_slot), _ptr(n_miss), _stream(stream)),
           "kvswap_reuse_fill")


def reuse_attention_shape(shape: kvswap_shape, n_slots: int) -> kvswap_shape:
    """The shape that describes the reuse store to kvswap_sparse_decode: n_slots groups plus the
    rolling-buffer rows, dense [B, H_kv, (n_slots + 1) G, d]."""
    G, d, Hkv = shape.group_size, shape.head_dim, shape.n_kv_heads
    R = (n_slots + 1) * G
    other = kvswap_shape.from_buffer_copy(shape)
    other.n_ctx = n_slots * G + shape.n_ctx % G
    other.kv_stride_b, other.kv_stride_h, other.kv_stride_n = Hkv * R * d, R * d, d
    return other


def kvswap_score_select(shape, q, proj, meta, group_idx, n_selected, group_scores_opt, ws, stream=None) -> None:
    _check(load().kvswap_score_select(ctypes.byref(shape), _ptr(q), _ptr(proj), _ptr(meta), _ptr(group_idx),
                                      _ptr(n_selected), _ptr(group_scores_opt), _ptr(ws),
                                      0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "kvswap_score_select")


def kvswap_sparse_decode(shape, q, K, V, group_idx, n_selected, out, lse_opt, ws, stream=None) -> None:
    _check(load().kvswap_sparse_decode(ctypes.byref(shape), _ptr(q), _ptr(K), _ptr(V), _ptr(group_idx),
                                       _ptr(n_selected), _ptr(out), _ptr(lse_opt), _ptr(ws),
                                       0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "kvswap_sparse_decode")


def kvswap_workspace_init(ws, stream=None) -> None:
    _check(load().kvswap_workspace_init(_ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "kvswap_workspace_init")


def kvswap_read_probe(buf, n_bytes: int, sink=None, stream=None) -> None:
    """One read-only pass over the first n_bytes of `buf` (the benchmark's calibration kernel)."""
    _check(load().kvswap_read_probe(_ptr(buf), int(n_bytes), _ptr(sink), _stream(stream)), "kvswap_read_probe")


def kvswap_read_device_status(ws, stream=None) -> int:
    """Synchronises the stream; returns 0, KVSWAP_ERR_TIMEOUT (10) if a kernel gave up a wait, or
    KVSWAP_ERR_INDEX (8) if a call with KVSWAP_CHECK_INDICES met an index out of range."""
    return int(load().kvswap_read_device_status(_ptr(ws), _stream(stream)))


def kvswap_version() -> int:
    return int(load().kvswap_version())


# ------------------------------------------------------------------------------------------------
# Whole decode step over L layers
# ------------------------------------------------------------------------------------------------
class kvswap_layers(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("max_lookahead", ctypes.c_int32),
                ("K", ctypes.POINTER(ctypes.c_void_p)),
                ("V", ctypes.POINTER(ctypes.c_void_p)), ("meta", ctypes.POINTER(ctypes.c_void_p)),
                ("proj", ctypes.POINTER(ctypes.c_void_p))]


class kvswap_tiers(ctypes.Structure):
    _fields_ = [("n_slots", ctypes.c_int32), ("max_groups", ctypes.c_int32),
                ("K_slow", ctypes.POINTER(ctypes.c_void_p)), ("V_slow", ctypes.POINTER(ctypes.c_void_p)),
                ("K_reuse", ctypes.POINTER(ctypes.c_void_p)), ("V_reuse", ctypes.POINTER(ctypes.c_void_p)),
                ("state", ctypes.POINTER(ctypes.c_void_p)), ("state_bytes", ctypes.c_size_t),
                ("slot_idx", ctypes.c_void_p), ("miss_group", ctypes.c_void_p), ("miss_slot", ctypes.c_void_p),
                ("n_miss", ctypes.c_void_p)]


def make_tiers(n_slots, max_groups, K_slow, V_slow, K_reuse, V_reuse, state, slot_idx, miss_group, miss_slot,
               n_miss) -> kvswap_tiers:
    """Pointer tables for lists of per-layer tensors (K_slow / V_slow: CUDA or pinned CPU tensors) and the
    [L, ...] output tensors.  The returned struct keeps everything alive."""
    n = len(K_slow)
    assert all(len(x) == n for x in (V_slow, K_reuse, V_reuse, state))

    def table(ts):
        return (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])

    tabs = [table(K_slow), table(V_slow), table(K_reuse), table(V_reuse), table(state)]
    cast = [ctypes.cast(t, ctypes.POINTER(ctypes.c_void_p)) for t in tabs]
    tiers = kvswap_tiers(int(n_slots), int(max_groups), *cast, state[0].numel() * state[0].element_size(),
                         slot_idx.data_ptr(), miss_group.data_ptr(), miss_slot.data_ptr(), n_miss.data_ptr())
    tiers._keep = (tabs, list(K_slow), list(V_slow), list(K_reuse), list(V_reuse), list(state), slot_idx, miss_group,
                   miss_slot, n_miss)
    return tiers


class kvswap_probe(ctypes.Structure):
    _fields_ = [("layer", ctypes.c_int32), ("ev_begin", ctypes.c_void_p), ("ev_mid", ctypes.c_void_p),
                ("ev_end", ctypes.c_void_p)]


def make_layers(K, V, meta, proj, max_lookahead: int = 0) -> kvswap_layers:
    """Pointer tables for lists of per-layer device tensors.  The returned struct keeps the
    tensors and the tables alive.  max_lookahead: layers the predictor of kvswap_decode_step may
    run ahead of the attention (0 = no limit, 1 = one layer, as a model allows)."""
    n = len(K)
    assert len(V) == n and len(meta) == n and len(proj) == n

    def table(ts):
        return (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])

    tabs = [table(K), table(V), table(meta), table(proj)]
    layers = kvswap_layers(n, int(max_lookahead), *[ctypes.cast(t, ctypes.POINTER(ctypes.c_void_p)) for t in tabs])
    layers._keep = (tabs, list(K), list(V), list(meta), list(proj))
    return layers


def make_probe(layer: int, ev_begin=None, ev_mid=None, ev_end=None) -> kvswap_probe:
    """Probe from torch.cuda.Event objects created with enable_timing=True.  An event's handle
    exists only once it has been recorded, so fresh events are recorded once here."""
    def handle(ev):
        if ev is None:
            return None
        if not ev.cuda_event:
            ev.record()
        return ev.cuda_event
    return kvswap_probe(int(layer), handle(ev_begin), handle(ev_mid), handle(ev_end))


def _declare_step(lib):
    if getattr(lib, "_step_declared", False):
        return lib
    V, SZ = ctypes.c_void_p, ctypes.c_size_t
    P, PL, PP = ctypes.POINTER(kvswap_shape), ctypes.POINTER(kvswap_layers), ctypes.POINTER(kvswap_probe)
    lib.kvswap_decode_step.restype = ctypes.c_int
    lib.kvswap_decode_step.argtypes = [P, PL, V, V, V, V, V, V, SZ, PP, V]
    lib.kvswap_append_step.restype = ctypes.c_int
    lib.kvswap_append_step.argtypes = [P, PL, V, V, ctypes.POINTER(ctypes.c_int32), V]
    PT = ctypes.POINTER(kvswap_tiers)
    lib.kvswap_tiered_workspace_bytes.restype = ctypes.c_size_t
    lib.kvswap_tiered_workspace_bytes.argtypes = [P, ctypes.c_int32]
    lib.kvswap_decode_step_tiered.restype = ctypes.c_int
    lib.kvswap_decode_step_tiered.argtypes = [P, PL, PT, V, V, V, V, V, V, SZ, V]
    lib.kvswap_append_step_tiered.restype = ctypes.c_int
    lib.kvswap_append_step_tiered.argtypes = [P, PL, PT, V, V, ctypes.POINTER(ctypes.c_int32), V]
    lib.kvswap_decode_step_host.restype = ctypes.c_int
    lib.kvswap_decode_step_host.argtypes = [P, PL, V, V, V, V, V, V, V, SZ, V]
    lib._step_declared = True
    return lib


def kvswap_decode_step(shape, layers, q, out, lse_opt, group_idx, n_selected, ws, probe_opt=None, stream=None) -> None:
    lib = _declare_step(load())
    _check(lib.kvswap_decode_step(ctypes.byref(shape), ctypes.byref(layers), _ptr(q), _ptr(out), _ptr(lse_opt),
                                  _ptr(group_idx), _ptr(n_selected), _ptr(ws), ws.numel() * ws.element_size(),
                                  None if probe_opt is None else ctypes.byref(probe_opt), _stream(stream)),
           "kvswap_decode_step")


def kvswap_append_step(shape, layers, k_new, v_new, stream=None) -> bool:
    """Appends one token per layer (k_new, v_new [L, B, H_kv, d]) at row shape.n_ctx; True if a group was flushed."""
    lib = _declare_step(load())
    flushed = ctypes.c_int32(0)
    _check(lib.kvswap_append_step(ctypes.byref(shape), ctypes.byref(layers), _ptr(k_new), _ptr(v_new),
                                  ctypes.byref(flushed), _stream(stream)), "kvswap_append_step")
    return bool(flushed.value)


def kvswap_tiered_workspace_bytes(shape, n_slots: int) -> int:
    return int(_declare_step(load()).kvswap_tiered_workspace_bytes(ctypes.byref(shape), n_slots))


def kvswap_decode_step_tiered(shape, layers, tiers, q, out, lse_opt, group_idx, n_selected, ws, stream=None) -> None:
    lib = _declare_step(load())
    _check(lib.kvswap_decode_step_tiered(ctypes.byref(shape), ctypes.byref(layers), ctypes.byref(tiers), _ptr(q),
                                         _ptr(out), _ptr(lse_opt), _ptr(group_idx), _ptr(n_selected), _ptr(ws),
                                         ws.numel() * ws.element_size(), _stream(stream)), "kvswap_decode_step_tiered")


def kvswap_append_step_tiered(shape, layers, tiers, k_new, v_new, stream=None) -> bool:
    lib = _declare_step(load())
    flushed = ctypes.c_int32(0)
    _check(lib.kvswap_append_step_tiered(ctypes.byref(shape), ctypes.byref(layers), ctypes.byref(tiers), _ptr(k_new),
                                         _ptr(v_new), ctypes.byref(flushed), _stream(stream)),
           "kvswap_append_step_tiered")
    return bool(flushed.value)


def kvswap_decode_step_host(shape, layers, q_host, out_host, q_dev, out_dev, group_idx, n_selected, ws,
                            stream=None) -> None:
    """q_host / out_host are CPU tensors (pinned for asynchronous copies)."""
    lib = _declare_step(load())
    _check(lib.kvswap_decode_step_host(ctypes.byref(shape), ctypes.byref(layers), _ptr(q_host), _ptr(out_host),
                                       _ptr(q_dev), _ptr(out_dev), _ptr(group_idx), _ptr(n_selected), _ptr(ws),
                                       ws.numel() * ws.element_size(), _stream(stream)), "kvswap_decode_step_host")


KVSWAP_STATIC_SCRATCH_BYTES = 8 << 20


def kvswap_sparse_decode_static(shape, q, K, V, group_idx, n_selected, out, lse_opt, stream=None) -> None:
    """kvswap_sparse_decode for callers that cannot hand over a workspace (they are not allowed
    to allocate device memory at the call site): the split-K partials go to a buffer built into
    the library.  Problems too large for that buffer raise KVSwapError (status 9).  Calls on one
    device share the buffer, so do not let two of them overlap on the GPU."""
    lib = load()
    if not getattr(lib, "_static_declared", False):
        V_ = ctypes.c_void_p
        lib.kvswap_sparse_decode_static.restype = ctypes.c_int
        lib.kvswap_sparse_decode_static.argtypes = [ctypes.POINTER(kvswap_shape), V_, V_, V_, V_, V_, V_, V_, V_]
        lib._static_declared = True
    _check(lib.kvswap_sparse_decode_static(ctypes.byref(shape), _ptr(q), _ptr(K), _ptr(V), _ptr(group_idx),
                                           _ptr(n_selected), _ptr(out), _ptr(lse_opt), _stream(stream)),
           "kvswap_sparse_decode_static")
