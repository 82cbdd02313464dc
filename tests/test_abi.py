"""The C-ABI library loads, exports every symbol declared in include/kvswap.h, and its host-side
validation returns the documented status codes.  No GPU needed: no compute entry point is reached
with valid arguments."""
import ctypes
import os
import re

import pytest

from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import build as kvbuild
from paper_2511_11907_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kvbuild.build()
    return kv.load()


def _declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(kvswap_\w+)\s*\(", text))
    return names


def good_shape(**kw):
    args = dict(batch=2, n_ctx=1024, n_q_heads=8, n_kv_heads=2, head_dim=64, rank=16, meta_heads=1,
                group_size=4, top_k=32, kv_dtype=W.F32, meta_dtype=W.F32, q_dtype=W.F32)
    args.update(kw)
    return kv.make_shape(**args)


def test_every_declared_symbol_is_exported(lib):
    declared = _declared_functions()
    assert {"kvswap_project_keys", "kvswap_score_select", "kvswap_sparse_decode",
            "kvswap_workspace_bytes", "kvswap_status_string"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"


def test_struct_layout_matches_header():
    assert ctypes.sizeof(kv.kvswap_shape) == 13 * 4 + 4 + 6 * 8   # 13 int32, padding, 6 int64


def test_layers_struct_layout_matches_header():
    # int32 n_layers, int32 max_lookahead, four pointers
    assert ctypes.sizeof(kv.kvswap_layers) == 8 + 4 * ctypes.sizeof(ctypes.c_void_p)
    assert kv.kvswap_layers.max_lookahead.offset == 4 and kv.kvswap_layers.K.offset == 8


def test_decode_step_rejects_bad_layer_tables(lib):
    kv._declare_step(lib)
    s = good_shape()
    fake = ctypes.c_void_p(4096)
    tab = (ctypes.c_void_p * 1)(4096)
    ptab = ctypes.cast(tab, ctypes.POINTER(ctypes.c_void_p))
    assert lib.kvswap_decode_step(ctypes.byref(s), None, fake, fake, None, fake, fake, fake, 1 << 30, None, None) == 1
    for bad in (kv.kvswap_layers(0, 0, ptab, ptab, ptab, ptab), kv.kvswap_layers(1, -1, ptab, ptab, ptab, ptab)):
        assert lib.kvswap_decode_step(ctypes.byref(s), ctypes.byref(bad), fake, fake, None, fake, fake, fake,
                                      1 << 30, None, None) == 2
    ok = kv.kvswap_layers(1, 0, ptab, ptab, ptab, ptab)
    assert lib.kvswap_decode_step(ctypes.byref(s), ctypes.byref(ok), fake, fake, None, fake, fake, fake, 16,
                                  None, None) == 5        # workspace too small: refused before any launch


def test_validation_status_codes(lib):
    assert kv.kvswap_validate_shape(good_shape()) == 0
    assert kv.kvswap_workspace_bytes(good_shape()) > 0
    bad = {
        2: [dict(batch=0), dict(n_ctx=0), dict(n_q_heads=7), dict(meta_heads=3), dict(group_size=0),
            dict(top_k=0), dict(scope=5), dict(kv_strides=(0, 0, 32))],
        3: [dict(kv_dtype=9), dict(meta_dtype=W.BF16), dict(kv_dtype=W.F32, q_dtype=W.BF16)],
        4: [dict(rank=4, meta_dtype=W.F16), dict(kv_strides=(0, 0, 66))],
        6: [dict(head_dim=96), dict(rank=18), dict(rank=512), dict(group_size=2048)],
    }
    for code, cases in bad.items():
        for c in cases:
            s = good_shape(**c)
            assert kv.kvswap_validate_shape(s) == code, (code, c)
            assert kv.kvswap_workspace_bytes(s) == 0
    assert lib.kvswap_validate_shape(None) == 1
    assert kv.kvswap_validate_shape(good_shape(flags=kv.KVSWAP_INPUTS_SETTLED)) == 0
    assert kv.kvswap_validate_shape(good_shape(flags=kv.KVSWAP_SCORE_SOFTMAX | kv.KVSWAP_INPUTS_SETTLED)) == 0
    assert kv.kvswap_validate_shape(good_shape(flags=kv.KVSWAP_CHECK_INDICES)) == 0
    assert kv.kvswap_validate_shape(good_shape(flags=8)) == 2          # unknown flag bit


def test_entry_points_reject_null_and_small_workspace_without_touching_the_gpu(lib):
    s = good_shape()
    ref = ctypes.byref(s)
    assert lib.kvswap_project_keys(ref, None, None, None, 0, 8, None, 0, None) == 1
    assert lib.kvswap_score_select(ref, None, None, None, None, None, None, None, 0, None) == 1
    assert lib.kvswap_sparse_decode(ref, None, None, None, None, None, None, None, None, 0, None) == 1
    fake = ctypes.c_void_p(4096)                     # aligned, never dereferenced on these paths
    assert lib.kvswap_project_keys(ref, fake, fake, fake, 8, 4, None, 0, None) == 2       # bad range
    assert lib.kvswap_project_keys(ref, fake, fake, fake, 0, 4096, None, 0, None) == 2    # beyond N
    assert lib.kvswap_project_keys(ref, fake, fake, fake, 5, 5, None, 0, None) == 0       # empty: no-op
    assert lib.kvswap_project_keys(ref, ctypes.c_void_p(4100), fake, fake, 0, 8, None, 0, None) == 4
    assert lib.kvswap_score_select(ref, fake, fake, fake, fake, fake, None, fake, 16, None) == 5
    assert lib.kvswap_sparse_decode(ref, fake, fake, fake, fake, fake, fake, None, fake, 16, None) == 5


def test_append_kv_validates_before_touching_the_gpu(lib):
    fake = ctypes.c_void_p(4096)
    flushed = ctypes.c_int32(7)
    dense = good_shape()
    assert lib.kvswap_append_kv(ctypes.byref(dense), fake, fake, fake, fake, fake, fake, ctypes.byref(flushed), None) == 2
    assert flushed.value == 0
    N, d, r = 1024, 64, 16
    roomy = good_shape(kv_strides=(2 * (N + 8) * d, (N + 8) * d, d), meta_strides=((N + 8) * r, (N + 8) * r, r))
    assert lib.kvswap_append_kv(ctypes.byref(roomy), None, fake, fake, fake, fake, fake, None, None) == 1
    assert lib.kvswap_append_kv(ctypes.byref(roomy), ctypes.c_void_p(4100), fake, fake, fake, fake, fake, None, None) == 4
    tight = good_shape(kv_strides=(2 * N * d, N * d, d), meta_strides=((N + 8) * r, (N + 8) * r, r))
    assert lib.kvswap_append_kv(ctypes.byref(tight), fake, fake, fake, fake, fake, fake, None, None) == 2   # K/V full
    tight_meta = good_shape(kv_strides=(2 * (N + 8) * d, (N + 8) * d, d), meta_strides=(N * r, N * r, r))
    assert lib.kvswap_append_kv(ctypes.byref(tight_meta), fake, fake, fake, fake, fake, fake, None, None) == 2
    assert lib.kvswap_append_kv(None, fake, fake, fake, fake, fake, fake, None, None) == 1
    kv._declare_step(lib)
    tab = (ctypes.c_void_p * 1)(4096)
    ptab = ctypes.cast(tab, ctypes.POINTER(ctypes.c_void_p))
    one = kv.kvswap_layers(1, 0, ptab, ptab, ptab, ptab)
    assert lib.kvswap_append_step(ctypes.byref(dense), ctypes.byref(one), fake, fake, None, None) == 2
    assert lib.kvswap_append_step(ctypes.byref(roomy), None, fake, fake, None, None) == 1
    assert lib.kvswap_append_step(ctypes.byref(roomy), ctypes.byref(one), None, fake, None, None) == 1
    none = kv.kvswap_layers(0, 0, ptab, ptab, ptab, ptab)
    assert lib.kvswap_append_step(ctypes.byref(roomy), ctypes.byref(none), fake, fake, None, None) == 2


def test_reuse_buffer_calls_validate_before_touching_the_gpu(lib):
    s = good_shape()                                       # M = 32, B = 2, S = 2
    ref = ctypes.byref(s)
    fake = ctypes.c_void_p(4096)
    assert kv.kvswap_reuse_state_bytes(s, 64, 256) == 4 * 2 * 2 * (1 + 64 + 256)
    assert kv.kvswap_reuse_state_bytes(s, 16, 256) == 0                  # fewer slots than a step selects
    assert kv.kvswap_reuse_state_bytes(s, 64, 0) == 0
    assert kv.kvswap_reuse_state_bytes(s, 1 << 16, 256) == 0             # beyond the supported slot count
    assert lib.kvswap_reuse_init(ref, 16, 256, fake, 1 << 20, None) == 2
    assert lib.kvswap_reuse_init(ref, 1 << 16, 256, fake, 1 << 20, None) == 6
    assert lib.kvswap_reuse_init(ref, 64, 256, None, 1 << 20, None) == 1
    assert lib.kvswap_reuse_init(ref, 64, 256, fake, 16, None) == 5
    assert lib.kvswap_reuse_lookup(ref, 64, 256, None, fake, fake, 1 << 20, fake, fake, fake, fake, None) == 1
    assert lib.kvswap_reuse_lookup(ref, 64, 256, ctypes.c_void_p(4098), fake, fake, 1 << 20, fake, fake, fake, fake,
                                   None) == 4
    assert lib.kvswap_reuse_lookup(ref, 64, 256, fake, fake, fake, 64, fake, fake, fake, fake, None) == 5
    assert lib.kvswap_reuse_lookup(ref, 8, 256, fake, fake, fake, 1 << 20, fake, fake, fake, fake, None) == 2
    # the context has floor(1024 / 4) = 256 complete groups: tables sized for fewer cannot record all of them
    assert lib.kvswap_reuse_lookup(ref, 64, 255, fake, fake, fake, 1 << 20, fake, fake, fake, fake, None) == 2
    assert lib.kvswap_reuse_init(ref, 64, 255, fake, 1 << 20, None) == 2
    assert kv.kvswap_reuse_state_bytes(s, 64, 255) == 0
    assert lib.kvswap_reuse_fill(ref, 64, None, fake, fake, fake, fake, fake, fake, None) == 1
    assert lib.kvswap_reuse_fill(ref, 64, ctypes.c_void_p(4100), fake, fake, fake, fake, fake, fake, None) == 4
    assert lib.kvswap_reuse_fill(ref, 8, fake, fake, fake, fake, fake, fake, fake, None) == 2


def test_tiered_step_validates_before_touching_the_gpu(lib):
    kv._declare_step(lib)
    s = good_shape()
    assert kv.kvswap_tiered_workspace_bytes(s, 64) > kv.kvswap_workspace_bytes(s)
    assert kv.kvswap_tiered_workspace_bytes(s, 8) == 0
    fake = ctypes.c_void_p(4096)
    tab = (ctypes.c_void_p * 1)(4096)
    ptab = ctypes.cast(tab, ctypes.POINTER(ctypes.c_void_p))
    layers = kv.kvswap_layers(1, 0, None, None, ptab, ptab)               # K and V tables are not needed
    tiers = kv.kvswap_tiers(64, 256, ptab, ptab, ptab, ptab, ptab, 1 << 20, 4096, 4096, 4096, 4096)
    call = lambda t, ws_bytes: lib.kvswap_decode_step_tiered(ctypes.byref(s), ctypes.byref(layers), t, fake, fake, None,
                                                             fake, fake, fake, ws_bytes, None)
    assert call(None, 1 << 30) == 1
    assert call(ctypes.byref(tiers), 1024) == 5                            # workspace too small
    small_state = kv.kvswap_tiers(64, 256, ptab, ptab, ptab, ptab, ptab, 64, 4096, 4096, 4096, 4096)
    assert call(ctypes.byref(small_state), 1 << 30) == 5
    few_slots = kv.kvswap_tiers(8, 256, ptab, ptab, ptab, ptab, ptab, 1 << 20, 4096, 4096, 4096, 4096)
    assert call(ctypes.byref(few_slots), 1 << 30) == 2
    no_out = kv.kvswap_tiers(64, 256, ptab, ptab, ptab, ptab, ptab, 1 << 20, None, 4096, 4096, 4096)
    assert call(ctypes.byref(no_out), 1 << 30) == 1
    short_tables = kv.kvswap_tiers(64, 255, ptab, ptab, ptab, ptab, ptab, 1 << 20, 4096, 4096, 4096, 4096)
    assert call(ctypes.byref(short_tables), 1 << 30) == 2                  # 256 complete groups, tables for 255
    # tiered append: capacity rule as for kvswap_append_kv, then the tables
    N, d, r = 1024, 64, 16
    roomy = good_shape(kv_strides=(2 * (N + 8) * d, (N + 8) * d, d), meta_strides=((N + 8) * r, (N + 8) * r, r))
    app = lambda sh, t: lib.kvswap_append_step_tiered(ctypes.byref(sh), ctypes.byref(layers), t, fake, fake, None, None)
    assert app(s, ctypes.byref(tiers)) == 2                                # dense strides: no room stated
    assert app(roomy, None) == 1
    no_store = kv.kvswap_tiers(64, 256, ptab, ptab, None, ptab, ptab, 1 << 20, 4096, 4096, 4096, 4096)
    assert app(roomy, ctypes.byref(no_store)) == 1
    assert app(roomy, ctypes.byref(short_tables)) == 2                     # the grown context outruns the tables


def test_8bit_metadata_shapes_are_validated(lib):
    ok = good_shape(kv_dtype=W.BF16, q_dtype=W.BF16, meta_dtype=W.E4M3, rank=32, head_dim=128, group_size=8)
    assert kv.kvswap_validate_shape(ok) == 0
    assert kv.kvswap_validate_shape(ok.with_flags(kv.KVSWAP_META_EXP(-3))) == 0
    assert kv.kvswap_workspace_bytes(ok) > 0
    bad_rank = good_shape(kv_dtype=W.BF16, q_dtype=W.BF16, meta_dtype=W.E4M3, rank=16, head_dim=128, group_size=8)
    assert kv.kvswap_validate_shape(bad_rank) == 6                     # the 8-bit rows are read by one scorer only
    odd_group = good_shape(kv_dtype=W.BF16, q_dtype=W.BF16, meta_dtype=W.E4M3, rank=32, head_dim=128, group_size=3)
    assert kv.kvswap_validate_shape(odd_group) == 6
    assert kv.kvswap_validate_shape(ok.with_flags(kv.KVSWAP_SCORE_SOFTMAX)) == 6
    assert kv.kvswap_validate_shape(good_shape().with_flags(kv.KVSWAP_META_EXP(2))) == 2     # an exponent without 8-bit metadata
    assert kv.kvswap_validate_shape(good_shape(kv_dtype=W.E4M3)) == 3
    assert kv.kvswap_validate_shape(good_shape(q_dtype=W.E4M3)) == 3
    assert kv.kvswap_validate_shape(ok.with_flags(1 << 16)) == 2           # unknown flag bit


def test_status_strings_and_version(lib):
    seen = {kv.status_string(i) for i in range(11)}
    assert len(seen) == 11 and "ok" in seen
    assert kv.status_string(123) == "unknown status"
    assert kv.kvswap_version() >= 100


def test_workspace_grows_with_the_problem(lib):
    small = kv.kvswap_workspace_bytes(good_shape())
    big = kv.kvswap_workspace_bytes(good_shape(batch=8, n_ctx=65536))
    assert big > small


def test_device_status_entry_points_validate_their_arguments(lib):
    assert lib.kvswap_workspace_init(None, 1024, None) == 1            # NULL workspace
    assert lib.kvswap_workspace_init(ctypes.c_void_p(4096), 16, None) == 5   # shorter than the header
    assert lib.kvswap_read_device_status(None, None) == 1


def test_selected_token_count_is_bounded(lib):
    """top_k * group_size beyond 2^30 is refused instead of overflowing the token arithmetic."""
    assert kv.kvswap_validate_shape(good_shape(top_k=1 << 29, group_size=4)) == 6
    assert kv.kvswap_validate_shape(good_shape(top_k=1 << 28, group_size=4)) == 0
