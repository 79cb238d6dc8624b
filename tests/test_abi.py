"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments
on the host before touching a device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def adit():
    from paper_2609_12075_b200 import build
    build.build()
    from paper_2609_12075_b200 import adit as mod
    return mod


def declared_functions():
    text = open(os.path.join(ROOT, "include", "adit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adit_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_stage_entry_points():
    names = declared_functions()
    for required in ("adit_create", "adit_load_weights", "adit_denoise", "adit_destroy"):
        assert required in names


def test_library_exports_every_declared_symbol(adit):
    for name in declared_functions():
        assert hasattr(adit.lib, name), name
    assert sorted(adit.EXPORTS) == declared_functions()


def test_strerror(adit):
    assert adit.lib.adit_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert len(adit.lib.adit_strerror(code)) > 0
    assert adit.lib.adit_strerror(-99) == b"unknown status"


def good_config(adit):
    from paper_2609_12075_b200 import workloads as W
    return adit.make_config(W.TINY, max_batch=2, max_prefix_len=64)


def test_create_rejects_bad_arguments_on_the_host(adit):
    h = C.c_void_p()
    assert adit.lib.adit_create(None, 0, C.byref(h)) == adit.E_INVALID
    assert adit.lib.adit_create(C.byref(good_config(adit)), 0, None) == adit.E_INVALID
    for field, value, want in [("n_layers", 0, adit.E_INVALID), ("n_kv_heads", 3, adit.E_INVALID),
                               ("time_emb_dim", 255, adit.E_INVALID), ("dtype", 7, adit.E_INVALID),
                               ("max_batch", 65, adit.E_CAPACITY), ("head_dim", 48, adit.E_UNSUPPORTED),
                               ("max_prefix_len", -1, adit.E_INVALID)]:
        c = good_config(adit)
        setattr(c, field, value)
        assert adit.lib.adit_create(C.byref(c), 0, C.byref(h)) == want, field
        assert not h.value


def test_null_handles(adit):
    assert adit.lib.adit_destroy(None) == adit.OK
    assert adit.lib.adit_poll_status(None) == adit.E_INVALID
    assert adit.lib.adit_load_weights(None, None, 0) == adit.E_INVALID
    assert adit.lib.adit_denoise(None, 1, None, None, None, None, 1, 0, None, None) == adit.E_INVALID
    assert adit.lib.adit_kernel_launches(None) == 0


def test_config_struct_matches_header(adit):
    # 13 int32 + 3 float + 1 int32, no padding
    assert C.sizeof(adit.Config) == 17 * 4
    assert C.sizeof(adit.Tensor) == 8 + 8 + 4 + 4 + 32 + 8


def test_attention_entry_points_reject_misaligned_buffers_on_the_host(adit):
    """16-byte copies and stores need 16-byte aligned qkv / out_att: a sliced bf16 pointer is refused before
    anything is enqueued (the pointers below are never dereferenced)."""
    kv = (C.c_void_p * 1)(0x10000)
    lens = (C.c_int32 * 1)(8)
    for fn in (adit.lib.adit_debug_attention, adit.lib.adit_attention_static):
        for qkv, out in ((0x20002, 0x30000), (0x20000, 0x30008)):
            assert fn(0, 1, 4, 2, 1, 64, 16, 0, C.c_void_p(qkv), kv, lens, 1, C.c_void_p(out), None) == adit.E_INVALID
    assert adit.lib.adit_attention_static_status(-1) == adit.E_INVALID
    assert adit.lib.adit_attention_static_status(5) == adit.OK      # never used on that device


def test_stamp_buffer_is_only_used_where_it_fits(adit):
    """The phase-stamp buffer holds 1024 blocks on the device it was armed on; larger grids (attention: 512, the
    per-block log starts there) and other devices must run the plain kernels instead of writing past it."""
    sel = adit.lib.adit_debug_stamps_selected
    assert sel(0, 0, 1024, 0) == 1 and sel(0, 0, 1025, 0) == 0
    assert sel(0, 0, 512, 1) == 1 and sel(0, 0, 513, 1) == 0 and sel(0, 0, 24576, 1) == 0
    assert sel(0, 1, 8, 0) == 0 and sel(-1, 0, 8, 0) == 0 and sel(0, 0, 0, 0) == 0


def test_persistent_loop_queries_are_host_only(adit):
    assert adit.lib.adit_uses_persistent_loop(None, 1, 0) == adit.E_INVALID
    assert adit.lib.adit_debug_wait_limit(None, 5, -1) == adit.E_INVALID
    assert adit.lib.adit_clear_status(None) == adit.E_INVALID
    assert adit.lib.adit_loop_trace_read(None, None, 0) == adit.E_INVALID
