"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, and its buffer/blob arithmetic agrees with the documented format."""
import ctypes
import os
import re

import numpy as np
import pytest

import hs_inputs as hi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hs():
    from paper_2605_01106_b200 import build, binding
    build.build()
    return binding


def test_exports_match_header(hs):
    text = open(os.path.join(ROOT, "include", "hs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(hs_[a-z_]+)\s*\(", text))
    assert declared, "no declarations found"
    L = hs.load_library()
    for name in declared:
        assert hasattr(L, name), "libhs.so does not export %s" % name
    assert declared == set(hs.EXPORTS)


@pytest.mark.parametrize("name", ["cfg1_tiny", "cfg2_0p5b", "cfg3_3b", "cfg4_seq", "cfg5_b64", "test_seq"])
def test_blob_format_agrees_with_generator(hs, name):
    s = hi.CONFIGS[name]
    cfg = hs.make_config(s, max_batch=s.batch, max_k=max(s.ks), kv_capacity=4096)
    table, total = hi.blob_layout(s)
    assert hs.query_sizes(cfg).weights == total
    L = hs.load_library()
    for (layer, tid), (off, shape, dt) in table.items():
        assert L.hs_weight_offset(ctypes.byref(cfg), layer, tid) == off, (layer, tid)
    # a tensor the layer kind does not have
    if s.arch == hi.ARCH_SEQUENTIAL:
        assert L.hs_weight_offset(ctypes.byref(cfg), 0, hi.T_A_LOG) == -1
        assert L.hs_weight_offset(ctypes.byref(cfg), 3, hi.T_W_OUT) == -1


def test_query_sizes_accounting(hs):
    s = hi.CONFIGS["cfg2_0p5b"]
    cfg = hs.make_config(s, max_batch=2, max_k=4, kv_capacity=1024)
    sz = hs.query_sizes(cfg)
    state = s.H * s.P * s.N * 4
    assert sz.snap == s.L * 2 * 5 * state
    assert sz.dstate == s.L * 2 * state
    assert sz.kv == 2 * s.L * 2 * s.kvh * 1024 * s.hd * 2
    assert sz.conv == s.L * 2 * s.convd * 4 * (3 + 5 + 6)


def test_invalid_configs_are_rejected(hs):
    s = hi.CONFIGS["cfg1_tiny"]
    L = hs.load_library()
    sz = hs.HsSizes()
    for kw in (dict(max_k=9), dict(max_batch=0), dict(kv_capacity=0)):
        cfg = hs.make_config(s, **{**dict(max_batch=1, max_k=2, kv_capacity=64), **kw})
        assert L.hs_query_sizes(ctypes.byref(cfg), ctypes.byref(sz)) == -1
    for bad in (s.replace(N=96), s.replace(hd=80), s.replace(d=200), s.replace(conv_w=3), s.replace(qh=3)):
        cfg = hs.make_config(bad, 1, 2, 64)
        assert L.hs_query_sizes(ctypes.byref(cfg), ctypes.byref(sz)) == -1
    assert L.hs_query_sizes(None, ctypes.byref(sz)) == -1
    assert L.hs_draft(None, 1) == -1 and L.hs_verify(None, 1, None) == -1
    assert L.hs_accept_rollback(None, None, None, None, None) == -1


def test_init_refuses_short_buffers_before_any_device_work(hs):
    # hs_init_model is told how many bytes each caller buffer really has; a short one is HS_ERR_SIZE, decided on
    # the host before any CUDA call (the pointers below are never dereferenced), and no handle is left behind
    s = hi.CONFIGS["cfg1_tiny"]
    cfg = hs.make_config(s, max_batch=1, max_k=2, kv_capacity=64)
    need = hs.query_sizes(cfg)
    L = hs.load_library()
    fake = hs.HsBuffers(*[0x10000 * (i + 1) for i in range(6)])
    for field in ("weights", "snap", "dstate", "conv", "kv", "work"):
        have = hs.HsSizes(*[getattr(need, f) for f in ("weights", "snap", "dstate", "conv", "kv", "work")])
        setattr(have, field, getattr(need, field) - 1)
        h = hs.vp(0xdead)
        assert L.hs_init_model(ctypes.byref(cfg), ctypes.byref(fake), ctypes.byref(have), None, ctypes.byref(h)) == -2, field
        assert not h.value
    # misaligned or null buffers and a missing size record are invalid arguments
    have = hs.HsSizes(*[getattr(need, f) for f in ("weights", "snap", "dstate", "conv", "kv", "work")])
    odd = hs.HsBuffers(0x10000, 0x20000, 0x30010, 0x40000, 0x50000, 0x60000)
    h = hs.vp()
    assert L.hs_init_model(ctypes.byref(cfg), ctypes.byref(odd), ctypes.byref(have), None, ctypes.byref(h)) == -1
    assert L.hs_init_model(ctypes.byref(cfg), ctypes.byref(fake), None, None, ctypes.byref(h)) == -1
    assert L.hs_round_host(None, 1, None, None, None, None) == -1
    assert L.hs_selftest_wait_timeout(None, 10) == -1 and L.hs_clear_status(None) == -1


def test_static_argmax_argument_checks_need_no_device(hs):
    # pointer, size and alignment checks of the allocation-free argmax come before any CUDA call
    L = hs.load_library()
    assert L.hs_argmax_static(None, 8, 1, 0x1000, None, None) == -1
    assert L.hs_argmax_static(0x1000, 8, 1, None, None, None) == -1
    assert L.hs_argmax_static(0x1000, 0, 1, 0x2000, None, None) == -1
    assert L.hs_argmax_static(0x1000, 8, 65, 0x2000, None, None) == -2
    assert L.hs_argmax_static(0x1004, 8, 1, 0x2000, None, None) == -1        # V % 4 == 0: rows are read 128 bits at a time
    assert L.hs_argmax_static(0x1000, 8, 1, 0x2002, None, None) == -1
    assert L.hs_argmax_static(0x1000, 8, 1, 0x2000, 0x3001, None) == -1
    assert L.hs_argmax_static(0x1002, 7, 1, 0x2000, None, None) == -1        # floats are 4-byte aligned at least
