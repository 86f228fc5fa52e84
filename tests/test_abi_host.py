"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, and its
host-side logic (shape validation, workspace sizing, call-order errors) behaves.  No compute calls."""
import ctypes
import os
import re

import numpy as np
import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b():
    entry.build()
    from paper_2609_03459_b200 import binding
    return binding


def _create(b, **kw):
    args = dict(num_rows=[1000], row_factors=[[10, 10, 10]], dim_factors=[[4, 4, 4]], ranks=[[1, 8, 8, 1]],
                max_batch=16, max_lookups=100)
    args.update(kw)
    cfg, keep = b.make_config(**args)
    h = ctypes.c_void_p()
    rc = b.lib.tt_emb_create(ctypes.byref(cfg), ctypes.byref(h))
    return rc, h


def test_header_symbols_are_exported(b):
    text = open(os.path.join(ROOT, "include", "tt_emb.h")).read()
    declared = set(re.findall(r"\b(tt_emb_[a-z0-9_]+)\s*\(", text))
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(b.lib, name), f"{name} declared in tt_emb.h but not exported"
    assert declared == set(b.EXPORTED_SYMBOLS)


def test_create_validates_shapes(b):
    rc, h = _create(b)
    assert rc == 0
    assert b.lib.tt_emb_destroy(h) == 0
    assert _create(b, row_factors=[[10, 10, 9]])[0] == b.TT_EMB_ERR_ARG          # prod(n) < N
    assert _create(b, ranks=[[2, 8, 8, 1]])[0] == b.TT_EMB_ERR_ARG               # r_0 != 1
    assert _create(b, ranks=[[1, 8, 200, 1]])[0] == b.TT_EMB_ERR_ARG             # rank limit
    assert _create(b, num_rows=[0])[0] == b.TT_EMB_ERR_ARG
    assert _create(b, max_batch=0)[0] == b.TT_EMB_ERR_ARG
    assert _create(b, row_factors=[[10, 100]], dim_factors=[[8, 8]], ranks=[[1, 4, 1]])[0] == 0  # K = 2
    # two tables must agree on D
    rc, _ = _create(b, num_rows=[1000, 1000], row_factors=[[10, 10, 10]] * 2, dim_factors=[[4, 4, 4], [4, 4, 2]],
                    ranks=[[1, 8, 8, 1]] * 2)
    assert rc == b.TT_EMB_ERR_ARG
    assert b.lib.tt_emb_create(None, None) == b.TT_EMB_ERR_ARG


def test_workspace_grows_with_capacity_and_backward(b):
    sizes = []
    for kw in (dict(max_lookups=100), dict(max_lookups=100000), dict(max_lookups=100000, enable_backward=True)):
        rc, h = _create(b, **kw)
        assert rc == 0
        n = ctypes.c_size_t()
        assert b.lib.tt_emb_workspace_bytes(h, ctypes.byref(n)) == 0
        sizes.append(n.value)
        d = ctypes.c_int32()
        assert b.lib.tt_emb_dim(h, ctypes.byref(d)) == 0 and d.value == 64
        c = ctypes.c_int64()
        assert b.lib.tt_emb_core_floats(h, 0, 1, ctypes.byref(c)) == 0 and c.value == 10 * 8 * 4 * 8
        b.lib.tt_emb_destroy(h)
    assert sizes[0] < sizes[1] < sizes[2]
    # max_unique_rows caps the row buffer
    rc, h = _create(b, max_lookups=100000, max_unique_rows=10)
    n = ctypes.c_size_t(); b.lib.tt_emb_workspace_bytes(h, ctypes.byref(n)); b.lib.tt_emb_destroy(h)
    assert n.value < sizes[1]


def test_call_order_and_missing_device_errors(b):
    rc, h = _create(b)
    out = np.zeros(4, np.float32)
    # forward before bind
    assert b.lib.tt_emb_forward(h, out.ctypes.data, out.ctypes.data, 1, 0, out.ctypes.data, None) == b.TT_EMB_ERR_STATE
    assert b.lib.tt_emb_bind(h, None, None, 0, None) == b.TT_EMB_ERR_ARG
    ptrs = (ctypes.c_void_p * 3)(256, 512, 768)
    assert b.lib.tt_emb_bind(h, ptrs, None, 0, None) == b.TT_EMB_ERR_WORKSPACE
    import torch
    if not torch.cuda.is_available():
        # no CPU fallback: binding on a machine without a B200 fails loudly
        assert b.lib.tt_emb_bind(h, ptrs, 256 * 1000, 1 << 40, None) == b.TT_EMB_ERR_ARCH
        v = ctypes.c_double()
        assert b.lib.tt_emb_probe_fp32(ctypes.byref(v), None) == b.TT_EMB_ERR_ARCH
        assert b.lib.tt_emb_probe_mma(ctypes.byref(v), None) == b.TT_EMB_ERR_ARCH
        v2 = ctypes.c_double()
        assert b.lib.tt_emb_probe_tcgen05(128, ctypes.byref(v), ctypes.byref(v2), None) == b.TT_EMB_ERR_ARCH
    assert b.lib.tt_emb_probe_tcgen05(64, ctypes.byref(ctypes.c_double()), ctypes.byref(ctypes.c_double()), None) == b.TT_EMB_ERR_ARG
    assert b.lib.tt_emb_backward(h, out.ctypes.data, ptrs, None) == b.TT_EMB_ERR_STATE
    assert b.lib.tt_emb_destroy(h) == 0
    assert b.lib.tt_emb_strerror(b.TT_EMB_ERR_ARCH).decode().startswith("no CUDA device")
