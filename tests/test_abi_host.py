"""CPU-only checks of the C ABI: the shared library loads, exports every function the header
declares, and rejects bad models on the host before touching a device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import build as build_mod
from paper_2309_06973_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def fake_model(wl, dtype=B.DNNS_F32, base=0x10000000):
    """Descriptors with made-up (aligned) device addresses: enough for host-side validation."""
    t = (B.dnns_tensor * len(wl.tensors))()
    for i, s in enumerate(wl.tensors):
        t[i] = B.dnns_tensor(base + i * 0x1000000, dtype, s.O, s.I, s.KH, s.KW, s.in_spatial, int(s.prunable),
                             s.out_group, s.in_group, (base + 0x100) if s.has_bias else None)
    b = (B.dnns_bn * max(1, len(wl.bns)))()
    for i, s in enumerate(wl.bns):
        b[i] = B.dnns_bn(base, base, base, base, s.C, s.tensor, s.eps)
    g = (B.dnns_group * len(wl.groups))()
    for i, s in enumerate(wl.groups):
        g[i] = B.dnns_group(s.C, s.flags)
    m = B.dnns_model(len(wl.tensors), t, len(wl.bns), b, len(wl.groups), g)
    m._keep = (t, b, g)
    return m


def test_library_exports_every_declared_function():
    header = open(os.path.join(ROOT, "include", "dnns.h")).read()
    declared = set(re.findall(r"\b(dnns_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_struct_sizes_match_the_header_layout():
    assert C.sizeof(B.dnns_threshold) == 32
    assert C.sizeof(B.dnns_tensor) == 56
    assert C.sizeof(B.dnns_bn) == 48
    assert C.sizeof(B.dnns_group) == 8


def test_workspace_query_is_host_only_and_scales():
    wl = W.toy()
    m = fake_model(wl)
    a = B.dnns_workspace_bytes(m, B.DNNS_SCOPE_GLOBAL, 1)
    b = B.dnns_workspace_bytes(m, B.DNNS_SCOPE_GLOBAL, 8)
    c = B.dnns_workspace_bytes(m, B.DNNS_SCOPE_PER_TENSOR, 1)
    assert 0 < a < b and a < c
    assert B.dnns_workspace_bytes(m, B.DNNS_SCOPE_GLOBAL, 0) == 0
    assert B.dnns_workspace_bytes(m, B.DNNS_SCOPE_GLOBAL, 65) == 0
    assert B.dnns_workspace_bytes(fake_model(wl, B.DNNS_BF16), B.DNNS_SCOPE_GLOBAL, 8) < b   # no low-digit histograms


def create_status(m, scope=B.DNNS_SCOPE_GLOBAL, maxv=1, ws=0x20000000, nbytes=1 << 40):
    plan = C.c_void_p()
    return B.lib().dnns_plan_create(C.byref(m), scope, maxv, ws, nbytes, None, C.byref(plan))


def test_bad_models_are_rejected_before_any_launch():
    wl = W.toy()
    m = fake_model(wl)
    m.tensors[1].O += 1
    assert create_status(m) == B.DNNS_ERR_BAD_GRAPH            # out-axis disagrees with its group
    m = fake_model(wl)
    m.tensors[2].I -= 1
    assert create_status(m) == B.DNNS_ERR_BAD_GRAPH            # in-axis disagrees with its group
    m = fake_model(wl)
    m.bns[0].C += 1
    assert create_status(m) == B.DNNS_ERR_BAD_GRAPH
    m = fake_model(wl)
    m.bns[1].tensor = 0
    assert create_status(m) == B.DNNS_ERR_BAD_GRAPH            # two BNs on one tensor
    m = fake_model(wl)
    m.tensors[0].data = None
    assert create_status(m) == B.DNNS_ERR_INVALID_ARG
    m = fake_model(wl)
    m.tensors[0].data = 0x10000004
    assert create_status(m) == B.DNNS_ERR_INVALID_ARG          # misaligned data
    m = fake_model(wl)
    m.tensors[0].KH = 0
    assert create_status(m) == B.DNNS_ERR_INVALID_ARG
    m = fake_model(wl)
    m.tensors[3].dtype = B.DNNS_BF16
    assert create_status(m) == B.DNNS_ERR_UNSUPPORTED          # mixed dtypes
    m = fake_model(wl)
    m.tensors[0].dtype = 7
    assert create_status(m) == B.DNNS_ERR_UNSUPPORTED
    m = fake_model(wl)
    m.tensors[4].out_group = 99
    assert create_status(m) == B.DNNS_ERR_BAD_GRAPH
    m = fake_model(wl)
    assert create_status(m, nbytes=1024) == B.DNNS_ERR_WORKSPACE
    assert create_status(m, ws=0x20000010) == B.DNNS_ERR_INVALID_ARG   # workspace not 256-byte aligned
    assert create_status(m, ws=0) == B.DNNS_ERR_INVALID_ARG


def test_null_plan_calls_return_invalid_arg():
    L = B.lib()
    assert L.dnns_magnitude_threshold(None, None, 1, None, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_apply_mask(None, None, 0, None, None, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_zero_structures(None, None, None, None, None, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_propagate_keep(None, None, None, 3, 1, None, None, None, None, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_compact(None, None, None, None, None, 0, None, None, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_zero_structures_portfolio(None, None, 0, 1, None, None, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_compact_masked_multi(None, None, 0, 1, None, None, None, 0, None, None, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_last_device_status(None, None) == B.DNNS_ERR_INVALID_ARG
    assert B.dnns_plan_launch_count(None) == 0
    assert B.dnns_status_string(B.DNNS_ERR_BAD_GRAPH) == "inconsistent model graph"
