"""ctypes access to the CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this module.  It compiles ``dnns_oracle.cpp`` with g++ on first use and
marshals numpy arrays into the oracle's own descriptor structs; it contains no
arithmetic of the method.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dnns_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

F32, BF16 = 0, 1
RULE_PRODUCER, RULE_CONSUMER, SHIFT_STRICT = 1, 2, 4

REC_DTYPE = np.dtype([("tau_bits", "<u4"), ("pad", "<u4"), ("n_below", "<u8"), ("n_tie", "<u8"),
                      ("n_equal", "<u8")])


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-Wall", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


class _Tensor(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("O", C.c_int32), ("I", C.c_int32),
                ("KH", C.c_int32), ("KW", C.c_int32), ("in_spatial", C.c_int32), ("prunable", C.c_int32),
                ("out_group", C.c_int32), ("in_group", C.c_int32), ("bias", C.c_void_p)]


class _BN(C.Structure):
    _fields_ = [("gamma", C.c_void_p), ("beta", C.c_void_p), ("mean", C.c_void_p), ("var", C.c_void_p),
                ("C", C.c_int32), ("tensor", C.c_int32), ("eps", C.c_float)]


class _Group(C.Structure):
    _fields_ = [("C", C.c_int32), ("flags", C.c_uint32)]


class _Model(C.Structure):
    _fields_ = [("n_tensors", C.c_int32), ("tensors", C.POINTER(_Tensor)), ("n_bn", C.c_int32),
                ("bns", C.POINTER(_BN)), ("n_groups", C.c_int32), ("groups", C.POINTER(_Group))]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_num_segments.restype = C.c_int
        _lib.orc_threshold.restype = C.c_int
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _ptr_array(arrs):
    return (C.c_void_p * len(arrs))(*[_ptr(a) for a in arrs])


class OracleModel:
    """A workload's descriptors bound to host arrays, in the oracle's own structs."""

    def __init__(self, wl, dtype: int = F32, weights: Optional[List[np.ndarray]] = None):
        self.wl = wl
        self.dtype = dtype
        self.weights = weights if weights is not None else wl.weights_as(dtype)
        self.weights = [np.ascontiguousarray(w) for w in self.weights]
        want = np.float32 if dtype == F32 else np.uint16
        assert all(w.dtype == want for w in self.weights)
        self.biases = [None if b is None else np.ascontiguousarray(b, np.float32) for b in wl.biases]
        self.bn_params = [tuple(np.ascontiguousarray(v, np.float32) for v in p) for p in wl.bn_params]
        self._t = (_Tensor * len(wl.tensors))()
        for i, t in enumerate(wl.tensors):
            self._t[i] = _Tensor(_ptr(self.weights[i]), dtype, t.O, t.I, t.KH, t.KW, t.in_spatial,
                                 int(t.prunable), t.out_group, t.in_group, _ptr(self.biases[i]))
        self._b = (_BN * max(1, len(wl.bns)))()
        for i, b in enumerate(wl.bns):
            g, be, mu, va = self.bn_params[i]
            self._b[i] = _BN(_ptr(g), _ptr(be), _ptr(mu), _ptr(va), b.C, b.tensor, b.eps)
        self._g = (_Group * len(wl.groups))()
        for i, g in enumerate(wl.groups):
            self._g[i] = _Group(g.C, g.flags)
        self.c = _Model(len(wl.tensors), self._t, len(wl.bns), self._b, len(wl.groups), self._g)

    def like(self, weights: List[np.ndarray]) -> "OracleModel":
        return OracleModel(self.wl, self.dtype, weights)


def num_segments(om: OracleModel, scope: int) -> int:
    return lib().orc_num_segments(C.byref(om.c), scope)


def threshold(om: OracleModel, scope: int, ks: np.ndarray) -> np.ndarray:
    """ks: uint64 (n_k, n_segments) -> records (n_k, n_segments)."""
    ks = np.ascontiguousarray(ks, np.uint64)
    S = num_segments(om, scope)
    assert ks.ndim == 2 and ks.shape[1] == S
    rec = np.zeros(ks.shape, REC_DTYPE)
    rc = lib().orc_threshold(C.byref(om.c), scope, C.c_void_p(ks.ctypes.data), ks.shape[0],
                             C.c_void_p(rec.ctypes.data))
    if rc:
        raise ValueError("k exceeds the segment size")
    return rec


def _bitwords(nbits: int) -> np.ndarray:
    return np.zeros((nbits + 31) // 32, np.uint32)


def apply_mask(om: OracleModel, scope: int, rec_row: np.ndarray):
    """rec_row: records of one variant (n_segments,). Returns (masked OracleModel, mask bit words per tensor)."""
    rec_row = np.ascontiguousarray(rec_row, REC_DTYPE)
    out = [np.empty_like(w) for w in om.weights]
    dst = om.like(out)
    bits = [_bitwords(w.size) for w in om.weights]
    lib().orc_apply_mask(C.byref(om.c), C.byref(dst.c), scope, C.c_void_p(rec_row.ctypes.data), _ptr_array(bits))
    return dst, bits


def zero_structures(om: OracleModel):
    wl = om.wl
    nz = [_bitwords(t.O * t.I) for t in wl.tensors]
    out_nz = [_bitwords(t.O) for t in wl.tensors]
    in_nz = [_bitwords(t.I) for t in wl.tensors]
    lib().orc_zero_structures(C.byref(om.c), _ptr_array(nz), _ptr_array(out_nz), _ptr_array(in_nz))
    return nz, out_nz, in_nz


def propagate_keep(om: OracleModel, out_nz, in_nz, policy: int = RULE_PRODUCER | RULE_CONSUMER, min_keep: int = 1):
    wl = om.wl
    keep_bits = [_bitwords(g.C) for g in wl.groups]
    keep_idx = [np.full(g.C, -1, np.int32) for g in wl.groups]
    keep_count = np.zeros(len(wl.groups), np.int32)
    stats = np.zeros(4, np.uint64)
    lib().orc_propagate_keep(C.byref(om.c), _ptr_array(out_nz), _ptr_array(in_nz), C.c_uint32(policy),
                             C.c_int32(min_keep), _ptr_array(keep_bits), _ptr_array(keep_idx),
                             C.c_void_p(keep_count.ctypes.data), C.c_void_p(stats.ctypes.data))
    return keep_bits, keep_idx, keep_count, stats


def compact(om: OracleModel, keep_idx, keep_count):
    """Returns (weights shaped (O', I', KH, KW), bn vectors [(g, b, m, v)], biases, shapes (T, 2))."""
    wl = om.wl
    keep_count = np.ascontiguousarray(keep_count, np.int32)
    dst_w, dst_bias = [], []
    for i, t in enumerate(wl.tensors):
        On, Cn = int(keep_count[t.out_group]), int(keep_count[t.in_group])
        dst_w.append(np.zeros((On, Cn * t.in_spatial, t.KH, t.KW), om.weights[i].dtype))
        dst_bias.append(np.zeros(On, np.float32) if om.biases[i] is not None else None)
    dst_bn = []
    for b in wl.bns:
        Cn = int(keep_count[wl.tensors[b.tensor].out_group])
        dst_bn.extend(np.zeros(Cn, np.float32) for _ in range(4))
    shapes = np.zeros((len(wl.tensors), 2), np.int32)
    lib().orc_compact(C.byref(om.c), _ptr_array(keep_idx), C.c_void_p(keep_count.ctypes.data), _ptr_array(dst_w),
                      _ptr_array(dst_bn) if dst_bn else None, _ptr_array(dst_bias), C.c_void_p(shapes.ctypes.data))
    bns = [tuple(dst_bn[4 * i: 4 * i + 4]) for i in range(len(wl.bns))]
    return dst_w, bns, dst_bias, shapes


def fold_batchnorm(om: OracleModel):
    """Returns (folded weights as float64 arrays or None per tensor, scale per BN, folded bias per BN)."""
    wl = om.wl
    has_bn = {b.tensor for b in wl.bns}
    fw = [np.zeros(w.shape, np.float64) if i in has_bn else None for i, w in enumerate(om.weights)]
    scale = [np.zeros(b.C, np.float64) for b in wl.bns]
    fbias = [np.zeros(b.C, np.float64) for b in wl.bns]
    lib().orc_fold_batchnorm(C.byref(om.c), _ptr_array(fw), _ptr_array(scale), _ptr_array(fbias))
    return fw, scale, fbias


def propagate_keep_cascade(om: OracleModel, nz_map, policy: int = RULE_PRODUCER | RULE_CONSUMER, min_keep: int = 1,
                           max_passes: int = 64):
    wl = om.wl
    keep_bits = [_bitwords(g.C) for g in wl.groups]
    keep_idx = [np.full(g.C, -1, np.int32) for g in wl.groups]
    keep_count = np.zeros(len(wl.groups), np.int32)
    stats = np.zeros(4, np.uint64)
    lib().orc_propagate_keep_cascade(C.byref(om.c), _ptr_array(nz_map), C.c_uint32(policy), C.c_int32(min_keep),
                                     C.c_int32(max_passes), _ptr_array(keep_bits), _ptr_array(keep_idx),
                                     C.c_void_p(keep_count.ctypes.data), C.c_void_p(stats.ctypes.data))
    return keep_bits, keep_idx, keep_count, stats
