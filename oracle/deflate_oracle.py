"""ctypes access to the CPU oracle of the deflation step (TEST INFRASTRUCTURE, not a product path).

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this module.
It compiles ``deflate_oracle.c`` with gcc on first use and marshals numpy arrays; it holds no
arithmetic of the method.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "deflate_oracle.c")
_LIB = os.path.join(_HERE, "libdeflate_oracle.so")

CHUNK, SUB = 16384, 512
SUBS_PER_CHUNK = CHUNK // SUB

_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_deflate_n_chunks.restype = C.c_size_t
        _lib.orc_deflate_n_chunks.argtypes = [C.c_size_t]
        _lib.orc_deflate_bound.restype = C.c_size_t
        _lib.orc_deflate_bound.argtypes = [C.c_size_t]
        _lib.orc_deflate.restype = C.c_size_t
        _lib.orc_deflate.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_inflate.restype = C.c_longlong
        _lib.orc_inflate.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t]
    return _lib


def _bytes_of(data) -> np.ndarray:
    a = np.frombuffer(bytes(data), np.uint8) if isinstance(data, (bytes, bytearray)) else np.ascontiguousarray(data)
    return a.view(np.uint8).ravel()


def deflate(data):
    """(stream uint8[size], chunk_offset uint64[n_chunks + 1], sub_bits uint32[32 * n_chunks])."""
    src = _bytes_of(data)
    n = src.size
    nc = lib().orc_deflate_n_chunks(n)
    stream = np.zeros(lib().orc_deflate_bound(n), np.uint8)
    chunk_offset = np.zeros(nc + 1, np.uint64)
    sub_bits = np.zeros(nc * SUBS_PER_CHUNK, np.uint32)
    keep = src if n else np.zeros(1, np.uint8)
    size = lib().orc_deflate(keep.ctypes.data, n, stream.ctypes.data, chunk_offset.ctypes.data, sub_bits.ctypes.data)
    return stream[:size].copy(), chunk_offset, sub_bits


def inflate(stream, capacity: int):
    """The decoded bytes, or None when the decoder rejects the stream."""
    s = _bytes_of(stream)
    dst = np.zeros(max(capacity, 1), np.uint8)
    keep = s if s.size else np.zeros(1, np.uint8)
    got = lib().orc_inflate(keep.ctypes.data, s.size, dst.ctypes.data, capacity)
    return None if got < 0 else dst[:got].copy()
