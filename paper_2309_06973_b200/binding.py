"""Thin ctypes binding of libdnns.so: the same entry points as include/dnns.h, argument
marshalling only.  Every step of the path runs in the library's CUDA kernels; there is no
fallback of any kind - if the shared library is missing the import fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
# DNNS_LIBRARY names another build of the same library (the tests' checked build); there is still no fallback
LIB_PATH = os.environ.get("DNNS_LIBRARY") or os.path.join(HERE, "libdnns.so")

DNNS_F32, DNNS_BF16 = 0, 1
DNNS_SCOPE_GLOBAL, DNNS_SCOPE_PER_TENSOR = 0, 1
DNNS_RULE_PRODUCER, DNNS_RULE_CONSUMER, DNNS_SHIFT_STRICT = 1, 2, 4
DNNS_GROUP_FROZEN = 1
(DNNS_OK, DNNS_ERR_INVALID_ARG, DNNS_ERR_BAD_GRAPH, DNNS_ERR_WORKSPACE, DNNS_ERR_UNSUPPORTED, DNNS_ERR_CUDA,
 DNNS_ERR_TIMEOUT, DNNS_ERR_STATIC_LIMIT) = range(8)
DNNS_STATIC_MAX_NUMEL = 1 << 26
DNNS_DEFLATE_CHUNK, DNNS_DEFLATE_SUB = 16384, 512
DNNS_MULTI_MAX = 4
DNNS_PORTFOLIO_MAX = 16

EXPORTS = ["dnns_status_string", "dnns_workspace_bytes", "dnns_plan_create", "dnns_plan_destroy", "dnns_plan_layout",
           "dnns_plan_launch_count", "dnns_magnitude_threshold", "dnns_apply_mask", "dnns_zero_structures",
           "dnns_propagate_keep", "dnns_compact", "dnns_last_device_status", "dnns_magnitude_threshold_static", "dnns_mask_and_structures", "dnns_fold_batchnorm", "dnns_propagate_keep_cascade",
           "dnns_plan_profile", "dnns_plan_profile_read", "dnns_plan_tie_sweep", "dnns_mask_and_structures_multi", "dnns_propagate_keep_multi", "dnns_compact_masked", "dnns_zero_structures_portfolio", "dnns_compact_masked_multi", "dnns_deflate_chunks", "dnns_deflate_bound", "dnns_deflate_workspace_bytes", "dnns_deflate", "dnns_inflate"]


class dnns_tensor(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("O", C.c_int32), ("I", C.c_int32), ("KH", C.c_int32),
                ("KW", C.c_int32), ("in_spatial", C.c_int32), ("prunable", C.c_int32), ("out_group", C.c_int32),
                ("in_group", C.c_int32), ("bias", C.c_void_p)]


class dnns_bn(C.Structure):
    _fields_ = [("gamma", C.c_void_p), ("beta", C.c_void_p), ("mean", C.c_void_p), ("var", C.c_void_p),
                ("C", C.c_int32), ("tensor", C.c_int32), ("eps", C.c_float)]


class dnns_group(C.Structure):
    _fields_ = [("C", C.c_int32), ("flags", C.c_uint32)]


class dnns_model(C.Structure):
    _fields_ = [("n_tensors", C.c_int32), ("tensors", C.POINTER(dnns_tensor)), ("n_bn", C.c_int32),
                ("bns", C.POINTER(dnns_bn)), ("n_groups", C.c_int32), ("groups", C.POINTER(dnns_group))]


class dnns_threshold(C.Structure):
    _fields_ = [("tau_bits", C.c_uint32), ("pad", C.c_uint32), ("n_below", C.c_uint64), ("n_tie", C.c_uint64),
                ("n_equal", C.c_uint64)]


class dnns_layout(C.Structure):
    _fields_ = [("n_tensors", C.c_int32), ("n_bn", C.c_int32), ("n_groups", C.c_int32), ("n_segments", C.c_int32),
                ("n_bias", C.c_int32), ("elem_bytes", C.c_int32), ("n_prunable", C.c_uint64),
                ("masked_arena_bytes", C.c_uint64), ("mask_words", C.c_uint64), ("nz_map_words", C.c_uint64),
                ("out_nz_words", C.c_uint64), ("in_nz_words", C.c_uint64), ("keep_words", C.c_uint64),
                ("keep_idx_len", C.c_uint64), ("compact_arena_bytes", C.c_uint64), ("n_compact_items", C.c_int32),
                ("arena_offset", C.POINTER(C.c_uint64)), ("mask_offset", C.POINTER(C.c_uint64)),
                ("nz_map_offset", C.POINTER(C.c_uint64)), ("out_nz_offset", C.POINTER(C.c_uint64)),
                ("in_nz_offset", C.POINTER(C.c_uint64)), ("keep_offset", C.POINTER(C.c_uint64)),
                ("keep_idx_offset", C.POINTER(C.c_uint64)), ("segment_size", C.POINTER(C.c_uint64)),
                ("segment_of_tensor", C.POINTER(C.c_int32))]


class DnnsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {dnns_status_string(status)} (status {status})")


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library.  Raises if it has not been built (python -m paper_2309_06973_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2309_06973_b200.build` "
                              "(nvcc, sm_100a); there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, i32, u32, u64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64
        L.dnns_status_string.restype = C.c_char_p
        L.dnns_status_string.argtypes = [C.c_int]
        L.dnns_workspace_bytes.restype = C.c_size_t
        L.dnns_workspace_bytes.argtypes = [C.POINTER(dnns_model), C.c_int, i32]
        L.dnns_plan_create.argtypes = [C.POINTER(dnns_model), C.c_int, i32, vp, C.c_size_t, vp, C.POINTER(vp)]
        L.dnns_plan_destroy.restype = None
        L.dnns_plan_destroy.argtypes = [vp]
        L.dnns_plan_layout.argtypes = [vp, C.POINTER(dnns_layout)]
        L.dnns_plan_launch_count.restype = u64
        L.dnns_plan_launch_count.argtypes = [vp]
        L.dnns_magnitude_threshold.argtypes = [vp, C.POINTER(u64), i32, vp, vp]
        L.dnns_apply_mask.argtypes = [vp, vp, i32, vp, vp, vp]
        L.dnns_zero_structures.argtypes = [vp, vp, vp, vp, vp, vp]
        L.dnns_mask_and_structures.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp]
        L.dnns_propagate_keep.argtypes = [vp, vp, vp, u32, i32, vp, vp, vp, vp, vp]
        L.dnns_compact.argtypes = [vp, vp, vp, vp, vp, C.c_size_t, vp, vp, vp]
        L.dnns_last_device_status.argtypes = [vp, vp]
        L.dnns_fold_batchnorm.argtypes = [vp, vp, vp, vp, vp]
        L.dnns_propagate_keep_cascade.argtypes = [vp, vp, u32, i32, i32, vp, vp, vp, vp, vp]
        L.dnns_magnitude_threshold_static.argtypes = [vp, i32, u64, u64, vp, vp]
        L.dnns_mask_and_structures_multi.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp, vp, vp]
        L.dnns_propagate_keep_multi.argtypes = [vp, i32, vp, vp, u32, i32, vp, vp, vp, vp, vp]
        L.dnns_compact_masked.argtypes = [vp, vp, i32, vp, vp, vp, C.c_size_t, vp, vp, vp]
        L.dnns_zero_structures_portfolio.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        L.dnns_compact_masked_multi.argtypes = [vp, vp, i32, i32, vp, vp, vp, C.c_size_t, vp, vp, vp]
        L.dnns_plan_profile.argtypes = [vp, i32]
        L.dnns_plan_tie_sweep.argtypes = [vp, C.POINTER(i32)]
        L.dnns_plan_profile_read.argtypes = [vp, C.c_char_p, C.POINTER(C.c_double), C.POINTER(u64)]
        for name in ("dnns_deflate_chunks", "dnns_deflate_bound", "dnns_deflate_workspace_bytes"):
            getattr(L, name).restype = C.c_size_t
            getattr(L, name).argtypes = [C.c_size_t]
        L.dnns_deflate.argtypes = [vp, C.c_size_t, vp, C.c_size_t, vp, vp, vp, C.c_size_t, vp]
        L.dnns_inflate.argtypes = [vp, C.c_size_t, vp, vp, C.c_size_t, vp, vp, vp]
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != DNNS_OK:
        raise DnnsError(status, where)


def dnns_status_string(status: int) -> str:
    return lib().dnns_status_string(status).decode()


def dnns_workspace_bytes(model: dnns_model, scope: int, max_variants: int) -> int:
    return lib().dnns_workspace_bytes(C.byref(model), scope, max_variants)


def dnns_plan_create(model: dnns_model, scope: int, max_variants: int, ws_dev: int, ws_bytes: int, stream: int = 0):
    plan = C.c_void_p()
    _check(lib().dnns_plan_create(C.byref(model), scope, max_variants, ws_dev, ws_bytes, stream, C.byref(plan)),
           "dnns_plan_create")
    return plan


def dnns_plan_destroy(plan) -> None:
    lib().dnns_plan_destroy(plan)


def dnns_plan_layout(plan) -> dnns_layout:
    out = dnns_layout()
    _check(lib().dnns_plan_layout(plan, C.byref(out)), "dnns_plan_layout")
    return out


def dnns_plan_launch_count(plan) -> int:
    return lib().dnns_plan_launch_count(plan)


def dnns_magnitude_threshold(plan, k, n_k: int, thr_dev: int, stream: int = 0) -> None:
    """k: sequence of n_k * n_segments prune counts, variant-major."""
    arr = (C.c_uint64 * len(k))(*[int(x) for x in k])
    _check(lib().dnns_magnitude_threshold(plan, arr, n_k, thr_dev, stream), "dnns_magnitude_threshold")


def dnns_apply_mask(plan, thr_dev: int, variant: int, masked_arena: int, mask_bits: int, stream: int = 0) -> None:
    _check(lib().dnns_apply_mask(plan, thr_dev, variant, masked_arena or None, mask_bits or None, stream),
           "dnns_apply_mask")


def dnns_zero_structures(plan, masked_arena: int, nz_map: int, out_nz: int, in_nz: int, stream: int = 0) -> None:
    _check(lib().dnns_zero_structures(plan, masked_arena or None, nz_map or None, out_nz, in_nz, stream),
           "dnns_zero_structures")


def dnns_mask_and_structures(plan, thr_dev: int, variant: int, masked_arena: int, mask_bits: int, nz_map: int,
                             out_nz: int, in_nz: int, stream: int = 0) -> None:
    _check(lib().dnns_mask_and_structures(plan, thr_dev, variant, masked_arena or None, mask_bits or None,
                                          nz_map or None, out_nz, in_nz, stream), "dnns_mask_and_structures")


def dnns_propagate_keep(plan, out_nz: int, in_nz: int, policy: int, min_keep: int, keep_bits: int, keep_idx: int,
                        keep_count: int, stats: int, stream: int = 0) -> None:
    _check(lib().dnns_propagate_keep(plan, out_nz, in_nz, policy, min_keep, keep_bits, keep_idx, keep_count,
                                     stats or None, stream), "dnns_propagate_keep")


def dnns_compact(plan, masked_arena: int, keep_idx: int, keep_count: int, dst_arena: int, dst_bytes: int,
                 dst_offsets_dev: int, dst_shapes_dev: int, stream: int = 0) -> None:
    _check(lib().dnns_compact(plan, masked_arena or None, keep_idx, keep_count, dst_arena, dst_bytes,
                              dst_offsets_dev, dst_shapes_dev, stream), "dnns_compact")


def dnns_last_device_status(plan, stream: int = 0) -> int:
    return lib().dnns_last_device_status(plan, stream)


def dnns_magnitude_threshold_static(weights_dev: int, dtype: int, numel: int, k: int, thr_dev: int,
                                    stream: int = 0) -> None:
    """Threshold of one tensor using the library's built-in scratch: nothing is allocated."""
    _check(lib().dnns_magnitude_threshold_static(weights_dev, dtype, numel, k, thr_dev, stream),
           "dnns_magnitude_threshold_static")


def dnns_fold_batchnorm(plan, dst_arena: int, dst_offsets_dev: int, dst_shapes_dev: int, stream: int = 0) -> None:
    _check(lib().dnns_fold_batchnorm(plan, dst_arena, dst_offsets_dev, dst_shapes_dev, stream), "dnns_fold_batchnorm")


def dnns_propagate_keep_cascade(plan, nz_map: int, policy: int, min_keep: int, max_passes: int, keep_bits: int,
                                keep_idx: int, keep_count: int, stats: int, stream: int = 0) -> None:
    _check(lib().dnns_propagate_keep_cascade(plan, nz_map, policy, min_keep, max_passes, keep_bits, keep_idx,
                                             keep_count, stats or None, stream), "dnns_propagate_keep_cascade")


def dnns_deflate_chunks(n_bytes: int) -> int:
    return lib().dnns_deflate_chunks(n_bytes)


def dnns_deflate_bound(n_bytes: int) -> int:
    return lib().dnns_deflate_bound(n_bytes)


def dnns_deflate_workspace_bytes(n_bytes: int) -> int:
    return lib().dnns_deflate_workspace_bytes(n_bytes)


def dnns_deflate(src_dev: int, n_bytes: int, stream_dev: int, stream_capacity: int, chunk_offset_dev: int,
                 sub_bits_dev: int, ws_dev: int, ws_bytes: int, stream: int = 0) -> None:
    _check(lib().dnns_deflate(src_dev or None, n_bytes, stream_dev, stream_capacity, chunk_offset_dev, sub_bits_dev,
                              ws_dev, ws_bytes, stream), "dnns_deflate")


def dnns_inflate(stream_dev: int, stream_bytes: int, chunk_offset_dev: int, sub_bits_dev: int, n_bytes: int,
                 dst_dev: int, status_dev: int, stream: int = 0) -> None:
    _check(lib().dnns_inflate(stream_dev, stream_bytes, chunk_offset_dev, sub_bits_dev, n_bytes, dst_dev or None,
                              status_dev, stream), "dnns_inflate")


def dnns_plan_profile(plan, enable: bool) -> None:
    _check(lib().dnns_plan_profile(plan, int(enable)), "dnns_plan_profile")


def dnns_plan_tie_sweep(plan) -> bool:
    """Whether the latest threshold call (or a masking sweep after it) read the weights once more for the tie tables."""
    flag = C.c_int32(0)
    _check(lib().dnns_plan_tie_sweep(plan, C.byref(flag)), "dnns_plan_tie_sweep")
    return bool(flag.value)


def dnns_plan_profile_read(plan, kernel: str):
    """(total device milliseconds, launches) of the recorded kernels whose name starts with `kernel`."""
    ms, n = C.c_double(0), C.c_uint64(0)
    _check(lib().dnns_plan_profile_read(plan, kernel.encode(), C.byref(ms), C.byref(n)), "dnns_plan_profile_read")
    return ms.value, n.value


def _ptr_array(ptrs):
    """A host array of device pointers (None -> NULL entry); None for the whole list -> NULL."""
    if ptrs is None:
        return None
    return (C.c_void_p * len(ptrs))(*[p or None for p in ptrs])


def dnns_mask_and_structures_multi(plan, thr_dev: int, first_variant: int, n_variants: int, masked_arenas, mask_bits,
                                   nz_map, out_nz, in_nz, stream: int = 0) -> None:
    """masked_arenas, out_nz, in_nz: lists of n_variants device addresses; mask_bits, nz_map: lists or None."""
    arrays = [_ptr_array(a) for a in (masked_arenas, mask_bits, nz_map, out_nz, in_nz)]
    _check(lib().dnns_mask_and_structures_multi(plan, thr_dev, first_variant, n_variants, *arrays, stream),
           "dnns_mask_and_structures_multi")


def dnns_propagate_keep_multi(plan, n_variants: int, out_nz, in_nz, policy: int, min_keep: int, keep_bits, keep_idx,
                              keep_count, stats: int, stream: int = 0) -> None:
    """out_nz ... keep_count: lists of n_variants device addresses; stats: one address (4 words per variant) or 0."""
    arrays = [_ptr_array(a) for a in (out_nz, in_nz)]
    outs = [_ptr_array(a) for a in (keep_bits, keep_idx, keep_count)]
    _check(lib().dnns_propagate_keep_multi(plan, n_variants, arrays[0], arrays[1], policy, min_keep, *outs, stats or None,
                                           stream), "dnns_propagate_keep_multi")


def dnns_zero_structures_portfolio(plan, thr_dev: int, first_variant: int, n_variants: int, out_nz, in_nz,
                                   stream: int = 0) -> None:
    """out_nz, in_nz: lists of n_variants device addresses."""
    _check(lib().dnns_zero_structures_portfolio(plan, thr_dev, first_variant, n_variants, _ptr_array(out_nz),
                                                _ptr_array(in_nz), stream), "dnns_zero_structures_portfolio")


def dnns_compact_masked_multi(plan, thr_dev: int, first_variant: int, n_variants: int, keep_idx, keep_count, dst_arenas,
                              dst_bytes: int, dst_offsets_dev, dst_shapes_dev, stream: int = 0) -> None:
    """keep_idx ... dst_shapes_dev: lists of n_variants device addresses (dst_bytes: size of every arena)."""
    a = [_ptr_array(x) for x in (keep_idx, keep_count, dst_arenas)]
    b = [_ptr_array(x) for x in (dst_offsets_dev, dst_shapes_dev)]
    _check(lib().dnns_compact_masked_multi(plan, thr_dev, first_variant, n_variants, a[0], a[1], a[2], dst_bytes, b[0], b[1],
                                           stream), "dnns_compact_masked_multi")


def dnns_compact_masked(plan, thr_dev: int, variant: int, keep_idx: int, keep_count: int, dst_arena: int,
                        dst_bytes: int, dst_offsets_dev: int, dst_shapes_dev: int, stream: int = 0) -> None:
    _check(lib().dnns_compact_masked(plan, thr_dev, variant, keep_idx, keep_count, dst_arena, dst_bytes,
                                     dst_offsets_dev, dst_shapes_dev, stream), "dnns_compact_masked")
