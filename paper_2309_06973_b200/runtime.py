"""Device-side plumbing around the C ABI: torch is used for device memory and streams only.

``DeviceModel`` puts a workload's arrays on the GPU and fills the ``dnns_model`` descriptors;
``Session`` owns a plan, its workspace and one set of output buffers, and exposes the five
steps plus read-back helpers.  No step of the method is computed here.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional

import numpy as np
import torch

from . import binding as B

REC_DTYPE = np.dtype([("tau_bits", "<u4"), ("pad", "<u4"), ("n_below", "<u8"), ("n_tie", "<u8"), ("n_equal", "<u8")])


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _to_dev(a: np.ndarray, device) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    elif a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(a).to(device)


class DeviceModel:
    """A workload's tensors, BatchNorm vectors and biases resident on one GPU."""

    def __init__(self, wl, dtype: int = B.DNNS_F32, device="cuda:0", weights: Optional[List[np.ndarray]] = None,
                 pinned_host: bool = False):
        self.wl, self.dtype, self.device = wl, dtype, torch.device(device)
        host_w = weights if weights is not None else wl.weights_as(dtype)
        self.elem_bytes = 4 if dtype == B.DNNS_F32 else 2
        # one allocation for all weights (256-byte aligned pieces) so that a host copy is one transfer
        offs, o = [], 0
        for w in host_w:
            offs.append(o)
            o = (o + w.size * self.elem_bytes + 255) // 256 * 256
        self.weight_offsets, self.weight_bytes = offs, o
        host = torch.zeros(o, dtype=torch.uint8)
        hv = host.numpy()
        for w, off in zip(host_w, offs):
            hv[off: off + w.size * self.elem_bytes] = np.ascontiguousarray(w).view(np.uint8).ravel()
        self.host_weights = host.pin_memory() if pinned_host else host
        self.weights = torch.empty(o, dtype=torch.uint8, device=self.device)
        self.weights.copy_(self.host_weights)
        self.biases = [None if b is None else _to_dev(b.astype(np.float32), self.device) for b in wl.biases]
        self.bn = [tuple(_to_dev(np.asarray(v, np.float32), self.device) for v in p) for p in wl.bn_params]
        self._t = (B.dnns_tensor * len(wl.tensors))()
        base = self.weights.data_ptr()
        for i, t in enumerate(wl.tensors):
            self._t[i] = B.dnns_tensor(base + offs[i], dtype, t.O, t.I, t.KH, t.KW, t.in_spatial, int(t.prunable),
                                       t.out_group, t.in_group,
                                       None if self.biases[i] is None else self.biases[i].data_ptr())
        self._b = (B.dnns_bn * max(1, len(wl.bns)))()
        for i, b in enumerate(wl.bns):
            g, be, mu, va = self.bn[i]
            self._b[i] = B.dnns_bn(g.data_ptr(), be.data_ptr(), mu.data_ptr(), va.data_ptr(), b.C, b.tensor, b.eps)
        self._g = (B.dnns_group * len(wl.groups))()
        for i, g in enumerate(wl.groups):
            self._g[i] = B.dnns_group(g.C, g.flags)
        self.c = B.dnns_model(len(wl.tensors), self._t, len(wl.bns), self._b, len(wl.groups), self._g)

    def upload_weights(self):
        """Host-to-device copy of all weights (one transfer from the host staging buffer)."""
        self.weights.copy_(self.host_weights, non_blocking=True)


class Session:
    """A plan with its workspace and one set of output buffers for one variant at a time."""

    def __init__(self, dm: DeviceModel, scope: int, max_variants: int, want_mask_bits: bool = True,
                 want_nz_map: bool = True, slots: int = 1, portfolio_slots: int = 0, portfolio_arenas: bool = False):
        """slots > 1 adds that many more sets of per-variant buffers for the multi-variant sweep;
        portfolio_slots adds sets of flags and keep sets only (no sparse model) for the portfolio-wide calls;
        portfolio_arenas gives each of those a destination arena of its own (rebuild of all variants in one launch)."""
        self.dm, self.scope, self.max_variants, self.slots = dm, scope, max_variants, slots
        dev = dm.device
        nbytes = B.dnns_workspace_bytes(dm.c, scope, max_variants)
        if nbytes == 0:
            raise B.DnnsError(B.DNNS_ERR_INVALID_ARG, "dnns_workspace_bytes")
        self.ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        self.plan = B.dnns_plan_create(dm.c, scope, max_variants, self.ws.data_ptr(), nbytes, _stream())
        L = B.dnns_plan_layout(self.plan)
        self.L = L
        T, G, S = L.n_tensors, L.n_groups, L.n_segments
        self.n_segments = S
        arr = lambda p, n, dt: np.array([p[i] for i in range(n)], dt)
        self.arena_offset = arr(L.arena_offset, T, np.uint64)
        self.mask_offset = arr(L.mask_offset, T, np.uint64)
        self.nz_map_offset = arr(L.nz_map_offset, T, np.uint64)
        self.out_nz_offset = arr(L.out_nz_offset, T, np.uint64)
        self.in_nz_offset = arr(L.in_nz_offset, T, np.uint64)
        self.keep_offset = arr(L.keep_offset, G, np.uint64)
        self.keep_idx_offset = arr(L.keep_idx_offset, G, np.uint64)
        self.segment_size = arr(L.segment_size, max(S, 1), np.uint64)
        i32 = lambda n: torch.zeros(max(int(n), 1), dtype=torch.int32, device=dev)
        self.thr = torch.zeros(max_variants * max(S, 1) * REC_DTYPE.itemsize, dtype=torch.uint8, device=dev)
        self.masked = torch.empty(int(L.masked_arena_bytes), dtype=torch.uint8, device=dev)
        self.mask_bits = i32(L.mask_words) if want_mask_bits else None
        self.nz_map = i32(L.nz_map_words) if want_nz_map else None
        self.out_nz, self.in_nz = i32(L.out_nz_words), i32(L.in_nz_words)
        self.keep_bits, self.keep_idx = i32(L.keep_words), i32(L.keep_idx_len)
        self.keep_count = i32(G)
        self.stats = torch.zeros(4, dtype=torch.int64, device=dev)
        self.compact_arena = torch.empty(int(L.compact_arena_bytes), dtype=torch.uint8, device=dev)
        self.dst_offsets = torch.zeros(L.n_compact_items, dtype=torch.int64, device=dev)
        self.dst_shapes = i32(2 * T)
        # slot 0 is the set above; slots 1.. are further sets of what differs per variant before the rebuild
        self.extra = []
        for _ in range(1, slots):
            self.extra.append({
                "masked": torch.empty(int(L.masked_arena_bytes), dtype=torch.uint8, device=dev),
                "mask_bits": i32(L.mask_words) if want_mask_bits else None,
                "nz_map": i32(L.nz_map_words) if want_nz_map else None,
                "out_nz": i32(L.out_nz_words), "in_nz": i32(L.in_nz_words),
                "keep_bits": i32(L.keep_words), "keep_idx": i32(L.keep_idx_len), "keep_count": i32(G)})
        self.stats_multi = torch.zeros(4 * max(slots, portfolio_slots, 1), dtype=torch.int64, device=dev)
        self.pf = [{"out_nz": i32(L.out_nz_words), "in_nz": i32(L.in_nz_words), "keep_bits": i32(L.keep_words),
                    "keep_idx": i32(L.keep_idx_len), "keep_count": i32(G)} for _ in range(portfolio_slots)]
        if portfolio_arenas:
            for slot in self.pf:
                slot["arena"] = torch.empty(int(L.compact_arena_bytes), dtype=torch.uint8, device=dev)
                slot["dst_offsets"] = torch.zeros(L.n_compact_items, dtype=torch.int64, device=dev)
                slot["dst_shapes"] = i32(2 * T)

    def _slot(self, name: str, slot: int):
        return getattr(self, name) if slot == 0 else self.extra[slot - 1][name]

    def close(self):
        if self.plan is not None:
            B.dnns_plan_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the five steps -------------------------------------------------------------
    def magnitude_threshold(self, ks: np.ndarray):
        ks = np.ascontiguousarray(ks, np.uint64)
        assert ks.ndim == 2 and ks.shape[1] == self.n_segments
        self.n_k = ks.shape[0]
        B.dnns_magnitude_threshold(self.plan, ks.ravel().tolist(), ks.shape[0], self.thr.data_ptr(), _stream())

    def apply_mask(self, variant: int, in_place: bool = False):
        B.dnns_apply_mask(self.plan, self.thr.data_ptr(), variant, 0 if in_place else self.masked.data_ptr(),
                          0 if self.mask_bits is None else self.mask_bits.data_ptr(), _stream())

    def zero_structures(self, from_model: bool = False):
        B.dnns_zero_structures(self.plan, 0 if from_model else self.masked.data_ptr(),
                               0 if self.nz_map is None else self.nz_map.data_ptr(), self.out_nz.data_ptr(),
                               self.in_nz.data_ptr(), _stream())

    def mask_and_structures(self, variant: int, in_place: bool = False):
        B.dnns_mask_and_structures(self.plan, self.thr.data_ptr(), variant, 0 if in_place else self.masked.data_ptr(),
                                   0 if self.mask_bits is None else self.mask_bits.data_ptr(),
                                   0 if self.nz_map is None else self.nz_map.data_ptr(), self.out_nz.data_ptr(),
                                   self.in_nz.data_ptr(), _stream())

    def mask_and_structures_multi(self, first_variant: int, n_variants: int, store_masked: bool = True):
        """Steps 2 and 3 of n_variants consecutive variants in one sweep; variant first_variant + g lands in slot g.
        store_masked = False: only mask bits and zero structures are written (rebuild with compact_masked)."""
        ptrs = lambda name: [None if self._slot(name, g) is None else self._slot(name, g).data_ptr() for g in range(n_variants)]
        B.dnns_mask_and_structures_multi(self.plan, self.thr.data_ptr(), first_variant, n_variants,
                                         ptrs("masked") if store_masked else [None] * n_variants,
                                         None if self.mask_bits is None else ptrs("mask_bits"),
                                         None if self.nz_map is None else ptrs("nz_map"), ptrs("out_nz"), ptrs("in_nz"),
                                         _stream())

    def propagate_keep(self, policy: int = B.DNNS_RULE_PRODUCER | B.DNNS_RULE_CONSUMER, min_keep: int = 1, slot: int = 0):
        B.dnns_propagate_keep(self.plan, self._slot("out_nz", slot).data_ptr(), self._slot("in_nz", slot).data_ptr(), policy, min_keep,
                              self.keep_bits.data_ptr(), self.keep_idx.data_ptr(), self.keep_count.data_ptr(),
                              self.stats.data_ptr(), _stream())

    def propagate_keep_multi(self, n_variants: int, policy: int = B.DNNS_RULE_PRODUCER | B.DNNS_RULE_CONSUMER,
                             min_keep: int = 1):
        """Step 4 of the n_variants variants of the latest multi-variant sweep in one launch; slot g keeps its own
        keep sets (slot 0: the session's), read by compact(slot=g, own_keep=True)."""
        ptrs = lambda name: [self._slot(name, g).data_ptr() for g in range(n_variants)]
        B.dnns_propagate_keep_multi(self.plan, n_variants, ptrs("out_nz"), ptrs("in_nz"), policy, min_keep,
                                    ptrs("keep_bits"), ptrs("keep_idx"), ptrs("keep_count"), self.stats_multi.data_ptr(),
                                    _stream())

    def compact(self, from_model: bool = False, dst_bytes: Optional[int] = None, slot: int = 0, own_keep: bool = False):
        """own_keep: rebuild from the keep sets of the slot itself (written by propagate_keep_multi)."""
        keep_slot = slot if own_keep else 0
        B.dnns_compact(self.plan, 0 if from_model else self._slot("masked", slot).data_ptr(),
                       self._slot("keep_idx", keep_slot).data_ptr(),
                       self._slot("keep_count", keep_slot).data_ptr(), self.compact_arena.data_ptr(),
                       self.compact_arena.numel() if dst_bytes is None else dst_bytes, self.dst_offsets.data_ptr(),
                       self.dst_shapes.data_ptr(), _stream())

    def compact_masked(self, variant: int, slot: int = 0, own_keep: bool = False):
        """Rebuild `variant` straight from the dense model, masking on the way (keep sets of `slot` with own_keep)."""
        keep_slot = slot if own_keep else 0
        B.dnns_compact_masked(self.plan, self.thr.data_ptr(), variant,
                              self._slot("keep_idx", keep_slot).data_ptr(), self._slot("keep_count", keep_slot).data_ptr(),
                              self.compact_arena.data_ptr(), self.compact_arena.numel(), self.dst_offsets.data_ptr(),
                              self.dst_shapes.data_ptr(), _stream())

    # ---- the whole portfolio without a sparse model: flags of all variants from one sweep, keep sets in one launch,
    # then a masking rebuild per variant (slot i holds variant first_variant + i)
    def zero_structures_portfolio(self, first_variant: int, n_variants: int):
        B.dnns_zero_structures_portfolio(self.plan, self.thr.data_ptr(), first_variant, n_variants,
                                         [self.pf[i]["out_nz"].data_ptr() for i in range(n_variants)],
                                         [self.pf[i]["in_nz"].data_ptr() for i in range(n_variants)], _stream())

    def propagate_keep_portfolio(self, n_variants: int, policy: int = B.DNNS_RULE_PRODUCER | B.DNNS_RULE_CONSUMER,
                                 min_keep: int = 1):
        ptrs = lambda name: [self.pf[i][name].data_ptr() for i in range(n_variants)]
        B.dnns_propagate_keep_multi(self.plan, n_variants, ptrs("out_nz"), ptrs("in_nz"), policy, min_keep,
                                    ptrs("keep_bits"), ptrs("keep_idx"), ptrs("keep_count"), self.stats_multi.data_ptr(),
                                    _stream())

    def compact_portfolio(self, variant: int, slot: int, arena: Optional[torch.Tensor] = None):
        """Rebuild `variant` from the dense model with the keep sets of portfolio slot `slot` (arena: another
        destination than the session's own)."""
        arena = self.compact_arena if arena is None else arena
        B.dnns_compact_masked(self.plan, self.thr.data_ptr(), variant, self.pf[slot]["keep_idx"].data_ptr(),
                              self.pf[slot]["keep_count"].data_ptr(), arena.data_ptr(), arena.numel(),
                              self.dst_offsets.data_ptr(), self.dst_shapes.data_ptr(), _stream())

    def compact_portfolio_multi(self, first_variant: int, n_variants: int):
        """Rebuild variants first_variant .. from the dense model in one launch, slot i into its own arena."""
        ptrs = lambda name: [self.pf[i][name].data_ptr() for i in range(n_variants)]
        B.dnns_compact_masked_multi(self.plan, self.thr.data_ptr(), first_variant, n_variants, ptrs("keep_idx"),
                                    ptrs("keep_count"), ptrs("arena"), self.pf[0]["arena"].numel(), ptrs("dst_offsets"),
                                    ptrs("dst_shapes"), _stream())

    def propagate_keep_cascade(self, policy: int = B.DNNS_RULE_PRODUCER | B.DNNS_RULE_CONSUMER, min_keep: int = 1,
                               max_passes: int = 8):
        B.dnns_propagate_keep_cascade(self.plan, self.nz_map.data_ptr(), policy, min_keep, max_passes,
                                      self.keep_bits.data_ptr(), self.keep_idx.data_ptr(), self.keep_count.data_ptr(),
                                      self.stats.data_ptr(), _stream())

    def fold_batchnorm(self):
        """Fold the BatchNorms of the variant in the destination arena into its convolutions (in place)."""
        B.dnns_fold_batchnorm(self.plan, self.compact_arena.data_ptr(), self.dst_offsets.data_ptr(),
                              self.dst_shapes.data_ptr(), _stream())

    def variant(self, v: int, policy: int = B.DNNS_RULE_PRODUCER | B.DNNS_RULE_CONSUMER, min_keep: int = 1,
                fused: bool = False):
        """Steps 2-5 for variant v of the latest threshold call (fused: steps 2 and 3 in one sweep)."""
        if fused:
            self.mask_and_structures(v)
        else:
            self.apply_mask(v)
            self.zero_structures()
        self.propagate_keep(policy, min_keep)
        self.compact()

    def device_status(self) -> int:
        return B.dnns_last_device_status(self.plan, _stream())

    def launch_count(self) -> int:
        return B.dnns_plan_launch_count(self.plan)

    def tie_sweep_ran(self) -> bool:
        return B.dnns_plan_tie_sweep(self.plan)

    def profile(self, enable: bool):
        B.dnns_plan_profile(self.plan, enable)

    def kernel_time(self, kernel: str):
        """(total ms, launches) of a kernel since the profile was switched on."""
        return B.dnns_plan_profile_read(self.plan, kernel)

    # ---- read-back (host copies, for tests and reports) ------------------------------------
    def records(self) -> np.ndarray:
        n = self.n_k * self.n_segments
        raw = self.thr.cpu().numpy()[: n * REC_DTYPE.itemsize]
        return raw.view(REC_DTYPE).reshape(self.n_k, self.n_segments).copy()

    def _np_dtype(self):
        return np.float32 if self.dm.dtype == B.DNNS_F32 else np.uint16

    def masked_tensors(self, in_place: bool = False, slot: int = 0) -> List[np.ndarray]:
        wl, eb = self.dm.wl, self.dm.elem_bytes
        if in_place:
            raw, offs = self.dm.weights.cpu().numpy(), self.dm.weight_offsets
        else:
            raw, offs = self._slot("masked", slot).cpu().numpy(), self.arena_offset
        return [raw[int(o): int(o) + t.numel * eb].view(self._np_dtype()).reshape(t.O, t.I, t.KH, t.KW).copy()
                for t, o in zip(wl.tensors, offs)]

    def _split_words(self, buf, offsets, nbits) -> List[np.ndarray]:
        raw = buf.cpu().numpy().view(np.uint32)
        return [raw[int(o): int(o) + (n + 31) // 32].copy() for o, n in zip(offsets, nbits)]

    def mask_words(self, slot: int = 0):
        return self._split_words(self._slot("mask_bits", slot), self.mask_offset, [t.numel for t in self.dm.wl.tensors])

    def structure_words(self, slot: int = 0, portfolio: bool = False):
        wl = self.dm.wl
        get = (lambda n: self.pf[slot][n]) if portfolio else (lambda n: self._slot(n, slot))
        nz = None if self.nz_map is None or portfolio else self._split_words(get("nz_map"), self.nz_map_offset,
                                                                              [t.O * t.I for t in wl.tensors])
        return (nz, self._split_words(get("out_nz"), self.out_nz_offset, [t.O for t in wl.tensors]),
                self._split_words(get("in_nz"), self.in_nz_offset, [t.I for t in wl.tensors]))

    def keep_sets(self, slot: int = 0, multi_stats: bool = False, portfolio: bool = False):
        """multi_stats: the statistics written by propagate_keep_multi for this slot."""
        wl = self.dm.wl
        get = (lambda n: self.pf[slot][n]) if portfolio else (lambda n: self._slot(n, slot))
        bits = self._split_words(get("keep_bits"), self.keep_offset, [g.C for g in wl.groups])
        cnt = get("keep_count").cpu().numpy()[: len(wl.groups)].copy()
        idx_raw = get("keep_idx").cpu().numpy()
        idx = [idx_raw[int(o): int(o) + int(c)].copy() for o, c in zip(self.keep_idx_offset, cnt)]
        st = self.stats_multi[4 * slot: 4 * slot + 4] if multi_stats else self.stats
        return bits, idx, cnt, st.cpu().numpy().view(np.uint64).copy()

    def compacted(self, keep_slot: int = 0, portfolio: bool = False, own_arena: bool = False):
        """(weights [(O', I', KH, KW)], bn [(g, b, m, v)], biases, shapes (T, 2), offsets) of the variant rebuilt
        last; keep_slot: the slot whose keep sets it was rebuilt from."""
        wl, eb = self.dm.wl, self.dm.elem_bytes
        T = len(wl.tensors)
        src = self.pf[keep_slot] if own_arena else {"dst_offsets": self.dst_offsets, "dst_shapes": self.dst_shapes,
                                                      "arena": self.compact_arena}
        offs = src["dst_offsets"].cpu().numpy().view(np.uint64)
        shapes = src["dst_shapes"].cpu().numpy()[: 2 * T].reshape(T, 2).copy()
        raw = src["arena"].cpu().numpy()
        ws = []
        for i, t in enumerate(wl.tensors):
            On, In = int(shapes[i, 0]), int(shapes[i, 1])
            n = On * In * t.KH * t.KW
            ws.append(raw[int(offs[i]): int(offs[i]) + n * eb].view(self._np_dtype()).reshape(On, In, t.KH, t.KW).copy())
        cnt = (self.pf[keep_slot]["keep_count"] if portfolio else self._slot("keep_count", keep_slot)).cpu().numpy()
        bns, k = [], T
        for b in wl.bns:
            Cn = int(cnt[wl.tensors[b.tensor].out_group])
            vecs = []
            for _ in range(4):
                vecs.append(raw[int(offs[k]): int(offs[k]) + 4 * Cn].view(np.float32).copy())
                k += 1
            bns.append(tuple(vecs))
        biases = []
        for i, t in enumerate(wl.tensors):
            if wl.biases[i] is None:
                biases.append(None)
            else:
                On = int(shapes[i, 0])
                biases.append(raw[int(offs[k]): int(offs[k]) + 4 * On].view(np.float32).copy())
                k += 1
        return ws, bns, biases, shapes, offs.copy()


class Deflater:
    """Buffers for dnns_deflate / dnns_inflate of byte strings of up to `max_bytes` (device memory only)."""

    def __init__(self, max_bytes: int, device="cuda:0"):
        self.device, self.max_bytes = torch.device(device), max_bytes
        nc = B.dnns_deflate_chunks(max_bytes)
        u8 = lambda n: torch.empty(max(int(n), 16), dtype=torch.uint8, device=self.device)
        self.capacity = (B.dnns_deflate_bound(max_bytes) + 3) // 4 * 4
        self.stream = u8(self.capacity)
        self.ws_bytes = B.dnns_deflate_workspace_bytes(max_bytes)
        self.ws = u8(self.ws_bytes)
        self.chunk_offset = torch.zeros(nc + 1, dtype=torch.int64, device=self.device)
        self.sub_bits = torch.zeros(32 * nc, dtype=torch.int32, device=self.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.n_bytes = 0

    def deflate(self, src: torch.Tensor, n_bytes: int):
        assert n_bytes <= self.max_bytes
        self.n_bytes = n_bytes
        B.dnns_deflate(src.data_ptr() if n_bytes else 0, n_bytes, self.stream.data_ptr(), self.capacity,
                       self.chunk_offset.data_ptr(), self.sub_bits.data_ptr(), self.ws.data_ptr(), self.ws_bytes, _stream())

    def stream_bytes(self) -> int:
        """Size of the latest stream (synchronises: the size is computed on the device)."""
        return int(self.chunk_offset[B.dnns_deflate_chunks(self.n_bytes)].item())

    def inflate(self, dst: torch.Tensor, stream_bytes: int):
        B.dnns_inflate(self.stream.data_ptr(), stream_bytes, self.chunk_offset.data_ptr(), self.sub_bits.data_ptr(),
                       self.n_bytes, dst.data_ptr() if self.n_bytes else 0, self.status.data_ptr(), _stream())

    def index(self):
        nc = B.dnns_deflate_chunks(self.n_bytes)
        return (self.chunk_offset[: nc + 1].cpu().numpy().view(np.uint64).copy(),
                self.sub_bits[: 32 * nc].cpu().numpy().view(np.uint32).copy())
