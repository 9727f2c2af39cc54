"""No kernel writes outside its outputs: every output buffer of a session is re-allocated with guard
words before and after it, the whole path runs (both dtypes, ragged shapes, every entry point), and
the guards must still hold their pattern.  Out-of-bounds reads cannot be seen this way; the index
arithmetic of the ragged paths is what the odd shapes are there to exercise."""
import numpy as np
import pytest
import torch

from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W
from paper_2309_06973_b200.runtime import DeviceModel, Session

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on each side, a multiple of 256 so the payload keeps its alignment
PATTERN = 0x5A


class Guarded:
    def __init__(self, tensor):
        self.dtype, self.n = tensor.dtype, tensor.numel()
        nbytes = tensor.numel() * tensor.element_size()
        self.raw = torch.full((nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device=tensor.device)
        self.view = self.raw[GUARD: GUARD + nbytes].view(tensor.dtype)
        assert self.view.data_ptr() % 256 == 0

    def intact(self):
        r = self.raw.cpu().numpy()
        return bool(np.all(r[:GUARD] == PATTERN) and np.all(r[-GUARD:] == PATTERN))


def guard_session(ses):
    names = ["thr", "masked", "mask_bits", "nz_map", "out_nz", "in_nz", "keep_bits", "keep_idx", "keep_count", "stats",
             "compact_arena", "dst_offsets", "dst_shapes"]
    guards = {}
    for n in names:
        g = Guarded(getattr(ses, n))
        setattr(ses, n, g.view)
        guards[n] = g
    for i, extra in enumerate(ses.extra):           # the further buffer sets of the multi-variant sweep
        for n in list(extra):
            if extra[n] is not None:
                g = Guarded(extra[n])
                extra[n] = g.view
                guards[f"slot{i + 1}.{n}"] = g
    return guards


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
@pytest.mark.parametrize("make", [W.toy, lambda: W.chain([37, 70, 129, 33], seed=5, kernel=5, planted_frac=0.2),
                                  lambda: W.small_resnet(seed=3), W.resnet56])
def test_guards_survive_every_entry_point(make, dtype):
    wl = make()
    dm = DeviceModel(wl, dtype)
    n_multi = min(len(wl.ks), B.DNNS_MULTI_MAX)
    ses = Session(dm, wl.scope, len(wl.ks), slots=n_multi)
    guards = guard_session(ses)
    ses.magnitude_threshold(wl.ks)
    ses.mask_and_structures_multi(len(wl.ks) - n_multi, n_multi)
    for g in range(n_multi):
        ses.propagate_keep(slot=g)
        ses.compact(slot=g)
    ses.propagate_keep_multi(n_multi)
    for g in range(n_multi):
        ses.compact(slot=g, own_keep=True)
    ses.mask_and_structures_multi(len(wl.ks) - n_multi, n_multi, store_masked=False)
    for g in range(n_multi):
        ses.compact_masked(len(wl.ks) - n_multi + g, slot=g, own_keep=True)
    for v in sorted({0, len(wl.ks) - 1}):
        ses.apply_mask(v)
        ses.zero_structures()
        ses.propagate_keep()
        ses.compact()
        ses.mask_and_structures(v)
        ses.propagate_keep_cascade(max_passes=4)
        ses.compact()
        ses.fold_batchnorm()
    assert ses.device_status() == B.DNNS_OK
    torch.cuda.synchronize()
    for name, g in guards.items():
        assert g.intact(), name


def test_workspace_is_not_overrun():
    """The plan's own workspace: same check, with the workspace placed between guards."""
    wl = W.small_resnet(seed=4, bottleneck=False)
    dm = DeviceModel(wl, B.DNNS_F32)
    nbytes = B.dnns_workspace_bytes(dm.c, wl.scope, len(wl.ks))
    raw = torch.full((nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device=dm.device)
    ses = Session.__new__(Session)
    Session.__init__(ses, dm, wl.scope, len(wl.ks))                   # builds its own plan; replace it by a guarded one
    ses.close()
    ses.ws = raw[GUARD: GUARD + nbytes]
    ses.plan = B.dnns_plan_create(dm.c, wl.scope, len(wl.ks), ses.ws.data_ptr(), nbytes,
                                  torch.cuda.current_stream().cuda_stream)
    ses.magnitude_threshold(wl.ks)
    for v in range(len(wl.ks)):
        ses.variant(v, fused=True)
        ses.propagate_keep_cascade(max_passes=3)
    assert ses.device_status() == B.DNNS_OK
    torch.cuda.synchronize()
    r = raw.cpu().numpy()
    assert np.all(r[:GUARD] == PATTERN) and np.all(r[-GUARD:] == PATTERN)


def test_codec_buffers_are_not_overrun():
    """dnns_deflate / dnns_inflate with every buffer sized exactly as the size queries say, between guards:
    dense bytes (every chunk stored, the largest stream and the fullest slots), sparse bytes, a ragged end."""
    from runtime_guard_codec import run_guarded_codec
    rng = np.random.default_rng(9)
    dense = rng.integers(0, 256, 5 * B.DNNS_DEFLATE_CHUNK + 333, dtype=np.uint8)
    sparse = dense.copy()
    sparse[rng.random(sparse.size) < 0.9] = 0
    for data in (dense, sparse, dense[:7], sparse[: B.DNNS_DEFLATE_CHUNK]):
        run_guarded_codec(data, Guarded)
