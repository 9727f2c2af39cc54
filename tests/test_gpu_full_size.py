"""GPU parity at the full benchmark sizes, in the launch configuration the benchmark uses: every
output of the chosen variants is still compared element by element (the oracle needs some tens
of seconds per model), plus the forward pass of the rebuilt model."""
import numpy as np
import pytest
import torch

from forward_ref import forward, silenced_reference
from gpu_compare import compare_portfolio, compare_sparse_free
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W

pytestmark = pytest.mark.gpu


def forward_check(wl, ses, dtype, slot=0, keep_slot=0):
    """slot: which buffer set of the session holds the masked weights of the variant rebuilt last;
    keep_slot: which one holds its keep sets."""
    is_bf16 = dtype == B.DNNS_BF16
    x = torch.from_numpy(np.random.default_rng(1).standard_normal((2, 3, wl.input_hw, wl.input_hw)).astype(np.float32))
    cw, cbn, cb, _, _ = ses.compacted(keep_slot)
    kb, _, _, _ = ses.keep_sets(keep_slot)
    mw, mbn, mb = silenced_reference(wl, ses.masked_tensors(slot=slot), wl.bn_params, wl.biases, kb)
    y_ref = forward(wl, mw, mbn, mb, x, is_bf16)
    y = forward(wl, cw, cbn, cb, x, is_bf16)
    assert float((y - y_ref).abs().max()) <= 1e-5 * float(y_ref.abs().max())
    assert float(y_ref.abs().max()) > 0


def forward_check_sparse_free(wl, ses, dtype):
    """The variant rebuilt last by the path that stores no sparse model, against the oracle's sparse model with the
    removed channels silenced."""
    is_bf16 = dtype == B.DNNS_BF16
    x = torch.from_numpy(np.random.default_rng(1).standard_normal((2, 3, wl.input_hw, wl.input_hw)).astype(np.float32))
    cw, cbn, cb, _, _ = ses.compacted(ses.last_slot, portfolio=True, own_arena="arena" in ses.pf[ses.last_slot])
    kb, _, _, _ = ses.keep_sets(ses.last_slot, portfolio=True)
    mw, mbn, mb = silenced_reference(wl, ses.last_masked, wl.bn_params, wl.biases, kb)
    y_ref = forward(wl, mw, mbn, mb, x, is_bf16)
    y = forward(wl, cw, cbn, cb, x, is_bf16)
    assert float((y - y_ref).abs().max()) <= 1e-5 * float(y_ref.abs().max())
    assert float(y_ref.abs().max()) > 0


def test_vgg16_per_layer_95():
    wl = W.vgg16()
    ses = compare_portfolio(wl, B.DNNS_F32, check_structure_maps=True)
    forward_check(wl, ses, B.DNNS_F32)
    ses = compare_sparse_free(wl, B.DNNS_F32)
    forward_check_sparse_free(wl, ses, B.DNNS_F32)


def test_resnet50_three_variants():
    wl = W.resnet50()
    ses = compare_portfolio(wl, B.DNNS_F32, fused=True)
    forward_check(wl, ses, B.DNNS_F32)
    ses = compare_portfolio(wl, B.DNNS_F32, multi=3)          # all three variants from one read of the weights
    forward_check(wl, ses, B.DNNS_F32, slot=2)
    ses = compare_sparse_free(wl, B.DNNS_F32)                 # the benchmark's path: no sparse model at all
    forward_check_sparse_free(wl, ses, B.DNNS_F32)


def test_resnet50_frozen_residual_streams():
    """ResNet-50 as the paper prunes it: residual streams frozen (Section IV-B-2)."""
    wl = W.freeze_streams(W.resnet50())
    ses = compare_sparse_free(wl, B.DNNS_F32, one_launch=True)
    forward_check_sparse_free(wl, ses, B.DNNS_F32)


def test_resnet50_bf16_sparse_free():
    compare_sparse_free(W.resnet50(), B.DNNS_BF16)


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
def test_resnet152_portfolio(dtype):
    wl = W.resnet152()
    ses = compare_portfolio(wl, dtype, variants=[0], fused=False)
    ses = compare_portfolio(wl, dtype, variants=[7], fused=True)
    forward_check(wl, ses, dtype)
    # every variant through the multi-variant sweep: four (fp32) or two (bf16) variants per read of the weights
    G = 4 if dtype == B.DNNS_F32 else 2
    ses = compare_portfolio(wl, dtype, multi=G, multi_plan=True)
    forward_check(wl, ses, dtype, slot=G - 1, keep_slot=G - 1)
    # ... and without the sparse model in memory: mask bits only, the rebuild masks the dense weights on its way
    compare_portfolio(wl, dtype, variants=list(range(8 - G, 8)), multi=G, multi_plan=True, no_store=True)


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
def test_resnet152_portfolio_sparse_free(dtype):
    """The benchmark's own configuration: all eight variants, zero structures from one sweep, keep sets in one
    launch, masking rebuild per variant."""
    wl = W.resnet152()
    ses = compare_sparse_free(wl, dtype, one_launch=True)      # the eight rebuilds in one launch, as the benchmark runs them
    forward_check_sparse_free(wl, ses, dtype)
    compare_sparse_free(wl, dtype)                             # ... and one launch per variant
