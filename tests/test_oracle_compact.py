"""Pins for the oracle's rebuild (O5) and the output-preservation property: Algorithm 2's
sizes, numpy fancy indexing as a library gather, scatter-back identity, "removed
channels carry only zeros", and the forward pass of the pruned model."""
import numpy as np
import pytest
import torch

from forward_ref import forward, silenced_reference
from oracle import oracle as O
from paper_2309_06973_b200 import workloads as W
from test_oracle_mask import bits_to_bool
from test_oracle_threshold import keys_f32


def run_variant(wl, v=0, policy=O.RULE_PRODUCER | O.RULE_CONSUMER, min_keep=1, dtype=O.F32):
    om = O.OracleModel(wl, dtype)
    rec = O.threshold(om, wl.scope, wl.ks)
    masked, _ = O.apply_mask(om, wl.scope, rec[v])
    _, out_nz, in_nz = O.zero_structures(masked)
    kb, ki, kc, st = O.propagate_keep(masked, out_nz, in_nz, policy, min_keep)
    cw, cbn, cbias, shapes = O.compact(masked, ki, kc)
    return masked, kb, ki, kc, st, cw, cbn, cbias, shapes


@pytest.mark.parametrize("policy", [O.RULE_PRODUCER, O.RULE_PRODUCER | O.RULE_CONSUMER])
@pytest.mark.parametrize("make", [W.toy, lambda: W.small_resnet(seed=3), lambda: W.small_resnet(seed=4, bottleneck=False)])
def test_rebuild_sizes_gather_and_scatter_back(make, policy):
    wl = make()
    v = len(wl.ks) - 1
    masked, kb, ki, kc, st, cw, cbn, cbias, shapes = run_variant(wl, v, policy)
    nnz_removed = 0
    for ti, t in enumerate(wl.tensors):
        ko = ki[t.out_group][: kc[t.out_group]]
        kin = ki[t.in_group][: kc[t.in_group]]
        n_out_removed = t.O - len(ko)
        n_in_removed = t.I - len(kin)
        # Algorithm 2: |C'_out| = |C_out(L)| - |C_out|, |C'_in| = |C_in(L)| - |C_in|
        assert tuple(shapes[ti]) == (t.O - n_out_removed, t.I - n_in_removed) == cw[ti].shape[:2]
        src = masked.weights[ti]
        assert np.array_equal(cw[ti], src[np.ix_(ko, kin)])              # numpy's gather
        back = np.zeros_like(src)
        back[np.ix_(ko, kin)] = cw[ti]
        gone = src.copy()
        gone[np.ix_(ko, kin)] = 0
        assert np.array_equal(back + gone, src)
        nnz_removed += int(np.count_nonzero(gone))
        if cbias[ti] is not None:
            assert np.array_equal(cbias[ti], wl.biases[ti][ko])
    for bi, b in enumerate(wl.bns):
        g = wl.tensors[b.tensor].out_group
        ko = ki[g][: kc[g]]
        for got, src in zip(cbn[bi], wl.bn_params[bi]):
            assert np.array_equal(got, src[ko])
    if policy == O.RULE_PRODUCER:
        # under the paper's rule a channel only goes when all its filters are zero, and then the
        # matching input slices of the consumers multiply a channel that is constant: every weight in a
        # removed *filter* is zero; weights in removed input slices may be non-zero
        for ti, t in enumerate(wl.tensors):
            ko = ki[t.out_group][: kc[t.out_group]]
            dead_rows = np.setdiff1d(np.arange(t.O), ko)
            assert not np.any(masked.weights[ti][dead_rows])


def test_nnz_preserved_when_both_axes_rules_agree():
    """On a plain chain with zero BN shift nothing non-zero is lost under the producer rule once the
    consumer slices of dead channels are zero as well (here: they are zeroed by hand)."""
    wl = W.chain([6, 8, 5], seed=2, planted_frac=0.4)
    for ti in range(1, len(wl.tensors)):
        wl.weights[ti][:, wl.planted[ti - 1]] = 0
    wl.ks[:] = 0
    masked, kb, ki, kc, st, cw, *_ = run_variant(wl, 0, O.RULE_PRODUCER)
    assert sum(int(np.count_nonzero(w)) for w in cw) == sum(int(np.count_nonzero(w)) for w in masked.weights)
    assert sum(w.size for w in cw) < sum(w.size for w in masked.weights)


def rel_err(a, b):
    return float((a - b).abs().max() / a.abs().max().clamp_min(1e-300))


@pytest.mark.parametrize("make,hw", [(W.toy, 32), (lambda: W.small_resnet(seed=6), 32),
                                      (lambda: W.small_resnet(seed=7, bottleneck=False), 16), (W.resnet56, 32)])
def test_pruned_model_computes_what_the_sparse_model_computes(make, hw):
    wl = make()
    x = torch.from_numpy(np.random.default_rng(99).standard_normal((2, 3, hw, hw)).astype(np.float32))
    for v in sorted({0, len(wl.ks) - 1}):
        masked, kb, ki, kc, st, cw, cbn, cbias, shapes = run_variant(wl, v)
        y_pruned = forward(wl, cw, cbn, cbias, x)
        mw, mbn, mb = silenced_reference(wl, masked.weights, wl.bn_params, wl.biases, kb)
        y_ref = forward(wl, mw, mbn, mb, x)
        assert rel_err(y_ref, y_pruned) <= 1e-5
        assert y_ref.abs().max() > 0


def test_strict_shift_policy_preserves_the_untouched_sparse_model():
    wl = W.small_resnet(seed=8)
    # make some shifts exactly zero so that the strict policy has something to remove
    for (g, be, mu, va) in wl.bn_params:
        be[::2] = 0.0
        mu[::2] = 0.0
    x = torch.from_numpy(np.random.default_rng(5).standard_normal((2, 3, 32, 32)).astype(np.float32))
    v = len(wl.ks) - 1
    masked, kb, ki, kc, st, cw, cbn, cbias, _ = run_variant(wl, v, O.RULE_PRODUCER | O.RULE_CONSUMER | O.SHIFT_STRICT)
    assert st[0] == 0 and st[1] > 0
    y_sparse = forward(wl, masked.weights, wl.bn_params, wl.biases, x)
    y_pruned = forward(wl, cw, cbn, cbias, x)
    assert rel_err(y_sparse, y_pruned) <= 1e-5


def test_fc_with_spatial_columns_drops_blocks_of_columns():
    """A linear layer fed by a flattened C x S map loses S consecutive columns per removed channel."""
    b = W._Builder()
    gi = b.group(2, frozen=True)
    g1 = b.group(5)
    gc = b.group(3, frozen=True)
    b.conv_bn("c", "x", "a", gi, g1, 1, 1, 0)
    b.fc("fc", "a", "out", g1, gc, in_spatial=4)
    wl = W.Workload("fcS", 0, W.SCOPE_GLOBAL, b.tensors, b.bns, b.groups, b.ops, 2)
    rng = np.random.default_rng(0)
    wl.weights = [rng.uniform(0.5, 1, (5, 2, 1, 1)).astype(np.float32), rng.uniform(0.5, 1, (3, 20, 1, 1)).astype(np.float32)]
    wl.weights[0][[1, 4]] = 0
    wl.biases = [None, np.arange(3, dtype=np.float32)]
    wl.bn_params = [(np.ones(5, np.float32), np.zeros(5, np.float32), np.zeros(5, np.float32), np.ones(5, np.float32))]
    wl.ks = np.zeros((1, 1), np.uint64)
    masked, kb, ki, kc, st, cw, cbn, cbias, shapes = run_variant(wl, 0, O.RULE_PRODUCER)
    assert ki[1][: kc[1]].tolist() == [0, 2, 3]
    cols = [0, 1, 2, 3, 8, 9, 10, 11, 12, 13, 14, 15]
    assert tuple(shapes[1]) == (3, 12)
    assert np.array_equal(cw[1], wl.weights[1][:, cols])
    # consumer rule on an FC with S > 1: a channel is unread only if all of its S columns are zero
    wl.weights[0][[1, 4]] = 1
    wl.weights[1][:, 8:11] = 0
    *_, kc2, _, _, _, _, _ = run_variant(wl, 0, O.RULE_CONSUMER)
    assert kc2[1] == 5
    wl.weights[1][:, 11] = 0
    _, _, ki3, kc3, *_ = run_variant(wl, 0, O.RULE_CONSUMER)
    assert ki3[1][: kc3[1]].tolist() == [0, 1, 3, 4]
