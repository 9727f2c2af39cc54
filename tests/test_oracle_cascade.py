"""Pins for the oracle's fixed-point keep propagation (O8): one pass is Algorithm 1's single pass,
a hand-built chain, a brute-force numpy re-statement, idempotence on the rebuilt model, and the
forward pass of the rebuilt model."""
import numpy as np
import pytest
import torch

from forward_ref import forward, silenced_reference
from oracle import oracle as O
from paper_2309_06973_b200 import workloads as W
from test_oracle_mask import bits_to_bool
from test_oracle_plan import plan as single_pass_plan


def masked_model(wl, v):
    om = O.OracleModel(wl)
    rec = O.threshold(om, wl.scope, wl.ks)
    masked, _ = O.apply_mask(om, wl.scope, rec[v])
    return masked


@pytest.mark.parametrize("policy", [O.RULE_PRODUCER, O.RULE_PRODUCER | O.RULE_CONSUMER])
def test_one_pass_is_the_single_pass_plan(policy):
    wl = W.small_resnet(seed=3)
    masked = masked_model(wl, len(wl.ks) - 1)
    nz, out_nz, in_nz = O.zero_structures(masked)
    a = O.propagate_keep(masked, out_nz, in_nz, policy, 1)
    b = O.propagate_keep_cascade(masked, nz, policy, 1, max_passes=1)
    assert np.array_equal(a[2], b[2])
    for x, y in zip(a[0], b[0]):
        assert np.array_equal(x, y)
    assert a[3][:3].tolist() == b[3][:3].tolist()


def hand_chain():
    """L0 2->3, L1 3->3, L2 3->2 (1x1).  L0's filter 1 is zero.  L1's filter 0 only reads channel 1.
    L2 only reads channel 0 of L1's output... through column 0."""
    b = W._Builder()
    g0 = b.group(2, frozen=True)
    g1, g2 = b.group(3), b.group(3)
    g3 = b.group(2, frozen=True)
    b.conv_bn("L0", "x", "a0", g0, g1, 1, 1, 0)
    b.conv_bn("L1", "a0", "a1", g1, g2, 1, 1, 0)
    b.conv_bn("L2", "a1", "out", g2, g3, 1, 1, 0)
    wl = W.Workload("hand", 0, W.SCOPE_GLOBAL, b.tensors, b.bns, b.groups, b.ops, 4)
    w0 = np.ones((3, 2, 1, 1), np.float32); w0[1] = 0                     # channel 1 of g1 is never produced
    w1 = np.ones((3, 3, 1, 1), np.float32); w1[0] = 0; w1[0, 1] = 5       # filter 0 of L1 only reads channel 1
    w2 = np.ones((2, 3, 1, 1), np.float32)
    wl.weights = [w0, w1, w2]
    wl.biases = [None] * 3
    wl.bn_params = [(np.ones(t.O, np.float32), np.zeros(t.O, np.float32), np.zeros(t.O, np.float32),
                     np.ones(t.O, np.float32)) for t in wl.tensors]
    wl.ks = np.zeros((1, 1), np.uint64)
    return wl


def test_hand_built_chain_cascades():
    wl = hand_chain()
    om = O.OracleModel(wl)
    nz, out_nz, in_nz = O.zero_structures(om)
    _, ki, kc, st = O.propagate_keep(om, out_nz, in_nz, O.RULE_PRODUCER, 1)
    assert ki[1][: kc[1]].tolist() == [0, 2] and kc[2] == 3               # single pass: only the zero filter goes
    _, ki, kc, st = O.propagate_keep_cascade(om, nz, O.RULE_PRODUCER, 1)
    assert ki[1][: kc[1]].tolist() == [0, 2]
    assert ki[2][: kc[2]].tolist() == [1, 2]                               # pass 2: L1's filter 0 read nothing that is left
    assert int(st[3]) == 2 and int(st[1]) == 2
    # consumer side: make L2 read only channel 2 of g2; then channels 0 and 1 of g2 go, and with them
    # everything in g1 that only fed those filters
    wl.weights[2][:, :2] = 0
    wl.weights[1][2] = 0; wl.weights[1][2, 2] = 1                          # filter 2 of L1 only reads channel 2 of g1
    om = O.OracleModel(wl)
    nz, _, _ = O.zero_structures(om)
    _, ki, kc, st = O.propagate_keep_cascade(om, nz, O.RULE_PRODUCER | O.RULE_CONSUMER, 1)
    assert ki[2][: kc[2]].tolist() == [2]
    assert ki[1][: kc[1]].tolist() == [2]                                  # channel 0 of g1 fed only removed filters


def brute_force(wl, weights, policy, max_passes=64):
    """Independent numpy re-statement on boolean kernel maps (no BatchNorm strictness, min_keep 0)."""
    nzs = [(w.reshape(w.shape[0], w.shape[1], -1) != 0).any(-1) for w in weights]
    removed = [np.zeros(g.C, bool) for g in wl.groups]
    for _ in range(max_passes):
        new = [r.copy() for r in removed]
        for g, grp in enumerate(wl.groups):
            if grp.flags & W.GROUP_FROZEN:
                continue
            prods = [i for i, t in enumerate(wl.tensors) if t.out_group == g]
            cons = [i for i, t in enumerate(wl.tensors) if t.in_group == g]
            pd = np.full(grp.C, bool(prods))
            for p in prods:
                t = wl.tensors[p]
                kept_cols = ~np.repeat(removed[t.in_group], t.in_spatial)
                pd &= ~(nzs[p][:, kept_cols].any(1))
            cd = np.full(grp.C, bool(cons))
            for q in cons:
                t = wl.tensors[q]
                live = nzs[q][~removed[t.out_group]].any(0).reshape(grp.C, t.in_spatial).any(1)
                cd &= ~live
            rule = (pd if policy & O.RULE_PRODUCER else False) | (cd if policy & O.RULE_CONSUMER else False)
            new[g] |= rule
        if all(np.array_equal(a, b) for a, b in zip(new, removed)):
            break
        removed = new
    return removed


@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("policy", [O.RULE_PRODUCER, O.RULE_CONSUMER, O.RULE_PRODUCER | O.RULE_CONSUMER])
def test_cascade_equals_brute_force(seed, policy):
    wl = W.small_resnet(seed=seed, bottleneck=bool(seed % 2))
    masked = masked_model(wl, len(wl.ks) - 1)
    nz, _, _ = O.zero_structures(masked)
    kb, ki, kc, st = O.propagate_keep_cascade(masked, nz, policy, 0)
    want = brute_force(wl, masked.weights, policy)
    for g, grp in enumerate(wl.groups):
        assert np.array_equal(~bits_to_bool(kb[g], grp.C), want[g]), g


def test_rebuilt_model_is_a_fixed_point_and_subset_of_single_pass():
    wl = W.resnet56()
    masked = masked_model(wl, 9)
    nz, out_nz, in_nz = O.zero_structures(masked)
    kb1, _, kc1, _ = O.propagate_keep(masked, out_nz, in_nz)
    kb, ki, kc, st = O.propagate_keep_cascade(masked, nz)
    assert int(st[2]) == 0
    for g, grp in enumerate(wl.groups):
        assert np.all(bits_to_bool(kb1[g], grp.C)[bits_to_bool(kb[g], grp.C)])          # cascade keeps a subset
    assert kc.sum() <= kc1.sum() and int(st[3]) >= 1
    # on the rebuilt model a single pass finds nothing more to remove
    from model_utils import compacted_workload
    cw, cbn, cb, _ = O.compact(masked, ki, kc)
    small = compacted_workload(wl, kc, cw, cbn, cb)
    om2 = O.OracleModel(small)
    _, o2, i2 = O.zero_structures(om2)
    _, _, kc2, _ = O.propagate_keep(om2, o2, i2)
    assert np.array_equal(kc2, kc)


@pytest.mark.parametrize("make,hw", [(lambda: W.small_resnet(seed=6), 32), (W.resnet56, 32)])
def test_cascaded_model_computes_what_the_sparse_model_computes(make, hw):
    wl = make()
    x = torch.from_numpy(np.random.default_rng(9).standard_normal((2, 3, hw, hw)).astype(np.float32))
    masked = masked_model(wl, len(wl.ks) - 1)
    nz, _, _ = O.zero_structures(masked)
    kb, ki, kc, st = O.propagate_keep_cascade(masked, nz)
    cw, cbn, cb, _ = O.compact(masked, ki, kc)
    y = forward(wl, cw, cbn, cb, x)
    mw, mbn, mb = silenced_reference(wl, masked.weights, wl.bn_params, wl.biases, kb)
    y_ref = forward(wl, mw, mbn, mb, x)
    assert float((y - y_ref).abs().max()) <= 1e-5 * float(y_ref.abs().max())
