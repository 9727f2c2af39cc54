"""Pins for the oracle's keep propagation (O4): Algorithm 1 on a chain, hand-built
residual coupling, frozen groups, min_keep, the strict-shift policy."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2309_06973_b200 import workloads as W
from test_oracle_mask import bits_to_bool, read_golden


def plan(wl, policy=O.RULE_PRODUCER | O.RULE_CONSUMER, min_keep=1, weights=None):
    om = O.OracleModel(wl, O.F32, weights)
    _, out_nz, in_nz = O.zero_structures(om)
    kb, ki, kc, st = O.propagate_keep(om, out_nz, in_nz, policy, min_keep)
    return om, kb, ki, kc, st


def chain_from_golden():
    g = read_golden("chain_plan.txt")
    b = W._Builder()
    g0 = b.group(2, frozen=True)
    g1, g2 = b.group(4), b.group(3)
    g3 = b.group(2, frozen=True)
    b.conv_bn("L0", "x", "a0", g0, g1, 1, 1, 0)
    b.conv_bn("L1", "a0", "a1", g1, g2, 1, 1, 0)
    b.conv_bn("L2", "a1", "out", g2, g3, 1, 1, 0)
    wl = W.Workload("golden_chain", 0, W.SCOPE_GLOBAL, b.tensors, b.bns, b.groups, b.ops, 4)
    rng = np.random.default_rng(0)
    wl.weights = [rng.uniform(0.5, 1.0, (t.O, t.I, 1, 1)).astype(np.float32) for t in wl.tensors]
    for row in g["zero_filters"]:
        wl.weights[int(row[0])][[int(v) for v in row[1:]]] = 0.0
    wl.biases = [None] * 3
    wl.bn_params = [(np.ones(t.O, np.float32), np.full(t.O, 0.25, np.float32), np.zeros(t.O, np.float32),
                     np.ones(t.O, np.float32)) for t in wl.tensors]
    return wl, g


def test_chain_plan_is_algorithm_1_worked_example():
    wl, g = chain_from_golden()
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER)
    for row in g["plan"]:
        n = int(row[0])
        cin = [int(v) for v in row[row.index("cin") + 1: row.index("cout")] if v != "-"]
        cout = [int(v) for v in row[row.index("cout") + 1:] if v != "-"]
        t = wl.tensors[n]
        removed_out = np.flatnonzero(~bits_to_bool(kb[t.out_group], t.O)).tolist()
        removed_in = np.flatnonzero(~bits_to_bool(kb[t.in_group], t.I)).tolist()
        if n == len(wl.tensors) - 1:
            removed_out_expected = []          # the class axis is never pruned
        else:
            removed_out_expected = cout
        assert removed_out == removed_out_expected and removed_in == cin
    for row in g["size"]:
        t = wl.tensors[int(row[0])]
        assert (int(kc[t.in_group]), int(kc[t.out_group])) == (int(row[2]), int(row[4]))
    # beta = 0.25 on every removed channel: three removed (producer, channel) pairs carry a non-zero shift
    assert st.tolist() == [3, 3, 0, 0]


@pytest.mark.parametrize("seed", range(3))
def test_chain_reduces_to_algorithm_1(seed):
    """Producer rule on a plain chain: C_out(L_n) = zero filters of L_n, C_in(L_n) = C_out(L_{n-1}), none for n = 0."""
    wl = W.chain([6, 9, 7, 12], seed=seed, planted_frac=0.34)
    _, kb, ki, kc, _ = plan(wl, O.RULE_PRODUCER)
    convs = [i for i, t in enumerate(wl.tensors) if not t.has_bias]
    zero_ch = {n: set(wl.planted[n].tolist()) for n in convs}            # C_Zero per layer, from the generator
    for n in convs:
        t = wl.tensors[n]
        c_out = zero_ch[n]
        c_in = zero_ch[n - 1] if n > 0 else set()
        assert set(np.flatnonzero(~bits_to_bool(kb[t.out_group], t.O)).tolist()) == c_out
        assert set(np.flatnonzero(~bits_to_bool(kb[t.in_group], t.I)).tolist()) == c_in
        assert int(kc[t.out_group]) == t.O - len(c_out) and int(kc[t.in_group]) == t.I - len(c_in)
    for g_, idx, cnt in zip(wl.groups, ki, kc):
        kept = idx[:cnt]
        assert np.all(np.diff(kept) > 0) and cnt == len(kept)            # strictly ascending


def residual_pair():
    """x -> A (3->4) -> stream; B (4->4, on the stream) ; out = A + B(A); consumer D (4->2)."""
    b = W._Builder()
    gi = b.group(3, frozen=True)
    s = b.group(4)
    go = b.group(2, frozen=True)
    b.conv_bn("A", "x", "a", gi, s, 1, 1, 0)
    b.conv_bn("B", "a", "r", s, s, 1, 1, 0, relu=False)
    b.ops.append(("add", "r", "a", "o"))
    b.conv_bn("D", "o", "out", s, go, 1, 1, 0)
    wl = W.Workload("res", 0, W.SCOPE_GLOBAL, b.tensors, b.bns, b.groups, b.ops, 4)
    rng = np.random.default_rng(1)
    wl.weights = [rng.uniform(0.5, 1.0, (t.O, t.I, 1, 1)).astype(np.float32) for t in wl.tensors]
    wl.biases = [None] * 3
    wl.bn_params = [(np.ones(t.O, np.float32), np.zeros(t.O, np.float32), np.zeros(t.O, np.float32),
                     np.ones(t.O, np.float32)) for t in wl.tensors]
    return wl


def test_stream_channel_needs_every_producer_dead():
    wl = residual_pair()
    wl.weights[0][1] = 0          # A's filter 1 zero, B's filter 1 alive -> channel 1 stays
    wl.weights[0][2] = 0
    wl.weights[1][2] = 0          # both producers' filter 2 zero -> channel 2 goes
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER)
    assert ki[1][: kc[1]].tolist() == [0, 1, 3]
    assert st.tolist() == [0, 1, 0, 0]                                   # beta = 0, mean = 0: shift is zero


def test_consumer_rule_needs_every_consumer_blind():
    wl = residual_pair()
    wl.weights[1][:, 3] = 0       # B does not read channel 3, D still does
    _, kb, ki, kc, _ = plan(wl, O.RULE_CONSUMER)
    assert kc[1] == 4
    wl.weights[2][:, 3] = 0       # now nobody reads it
    _, kb, ki, kc, _ = plan(wl, O.RULE_CONSUMER)
    assert ki[1][: kc[1]].tolist() == [0, 1, 2]
    _, kb, ki, kc, _ = plan(wl, O.RULE_PRODUCER)
    assert kc[1] == 4                                                    # the producer rule alone ignores it


def test_frozen_min_keep_and_strict_shift():
    wl = residual_pair()
    for w in wl.weights[:2]:
        w[:] = 0                   # the whole stream is dead
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER, min_keep=1)
    assert ki[1][: kc[1]].tolist() == [0] and st.tolist() == [0, 3, 1, 0]   # layer collapse: lowest index taken back
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER, min_keep=3)
    assert ki[1][: kc[1]].tolist() == [0, 1, 2]
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER, min_keep=0)
    assert kc[1] == 0
    assert kc[0] == 3 and kc[2] == 2                                     # frozen groups keep everything
    wl.groups[1].flags = W.GROUP_FROZEN
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER)
    assert kc[1] == 4
    wl.groups[1].flags = 0
    # strict: a non-zero BN shift on one producer of channel 2 keeps the channel
    wl.bn_params[1][1][2] = 0.5
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER | O.SHIFT_STRICT, min_keep=0)
    assert ki[1][: kc[1]].tolist() == [2]
    _, kb, ki, kc, st = plan(wl, O.RULE_PRODUCER, min_keep=0)
    assert kc[1] == 0 and st[0] == 1                                     # default drops it and counts it
    # gamma = 0 makes the mean irrelevant; mean == bias cancels
    wl.bn_params[1][1][2] = 0.0
    wl.bn_params[0][2][1] = 0.7                                          # mean of A's channel 1 non-zero
    _, _, _, _, st = plan(wl, O.RULE_PRODUCER, min_keep=0)
    assert st[0] == 1
    wl.bn_params[0][0][1] = 0.0                                          # gamma = 0
    _, _, _, _, st = plan(wl, O.RULE_PRODUCER, min_keep=0)
    assert st[0] == 0


def test_keep_sets_are_nested_across_a_portfolio():
    wl = W.resnet56()
    om = O.OracleModel(wl)
    rec = O.threshold(om, wl.scope, wl.ks)
    prev = None
    for v in range(0, len(wl.ks), 3):
        masked, _ = O.apply_mask(om, wl.scope, rec[v])
        _, out_nz, in_nz = O.zero_structures(masked)
        kb, ki, kc, st = O.propagate_keep(masked, out_nz, in_nz)
        cur = [bits_to_bool(b, g.C) for b, g in zip(kb, wl.groups)]
        if prev is not None and st[2] == 0:
            assert all(np.all(p[c]) for p, c in zip(prev, cur))
        prev = cur
    # the planted stream channels are dead in every producer: the producer rule removes exactly those at low sparsity
    masked, _ = O.apply_mask(om, wl.scope, rec[0])
    _, out_nz, in_nz = O.zero_structures(masked)
    kb, ki, kc, st = O.propagate_keep(masked, out_nz, in_nz, O.RULE_PRODUCER)
    streams = {}
    for ti, t in enumerate(wl.tensors):
        streams.setdefault(t.out_group, []).append(ti)
    for g, tis in streams.items():
        if len(tis) > 1:
            removed = np.flatnonzero(~bits_to_bool(kb[g], wl.groups[g].C))
            assert set(wl.planted[tis[0]].tolist()) <= set(removed.tolist())
