"""Pins for the oracle's mask step (O2): the worked tie example, exact counts,
bit-exact survivors, nesting and the iterative = one-shot equivalence."""
import os

import numpy as np
import pytest

from oracle import oracle as O
from paper_2309_06973_b200 import workloads as W
from test_oracle_threshold import keys_f32, one_tensor_workload, special_values

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].split()
        if line:
            out.setdefault(line[0], []).append(line[1:])
    return out


def popcount(words):
    return int(np.unpackbits(np.ascontiguousarray(words).view(np.uint8)).sum())


def bits_to_bool(words, n):
    return np.unpackbits(np.ascontiguousarray(words).view(np.uint8), bitorder="little")[:n].astype(bool)


def test_worked_tie_example():
    g = read_golden("tie_example.txt")
    x = np.array([float(v) for v in g["weights"][0]], np.float32)
    k = int(g["k"][0][0])
    _, om = one_tensor_workload(x)
    rec = O.threshold(om, W.SCOPE_GLOBAL, np.array([[k]], np.uint64))
    r = rec[0, 0]
    assert int(r["tau_bits"]) == int(np.array([float(g["tau_value"][0][0])], np.float32).view(np.uint32)[0])
    assert int(r["n_below"]) == int(g["n_below"][0][0])
    assert int(r["n_tie"]) == int(g["n_tie"][0][0])
    assert int(r["n_equal"]) == int(g["n_equal"][0][0])
    masked, bits = O.apply_mask(om, W.SCOPE_GLOBAL, rec[0])
    kept = bits_to_bool(bits[0], x.size)
    assert sorted(np.flatnonzero(~kept).tolist()) == [int(v) for v in g["masked"][0]]
    out = masked.weights[0].ravel()
    assert out.view(np.uint32)[~kept].tolist() == [0, 0, 0]          # masked weights are +0
    assert out.view(np.uint32)[kept].tolist() == x.view(np.uint32)[kept].tolist()


@pytest.mark.parametrize("seed", range(4))
def test_mask_counts_survivors_and_order(seed):
    rng = np.random.default_rng(100 + seed)
    n = 4000
    x = special_values(rng, n)
    _, om = one_tensor_workload(x, shape=(40, 100))
    ks = np.array([0, 1, 900, 2500, 3999, 4000], np.uint64)
    rec = O.threshold(om, W.SCOPE_GLOBAL, ks[:, None])
    keys = keys_f32(x)
    prev_kept = np.ones(n, bool)
    for k, r in zip(ks, rec):
        masked, bits = O.apply_mask(om, W.SCOPE_GLOBAL, r)
        kept = bits_to_bool(bits[0], n)
        assert kept.sum() == n - int(k) == popcount(bits[0])           # exactly k masked
        out = masked.weights[0].ravel().view(np.uint32)
        assert np.all(out[kept] == x.view(np.uint32)[kept])            # survivors bit-identical (NaN payload, -0)
        assert np.all(out[~kept] == 0)
        tau = int(r[0]["tau_bits"])
        assert np.all(keys[~kept] <= tau) and np.all(keys[kept] >= tau)
        # ties: the masked ones are exactly the first n_tie in index order
        ties = np.flatnonzero(keys == tau)
        if k > 0:
            assert np.all(~kept[ties[: int(r[0]["n_tie"])]]) and np.all(kept[ties[int(r[0]["n_tie"]):]])
        assert np.all(prev_kept[kept])                                  # masks nested across increasing k
        prev_kept = kept


def test_mask_python_walk_brute_force():
    """A second, independent walk in pure Python over a multi-tensor, per-tensor-scope model."""
    wl = W.chain([5, 6], seed=3, planted_frac=0.4)
    wl.scope = W.SCOPE_PER_TENSOR
    om = O.OracleModel(wl)
    sizes = [t.numel for t in wl.tensors]
    ks = np.array([[n // 3 for n in sizes], [n - 1 for n in sizes]], np.uint64)
    rec = O.threshold(om, wl.scope, ks)
    for v in range(2):
        masked, bits = O.apply_mask(om, wl.scope, rec[v])
        for ti, w in enumerate(wl.weights):
            keys = [int(a) for a in keys_f32(w)]
            order = sorted(range(len(keys)), key=lambda i: (keys[i], i))   # magnitude, then index
            gone = set(order[: int(ks[v, ti])])
            kept = bits_to_bool(bits[ti], len(keys))
            assert set(np.flatnonzero(~kept).tolist()) == gone


def test_iterative_rounds_equal_one_shot_on_dense():
    """Pruning a fifth of what remains, round after round, on the previous round's sparse model
    gives the same sparse models as one-shot pruning of the dense weights at the cumulative counts."""
    for wl in (W.toy(), W.small_resnet(seed=1)):
        n = wl.n_prunable
        ks = np.array(W.k_iterative(n, list(range(1, 8))), np.uint64)[:, None]
        om = O.OracleModel(wl)
        rec = O.threshold(om, W.SCOPE_GLOBAL, ks)
        cur = om
        for v in range(len(ks)):
            one_shot, _ = O.apply_mask(om, W.SCOPE_GLOBAL, rec[v])
            rec_it = O.threshold(cur, W.SCOPE_GLOBAL, ks[v:v + 1])
            cur, _ = O.apply_mask(cur, W.SCOPE_GLOBAL, rec_it[0])
            for a, b in zip(one_shot.weights, cur.weights):
                assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
            nnz = sum(int(np.count_nonzero(keys_f32(w))) for w in cur.weights)
            assert nnz <= n - int(ks[v, 0])


def test_non_prunable_tensors_are_copied_and_fully_kept():
    wl = W.chain([4, 4], seed=9)
    wl.tensors[0].prunable = False
    om = O.OracleModel(wl)
    n = wl.n_prunable
    rec = O.threshold(om, W.SCOPE_GLOBAL, np.array([[n]], np.uint64))
    masked, bits = O.apply_mask(om, W.SCOPE_GLOBAL, rec[0])
    assert np.array_equal(masked.weights[0], wl.weights[0])
    assert popcount(bits[0]) == wl.tensors[0].numel
    assert all(not np.any(w) for w in masked.weights[1:])


def test_bf16_mask_counts_with_heavy_ties():
    wl = W.small_resnet(seed=2)
    om = O.OracleModel(wl, O.BF16)
    n = wl.n_prunable
    ks = np.array(W.k_iterative(n, [1, 4, 9]), np.uint64)[:, None]
    rec = O.threshold(om, W.SCOPE_GLOBAL, ks)
    assert int(rec["n_equal"].max()) > 1                                # bf16 magnitudes collide
    for v in range(3):
        _, bits = O.apply_mask(om, W.SCOPE_GLOBAL, rec[v])
        assert sum(popcount(b) for b in bits) == n - int(ks[v, 0])
