"""Pins for the oracle's threshold step (O1): brute force, a library selection
routine, the Gaussian closed form and order invariants."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2309_06973_b200 import workloads as W


def one_tensor_workload(values, dtype=W.F32, shape=None):
    """A single FC tensor [O][I] holding `values` (float32 array or uint16 bf16 words)."""
    values = np.asarray(values)
    n = values.size
    shape = shape or (1, n)
    wl = W.Workload("t", 0, W.SCOPE_GLOBAL,
                    [W.TensorSpec("w", shape[0], shape[1], 1, 1, 1, 0)], [],
                    [W.GroupSpec(shape[1], W.GROUP_FROZEN), W.GroupSpec(shape[0], W.GROUP_FROZEN)], [], 1)
    wl.biases = [None]
    wl.bn_params = []
    if dtype == W.F32:
        wl.weights = [np.ascontiguousarray(values, np.float32).reshape(shape[0], shape[1], 1, 1)]
        return wl, O.OracleModel(wl, O.F32)
    wl.weights = [np.zeros((shape[0], shape[1], 1, 1), np.float32)]
    return wl, O.OracleModel(wl, O.BF16, [np.ascontiguousarray(values, np.uint16).reshape(shape[0], shape[1], 1, 1)])


def keys_f32(x):
    return np.ascontiguousarray(x, np.float32).view(np.uint32).ravel() & 0x7FFFFFFF


def special_values(rng, n):
    x = rng.standard_normal(n).astype(np.float32)
    x[rng.integers(0, n, n // 5)] = 0.0
    x[rng.integers(0, n, n // 10)] = -0.0
    x[rng.integers(0, n, n // 10)] = np.float32(1e-42)      # denormal
    x[rng.integers(0, n, n // 20)] = np.inf
    x[rng.integers(0, n, n // 20)] = -np.inf
    x[rng.integers(0, n, n // 20)] = np.nan
    dup = rng.integers(0, n, n // 4)
    x[dup] = x[rng.integers(0, n, n // 4)] * np.float32(-1.0)  # duplicates of opposite sign
    return x


@pytest.mark.parametrize("seed", range(6))
def test_threshold_equals_full_sort_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 3000))
    x = special_values(rng, max(n, 20))[:n]
    _, om = one_tensor_workload(x)
    ks = np.unique(np.concatenate([[0, 1, n], rng.integers(0, n + 1, 12)])).astype(np.uint64)
    rec = O.threshold(om, W.SCOPE_GLOBAL, ks[:, None])
    srt = sorted(int(v) for v in keys_f32(x))     # python's sort, integers
    for k, r in zip(ks, rec[:, 0]):
        k = int(k)
        if k == 0:
            assert (r["tau_bits"], r["n_below"], r["n_tie"], r["n_equal"]) == (0, 0, 0, 0)
            continue
        tau = srt[k - 1]
        below = sum(1 for v in srt if v < tau)
        equal = sum(1 for v in srt if v == tau)
        assert int(r["tau_bits"]) == tau
        assert int(r["n_below"]) == below
        assert int(r["n_tie"]) == k - below and 1 <= int(r["n_tie"]) <= equal
        assert int(r["n_equal"]) == equal


def test_threshold_bf16_keys_brute_force():
    rng = np.random.default_rng(7)
    words = rng.integers(0, 1 << 16, 5000).astype(np.uint16)
    words[::7] = 0x8000      # -0
    words[::11] = 0x7F80     # +inf
    _, om = one_tensor_workload(words, W.BF16)
    ks = np.array([1, 17, 2500, 4999, 5000], np.uint64)
    rec = O.threshold(om, W.SCOPE_GLOBAL, ks[:, None])
    srt = sorted(int(w) & 0x7FFF for w in words)
    for k, r in zip(ks, rec[:, 0]):
        tau = srt[int(k) - 1]
        assert int(r["tau_bits"]) == tau
        assert int(r["n_below"]) == sum(1 for v in srt if v < tau)
        assert int(r["n_equal"]) == srt.count(tau)


def test_threshold_value_matches_library_kthvalue():
    """tau, read back as a float, is the k-th smallest |w| according to torch.kthvalue."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal(200_000).astype(np.float32)
    _, om = one_tensor_workload(x)
    ks = np.array([1, 1000, 100_000, 160_000, 199_999, 200_000], np.uint64)
    rec = O.threshold(om, W.SCOPE_GLOBAL, ks[:, None])
    a = torch.from_numpy(np.abs(x))
    for k, r in zip(ks, rec[:, 0]):
        want = torch.kthvalue(a, int(k)).values.item()
        got = np.array([r["tau_bits"]], np.uint32).view(np.float32)[0]
        assert got == np.float32(want)


def test_threshold_gaussian_closed_form():
    """For i.i.d. N(0, s^2) weights the s-quantile of |w| is s * Phi^-1((1+p)/2)."""
    rng = np.random.default_rng(11)
    n, sigma = 2_000_000, 0.037
    x = (sigma * rng.standard_normal(n)).astype(np.float32)
    _, om = one_tensor_workload(x)
    fr = [(4, 5, 1.2816), (9, 10, 1.6449), (19, 20, 1.9600), (49, 50, 2.3263)]
    ks = np.array([W.k_fraction(n, p, q) for p, q, _ in fr], np.uint64)
    rec = O.threshold(om, W.SCOPE_GLOBAL, ks[:, None])
    for (p, q, z), r in zip(fr, rec[:, 0]):
        tau = float(np.array([r["tau_bits"]], np.uint32).view(np.float32)[0])
        assert abs(tau / sigma - z) < 0.01 * z


def test_threshold_order_invariants_and_per_tensor_scope():
    wl = W.small_resnet(seed=5)
    wl.scope = W.SCOPE_PER_TENSOR
    om = O.OracleModel(wl)
    segs = wl.segments()
    sizes = [sum(wl.tensors[i].numel for i in s) for s in segs]
    fracs = [(0, 1), (1, 7), (1, 2), (9, 10), (1, 1)]
    ks = np.array([[W.k_fraction(n, p, q) for n in sizes] for p, q in fracs], np.uint64)
    rec = O.threshold(om, W.SCOPE_PER_TENSOR, ks)
    for s, idx in enumerate(segs):
        keys = np.sort(np.concatenate([keys_f32(wl.weights[i]) for i in idx]))
        taus = rec["tau_bits"][:, s]
        assert np.all(np.diff(taus.astype(np.int64)) >= 0)              # tau non-decreasing in k
        assert int(taus[-1]) == int(keys[-1])                           # k = N gives the maximum key
        for v in range(len(fracs)):
            k = int(ks[v, s])
            r = rec[v, s]
            if k == 0:
                continue
            assert int(r["n_below"]) < k <= int(r["n_below"]) + int(r["n_equal"])
            assert int(r["tau_bits"]) == int(keys[k - 1])               # numpy's sort as a second sorter


def test_threshold_rejects_k_above_segment():
    _, om = one_tensor_workload(np.ones(10, np.float32))
    with pytest.raises(ValueError):
        O.threshold(om, W.SCOPE_GLOBAL, np.array([[11]], np.uint64))


def test_vgg_per_layer_thresholds_follow_the_truncated_gaussian_quantile():
    """With 30 % exact zeros and 95 % pruned per layer, the non-zero N(0, 2/fan_in) weights are
    pruned at rate 0.65/0.70, so tau_l is close to Phi^-1((1 + 0.65/0.70)/2) * sqrt(2/fan_in)."""
    wl = W.vgg16()
    om = O.OracleModel(wl)
    rec = O.threshold(om, wl.scope, wl.ks)
    z = 1.8027
    for s, t in enumerate(wl.tensors[:13]):
        if t.numel < 500_000:
            continue
        frac_zero = len(wl.planted[s]) / t.O
        sigma = np.sqrt(2.0 / (t.I * t.KH * t.KW))
        tau = float(np.array([rec[0, s]["tau_bits"]], np.uint32).view(np.float32)[0])
        # quantile of the non-zero part that is pruned, with the layer's exact planted fraction
        from statistics import NormalDist
        p = (0.95 - frac_zero) / (1 - frac_zero)
        zl = NormalDist().inv_cdf((1 + p) / 2)
        assert abs(zl - z) < 0.03
        assert abs(tau / sigma - zl) < 0.02 * zl
