"""Where a variant stops masking the weights equal to tau (32-bit weights): found in the list that the second ranking
sweep keeps of the keys it counts, or - when the list cannot say - by the sweep that counts those weights tile by tile.
Either way the records, the masks and the rebuilt variants are the oracle's; these cases pin down WHICH way ran."""
import numpy as np
import pytest

from gpu_compare import compare_portfolio, compare_sparse_free
from oracle import oracle as O
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W
from paper_2309_06973_b200.runtime import DeviceModel, Session

pytestmark = pytest.mark.gpu


def with_duplicates(copies):
    """A small ResNet whose k-th weights have `copies` equal twins: every variant splits its ties."""
    wl = W.small_resnet(seed=21)
    flat = np.concatenate([w.reshape(-1) for w in wl.weights])
    order = np.argsort(np.abs(flat), kind="stable")
    ks = [int(k[0]) for k in wl.ks]
    rng = np.random.default_rng(3)
    for k in ks:
        val = np.abs(flat[order[k - 1]])
        for j in rng.choice(np.arange(k + 50, min(len(flat), k + 5000)), copies, replace=False):
            flat[order[j]] = val if j % 2 else -val
    at = 0
    for w in wl.weights:
        w[...] = flat[at:at + w.size].reshape(w.shape)
        at += w.size
    # the k-th smallest magnitudes moved: take prune counts that land inside the groups of equal weights
    key = np.sort(np.abs(flat).view(np.uint32))
    new_ks = []
    for k in ks:
        tau = key[k - 1]
        lo, hi = int(np.searchsorted(key, tau, "left")), int(np.searchsorted(key, tau, "right"))
        new_ks.append([lo + max(1, (hi - lo) // 2)])
    wl.ks = np.array(new_ks, np.uint64)
    return wl


def test_few_equal_weights_are_found_in_the_list():
    wl = with_duplicates(5)
    ses = compare_sparse_free(wl, B.DNNS_F32)
    rec = ses.records()
    assert (rec["n_tie"] < rec["n_equal"]).any()          # the ties really split
    assert not ses.tie_sweep_ran()                        # ... and no sweep counted them tile by tile
    # the sweeps that mask tile by tile get their tables on demand, and mask the same weights
    ses2 = compare_portfolio(with_duplicates(5), B.DNNS_F32, fused=True)
    assert ses2.tie_sweep_ran()


def test_many_equal_weights_fall_back_to_the_tie_sweep():
    wl = with_duplicates(1500)                            # more than a short list holds
    ses = compare_sparse_free(wl, B.DNNS_F32)
    rec = ses.records()
    assert (rec["n_equal"] > 1024).any() and (rec["n_tie"] < rec["n_equal"]).any()
    assert ses.tie_sweep_ran()


def test_tau_zero_falls_back_to_the_tie_sweep():
    wl = W.small_resnet(seed=22)
    for w in wl.weights:
        w.reshape(-1)[::3] = 0.0
    nz = sum(int(np.count_nonzero(w == 0)) for w in wl.weights)
    wl.ks = np.array([[nz // 2], [nz - 1]], np.uint64)    # stop masking inside the zeros
    ses = compare_sparse_free(wl, B.DNNS_F32)
    assert ses.tie_sweep_ran()


def test_sixteen_bit_weights_always_take_the_tie_sweep():
    ses = compare_sparse_free(with_duplicates(5), B.DNNS_BF16)
    rec = ses.records()
    assert ses.tie_sweep_ran() == bool((rec["n_tie"] < rec["n_equal"]).any())


def test_no_split_no_sweep():
    wl = W.chain([16, 24, 16], seed=23, planted_frac=0.0)
    n = wl.n_prunable
    wl.ks = np.array([[n]], np.uint64)                    # everything masked: no weight equal to tau stays
    ses = compare_sparse_free(wl, B.DNNS_F32)
    assert not ses.tie_sweep_ran()
