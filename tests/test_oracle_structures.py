"""Pins for the oracle's zero-structure flags (O3): hand-built tensors, planted zero
filters of the workloads and the row/column OR relations."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2309_06973_b200 import workloads as W
from test_oracle_mask import bits_to_bool


def single_conv(w):
    O_, I_, KH, KW = w.shape
    wl = W.Workload("c", 0, W.SCOPE_GLOBAL, [W.TensorSpec("w", O_, I_, KH, KW, 1, 0)], [],
                    [W.GroupSpec(I_, 1), W.GroupSpec(O_, 1)], [], 1)
    wl.weights, wl.biases, wl.bn_params = [np.ascontiguousarray(w, np.float32)], [None], []
    return wl, O.OracleModel(wl)


def test_hand_built_kernel_map():
    w = np.zeros((3, 4, 3, 3), np.float32)
    w[0, 1, 2, 2] = 5.0          # last element of kernel (0,1)
    w[0, 3, 0, 0] = -0.0         # a negative zero is a zero
    w[2, 0, 1, 1] = 1e-42        # a denormal is not
    w[2, 2, 0, 2] = np.nan       # neither is a NaN
    wl, om = single_conv(w)
    nz, out_nz, in_nz = O.zero_structures(om)
    m = bits_to_bool(nz[0], 12).reshape(3, 4)
    want = np.zeros((3, 4), bool)
    want[0, 1] = want[2, 0] = want[2, 2] = True
    assert np.array_equal(m, want)
    assert bits_to_bool(out_nz[0], 3).tolist() == [True, False, True]   # filter 1 is all zero
    assert bits_to_bool(in_nz[0], 4).tolist() == [True, True, True, False]  # nobody reads column 3


def test_single_nonzero_in_last_element_of_filter():
    w = np.zeros((2, 5, 3, 3), np.float32)
    w[1, 4, 2, 2] = 1.0
    _, om = single_conv(w)
    nz, out_nz, in_nz = O.zero_structures(om)
    assert bits_to_bool(out_nz[0], 2).tolist() == [False, True]
    assert bits_to_bool(in_nz[0], 5).tolist() == [False] * 4 + [True]
    assert np.flatnonzero(bits_to_bool(nz[0], 10)).tolist() == [9]


@pytest.mark.parametrize("name", ["toy", "resnet56"])
def test_planted_zero_filters_are_flagged_and_flags_are_row_col_ors(name):
    wl = W.BY_NAME[name]()
    om = O.OracleModel(wl)
    nz, out_nz, in_nz = O.zero_structures(om)
    for ti, t in enumerate(wl.tensors):
        m = bits_to_bool(nz[ti], t.O * t.I).reshape(t.O, t.I)
        # numpy's own reductions on float values as an independent evaluation
        assert np.array_equal(m, (wl.weights[ti] != 0).any(axis=(2, 3)))
        o = bits_to_bool(out_nz[ti], t.O)
        i = bits_to_bool(in_nz[ti], t.I)
        assert np.array_equal(o, m.any(axis=1)) and np.array_equal(i, m.any(axis=0))
        assert np.array_equal(np.flatnonzero(~o), wl.planted[ti])        # dense Gaussian: only planted filters are zero


def test_planted_filters_stay_flagged_after_masking():
    wl = W.toy()
    om = O.OracleModel(wl)
    rec = O.threshold(om, wl.scope, wl.ks)
    masked, _ = O.apply_mask(om, wl.scope, rec[0])
    _, out_nz, _ = O.zero_structures(masked)
    for ti, t in enumerate(wl.tensors):
        dead = np.flatnonzero(~bits_to_bool(out_nz[ti], t.O))
        assert set(wl.planted[ti].tolist()) <= set(dead.tolist())
        assert len(dead) >= int(0.25 * t.O) or t.has_bias
