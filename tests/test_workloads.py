"""The synthetic workloads have the shapes of the paper's models: parameter counts, tensor and group counts.

Table II of the paper lists 14.72 M parameters for VGG-16 (CIFAR shapes, one linear layer) and 25.56 M for
ResNet-50; the other counts follow from the stated architectures.  A refactor of the generators must not move them."""
import numpy as np
import pytest

from paper_2309_06973_b200 import workloads as W


@pytest.mark.parametrize("name, prunable, params, tensors, prunable_groups", [
    ("toy", 33_328, 33_626, 5, 4),
    ("vgg16", 14_715_584, 14_724_042, 14, 13),
    ("resnet56", 851_504, 855_770, 58, 30),
    ("resnet50", 25_502_912, 25_557_032, 54, 37),
    ("resnet152", 60_040_384, 60_192_808, 156, 105),
])
def test_parameter_counts(name, prunable, params, tensors, prunable_groups):
    wl = W.BY_NAME[name]()
    assert wl.n_prunable == prunable and wl.n_params == params
    assert len(wl.tensors) == tensors
    assert sum(1 for g in wl.groups if not (g.flags & W.GROUP_FROZEN)) == prunable_groups
    assert abs(params / 1e6 - {"vgg16": 14.72, "resnet50": 25.56}.get(name, params / 1e6)) < 0.005   # Table II


def test_prune_counts_are_integers_of_the_stated_rules():
    n = W.resnet152().n_prunable
    ks = W.resnet152().ks[:, 0].tolist()
    rem, want = n, []
    for r in range(1, 11):
        rem -= (rem + 4) // 5                    # a fifth of what remains, rounded up
        if r >= 3:
            want.append(n - rem)
    assert ks == want
    assert W.resnet50().ks[:, 0].tolist() == [n50 * p // q for n50 in [W.resnet50().n_prunable] for p, q in ((4, 5), (9, 10), (49, 50))]


def test_freeze_streams_marks_exactly_the_groups_several_layers_write():
    wl = W.freeze_streams(W.resnet50())
    writers = np.zeros(len(wl.groups), int)
    for t in wl.tensors:
        writers[t.out_group] += 1
    for g, n in zip(wl.groups, writers):
        if n > 1:
            assert g.flags & W.GROUP_FROZEN
    # stem output (maxpool feeds layer1's projection and first block only reads it) stays prunable; 4 streams are frozen
    assert sum(1 for g in wl.groups if not (g.flags & W.GROUP_FROZEN)) == 37 - 4
    chain = W.freeze_streams(W.vgg16())
    assert sum(1 for g in chain.groups if not (g.flags & W.GROUP_FROZEN)) == 13      # a chain has no such group
