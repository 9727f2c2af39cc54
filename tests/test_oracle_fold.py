"""Pins for the oracle's conv + BatchNorm fusion (O7): the fused layer computes what conv followed
by BN computes (torch's batch_norm as the independent definition), the identity BN, a hand example."""
import numpy as np
import torch
import torch.nn.functional as F

from oracle import oracle as O
from paper_2309_06973_b200 import workloads as W


def test_fused_layer_equals_conv_then_batchnorm():
    wl = W.toy()
    wl.tensors[1].has_bias = True
    wl.biases[1] = np.linspace(-1, 1, wl.tensors[1].O).astype(np.float32)     # one conv with a bias
    om = O.OracleModel(wl)
    fw, scale, fbias = O.fold_batchnorm(om)
    rng = np.random.default_rng(0)
    for bi, b in enumerate(wl.bns):
        t = wl.tensors[b.tensor]
        x = torch.from_numpy(rng.standard_normal((2, t.I, 6, 6)))
        w = torch.from_numpy(wl.weights[b.tensor]).double()
        bias = None if wl.biases[b.tensor] is None else torch.from_numpy(wl.biases[b.tensor]).double()
        g, be, mu, va = [torch.from_numpy(v).double() for v in wl.bn_params[bi]]
        want = F.batch_norm(F.conv2d(x, w, bias, 1, 1), mu, va, g, be, False, 0.0, b.eps)
        got = F.conv2d(x, torch.from_numpy(fw[b.tensor]), torch.from_numpy(fbias[bi]), 1, 1)
        assert float((want - got).abs().max()) <= 1e-12 * float(want.abs().max())
    assert fw[-1] is None                                  # the linear layer has no BN: nothing to fold


def test_identity_batchnorm_and_hand_example():
    wl = W.chain([3], seed=1, kernel=1, planted_frac=0.0)
    eps = wl.bns[0].eps
    wl.bn_params[0] = (np.ones(3, np.float32), np.zeros(3, np.float32), np.zeros(3, np.float32),
                       np.full(3, 1.0, np.float32))
    wl.bns[0].eps = 0.0
    fw, scale, fbias = O.fold_batchnorm(O.OracleModel(wl))
    assert np.array_equal(fw[0], wl.weights[0].astype(np.float64)) and not fbias[0].any() and np.all(scale[0] == 1)
    # gamma 2, var 3 + eps 1 -> scale 1; gamma 3, var 8 + eps 1 -> scale 1; beta 0.5, mean 0.25 -> bias 0.5 - 0.25 * s
    wl.bns[0].eps = 1.0
    wl.bn_params[0] = (np.array([2, 3, 0], np.float32), np.array([0.5, 0.5, 0.5], np.float32),
                       np.array([0.25, -1, 7], np.float32), np.array([3, 8, 0], np.float32))
    fw, scale, fbias = O.fold_batchnorm(O.OracleModel(wl))
    assert scale[0].tolist() == [1.0, 1.0, 0.0]
    assert fbias[0].tolist() == [0.25, 1.5, 0.5]
    assert np.array_equal(fw[0][0], wl.weights[0][0].astype(np.float64)) and not fw[0][2].any()
    wl.bns[0].eps = eps


def test_bf16_weights_are_widened_exactly():
    wl = W.chain([4], seed=2, kernel=3, planted_frac=0.0)
    om = O.OracleModel(wl, O.BF16)
    fw, scale, _ = O.fold_batchnorm(om)
    wide = W.bf16_bits_to_f32(om.weights[0]).astype(np.float64)
    assert np.array_equal(fw[0], wide * scale[0][:, None, None, None])
