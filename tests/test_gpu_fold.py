"""GPU parity of the conv + BatchNorm fusion on rebuilt variants, against the fp64 oracle.
Tolerance: the kernel works in fp32 (one division, one square root, one multiply per value), so a
result may differ from the fp64 value by a few fp32 units in the last place; bf16 weights add the
final rounding to 8 significant bits."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W
from paper_2309_06973_b200.runtime import DeviceModel, Session
from model_utils import compacted_workload

pytestmark = pytest.mark.gpu  # (compacted_workload below is also used by CPU tests)

F32_RTOL = 4 * 2.0 ** -24      # division, square root and product, each within half an ulp
BF16_RTOL = 2.0 ** -8 + F32_RTOL


def close(got, want, rtol):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    return np.all(np.abs(got - want) <= rtol * np.abs(want) + 1e-300)


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
@pytest.mark.parametrize("make", [W.toy, lambda: W.small_resnet(seed=3), W.resnet56,
                                  lambda: W.chain([37, 70, 129, 33], seed=5, kernel=5, planted_frac=0.2)])
def test_fold_matches_fp64_oracle(make, dtype):
    wl = make()
    if wl.name == "toy":                       # one conv with a bias in front of its BN
        wl.tensors[1].has_bias = True
        wl.biases[1] = np.linspace(-1, 1, wl.tensors[1].O).astype(np.float32)
    dm = DeviceModel(wl, dtype)
    ses = Session(dm, wl.scope, len(wl.ks))
    ses.magnitude_threshold(wl.ks)
    v = len(wl.ks) - 1
    ses.variant(v, fused=True)
    cw, cbn, cb, shapes, _ = ses.compacted()          # the rebuilt variant before folding (parity-checked elsewhere)
    _, _, kc, _ = ses.keep_sets()
    ses.fold_batchnorm()
    assert ses.device_status() == B.DNNS_OK
    fw, fbn, fb, shapes2, _ = ses.compacted()
    assert np.array_equal(shapes, shapes2)

    small = compacted_workload(wl, kc, [w if dtype == B.DNNS_F32 else W.bf16_bits_to_f32(w) for w in cw], cbn, cb)
    om = O.OracleModel(small, dtype, weights=cw)
    ow, oscale, obias = O.fold_batchnorm(om)
    has_bn = {b.tensor: i for i, b in enumerate(wl.bns)}
    for ti in range(len(wl.tensors)):
        if ti in has_bn:
            got = fw[ti] if dtype == B.DNNS_F32 else W.bf16_bits_to_f32(fw[ti])
            assert close(got, ow[ti], F32_RTOL if dtype == B.DNNS_F32 else BF16_RTOL), f"weights {ti}"
        else:
            assert np.array_equal(fw[ti].view(np.uint8), cw[ti].view(np.uint8))       # no BN: untouched
    for bi in range(len(wl.bns)):
        assert close(fbn[bi][0], oscale[bi], F32_RTOL), f"scale {bi}"
        # the folded bias is a sum: absolute error is bounded by the larger of its two terms
        bound = F32_RTOL * (np.abs(cbn[bi][1]) + np.abs(obias[bi] - cbn[bi][1])) * 2 + 1e-30
        assert np.all(np.abs(fbn[bi][1].astype(np.float64) - obias[bi]) <= bound), f"folded bias {bi}"
        assert np.array_equal(fbn[bi][2], cbn[bi][2]) and np.array_equal(fbn[bi][3], cbn[bi][3])   # mean, var kept
