"""GPU parity of the fixed-point keep propagation against the oracle: keep sets, index lists, counts,
statistics (including the number of passes) and the variant rebuilt from them, bit for bit."""
import numpy as np
import pytest

from gpu_compare import assert_words, bits_eq
from oracle import oracle as O
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W
from paper_2309_06973_b200.runtime import DeviceModel, Session

pytestmark = pytest.mark.gpu


def run_case(wl, dtype, v, policy, min_keep, max_passes):
    om = O.OracleModel(wl, dtype)
    rec = O.threshold(om, wl.scope, wl.ks)
    masked, _ = O.apply_mask(om, wl.scope, rec[v])
    nz, _, _ = O.zero_structures(masked)
    kb_c, ki_c, kc_c, st_c = O.propagate_keep_cascade(masked, nz, policy, min_keep, max_passes)
    cw_c, cbn_c, cb_c, sh_c = O.compact(masked, ki_c, kc_c)

    dm = DeviceModel(wl, dtype)
    ses = Session(dm, wl.scope, len(wl.ks))
    ses.magnitude_threshold(wl.ks)
    ses.mask_and_structures(v)
    ses.propagate_keep_cascade(policy, min_keep, max_passes)
    ses.compact()
    assert ses.device_status() == B.DNNS_OK
    kb_g, ki_g, kc_g, st_g = ses.keep_sets()
    assert np.array_equal(kc_g, kc_c)
    assert_words(kb_g, kb_c, "keep bits")
    for g, (a, b) in enumerate(zip(ki_g, ki_c)):
        assert np.array_equal(a, b[: kc_c[g]]), g
    assert st_g.tolist() == st_c.tolist()
    cw_g, cbn_g, cb_g, sh_g, _ = ses.compacted()
    assert np.array_equal(sh_g, sh_c)
    for a, b in zip(cw_g, cw_c):
        assert bits_eq(a, b)
    return st_c, kc_c


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
@pytest.mark.parametrize("make", [W.toy, lambda: W.small_resnet(seed=3), lambda: W.small_resnet(seed=4, bottleneck=False),
                                  W.resnet56, lambda: W.chain([37, 70, 129, 33], seed=5, kernel=5, planted_frac=0.2)])
def test_cascade_to_convergence(make, dtype):
    wl = make()
    for v in sorted({0, len(wl.ks) - 1}):
        run_case(wl, dtype, v, O.RULE_PRODUCER | O.RULE_CONSUMER, 1, 16)


@pytest.mark.parametrize("policy", [O.RULE_PRODUCER, O.RULE_CONSUMER, O.RULE_PRODUCER | O.RULE_CONSUMER | O.SHIFT_STRICT])
@pytest.mark.parametrize("max_passes", [1, 2, 3])
def test_cascade_cut_short_and_policies(policy, max_passes):
    wl = W.resnet56()
    for (g, be, mu, va) in wl.bn_params:
        be[::2] = 0.0
        mu[::2] = 0.0
    run_case(wl, B.DNNS_F32, 9, policy, 0, max_passes)


def test_hand_chain_takes_two_passes():
    from test_oracle_cascade import hand_chain
    st, kc = run_case(hand_chain(), B.DNNS_F32, 0, O.RULE_PRODUCER, 1, 8)
    assert int(st[3]) == 2 and kc.tolist() == [2, 2, 2, 2]


def test_fc_with_spatial_columns_cascade():
    b = W._Builder()
    gi = b.group(3, frozen=True)
    g1 = b.group(64)
    gc = b.group(7, frozen=True)
    b.conv_bn("c", "x", "a", gi, g1, 3, 1, 1)
    b.fc("fc", "a", "out", g1, gc, in_spatial=2)          # 128 columns: whole words, but two columns per channel
    wl = W.Workload("fcS", 11, W.SCOPE_GLOBAL, b.tensors, b.bns, b.groups, b.ops, 3)
    W._draw(wl, True, 0.5, 0.3)
    W._set_ks(wl, lambda n: [n * 9 // 10])
    run_case(wl, B.DNNS_F32, 0, O.RULE_PRODUCER | O.RULE_CONSUMER, 1, 8)


def test_resnet50_cascade_full_size():
    wl = W.resnet50()
    st, kc = run_case(wl, B.DNNS_F32, 2, O.RULE_PRODUCER | O.RULE_CONSUMER, 1, 8)
    assert int(st[3]) >= 1
