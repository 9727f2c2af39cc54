"""GPU parity of the portfolio path that never forms a sparse model: zero structures of all variants from one
sweep over the dense weights (largest key per filter and input column against every variant's threshold), keep
sets of all variants in one launch, masking rebuild per variant.  Every output is compared with the oracle's
step-by-step result: mask, zero structures, keep propagation, compaction."""
import numpy as np
import pytest

from gpu_compare import compare_sparse_free
from oracle import oracle as O
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
@pytest.mark.parametrize("make", [W.toy, lambda: W.small_resnet(seed=3), lambda: W.small_resnet(seed=4, bottleneck=False),
                                  W.resnet56])
def test_small_configs_every_variant(make, dtype):
    compare_sparse_free(make(), dtype)
    compare_sparse_free(make(), dtype, one_launch=True)     # all variants rebuilt by one launch


@pytest.mark.parametrize("policy", [O.RULE_PRODUCER, O.RULE_CONSUMER, O.RULE_PRODUCER | O.RULE_CONSUMER | O.SHIFT_STRICT])
@pytest.mark.parametrize("min_keep", [0, 1, 5])
def test_policies_and_min_keep(policy, min_keep):
    wl = W.small_resnet(seed=8)
    for (g, be, mu, va) in wl.bn_params:
        be[::2] = 0.0
        mu[::2] = 0.0
    wl.ks = np.array([[W.k_fraction(wl.n_prunable, 97, 100)], [wl.n_prunable]], np.uint64)
    compare_sparse_free(wl, B.DNNS_F32, policy=policy, min_keep=min_keep)


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
def test_per_tensor_scope_and_odd_shapes(dtype):
    # widths that are not multiples of 32, 5x5 kernels, rows that are not multiples of 16 bytes, ragged tiles
    wl = W.chain([37, 70, 129, 33], seed=5, kernel=5, planted_frac=0.2)
    wl.scope = W.SCOPE_PER_TENSOR
    sizes = [t.numel for t in wl.tensors]
    wl.ks = np.array([[0] * len(sizes), [n // 2 for n in sizes], [n * 9 // 10 for n in sizes],
                      [n - 1 for n in sizes], sizes], np.uint64)
    compare_sparse_free(wl, dtype)
    compare_sparse_free(wl, dtype, one_launch=True)


def test_non_prunable_tensor_and_1x1_chain():
    wl = W.chain([64, 96, 64, 256], seed=6, kernel=1, planted_frac=0.3)
    wl.tensors[1].prunable = False
    n = wl.n_prunable
    wl.ks = np.array([[n // 3], [n * 19 // 20]], np.uint64)
    compare_sparse_free(wl, B.DNNS_F32)
    compare_sparse_free(wl, B.DNNS_BF16)


def test_special_values_and_heavy_ties():
    """Zeros, negative zeros, denormals, infinities, NaNs and big blocks of equal magnitudes: many filters and input
    columns whose largest key equals the threshold, in the tensor where the equal weights split and around it."""
    wl = W.chain([48, 64, 80], seed=7, planted_frac=0.5)
    rng = np.random.default_rng(0)
    for w in wl.weights:
        flat = w.reshape(-1)
        n = flat.size
        flat[rng.integers(0, n, n // 8)] = -0.0
        flat[rng.integers(0, n, n // 16)] = np.float32(1e-42)
        flat[rng.integers(0, n, n // 32)] = np.inf
        flat[rng.integers(0, n, n // 32)] = np.nan
        flat[rng.integers(0, n, n // 4)] = np.float32(0.125)
        flat[rng.integers(0, n, n // 8)] = np.float32(-0.125)
    n = wl.n_prunable
    nz0 = sum(int(np.count_nonzero(w.view(np.uint32) & 0x7FFFFFFF == 0)) for w in wl.weights)
    ks = [1, nz0 // 2, nz0, nz0 + 5, n // 2, n * 3 // 4, n - 3, n]
    wl.ks = np.array(ks, np.uint64)[:, None]
    ses = compare_sparse_free(wl, B.DNNS_F32)
    rec = ses.records()
    assert (rec["n_tie"] < rec["n_equal"]).any()                   # the equal weights really split
    compare_sparse_free(wl, B.DNNS_BF16)
    compare_sparse_free(wl, B.DNNS_BF16, one_launch=True)


def test_filters_whose_largest_weight_equals_the_threshold():
    """Whole filters and whole input columns made of one magnitude that is also the threshold: whether such a
    filter survives depends on where, in index order, the variant stops masking the equal weights."""
    wl = W.chain([32, 40, 48], seed=9, planted_frac=0.0)
    for w in wl.weights:
        w[...] = np.where(np.abs(w) < 0.05, np.float32(0.03125), w).astype(np.float32)   # a third of all weights equal
        w[::3] = np.float32(-0.03125)                                                     # whole filters of that value
        w[:, ::4] = np.float32(0.03125)                                                   # whole input columns
    n = wl.n_prunable
    eq = sum(int(np.count_nonzero(np.abs(w) == np.float32(0.03125))) for w in wl.weights)
    ks = [eq // 7, eq // 3, eq // 2, eq - 1, eq, eq + 1]
    wl.ks = np.array(ks, np.uint64)[:, None]
    compare_sparse_free(wl, B.DNNS_F32)
    compare_sparse_free(wl, B.DNNS_BF16)


def test_more_variants_than_one_call_takes():
    wl = W.small_resnet(seed=13)
    n = wl.n_prunable
    wl.ks = np.array([[n * (i + 1) // 21] for i in range(20)], np.uint64)
    compare_sparse_free(wl, B.DNNS_F32)
    compare_sparse_free(wl, B.DNNS_F32, one_launch=True)


def test_fc_with_spatial_columns():
    b = W._Builder()
    gi = b.group(3, frozen=True)
    g1 = b.group(40)
    gc = b.group(7, frozen=True)
    b.conv_bn("c", "x", "a", gi, g1, 3, 1, 1)
    b.fc("fc", "a", "out", g1, gc, in_spatial=9)
    wl = W.Workload("fcS", 11, W.SCOPE_GLOBAL, b.tensors, b.bns, b.groups, b.ops, 3)
    W._draw(wl, True, 0.5, 0.3)
    wl.biases[1][:] = np.arange(7)
    W._set_ks(wl, lambda n: [n // 2, n * 9 // 10])
    compare_sparse_free(wl, B.DNNS_F32)


@pytest.mark.parametrize("make", [W.resnet56, lambda: W.small_resnet(seed=3)])
def test_frozen_residual_streams(make):
    """The paper's own setting (Section IV-B-2): skip connections and downsampling layers are left alone - every
    group that several layers write is frozen, only plain layer-to-layer channels are pruned."""
    from gpu_compare import compare_portfolio
    wl = W.freeze_streams(make())
    ses = compare_sparse_free(wl, B.DNNS_F32)
    _, _, kc, _ = ses.keep_sets(ses.last_slot, portfolio=True)
    for g, c in zip(wl.groups, kc):
        if g.flags & W.GROUP_FROZEN:
            assert c == g.C
    compare_sparse_free(W.freeze_streams(make()), B.DNNS_BF16, one_launch=True)
    compare_portfolio(W.freeze_streams(make()), B.DNNS_F32, multi=2, multi_plan=True)


def test_variants_outside_the_latest_threshold_call_are_rejected():
    from paper_2309_06973_b200.runtime import DeviceModel, Session
    wl = W.toy()
    dm = DeviceModel(wl, B.DNNS_F32)
    ses = Session(dm, wl.scope, 4, portfolio_slots=4)
    n = wl.n_prunable
    ses.magnitude_threshold(np.array([[n // 2], [n // 3]], np.uint64))      # two of at most four variants
    L = B.lib()
    thr, s = ses.thr.data_ptr(), 0
    assert L.dnns_apply_mask(ses.plan, thr, 2, ses.masked.data_ptr(), None, s) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_mask_and_structures(ses.plan, thr, 3, ses.masked.data_ptr(), None, None, ses.out_nz.data_ptr(),
                                      ses.in_nz.data_ptr(), s) == B.DNNS_ERR_INVALID_ARG
    with pytest.raises(B.DnnsError):
        ses.zero_structures_portfolio(1, 2)
    with pytest.raises(B.DnnsError):
        ses.compact_portfolio(2, 0)
    ses.zero_structures_portfolio(0, 2)                                      # inside the call: fine
    ses.propagate_keep_portfolio(2)
    ses.compact_portfolio(1, 1)
    assert ses.device_status() == B.DNNS_OK
