"""GPU parity: the CUDA path against the CPU oracle, element by element, on seeded workloads that
span several tiles, ragged tails, odd shapes, both dtypes, both scopes and every policy."""
import numpy as np
import pytest
import torch

from gpu_compare import compare_portfolio
from oracle import oracle as O
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
@pytest.mark.parametrize("make", [W.toy, lambda: W.small_resnet(seed=3), lambda: W.small_resnet(seed=4, bottleneck=False),
                                  W.resnet56])
def test_small_configs_every_variant(make, dtype, fused):
    compare_portfolio(make(), dtype, fused=fused)


@pytest.mark.parametrize("multi", [1, 2, 3, 4])
@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
@pytest.mark.parametrize("make", [W.toy, lambda: W.small_resnet(seed=3), W.resnet56])
def test_multi_variant_sweep_every_variant(make, dtype, multi):
    """Groups of up to four variants masked and analysed in one sweep: each variant as from its own sweep."""
    compare_portfolio(make(), dtype, multi=multi)
    compare_portfolio(make(), dtype, multi=multi, multi_plan=True)     # ... and planned in one launch
    compare_portfolio(make(), dtype, multi=multi, multi_plan=True, no_store=True)   # ... rebuilt from the dense model


@pytest.mark.parametrize("policy", [O.RULE_PRODUCER, O.RULE_CONSUMER, O.RULE_PRODUCER | O.RULE_CONSUMER | O.SHIFT_STRICT])
@pytest.mark.parametrize("min_keep", [0, 1, 5])
def test_policies_and_min_keep(policy, min_keep):
    wl = W.small_resnet(seed=8)
    for (g, be, mu, va) in wl.bn_params:
        be[::2] = 0.0
        mu[::2] = 0.0
    wl.ks = np.array([[W.k_fraction(wl.n_prunable, 97, 100)], [wl.n_prunable]], np.uint64)
    compare_portfolio(wl, B.DNNS_F32, policy=policy, min_keep=min_keep)
    compare_portfolio(wl, B.DNNS_F32, policy=policy, min_keep=min_keep, multi=2, multi_plan=True)


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
def test_per_tensor_scope_and_odd_shapes(dtype):
    # widths that are not multiples of 32, 5x5 kernels, ragged tiles
    wl = W.chain([37, 70, 129, 33], seed=5, kernel=5, planted_frac=0.2)
    wl.scope = W.SCOPE_PER_TENSOR
    sizes = [t.numel for t in wl.tensors]
    wl.ks = np.array([[0] * len(sizes), [n // 2 for n in sizes], [n * 9 // 10 for n in sizes],
                      [n - 1 for n in sizes], sizes], np.uint64)
    compare_portfolio(wl, dtype)
    compare_portfolio(wl, dtype, variants=[1, 3], fused=True)
    compare_portfolio(wl, dtype, multi=2)
    compare_portfolio(wl, dtype, multi=3, no_store=True)


def test_non_prunable_tensor_and_1x1_chain():
    wl = W.chain([64, 96, 64, 256], seed=6, kernel=1, planted_frac=0.3)
    wl.tensors[1].prunable = False
    n = wl.n_prunable
    wl.ks = np.array([[n // 3], [n * 19 // 20]], np.uint64)
    compare_portfolio(wl, B.DNNS_F32)
    compare_portfolio(wl, B.DNNS_BF16)


def test_special_values_and_heavy_ties():
    """Zeros, negative zeros, denormals, infinities, NaNs and many duplicates: ties split inside tiles."""
    wl = W.chain([48, 64, 80], seed=7, planted_frac=0.5)
    rng = np.random.default_rng(0)
    for w in wl.weights:
        flat = w.reshape(-1)
        n = flat.size
        flat[rng.integers(0, n, n // 8)] = -0.0
        flat[rng.integers(0, n, n // 16)] = np.float32(1e-42)
        flat[rng.integers(0, n, n // 32)] = np.inf
        flat[rng.integers(0, n, n // 32)] = np.nan
        flat[rng.integers(0, n, n // 4)] = np.float32(0.125)      # a big block of equal magnitudes
        flat[rng.integers(0, n, n // 8)] = np.float32(-0.125)
    n = wl.n_prunable
    nz0 = sum(int(np.count_nonzero(w.view(np.uint32) & 0x7FFFFFFF == 0)) for w in wl.weights)
    ks = [1, nz0 // 2, nz0, nz0 + 5, n // 2, n * 3 // 4, n - 3, n]
    wl.ks = np.array(ks, np.uint64)[:, None]
    ses = compare_portfolio(wl, B.DNNS_F32)
    rec = ses.records()
    assert (rec["n_tie"] < rec["n_equal"]).any()                   # the split-tie path really ran
    compare_portfolio(wl, B.DNNS_BF16)
    compare_portfolio(wl, B.DNNS_F32, fused=True)
    compare_portfolio(wl, B.DNNS_F32, multi=4)     # tiles that rank the ties of several variants at once
    compare_portfolio(wl, B.DNNS_BF16, multi=3)
    compare_portfolio(wl, B.DNNS_F32, multi=4, no_store=True)      # ties decided by the mask bits during the rebuild
    compare_portfolio(wl, B.DNNS_BF16, multi=2, multi_plan=True, no_store=True)


def test_deep_chain_with_more_than_1024_gather_items():
    """260 convs + BN = 1300 gather items: the layout is then computed by its own kernel."""
    wl = W.chain([8] * 260, seed=21, kernel=1, planted_frac=0.25)
    n = wl.n_prunable
    wl.ks = np.array([[n // 2]], np.uint64)
    compare_portfolio(wl, B.DNNS_F32, fused=True)


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
    compare_portfolio(wl, B.DNNS_F32)


def test_sparse_model_straight_from_the_model_tensors():
    """Phase 2 alone: structures and rebuild read the model's own (already sparse) tensors."""
    from paper_2309_06973_b200.runtime import DeviceModel, Session
    from gpu_compare import bits_eq
    wl = W.small_resnet(seed=12)
    om = O.OracleModel(wl)
    rec = O.threshold(om, wl.scope, wl.ks)
    sparse, _ = O.apply_mask(om, wl.scope, rec[-1])
    dm = DeviceModel(wl, B.DNNS_F32, weights=sparse.weights)
    ses = Session(dm, wl.scope, 1)
    ses.zero_structures(from_model=True)
    ses.propagate_keep()
    ses.compact(from_model=True)
    _, out_c, in_c = O.zero_structures(sparse)
    kb, ki, kc, st = O.propagate_keep(sparse, out_c, in_c)
    cw, *_ = O.compact(sparse, ki, kc)
    for a, b in zip(ses.compacted()[0], cw):
        assert bits_eq(a, b)


def test_in_place_mask_and_small_destination_arena():
    from paper_2309_06973_b200.runtime import DeviceModel, Session
    from gpu_compare import bits_eq
    wl = W.toy()
    om = O.OracleModel(wl)
    dm = DeviceModel(wl)
    ses = Session(dm, wl.scope, 1)
    ses.magnitude_threshold(wl.ks)
    ses.apply_mask(0, in_place=True)
    rec = O.threshold(om, wl.scope, wl.ks)
    masked, _ = O.apply_mask(om, wl.scope, rec[0])
    for a, b in zip(ses.masked_tensors(in_place=True), masked.weights):
        assert bits_eq(a, b)
    ses.zero_structures(from_model=True)
    ses.propagate_keep()
    ses.compact(from_model=True, dst_bytes=256)
    assert ses.device_status() == B.DNNS_ERR_WORKSPACE            # reported, nothing copied
    assert ses.device_status() == B.DNNS_OK                       # and cleared
    with pytest.raises(B.DnnsError):
        ses.magnitude_threshold(np.array([[wl.n_prunable + 1]], np.uint64))


def test_two_runs_are_bit_identical():
    wl = W.resnet56()
    from paper_2309_06973_b200.runtime import DeviceModel, Session
    outs = []
    for _ in range(2):
        dm = DeviceModel(wl, B.DNNS_BF16)
        ses = Session(dm, wl.scope, len(wl.ks))
        ses.magnitude_threshold(wl.ks)
        ses.variant(7)
        torch.cuda.synchronize()
        # padding between arena items is never written: compare the tensors, not the raw arenas
        outs.append(ses.masked_tensors() + ses.compacted()[0] + [ses.keep_idx.cpu().numpy(), ses.records()])
    for a, b in zip(*outs):
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8))


def test_multi_variant_calls_reject_bad_arguments():
    """Host-side checks of the multi-variant entry points: too many variants, shared output buffers."""
    from paper_2309_06973_b200.runtime import DeviceModel, Session
    wl = W.resnet56()
    ses = Session(DeviceModel(wl, B.DNNS_F32), wl.scope, len(wl.ks), slots=2)
    ses.magnitude_threshold(wl.ks)
    p = lambda name, g: ses._slot(name, g).data_ptr()
    def sweep(first, n, arenas, outs, ins):
        B.dnns_mask_and_structures_multi(ses.plan, ses.thr.data_ptr(), first, n, arenas, None, None, outs, ins)
    good = ([p("masked", 0), p("masked", 1)], [p("out_nz", 0), p("out_nz", 1)], [p("in_nz", 0), p("in_nz", 1)])
    sweep(0, 2, *good)                                                    # fine
    for bad in [(0, 2, [p("masked", 0)] * 2, good[1], good[2]),           # one arena for two variants
                (0, 2, good[0], [p("out_nz", 0)] * 2, good[2]),           # shared flags
                (len(wl.ks) - 1, 2, *good),                               # runs past the last variant
                (0, 5, good[0] * 3, good[1] * 3, good[2] * 3)]:           # more than DNNS_MULTI_MAX
        with pytest.raises(B.DnnsError) as e:
            sweep(*bad)
        assert e.value.status == B.DNNS_ERR_INVALID_ARG
    kb, ki, kc = ([p(n, 0), p(n, 1)] for n in ("keep_bits", "keep_idx", "keep_count"))
    B.dnns_propagate_keep_multi(ses.plan, 2, good[1], good[2], 3, 1, kb, ki, kc, ses.stats_multi.data_ptr())
    with pytest.raises(B.DnnsError) as e:
        B.dnns_propagate_keep_multi(ses.plan, 2, good[1], good[2], 3, 1, kb, [p("keep_idx", 0)] * 2, kc, 0)
    assert e.value.status == B.DNNS_ERR_INVALID_ARG
    with pytest.raises(B.DnnsError) as e:
        B.dnns_propagate_keep_multi(ses.plan, 2, good[1], good[2], 64, 1, kb, ki, kc, 0)    # unknown policy bit
    assert e.value.status == B.DNNS_ERR_INVALID_ARG
    assert ses.device_status() == B.DNNS_OK
    ses.close()


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
def test_rebuild_from_the_dense_model_equals_rebuild_from_the_masked_one(dtype):
    """dnns_compact_masked after dnns_apply_mask gives the destination arena of dnns_compact, byte for byte."""
    from paper_2309_06973_b200.runtime import DeviceModel, Session
    wl = W.small_resnet(seed=11)
    ses = Session(DeviceModel(wl, dtype), wl.scope, len(wl.ks))
    ses.magnitude_threshold(wl.ks)
    for v in range(len(wl.ks)):
        ses.apply_mask(v)
        ses.zero_structures()
        ses.propagate_keep()
        ses.compact_arena.fill_(0x5A)              # the gaps between items keep the fill in both runs
        ses.compact()
        torch.cuda.synchronize()
        want, offs, shapes = ses.compact_arena.clone(), ses.dst_offsets.clone(), ses.dst_shapes.clone()
        ses.compact_arena.fill_(0x5A)
        ses.compact_masked(v)
        torch.cuda.synchronize()
        assert torch.equal(ses.dst_offsets, offs) and torch.equal(ses.dst_shapes, shapes)
        assert torch.equal(ses.compact_arena, want)
    assert ses.device_status() == B.DNNS_OK
    ses.close()


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
def test_two_runs_give_identical_bytes(dtype):
    """Determinism: the same portfolio generated twice (fresh plans, atomics and all) - every mask bit, keep list
    and rebuilt byte is the same, although histograms, tie counts and flags are accumulated with atomics."""
    from paper_2309_06973_b200.runtime import DeviceModel, Session
    wl = W.resnet56()
    V = len(wl.ks)

    def run():
        ses = Session(DeviceModel(wl, dtype), wl.scope, V, slots=2)
        ses.compact_arena.fill_(0)
        ses.magnitude_threshold(wl.ks)
        out = [ses.thr.clone()]
        for v0 in range(0, V, 2):
            ses.mask_and_structures_multi(v0, 2)
            ses.propagate_keep_multi(2)
            for g in range(2):
                ses.compact(slot=g, own_keep=True)
                torch.cuda.synchronize()
                used = int(ses.dst_offsets[-1].item()) + 4
                out += [ses._slot("mask_bits", g).clone(), ses._slot("out_nz", g).clone(), ses._slot("in_nz", g).clone(),
                        ses._slot("keep_bits", g).clone(), ses._slot("keep_count", g).clone(), ses.dst_offsets.clone(),
                        ses.dst_shapes.clone(), ses.compact_arena[:used].clone()]
        assert ses.device_status() == B.DNNS_OK
        ses.close()
        return out

    first, second = run(), run()
    assert len(first) == len(second) and all(torch.equal(a, b) for a, b in zip(first, second))
