"""Shared driver of the GPU parity tests: run the CUDA path and the oracle on the same seeded
workload and compare every output bit for bit."""
import numpy as np

from oracle import oracle as O
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200.runtime import DeviceModel, Session


def assert_words(a, b, what):
    assert len(a) == len(b), what
    for i, (x, y) in enumerate(zip(a, b)):
        assert np.array_equal(np.asarray(x).view(np.uint32), np.asarray(y).view(np.uint32)), f"{what}[{i}]"


def bits_eq(a, b):
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    return a.shape == b.shape and np.array_equal(a.view(np.uint8), b.view(np.uint8))


def expected_offsets(sizes_bytes):
    """Destination offsets rule: items in order, each at the next multiple of 256 bytes."""
    out, o = [], 0
    for s in sizes_bytes:
        out.append(o)
        o = (o + s + 255) // 256 * 256
    return out


def compare_portfolio(wl, dtype=B.DNNS_F32, variants=None, policy=O.RULE_PRODUCER | O.RULE_CONSUMER, min_keep=1,
                      weights=None, check_structure_maps=True, fused=False, multi=0, multi_plan=False, no_store=False):
    """Thresholds for all of wl.ks in one call, then steps 2-5 for the chosen variants.
    multi = G > 0: steps 2 and 3 of G consecutive variants at a time through the multi-variant sweep;
    multi_plan: step 4 of those variants in one launch as well (dnns_propagate_keep_multi);
    no_store: the sweep writes no masked weights and the rebuild masks the dense model on its way
    (dnns_compact_masked) - everything but the masked weights themselves is still compared."""
    om = O.OracleModel(wl, dtype, weights)
    dm = DeviceModel(wl, dtype, weights=weights)
    ses = Session(dm, wl.scope, len(wl.ks), slots=max(multi, 1))
    ses.magnitude_threshold(wl.ks)
    rec_gpu = ses.records()
    rec_cpu = O.threshold(om, wl.scope, wl.ks)
    for f in ("tau_bits", "n_below", "n_tie", "n_equal"):
        assert np.array_equal(rec_gpu[f], rec_cpu[f]), f
    eb = 4 if dtype == B.DNNS_F32 else 2
    todo = list(range(len(wl.ks)) if variants is None else variants)
    for pos, v in enumerate(todo):
        slot = 0
        if multi:
            slot = pos % multi
            if slot == 0:
                n = min(multi, len(todo) - pos)
                assert todo[pos: pos + n] == list(range(v, v + n)), "the multi-variant sweep takes consecutive variants"
                ses.mask_and_structures_multi(v, n, store_masked=not no_store)
                if multi_plan:
                    ses.propagate_keep_multi(n, policy, min_keep)
            if no_store:
                if not multi_plan:
                    ses.propagate_keep(policy, min_keep, slot=slot)
                ses.compact_masked(v, slot=slot, own_keep=multi_plan)
            elif multi_plan:
                ses.compact(slot=slot, own_keep=True)
            else:
                ses.propagate_keep(policy, min_keep, slot=slot)
                ses.compact(slot=slot)
        else:
            ses.variant(v, policy, min_keep, fused=fused)
        assert ses.device_status() == B.DNNS_OK
        masked_cpu, bits_cpu = O.apply_mask(om, wl.scope, rec_cpu[v])
        if not no_store:
            for i, (a, b) in enumerate(zip(ses.masked_tensors(slot=slot), masked_cpu.weights)):
                assert bits_eq(a, b), f"masked weights, variant {v}, tensor {i}"
        assert_words(ses.mask_words(slot), bits_cpu, f"mask bits v{v}")
        nz_c, out_c, in_c = O.zero_structures(masked_cpu)
        nz_g, out_g, in_g = ses.structure_words(slot)
        if check_structure_maps:
            assert_words(nz_g, nz_c, f"kernel map v{v}")
        assert_words(out_g, out_c, f"out flags v{v}")
        assert_words(in_g, in_c, f"in flags v{v}")
        kb_c, ki_c, kc_c, st_c = O.propagate_keep(masked_cpu, out_c, in_c, policy, min_keep)
        kb_g, ki_g, kc_g, st_g = ses.keep_sets(slot if multi_plan else 0, multi_stats=multi_plan)
        assert np.array_equal(kc_g, kc_c), f"keep counts v{v}"
        assert_words(kb_g, kb_c, f"keep bits v{v}")
        for g, (a, b) in enumerate(zip(ki_g, ki_c)):
            assert np.array_equal(a, b[: kc_c[g]]), f"keep idx v{v} group {g}"
        assert st_g.tolist() == st_c.tolist(), f"stats v{v}"
        cw_c, cbn_c, cb_c, sh_c = O.compact(masked_cpu, ki_c, kc_c)
        cw_g, cbn_g, cb_g, sh_g, offs = ses.compacted(slot if multi_plan else 0)
        assert np.array_equal(sh_g, sh_c), f"shapes v{v}"
        for i, (a, b) in enumerate(zip(cw_g, cw_c)):
            assert bits_eq(a, b), f"compacted weights v{v} tensor {i}"
        for i, (a, b) in enumerate(zip(cbn_g, cbn_c)):
            for x, y in zip(a, b):
                assert bits_eq(x, y), f"compacted bn v{v} {i}"
        for a, b in zip(cb_g, cb_c):
            assert (a is None and b is None) or bits_eq(a, b)
        sizes = [w.size * eb for w in cw_c] + [4 * len(x) for p in cbn_c for x in p] + \
                [4 * len(b) for b in cb_c if b is not None]
        assert offs.tolist() == expected_offsets(sizes), f"arena offsets v{v}"
    return ses


def compare_sparse_free(wl, dtype=B.DNNS_F32, policy=O.RULE_PRODUCER | O.RULE_CONSUMER, min_keep=1, weights=None,
                        one_launch=False):
    """The portfolio without any sparse model: thresholds once, the zero structures of every variant from one sweep
    over the dense weights (dnns_zero_structures_portfolio), keep sets of all variants in one launch, then a masking
    rebuild per variant (dnns_compact_masked; one_launch: of all variants of a call at once, each into an arena of
    its own, dnns_compact_masked_multi).  Flags, keep sets, statistics and every rebuilt item are compared
    with the oracle's step-by-step result (mask, zero structures, keep propagation, compaction)."""
    om = O.OracleModel(wl, dtype, weights)
    dm = DeviceModel(wl, dtype, weights=weights)
    V = len(wl.ks)
    per_call = min(V, B.DNNS_PORTFOLIO_MAX)
    ses = Session(dm, wl.scope, V, want_mask_bits=False, want_nz_map=False, portfolio_slots=per_call,
                  portfolio_arenas=one_launch)
    ses.magnitude_threshold(wl.ks)
    rec_gpu, rec_cpu = ses.records(), O.threshold(om, wl.scope, wl.ks)
    for f in ("tau_bits", "n_below", "n_tie", "n_equal"):
        assert np.array_equal(rec_gpu[f], rec_cpu[f]), f
    eb = 4 if dtype == B.DNNS_F32 else 2
    for v0 in range(0, V, per_call):
        n = min(per_call, V - v0)
        ses.zero_structures_portfolio(v0, n)
        ses.propagate_keep_portfolio(n, policy, min_keep)
        if one_launch:
            ses.compact_portfolio_multi(v0, n)
        for s in range(n):
            v = v0 + s
            if not one_launch:
                ses.compact_portfolio(v, s)
            assert ses.device_status() == B.DNNS_OK
            masked_cpu, _ = O.apply_mask(om, wl.scope, rec_cpu[v])
            _, out_c, in_c = O.zero_structures(masked_cpu)
            _, out_g, in_g = ses.structure_words(s, portfolio=True)
            assert_words(out_g, out_c, f"out flags v{v}")
            assert_words(in_g, in_c, f"in flags v{v}")
            kb_c, ki_c, kc_c, st_c = O.propagate_keep(masked_cpu, out_c, in_c, policy, min_keep)
            kb_g, ki_g, kc_g, st_g = ses.keep_sets(s, multi_stats=True, portfolio=True)
            assert np.array_equal(kc_g, kc_c), f"keep counts v{v}"
            assert_words(kb_g, kb_c, f"keep bits v{v}")
            for g, (a, b) in enumerate(zip(ki_g, ki_c)):
                assert np.array_equal(a, b[: kc_c[g]]), f"keep idx v{v} group {g}"
            assert st_g.tolist() == st_c.tolist(), f"stats v{v}"
            cw_c, cbn_c, cb_c, sh_c = O.compact(masked_cpu, ki_c, kc_c)
            cw_g, cbn_g, cb_g, sh_g, offs = ses.compacted(s, portfolio=True, own_arena=one_launch)
            assert np.array_equal(sh_g, sh_c), f"shapes v{v}"
            for i, (a, b) in enumerate(zip(cw_g, cw_c)):
                assert bits_eq(a, b), f"compacted weights v{v} tensor {i}"
            for i, (a, b) in enumerate(zip(cbn_g, cbn_c)):
                for x, y in zip(a, b):
                    assert bits_eq(x, y), f"compacted bn v{v} {i}"
            for a, b in zip(cb_g, cb_c):
                assert (a is None and b is None) or bits_eq(a, b)
            sizes = [w.size * eb for w in cw_c] + [4 * len(x) for p in cbn_c for x in p] + \
                    [4 * len(b) for b in cb_c if b is not None]
            assert offs.tolist() == expected_offsets(sizes), f"arena offsets v{v}"
            ses.last_masked, ses.last_slot = masked_cpu.weights, s   # the oracle's sparse model of the variant rebuilt last
    return ses
