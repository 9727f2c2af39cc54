#!/usr/bin/env python
"""Benchmark of the portfolio-generation hot path: threshold once, then mask, zero-structure
detection, keep propagation and compaction for every variant.

One "step" is one whole portfolio on one model.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet152] [--dtype f32|bf16] [--path sparse_free]
  python bench.py --impl reference ...     # the CPU oracle, as it stands, on the host cores

The default path stores no sparse model: thresholds of all variants from one ranking, the zero structures of all
variants from one sweep over the dense weights, keep sets of all variants in one launch, then one masking rebuild
per variant.  --path multi / fused / stepwise time the paths that write the sparse model of every variant.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "ms per pruned variant (portfolio generation: threshold, mask, zero structures, keep propagation, compaction)"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def measured_traffic(workload: str, dtype: str, kernel: str):
    """DRAM bytes per launch of `kernel` from the committed ncu summary, or None when there is none."""
    try:
        table = json.load(open(os.path.join(ROOT, "profiles", "dram_traffic.json")))
        return table[f"{workload}_{dtype}"][kernel]
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return None
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            p = [x.strip() for x in line.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0]))
                mx.append(float(p[1]))
            except ValueError:
                continue
            for n, v in zip(names, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------
# reference arm / CPU baseline: the oracle, unchanged, on the host
# --------------------------------------------------------------------------------------------

def oracle_portfolio(wl, dtype, variants):
    """One pass of the whole path in the oracle for the given variant indices. Returns seconds."""
    from oracle import oracle as O
    om = O.OracleModel(wl, dtype)
    t0 = time.perf_counter()
    rec = O.threshold(om, wl.scope, wl.ks[variants])
    for i in range(len(variants)):
        masked, _ = O.apply_mask(om, wl.scope, rec[i])
        _, out_nz, in_nz = O.zero_structures(masked)
        _, ki, kc, _ = O.propagate_keep(masked, out_nz, in_nz)
        O.compact(masked, ki, kc)
    return time.perf_counter() - t0


def dtype_label(dtype):
    return "u32 keys / fp32 words" if dtype == 0 else "u16 keys / bf16 words"


def config_of(wl, dtype):
    return {"workload": f"{wl.name} ({'fp32' if dtype == 0 else 'bf16'}), {wl.n_prunable} prunable weights, "
                        f"{len(wl.ks)} variants, {'global' if wl.scope == 0 else 'per-tensor'} ranking, seed {wl.seed}",
            "variants": len(wl.ks), "prunable_weights": wl.n_prunable,
            "l2": f"L2 flushed before every timed step ({FLUSH_BYTES >> 20} MiB scratch write, outside the timed region)"}


def run_reference(args, wl, dtype):
    """The whole workload (every variant) per step, as the cpu_baseline leg of the main arm times it."""
    V = len(wl.ks)
    variants = list(range(V))
    for _ in range(args.warmup):
        oracle_portfolio(wl, dtype, variants)
    times = [oracle_portfolio(wl, dtype, variants) for _ in range(args.steps)]
    ms = [1e3 * t / V for t in times]
    sample = f"the whole workload per step: all {V} variants, full weights"
    line = {
        "impl": "reference", "metric": METRIC, "value": statistics.median(ms), "unit": "ms", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * statistics.median(times),
        "ms_per_variant_min": min(ms), "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": dtype_label(dtype), "data": "synthetic", "config": config_of(wl, dtype),
        "cpu_baseline": {"value": statistics.median(ms), "unit": "ms", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": statistics.median(ms), "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


FLUSH_BYTES = 512 << 20
KERNELS = ["k_hist1", "k_select1", "k_hist2", "k_select2", "k_tie_find", "k_tie_pick", "k_ties", "k_tie_scan", "k_extrema_rows", "k_extrema_sweep", "k_extrema_flags",
           "k_sweep<", "k_sweep_multi", "k_flags", "k_shift_zero", "k_propagate", "k_rebuild_layout", "k_compact_gather"]


def item_sizes(wl, keep_count, eb):
    """Bytes of every rebuilt item (weights, BatchNorm vectors, biases) for one array of keep counts, R and N'."""
    R = Nn = 0
    sizes = []
    for t in wl.tensors:
        On, Cn = int(keep_count[t.out_group]), int(keep_count[t.in_group])
        R += On * t.I * t.KH * t.KW
        Nn += On * Cn * t.in_spatial * t.KH * t.KW
        sizes.append(On * Cn * t.in_spatial * t.KH * t.KW * eb)
    for b in wl.bns:
        sizes += [4 * int(keep_count[wl.tensors[b.tensor].out_group])] * 4
    for t in wl.tensors:
        if t.has_bias:
            sizes.append(4 * int(keep_count[t.out_group]))
    used = 0
    for s in sizes:                      # items in order, each at the next multiple of 256 bytes
        used = (used + 255) // 256 * 256 + s
    return R, Nn, (used + 255) // 256 * 256


class Config:
    """One (workload, dtype) on the GPU: buffers, the step of the chosen path, timing."""

    def __init__(self, args, name, dtype, device, pinned_host=False, freeze=False):
        import torch
        from paper_2309_06973_b200 import workloads as W
        from paper_2309_06973_b200.runtime import DeviceModel, Session
        self.torch, self.args, self.dtype = torch, args, dtype
        wl = W.BY_NAME[name]()
        if freeze:
            W.freeze_streams(wl)
        self.wl, self.V, self.eb, self.N = wl, len(wl.ks), 4 if dtype == 0 else 2, wl.n_prunable
        V = self.V
        self.path = args.path
        self.dm = DeviceModel(wl, dtype, device=device, pinned_host=pinned_host)
        G = args.multi if args.multi >= 0 else (4 if dtype == 0 else 2)
        self.G = min(G, 4, V) if self.path == "multi" else 0
        self.groups = [(v0, min(self.G, V - v0)) for v0 in range(0, V, self.G)] if self.G else []
        sparse_free = self.path == "sparse_free"
        self.ses = Session(self.dm, wl.scope, V, want_mask_bits=not sparse_free, want_nz_map=False,
                           slots=max(self.G, 1), portfolio_slots=V if sparse_free else 0,
                           portfolio_arenas=sparse_free and not args.rebuild_per_variant)
        self.flush_buf = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=self.dm.device)
        self.call_names = {"sparse_free": ["threshold", "structures(portfolio)", "propagate", "compact"],
                           "multi": ["threshold", "mask+structures", "propagate", "compact"],
                           "fused": ["threshold", "mask+structures", "propagate", "compact"],
                           "stepwise": ["threshold", "mask", "structures", "propagate", "compact"]}[self.path]
        self.spans = {n: [] for n in self.call_names}

    def step(self, record=False):
        torch, ses, wl, V = self.torch, self.ses, self.wl, self.V

        def timed(name, fn, *a):
            if not record:
                return fn(*a)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(*a)
            e1.record()
            self.spans[name].append((e0, e1))
        timed("threshold", ses.magnitude_threshold, wl.ks)
        if self.path == "sparse_free":
            for v0 in range(0, V, 16):                        # the portfolio-wide calls take up to 16 variants
                n = min(16, V - v0)
                timed("structures(portfolio)", ses.zero_structures_portfolio, v0, n)
                timed("propagate", ses.propagate_keep_portfolio, n)
                if self.args.rebuild_per_variant:
                    for s in range(n):
                        timed("compact", ses.compact_portfolio, v0 + s, s)
                else:                                         # the n rebuilds in one launch, each into its own arena
                    timed("compact", ses.compact_portfolio_multi, v0, n)
            return
        for v0, n in self.groups:                             # n variants per read of the dense weights
            timed("mask+structures", ses.mask_and_structures_multi, v0, n)
            timed("propagate", ses.propagate_keep_multi, n)
            for g in range(n):
                timed("compact", lambda: ses.compact(slot=g, own_keep=True))
        for v in (range(V) if not self.G else ()):
            if self.path == "stepwise":
                timed("mask", ses.apply_mask, v)
                timed("structures", ses.zero_structures)
            else:
                timed("mask+structures", ses.mask_and_structures, v)
            timed("propagate", ses.propagate_keep)
            timed("compact", ses.compact)

    def timed_steps(self, run, steps):
        """`steps` runs, the L2 flushed before each, one event pair per run. Returns the list of ms."""
        torch = self.torch
        pairs = []
        for _ in range(steps):
            self.flush_buf.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            run()
            b.record()
            pairs.append((a, b))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in pairs]

    def variant_sizes(self):
        """Per variant: R (weights in kept filter rows), N' (rebuilt weights), used arena bytes, keep counts, stats."""
        ses, wl, V = self.ses, self.wl, self.V
        out = []
        if self.path == "sparse_free":
            assert V <= 16
            ses.magnitude_threshold(wl.ks)
            ses.zero_structures_portfolio(0, V)
            ses.propagate_keep_portfolio(V)
            self.torch.cuda.synchronize()
            st = ses.stats_multi.cpu().numpy().view(np.uint64)
            for v in range(V):
                kc = ses.pf[v]["keep_count"].cpu().numpy()
                out.append((kc, st[4 * v: 4 * v + 4].copy()))
        else:
            ses.magnitude_threshold(wl.ks)
            for v in range(V):
                ses.variant(v, fused=self.path != "stepwise")
                self.torch.cuda.synchronize()
                out.append((ses.keep_count.cpu().numpy().copy(), ses.stats.cpu().numpy().view(np.uint64).copy()))
        res = []
        for kc, st in out:
            R, Nn, used = item_sizes(wl, kc, self.eb)
            res.append({"R": R, "Nn": Nn, "used": used, "keep_count": kc, "stats": st})
        return res


def measure(cfg, steps, warmup, barrier, max_over_ranks, ms_per_variant_of, peak, peak_kind, workload_key):
    """Device-resident timing of one configuration: whole-portfolio steps (CUDA graph replay), per-call and
    per-kernel durations (plain launches), bytes moved, roofline of the dominant kernel."""
    import torch
    from paper_2309_06973_b200 import binding as B
    ses, wl, V, N, eb, args = cfg.ses, cfg.wl, cfg.V, cfg.N, cfg.eb, cfg.args
    for _ in range(max(warmup, 3)):
        cfg.step()
    torch.cuda.synchronize()
    assert ses.device_status() == B.DNNS_OK
    sizes = cfg.variant_sizes()
    rec = ses.records()
    ties_swept = ses.tie_sweep_ran()     # the tie sweep reads the weights only when some variant splits its ties and the lists of the second sweep cannot say where

    graph, launches_per_step = None, None
    if not args.no_graph:
        try:
            l0 = ses.launch_count()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                cfg.step()
            launches_per_step = ses.launch_count() - l0
            graph.replay()
            torch.cuda.synchronize()
        except Exception as e:  # capture refused: fall back to plain launches and say so
            print(f"bench: CUDA graph capture failed ({e}); timing plain launches", file=sys.stderr)
            graph = None

    barrier()
    launches0 = ses.launch_count()
    plain = cfg.timed_steps(lambda: cfg.step(True), steps)
    launches_plain = ses.launch_count() - launches0
    ses.profile(True)                                 # the same steps with an event pair around every single kernel
    cfg.timed_steps(cfg.step, steps)
    ses.profile(False)
    kernel_ms = {}
    for kn in KERNELS:
        ms, n = ses.kernel_time(kn)
        if n:
            kernel_ms[kn] = {"avg_ms": ms / n, "launches_per_step": n / steps, "ms_per_step": ms / steps}
    if graph is not None:
        barrier()
        timed = cfg.timed_steps(graph.replay, steps)
        launches = launches_per_step * steps
    else:
        timed, launches = plain, launches_plain
    barrier()
    med, mn, mean, plain_med = max_over_ranks([statistics.median(timed), min(timed), statistics.mean(timed),
                                               statistics.median(plain)])
    assert ses.device_status() == B.DNNS_OK

    # ---- bytes: what the kernels of this path really read and write, and the step-by-step accounting
    thr_sweeps = (2 if cfg.dtype == 0 else 1) + (1 if ties_swept else 0)
    rebuild = [(s["R"] + s["Nn"]) * eb for s in sizes]
    if cfg.path == "sparse_free":
        moved = (thr_sweeps + 1) * N * eb + sum(rebuild)
        sweeps = (f"no sparse model: {thr_sweeps} ranking sweeps and one sweep for the zero structures of all {V} variants, "
                  + ("then one masking rebuild per variant" if args.rebuild_per_variant else "then the masking rebuilds of all variants in one launch"))
    elif cfg.path == "multi":
        moved = thr_sweeps * N * eb + sum(N * eb + n * (N * eb + N / 4) for _, n in cfg.groups) + sum(rebuild)
        sweeps = f"fused mask+structures, {cfg.G} variants per read of the dense weights; {thr_sweeps} ranking sweeps"
    elif cfg.path == "fused":
        moved = thr_sweeps * N * eb + V * (2 * N * eb + N / 4) + sum(rebuild)
        sweeps = f"fused mask+structures, one variant per sweep; {thr_sweeps} ranking sweeps"
    else:
        moved = thr_sweeps * N * eb + V * (3 * N * eb + N / 4) + sum(rebuild)
        sweeps = f"stepwise: mask sweep and structure sweep per variant; {thr_sweeps} ranking sweeps"
    stepwise_bytes = N * eb * (1 + 3 * V) + V * N / 8 + sum(rebuild)   # one read per input, one write per output of every step

    # the sweep for the largest keys walks tensors with long rows of whole 16-byte vectors row by row, the rest tile by tile
    by_rows = sum(t.numel for t in wl.tensors if (t.I * t.KH * t.KW * eb) % 16 == 0 and t.I * t.KH * t.KW * eb // 16 >= 96)
    all_weights = sum(t.numel for t in wl.tensors)
    kernel_alg = {"k_hist1": N * eb, "k_hist2": N * eb, "k_ties": N * eb if ties_swept else 0,
                  "k_extrema_rows": by_rows * eb, "k_extrema_sweep": (all_weights - by_rows) * eb,
                  "k_compact_gather": statistics.mean(rebuild) if (cfg.path != "sparse_free" or args.rebuild_per_variant)
                  else sum(rebuild) / ((V + 15) // 16),      # one launch rebuilds up to 16 variants
                  "k_sweep<": (3 * N * eb + N / 4) / 2 if cfg.path == "stepwise" else 2 * N * eb + N / 4}
    if cfg.groups:
        kernel_alg["k_sweep_multi"] = sum(N * eb + n * (N * eb + N / 4) for _, n in cfg.groups) / len(cfg.groups)
    total_k = sum(k["ms_per_step"] for k in kernel_ms.values())
    for kn, k in kernel_ms.items():
        k["share"] = k["ms_per_step"] / total_k
        if kernel_alg.get(kn):
            k["gbs"] = kernel_alg[kn] / (k["avg_ms"] * 1e-3) / 1e9
            k["frac_of_peak"] = k["gbs"] / peak
    dominant = max((kn for kn in kernel_ms if kernel_alg.get(kn)), key=lambda kn: kernel_ms[kn]["ms_per_step"])
    label = {"k_sweep<": "k_sweep", "k_sweep_multi": f"k_sweep_multi<{cfg.G}>"}.get(dominant, dominant)
    traffic = measured_traffic(workload_key, "f32" if cfg.dtype == 0 else "bf16", label)
    roof = {"bound": "hbm", "kernel": label, "achieved": kernel_ms[dominant]["gbs"], "peak": peak,
            "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": kernel_ms[dominant]["gbs"] / peak,
            "algorithmic_bytes": kernel_alg[dominant], "avg_launch_ms": kernel_ms[dominant]["avg_ms"],
            "timed_by": f"CUDA event pair around every launch of the kernel on its stream, {steps} steps of plain launches, "
                        "L2 flushed before every step",
            "traffic": traffic,
            "frac_measured": (traffic / (kernel_ms[dominant]["avg_ms"] * 1e-3) / 1e9 / peak) if traffic else None}
    per_call = {n: statistics.mean(a.elapsed_time(b) for a, b in cfg.spans[n]) for n in cfg.call_names if cfg.spans[n]}
    variants = []
    total_params = wl.n_params
    for v, s in enumerate(sizes):
        kept_params = s["Nn"] + sum(2 * int(s["keep_count"][wl.tensors[b.tensor].out_group]) for b in wl.bns) + \
            sum(int(s["keep_count"][t.out_group]) for t in wl.tensors if t.has_bias)
        variants.append({"k": [int(x) for x in wl.ks[v]], "tau_bits": [int(x) for x in rec["tau_bits"][v]],
                         "n_tie": [int(x) for x in rec["n_tie"][v]], "rebuilt_weights": s["Nn"], "kept_filter_row_weights": s["R"],
                         "channels_removed": int(s["stats"][1]), "dropped_nonzero_shift": int(s["stats"][0]),
                         "spatial_compression": total_params / max(kept_params, 1)})
    return {
        "ms_per_variant": ms_per_variant_of(med, V), "ms_per_variant_min": ms_per_variant_of(mn, V),
        "ms_per_step": med, "ms_per_step_min": mn, "ms_per_step_mean": mean, "ms_per_step_plain": plain_med,
        "steps": steps, "launch": "cuda graph replay" if graph is not None else "plain stream launches",
        "gpu_launches": launches, "sweeps": sweeps,
        "moved_bytes_per_step": moved, "moved_gbs": moved / (med * 1e-3) / 1e9, "moved_frac_of_peak": moved / (med * 1e-3) / 1e9 / peak,
        "stepwise_equivalent_gbs": stepwise_bytes / (med * 1e-3) / 1e9,
        "stepwise_equivalent_frac_of_peak": stepwise_bytes / (med * 1e-3) / 1e9 / peak,
        "stepwise_equivalent_note": "bytes a step-by-step run would move (one read per input and one write per output of "
                                    "every step) over the time of this path: not achieved bandwidth, can exceed the roofline",
        "per_call_ms": per_call, "kernel_ms": kernel_ms, "roofline": roof, "variants": variants, "_sizes": sizes,
    }


def end_to_end(cfg, steps, barrier, max_over_ranks, ms_per_variant_of):
    """The same portfolio through host buffers: every step copies the dense weights host -> device and every rebuilt
    variant (arena, offsets, shapes, keep counts) device -> host.  With the default path the rebuild of variant v+1
    runs while variant v travels back: two destination arenas, a copy stream, one host synchronisation per
    portfolio (for the keep counts, from which the host knows how many bytes every variant has)."""
    import torch
    ses, wl, V, dm = cfg.ses, cfg.wl, cfg.V, cfg.dm
    n_arena = ses.compact_arena.numel()
    host_out = [torch.empty(n_arena, dtype=torch.uint8).pin_memory() for _ in range(2)]
    host_small = [torch.empty(ses.dst_offsets.numel() * 8 + ses.dst_shapes.numel() * 4, dtype=torch.uint8).pin_memory()
                  for _ in range(V)]
    arenas = [ses.compact_arena, torch.empty_like(ses.compact_arena)]
    copy_stream = torch.cuda.Stream(device=dm.device)
    counters = {"h2d": 0, "d2h": 0}

    def step_overlapped():
        dm.upload_weights()
        counters["h2d"] += dm.weight_bytes
        ses.magnitude_threshold(wl.ks)
        ses.zero_structures_portfolio(0, V)
        ses.propagate_keep_portfolio(V)
        kcs = [ses.pf[v]["keep_count"].cpu().numpy() for v in range(V)]      # synchronises once: sizes are data
        counters["d2h"] += sum(k.nbytes for k in kcs)
        main = torch.cuda.current_stream()
        free = [None, None]
        for v in range(V):
            b = v & 1
            used = min(item_sizes(wl, kcs[v], cfg.eb)[2], n_arena)
            if free[b] is not None:
                main.wait_event(free[b])                  # the arena's previous variant has left the device
            ses.compact_portfolio(v, v, arenas[b])
            no, ns = ses.dst_offsets.numel() * 8, ses.dst_shapes.numel() * 4
            host_small[v][:no].copy_(ses.dst_offsets.view(torch.uint8), non_blocking=True)
            host_small[v][no:no + ns].copy_(ses.dst_shapes.view(torch.uint8), non_blocking=True)
            done = torch.cuda.Event()
            done.record(main)
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(done)
                host_out[b][:used].copy_(arenas[b][:used], non_blocking=True)
                free[b] = torch.cuda.Event()
                free[b].record(copy_stream)
            counters["d2h"] += used + no + ns
        copy_stream.synchronize()
        torch.cuda.synchronize()

    def step_sequential():
        dm.upload_weights()
        counters["h2d"] += dm.weight_bytes
        ses.magnitude_threshold(wl.ks)
        for v in range(V):
            if cfg.G:
                if v % cfg.G == 0:
                    ses.mask_and_structures_multi(v, min(cfg.G, V - v))
                    ses.propagate_keep_multi(min(cfg.G, V - v))
                ses.compact(slot=v % cfg.G, own_keep=True)
                cnt = ses._slot("keep_count", v % cfg.G).cpu()
            else:
                ses.variant(v, fused=cfg.path != "stepwise")
                cnt = ses.keep_count.cpu()
            offs, shp = ses.dst_offsets.cpu(), ses.dst_shapes.cpu()
            used = min(item_sizes(wl, cnt.numpy(), cfg.eb)[2], n_arena)
            host_out[0][:used].copy_(ses.compact_arena[:used], non_blocking=True)
            counters["d2h"] += used + offs.numel() * 8 + shp.numel() * 4 + cnt.numel() * 4
        torch.cuda.synchronize()

    # ---- steps in a pipeline: every variant has a destination arena of its own, so all rebuilds of a step are done
    # about a millisecond after its weights arrived; from then on the weights of the NEXT step travel up (a stream of
    # their own) while this step's variants travel down - PCIe carries both directions at once.  Every step still
    # uploads its own weights and reads back all of its variants; only the wall clock of the whole run is taken.
    pipelined = cfg.path == "sparse_free" and V <= 16 and "arena" in ses.pf[0]
    if pipelined:
        up_stream = torch.cuda.Stream(device=dm.device)
        host_var = [torch.empty(ses.pf[v]["arena"].numel(), dtype=torch.uint8).pin_memory() for v in range(V)]
        state = {"weights_free": None, "arenas_free": None}

        def step_pipelined():
            main = torch.cuda.current_stream()
            with torch.cuda.stream(up_stream):
                if state["weights_free"] is not None:
                    up_stream.wait_event(state["weights_free"])       # the last step's rebuilds have read the old weights
                dm.upload_weights()
                arrived = torch.cuda.Event()
                arrived.record(up_stream)
            counters["h2d"] += dm.weight_bytes
            main.wait_event(arrived)
            ses.magnitude_threshold(wl.ks)
            ses.zero_structures_portfolio(0, V)
            ses.propagate_keep_portfolio(V)
            kcs = [ses.pf[v]["keep_count"].cpu().numpy() for v in range(V)]      # synchronises once: sizes are data
            counters["d2h"] += sum(k.nbytes for k in kcs)
            if state["arenas_free"] is not None:
                main.wait_event(state["arenas_free"])                 # the last step's variants have left the device
            ses.compact_portfolio_multi(0, V)
            rebuilt = torch.cuda.Event()
            rebuilt.record(main)
            state["weights_free"] = rebuilt
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(rebuilt)
                for v in range(V):
                    used = min(item_sizes(wl, kcs[v], cfg.eb)[2], host_var[v].numel())
                    no, ns = ses.pf[v]["dst_offsets"].numel() * 8, ses.pf[v]["dst_shapes"].numel() * 4
                    host_small[v][:no].copy_(ses.pf[v]["dst_offsets"].view(torch.uint8), non_blocking=True)
                    host_small[v][no:no + ns].copy_(ses.pf[v]["dst_shapes"].view(torch.uint8), non_blocking=True)
                    host_var[v][:used].copy_(ses.pf[v]["arena"][:used], non_blocking=True)
                    counters["d2h"] += used + no + ns
                left = torch.cuda.Event()
                left.record(copy_stream)
                state["arenas_free"] = left

        for _ in range(2):
            step_pipelined()
        torch.cuda.synchronize()
        counters["h2d"] = counters["d2h"] = 0
        barrier()
        t0 = time.perf_counter()
        for _ in range(steps):
            step_pipelined()
        torch.cuda.synchronize()
        total = (time.perf_counter() - t0) * 1e3
        barrier()
        # what arrived is what the device holds (the smallest variant, byte for byte)
        used_last = min(item_sizes(wl, ses.pf[V - 1]["keep_count"].cpu().numpy(), cfg.eb)[2], host_var[V - 1].numel())
        assert torch.equal(host_var[V - 1][:used_last], ses.pf[V - 1]["arena"][:used_last].cpu()), "end-to-end copy differs"
        (per_step,) = max_over_ranks([total / steps])
        return {"value": ms_per_variant_of(per_step, V), "min": ms_per_variant_of(per_step, V), "unit": "ms",
                "h2d_bytes_per_step": counters["h2d"] // steps, "d2h_bytes_per_step": counters["d2h"] // steps,
                "how": f"host wall clock around {steps} whole portfolios through the C ABI with pinned host buffers, divided by "
                       f"{steps}: every step copies the weights up and every rebuilt variant down; the steps form a pipeline "
                       "(the next step's weights travel up while this step's variants travel down)"}

    run = step_overlapped if cfg.path == "sparse_free" and V <= 16 else step_sequential
    for _ in range(2):
        run()
    counters["h2d"] = counters["d2h"] = 0
    times = []
    for _ in range(steps):
        barrier()
        t0 = time.perf_counter()
        run()
        times.append((time.perf_counter() - t0) * 1e3)
    barrier()
    med, mn = max_over_ranks([statistics.median(times), min(times)])
    return {"value": ms_per_variant_of(med, V), "min": ms_per_variant_of(mn, V), "unit": "ms",
            "h2d_bytes_per_step": counters["h2d"] // steps, "d2h_bytes_per_step": counters["d2h"] // steps,
            "how": "host wall clock around a whole portfolio through the C ABI with pinned host buffers: weights up, "
                   "every rebuilt variant down" + (" (rebuild of the next variant overlaps the copy of the last)" if run is step_overlapped else "")}


def extras(cfg, sizes):
    """Rows beyond the five steps, on the rebuilt variants (not part of the timed portfolio step): conv+BN fusion,
    fixed-point keep propagation, deflation / inflation."""
    import torch
    from paper_2309_06973_b200 import binding as B
    from paper_2309_06973_b200.runtime import Deflater, Session
    ses, wl, V, eb, dm = cfg.ses, cfg.wl, cfg.V, cfg.eb, cfg.dm

    def rebuild(v):
        if cfg.path == "sparse_free":
            ses.compact_portfolio(v, v)
        else:
            ses.variant(v, fused=cfg.path != "stepwise")
    if cfg.path == "sparse_free":
        ses.magnitude_threshold(wl.ks)
        ses.zero_structures_portfolio(0, V)
        ses.propagate_keep_portfolio(V)

    fold_ms = []
    for _ in range(5):
        rebuild(V - 1)                      # a fresh rebuilt variant (the last one of the portfolio)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ses.fold_batchnorm()
        b.record()
        torch.cuda.synchronize()
        fold_ms.append(a.elapsed_time(b))
    fold_ms = statistics.median(fold_ms)
    fold = {"ms": fold_ms, "gbs": 2 * sizes[-1]["Nn"] * eb / (fold_ms * 1e-3) / 1e9,
            "what": "conv + BatchNorm fusion of the last variant in place (read + write of its weights)"}

    def params_of(session):
        sh = session.dst_shapes.cpu().numpy()[: 2 * len(wl.tensors)].reshape(-1, 2)
        return sum(int(sh[i, 0]) * int(sh[i, 1]) * t.KH * t.KW for i, t in enumerate(wl.tensors))
    ses2 = Session(dm, wl.scope, V, want_mask_bits=False, want_nz_map=True)
    ses2.magnitude_threshold(wl.ks)
    ses2.mask_and_structures(V - 1)
    ses2.propagate_keep()
    ses2.compact()
    torch.cuda.synchronize()
    params_single = params_of(ses2)
    casc_ms = []
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ses2.propagate_keep_cascade(max_passes=8)
        b.record()
        torch.cuda.synchronize()
        casc_ms.append(a.elapsed_time(b))
    ses2.compact()
    torch.cuda.synchronize()
    cascade = {"ms": statistics.median(casc_ms), "max_passes": 8,
               "passes_that_removed": int(ses2.stats.cpu().numpy().view(np.uint64)[3]),
               "weights_after_single_pass": params_single, "weights_after_cascade": params_of(ses2),
               "what": "last variant: rule of Algorithm 1 applied to a fixed point on the kernel maps"}
    ses2.close()

    deflater = Deflater(ses.compact_arena.numel(), dm.device)
    raw_sizes, packed_sizes, codec_ms = [], [], {"deflate": [], "inflate": []}
    restored = torch.empty_like(ses.compact_arena)
    for v in range(V):
        rebuild(v)
        torch.cuda.synchronize()
        used = min(sizes[v]["used"], ses.compact_arena.numel())
        for _ in range(5 if v == V - 1 else 1):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev[0].record()
            deflater.deflate(ses.compact_arena, used)
            ev[1].record()
            size = deflater.stream_bytes()
            ev[2].record()
            deflater.inflate(restored, size)
            ev[3].record()
            torch.cuda.synchronize()
            if v == V - 1:
                codec_ms["deflate"].append(ev[0].elapsed_time(ev[1]))
                codec_ms["inflate"].append(ev[2].elapsed_time(ev[3]))
        assert int(deflater.status.item()) == B.DNNS_OK and torch.equal(restored[:used], ses.compact_arena[:used])
        raw_sizes.append(used)
        packed_sizes.append(size + 8 * (B.dnns_deflate_chunks(used) + 1) + 4 * 32 * B.dnns_deflate_chunks(used))
    order = sorted(range(V), key=lambda v: raw_sizes[v])           # Module 7 sorts the portfolio by model size
    dms, ims = statistics.median(codec_ms["deflate"]), statistics.median(codec_ms["inflate"])
    deflate = {"package_order": order, "raw_bytes": [raw_sizes[v] for v in order],
               "packed_bytes_with_index": [packed_sizes[v] for v in order],
               "package_ratio": sum(packed_sizes) / sum(raw_sizes),
               "last_variant": {"deflate_ms": dms, "inflate_ms": ims,
                                "deflate_gbs": (raw_sizes[-1] + packed_sizes[-1]) / (dms * 1e-3) / 1e9,
                                "inflate_gbs": (raw_sizes[-1] + packed_sizes[-1]) / (ims * 1e-3) / 1e9},
               "what": "RFC 1951 streams (fixed Huffman / stored blocks, runs as distance-1 matches) plus chunk and "
                       "sub-block index; paper context: 43 ms to switch a VGG-16 variant in (Table V)"}
    return fold, cascade, deflate


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dnns", choices=["dnns", "reference"])
    ap.add_argument("--workload", default="resnet152", choices=["toy", "vgg16", "resnet56", "resnet50", "resnet152"])
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16"])
    ap.add_argument("--path", default="sparse_free", choices=["sparse_free", "multi", "fused", "stepwise"],
                    help="sparse_free: no sparse model is stored (default); multi: several variants per sweep, sparse models "
                         "written; fused: one fused sweep per variant; stepwise: the five calls one by one")
    ap.add_argument("--stepwise", action="store_true", help="same as --path stepwise")
    ap.add_argument("--multi", type=int, default=-1, help="--path multi: variants per sweep (1..4; default 4 for f32, 2 for bf16)")
    ap.add_argument("--rebuild-per-variant", action="store_true",
                    help="--path sparse_free: one rebuild launch per variant instead of one for all variants")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA graph replay")
    ap.add_argument("--no-also", action="store_true", help="skip the other target configurations (resnet152 bf16, resnet50 f32)")
    ap.add_argument("--no-extras", action="store_true", help="skip fold / cascade / deflate / frozen-streams figures")
    ap.add_argument("--extras-only", action="store_true",
                    help="one untimed portfolio step, then only the fold / cascade / deflate figures (a short run to profile those kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.stepwise:
        args.path = "stepwise"

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2309_06973_b200 import workloads as W
    dtype = 0 if args.dtype == "f32" else 1

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, W.BY_NAME[args.workload](), dtype)
        return

    import torch
    import torch.distributed as dist
    from paper_2309_06973_b200 import binding as B
    from paper_2309_06973_b200.dist_util import max_over_ranks as _max_over_ranks, ms_per_variant as whole_job_ms_per_variant

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    B.lib()  # fail loudly if the extension is missing
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    max_over_ranks = lambda xs: _max_over_ranks(xs, torch.device(device))
    ms_per_variant_of = lambda ms_per_step, V: whole_job_ms_per_variant(ms_per_step, V, world)
    peak, peak_kind = load_peaks()

    cfg = Config(args, args.workload, dtype, device, pinned_host=not args.extras_only)
    wl, V = cfg.wl, cfg.V
    if args.extras_only:
        cfg.step()
        torch.cuda.synchronize()
        fold, cascade, deflate = extras(cfg, cfg.variant_sizes())
        if rank == 0:
            print(json.dumps({"extras_only": True, "config": config_of(wl, dtype), "fold_batchnorm": fold, "cascade": cascade,
                              "deflate": deflate}))
        return
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    m = measure(cfg, args.steps, args.warmup, barrier, max_over_ranks, ms_per_variant_of, peak, peak_kind, args.workload)
    clocks = sampler.stop()
    sizes = m.pop("_sizes")
    e2e = end_to_end(cfg, max(3, min(args.steps, 10)), barrier, max_over_ranks, ms_per_variant_of)

    line = {
        "metric": METRIC, "value": m["ms_per_variant"], "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": m["ms_per_step"], "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": dtype_label(dtype), "data": "synthetic", "config": config_of(wl, dtype),
        "value_is": "median over the timed steps (one CUDA event pair per step, L2 flushed before each); ms_per_variant_min beside it",
    }
    line.update({k: v for k, v in m.items() if k not in ("ms_per_variant", "ms_per_step", "steps")})
    line["e2e"] = e2e
    line["clocks"] = clocks
    line["context"] = {"paper_pruning_time_ms": 120, "paper_hardware": "not stated for that figure"}

    if not args.no_extras:
        fold, cascade, deflate = extras(cfg, sizes)
        line["fold_batchnorm"], line["cascade"], line["deflate"] = fold, cascade, deflate
    del cfg
    torch.cuda.empty_cache()

    if not args.no_extras and any(sum(1 for t in wl.tensors if t.out_group == g) > 1 for g in range(len(wl.groups))):
        # the paper's own setting: residual streams (skip connections, downsampling layers) are left alone
        fz = Config(args, args.workload, dtype, device, freeze=True)
        mf = measure(fz, max(5, args.steps // 2), 3, barrier, max_over_ranks, ms_per_variant_of, peak, peak_kind, args.workload)
        line["frozen_streams_vs_coupled"] = {
            "what": "groups written by several layers (residual streams) frozen, as the paper leaves skip and downsampling "
                    "layers unpruned (Section IV-B-2), against the coupled keep sets of the headline run",
            "coupled": {"ms_per_variant": m["ms_per_variant"], "rebuilt_weights": [v["rebuilt_weights"] for v in m["variants"]]},
            "frozen": {"ms_per_variant": mf["ms_per_variant"], "rebuilt_weights": [v["rebuilt_weights"] for v in mf["variants"]]}}
        del fz
        torch.cuda.empty_cache()

    if not args.no_also and args.workload == "resnet152" and args.dtype == "f32":
        # the other configurations the target names, in the same record (device-resident timing only)
        also = {}
        for name, dt in (("resnet152", 1), ("resnet50", 0)):
            c2 = Config(args, name, dt, device)
            m2 = measure(c2, args.steps, 3, barrier, max_over_ranks, ms_per_variant_of, peak, peak_kind, name)
            m2.pop("_sizes")
            also[f"{name}_{'f32' if dt == 0 else 'bf16'}"] = {
                "config": config_of(c2.wl, dt), "dtype": dtype_label(dt),
                **{k: m2[k] for k in ("ms_per_variant", "ms_per_variant_min", "ms_per_step", "moved_gbs", "moved_frac_of_peak",
                                      "stepwise_equivalent_frac_of_peak", "sweeps", "launch", "kernel_ms", "roofline")},
                "spatial_compression": [v["spatial_compression"] for v in m2["variants"]]}
            del c2
            torch.cuda.empty_cache()
        line["also"] = also

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        t = oracle_portfolio(wl, dtype, list(range(V)))
        line["cpu_baseline"] = {"value": 1e3 * t / V, "unit": "ms", "cores": 1, "kind": "oracle",
                                "sample": f"the whole workload once: all {V} variants, full weights ({t:.1f} s)"}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
