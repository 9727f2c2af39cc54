#!/usr/bin/env python
"""Benchmark of the portfolio-generation hot path: threshold once, then mask, zero-structure
detection, keep propagation and compaction for every variant.

One "step" is one whole portfolio on one model.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet152] [--dtype f32|bf16]
  python bench.py --impl reference ...     # the CPU oracle, as it stands, on the host cores
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


def run_reference(args, wl, dtype):
    V = len(wl.ks)
    variants = sorted({0, V - 1})
    for _ in range(args.warmup):
        oracle_portfolio(wl, dtype, variants)
    times = [oracle_portfolio(wl, dtype, variants) for _ in range(args.steps)]
    total = sum(times)
    ms_per_variant = 1e3 * total / (args.steps * len(variants))
    sample = f"variants {variants} of {V} (threshold sort shared by {len(variants)} instead of {V}), full weights"
    line = {
        "impl": "reference", "metric": METRIC, "value": ms_per_variant, "unit": "ms", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32 keys / fp32 words" if dtype == 0 else "u16 keys / bf16 words", "data": "synthetic",
        "config": config_of(args, wl, dtype),
        "cpu_baseline": {"value": ms_per_variant, "unit": "ms", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": ms_per_variant, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def config_of(args, wl, dtype):
    return {"workload": f"{wl.name} ({'fp32' if dtype == 0 else 'bf16'}), {wl.n_prunable} prunable weights, "
                        f"{len(wl.ks)} variants, {'global' if wl.scope == 0 else 'per-tensor'} ranking, seed {wl.seed}",
            "variants": len(wl.ks), "prunable_weights": wl.n_prunable,
            "l2": "weights larger than L2 (no flush)" if wl.n_prunable * (4 if dtype == 0 else 2) > 126e6
                  else "L2 flushed between steps (256 MiB scratch write)"}


# --------------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="dnns", choices=["dnns", "reference"])
    ap.add_argument("--workload", default="resnet152", choices=["toy", "vgg16", "resnet56", "resnet50", "resnet152"])
    ap.add_argument("--dtype", default="f32", choices=["f32", "bf16"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stepwise", action="store_true", help="mask and zero-structure detection as two sweeps")
    ap.add_argument("--multi", type=int, default=-1,
                    help="variants per sweep over the dense weights (1..4; 0: one fused call per variant; default 4 for f32, 2 for bf16)")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA graph replay")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2309_06973_b200 import workloads as W
    dtype = 0 if args.dtype == "f32" else 1

    if args.impl == "reference":
        if rank != 0:
            return
        wl = W.BY_NAME[args.workload]()
        run_reference(args, wl, dtype)
        return

    import torch
    import torch.distributed as dist
    from paper_2309_06973_b200 import binding as B
    from paper_2309_06973_b200.runtime import Deflater, DeviceModel, Session
    from paper_2309_06973_b200.dist_util import max_over_ranks, ms_per_variant as whole_job_ms_per_variant

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    B.lib()  # fail loudly if the extension is missing
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl = W.BY_NAME[args.workload]()
    V = len(wl.ks)
    eb = 4 if dtype == 0 else 2
    N = wl.n_prunable
    dm = DeviceModel(wl, dtype, device=f"cuda:{local_rank}", pinned_host=True)
    G = args.multi if args.multi >= 0 else (4 if dtype == 0 else 2)
    G = 0 if args.stepwise else min(G, 4, V)
    groups = [(v0, min(G, V - v0)) for v0 in range(0, V, G)] if G else []
    ses = Session(dm, wl.scope, V, want_mask_bits=True, want_nz_map=False, slots=max(G, 1))
    need_flush = N * eb <= 126e6
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dm.device) if need_flush else None

    names = (["threshold", "mask", "structures", "propagate", "compact"] if args.stepwise
             else ["threshold", "mask+structures", "propagate", "compact"])
    spans = {n: [] for n in names}
    calls_per_step = {n: V for n in names}
    calls_per_step["threshold"] = 1
    if G:
        calls_per_step["mask+structures"] = calls_per_step["propagate"] = len(groups)

    def step(record: bool):
        def timed(name, fn, *a):
            if not record:
                return fn(*a)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(*a)
            e1.record()
            spans[name].append((e0, e1))
        timed("threshold", ses.magnitude_threshold, wl.ks)
        for v0, n in groups:                       # n variants per read of the dense weights
            timed("mask+structures", ses.mask_and_structures_multi, v0, n)
            timed("propagate", ses.propagate_keep_multi, n)        # the keep sets of the n variants in one launch
            for g in range(n):
                timed("compact", lambda: ses.compact(slot=g, own_keep=True))
        for v in (range(V) if not G else ()):
            if args.stepwise:
                timed("mask", ses.apply_mask, v)
                timed("structures", ses.zero_structures)
            else:
                timed("mask+structures", ses.mask_and_structures, v)
            timed("propagate", ses.propagate_keep)
            timed("compact", ses.compact)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing --------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step(False)
    torch.cuda.synchronize()
    assert ses.device_status() == B.DNNS_OK
    # data-dependent sizes of every variant (outside the timed region): R = kept filter rows, N' = rebuilt size
    R, Nn = [], []
    for v in range(V):
        ses.variant(v, fused=not args.stepwise)
        torch.cuda.synchronize()
        sh = ses.dst_shapes.cpu().numpy()[: 2 * len(wl.tensors)].reshape(-1, 2)
        R.append(sum(int(sh[i, 0]) * t.I * t.KH * t.KW for i, t in enumerate(wl.tensors)))
        Nn.append(sum(int(sh[i, 0]) * int(sh[i, 1]) * t.KH * t.KW for i, t in enumerate(wl.tensors)))

    # One portfolio captured once as a CUDA graph (the calls are plain stream work: no allocation, no
    # synchronisation), replayed for the timed steps.  A second, plain pass with an event pair around
    # every call gives the per-call durations; its total is reported as ms_per_step_plain.
    graph = None
    launches_per_step = None
    if not args.no_graph:
        try:
            l0 = ses.launch_count()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step(False)
            launches_per_step = ses.launch_count() - l0
            graph.replay()
            torch.cuda.synchronize()
        except Exception as e:  # capture refused: fall back to plain launches and say so
            print(f"bench: CUDA graph capture failed ({e}); timing plain launches", file=sys.stderr)
            graph = None

    def timed_steps(run_step):
        """K steps; returns total ms.  Models that fit in L2 get a flush before every step."""
        if need_flush:
            pairs = []
            for _ in range(args.steps):
                flush_buf.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                run_step()
                b.record()
                pairs.append((a, b))
            torch.cuda.synchronize()
            return sum(a.elapsed_time(b) for a, b in pairs)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            run_step()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    launches0 = ses.launch_count()
    plain_ms = timed_steps(lambda: step(True))
    launches_plain = ses.launch_count() - launches0
    # the same steps once more with an event pair around every single kernel (dnns_plan_profile)
    kernel_names = ["k_hist1", "k_select1", "k_hist2", "k_select2", "k_ties", "k_tie_scan", "k_sweep<", "k_sweep_multi", "k_flags",
                    "k_propagate", "k_compact_layout", "k_compact_gather"]
    ses.profile(True)
    timed_steps(lambda: step(False))
    ses.profile(False)
    kernel_ms = {}
    for kn in kernel_names:
        ms, n = ses.kernel_time(kn)
        if n:
            kernel_ms[kn] = {"avg_ms": ms / n, "launches_per_step": n / args.steps, "ms_per_step": ms / args.steps}
    if graph is not None:
        barrier()
        total_ms = timed_steps(graph.replay)
        launches = launches_per_step * args.steps
    else:
        total_ms = plain_ms
        launches = launches_plain
    clocks = sampler.stop()
    barrier()
    total_ms, plain_ms = max_over_ranks([total_ms, plain_ms], dm.device)
    assert ses.device_status() == B.DNNS_OK

    ms_per_step = total_ms / args.steps
    ms_per_variant = whole_job_ms_per_variant(ms_per_step, V, world)
    per_call = {n: statistics.mean(a.elapsed_time(b) for a, b in spans[n]) for n in names}
    plain_per_step = plain_ms / args.steps
    share = {n: per_call[n] * calls_per_step[n] / plain_per_step for n in names}

    # algorithmic bytes: one read of every input a step consumes, one write of every output
    # (the fused sweep moves 2*N*b + N/8 per launch; the stepwise accounting B_v charges the path 3*N*b + N/8)
    alg = {"threshold": N * eb, "mask": 2 * N * eb + N / 8, "structures": N * eb, "mask+structures": 2 * N * eb + N / 8,
           "propagate": 0, "compact": statistics.mean((r + n) * eb for r, n in zip(R, Nn))}
    portfolio_bytes = alg["threshold"] + V * (alg["mask"] + alg["structures"]) + sum((r + n) * eb for r, n in zip(R, Nn))
    moved_bytes = alg["threshold"] + V * (alg["mask"] + (alg["structures"] if args.stepwise else 0)) + \
        sum((r + n) * eb for r, n in zip(R, Nn))
    if G:   # one read of the dense weights per group, one write (+ mask bits) per variant
        multi_bytes = sum(N * eb + n * (N * eb + N / 8) for _, n in groups)
        alg["mask+structures"] = multi_bytes / len(groups)
        moved_bytes = alg["threshold"] + multi_bytes + sum((r + n) * eb for r, n in zip(R, Nn))
    peak, peak_kind = load_peaks()
    # the dominant kernel: largest share of the summed kernel time; its algorithmic bytes per launch
    kernel_alg = {"k_hist1": N * eb, "k_hist2": N * eb, "k_ties": N * eb,
                  "k_sweep<": 2 * N * eb + N / 4,          # weights in and out, mask bits, the element bits it packs
                  "k_compact_gather": alg["compact"]}
    if args.stepwise:
        kernel_alg["k_sweep<"] = (alg["mask"] + alg["structures"] + N / 8) / 2   # two sweeps per variant, averaged
    if G:   # per launch: one read, n writes with their mask and element bits
        kernel_alg["k_sweep_multi"] = sum(N * eb + n * (N * eb + N / 4) for _, n in groups) / len(groups)
    kernel_total = sum(k["ms_per_step"] for k in kernel_ms.values())
    for k in kernel_ms.values():
        k["share"] = k["ms_per_step"] / kernel_total
    dominant = max((kn for kn in kernel_ms if kn in kernel_alg), key=lambda kn: kernel_ms[kn]["ms_per_step"])
    achieved = kernel_alg[dominant] / (kernel_ms[dominant]["avg_ms"] * 1e-3) / 1e9
    for kn, k in kernel_ms.items():
        if kn in kernel_alg:
            k["gbs"] = kernel_alg[kn] / (k["avg_ms"] * 1e-3) / 1e9
    kernel_label = {"k_sweep<": "k_sweep<mask>+<structures>" if args.stepwise else "k_sweep<mask+structures>",
                    "k_sweep_multi": f"k_sweep_multi<{G}>"}

    # ---- Module 1 on a rebuilt variant (not part of the portfolio step): conv + BatchNorm fusion in place
    fold_ms = []
    for _ in range(5):
        ses.compact()                      # a fresh rebuilt variant (the last one of the portfolio)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ses.fold_batchnorm()
        b.record()
        torch.cuda.synchronize()
        fold_ms.append(a.elapsed_time(b))
    fold_ms = statistics.median(fold_ms)

    # ---- fixed-point keep propagation on the last variant (not part of the portfolio step)
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

    # ---- Module 7 / 8 on the rebuilt variants (not part of the portfolio step): every variant deflated into
    # one package, smallest first; timings for the last variant (deflate) and its inflation
    deflater = Deflater(ses.compact_arena.numel(), dm.device)
    raw_sizes, packed_sizes, codec_ms = [], [], {"deflate": [], "inflate": []}
    restored = torch.empty_like(ses.compact_arena)
    for v in range(V):
        ses.variant(v, fused=not args.stepwise)
        torch.cuda.synchronize()
        offs = ses.dst_offsets.cpu().numpy().view(np.uint64)
        cnt = ses.keep_count.cpu().numpy()
        used = min((int(offs[-1]) + 4 * max(int(cnt.max()), 1) + 255) // 256 * 256, ses.compact_arena.numel())
        reps = 5 if v == V - 1 else 1
        for _ in range(reps):
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
    deflate_info = {"package_order": order, "raw_bytes": [raw_sizes[v] for v in order],
                    "packed_bytes_with_index": [packed_sizes[v] for v in order],
                    "package_ratio": sum(packed_sizes) / sum(raw_sizes),
                    "last_variant": {"deflate_ms": dms, "inflate_ms": ims,
                                     "deflate_gbs": (raw_sizes[-1] + packed_sizes[-1]) / (dms * 1e-3) / 1e9,
                                     "inflate_gbs": (raw_sizes[-1] + packed_sizes[-1]) / (ims * 1e-3) / 1e9},
                    "what": "RFC 1951 streams (fixed Huffman / stored blocks, runs as distance-1 matches) plus chunk and "
                            "sub-block index; paper context: 43 ms to switch a VGG-16 variant in (Table V)"}
    del restored

    # ---- end to end through the C ABI with host buffers -----------------------------------------
    small = torch.empty(1 << 16, dtype=torch.uint8).pin_memory()
    host_out = torch.empty(ses.compact_arena.numel(), dtype=torch.uint8).pin_memory()
    h2d = d2h = 0

    def e2e_step():
        nonlocal h2d, d2h
        dm.upload_weights()
        h2d += dm.weight_bytes
        ses.magnitude_threshold(wl.ks)
        for v in range(V):
            if G:
                if v % G == 0:
                    ses.mask_and_structures_multi(v, min(G, V - v))
                    ses.propagate_keep_multi(min(G, V - v))
                ses.compact(slot=v % G, own_keep=True)
            else:
                ses.variant(v, fused=not args.stepwise)
            offs = ses.dst_offsets.cpu()           # synchronises: the sizes are only known on the device
            shp = ses.dst_shapes.cpu()
            cnt = ses._slot("keep_count", v % G if G else 0).cpu()
            last_w = len(wl.tensors) - 1
            used = int(offs[-1].item()) + 4 * max(int(cnt.max().item()), 1)
            used = min((used + 255) // 256 * 256, host_out.numel())
            host_out[:used].copy_(ses.compact_arena[:used], non_blocking=True)
            d2h += used + offs.numel() * 8 + shp.numel() * 4 + cnt.numel() * 4
        torch.cuda.synchronize()

    for _ in range(2):
        e2e_step()
    h2d = d2h = 0
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e2e_step()
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = max_over_ranks([e2e_ms], dm.device)[0]
    e2e_per_variant = whole_job_ms_per_variant(e2e_ms / args.steps, V, world)

    line = {
        "metric": METRIC, "value": ms_per_variant, "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "u32 keys / fp32 words" if dtype == 0 else "u16 keys / bf16 words",
        "data": "synthetic", "config": config_of(args, wl, dtype),
        "effective_gbs": portfolio_bytes / (ms_per_step * 1e-3) / 1e9,
        "effective_frac_of_peak": portfolio_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
        "algorithmic_bytes_per_variant": portfolio_bytes / V,
        "moved_gbs": moved_bytes / (ms_per_step * 1e-3) / 1e9,
        "sweeps": "stepwise" if args.stepwise else (f"fused mask+structures, {G} variants per read of the dense weights" if G
                                                    else "fused mask+structures"),
        "launch": "cuda graph replay" if graph is not None else "plain stream launches", "ms_per_step_plain": plain_per_step,
        "per_call_ms": per_call, "share": share,
        "per_call_gbs": {n: (alg[n] / (per_call[n] * 1e-3) / 1e9 if alg[n] else None) for n in names},
        "kernel_ms": kernel_ms,
        "roofline": {"bound": "hbm", "kernel": kernel_label.get(dominant, dominant), "achieved": achieved, "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                     "algorithmic_bytes": kernel_alg[dominant],
                     "avg_launch_ms": kernel_ms[dominant]["avg_ms"],
                     "timed_by": "CUDA event pair around every launch of the kernel on its stream, "
                                 f"{args.steps} steps of plain launches",
                     "traffic": measured_traffic(args.workload, args.dtype, kernel_label.get(dominant, dominant))},
        "e2e": {"value": e2e_per_variant, "unit": "ms", "h2d_bytes_per_step": h2d // args.steps,
                "d2h_bytes_per_step": d2h // args.steps},
        "gpu_launches": launches,
        "cascade": cascade,
        "fold_batchnorm": {"ms": fold_ms, "gbs": 2 * Nn[-1] * eb / (fold_ms * 1e-3) / 1e9,
                           "what": "conv + BatchNorm fusion of the last variant in place (read + write of its weights)"},
        "deflate": deflate_info,
        "clocks": clocks,
        "context": {"paper_pruning_time_ms": 120, "paper_hardware": "not stated for that figure"},
    }

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
