#!/usr/bin/env python
"""Benchmark of block-wise multi-hop feature aggregation on B200.

A step is one gnnpre_propagate call: all K hops over every edge block of one synthetic workload.
The metric is propagated edge-feature elements per second, K * |E| * F / t, where |E| counts the
edges of the operator's support.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the same
workload on its own GPU; the path has no exchange step, so there is no collective in it.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import gnnpre_inputs as gi

METRIC = "propagated edge-feature elems/s over K hops"
UNIT = "elems/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(gi.WORKLOADS))
    ap.add_argument("--scale-down", type=int, default=1, help="divide nodes and edges (debugging only)")
    ap.add_argument("--segment-edges", type=int, default=0)
    ap.add_argument("--blocks", type=int, default=-1, help="override the workload's block count")
    ap.add_argument("--per-block-launch", action="store_true")
    ap.add_argument("--no-bulk-copy", action="store_true", help="register-gather kernel for every width")
    ap.add_argument("--feat-dim", type=int, default=0, help="override the workload's F (sweeps)")
    ap.add_argument("--op", type=int, default=-1, help="override the workload's operator (sweeps)")
    ap.add_argument("--ld", type=int, default=0, help="leading dimension (floats) of X and of every hop, e.g. 128 for "
                                                      "F=100 so that rows start on 512-byte boundaries (0 = F)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--budget-gb", type=float, default=0.0, help="device-memory budget B_GPU of the streamed plan (0 = free memory)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "columns"],
                    help="N > 1: independent replicas of the workload (weak scaling, the default), or one workload with "
                         "the feature columns split over the ranks (strong scaling; no collective either)")
    ap.add_argument("--cuda-graph", action="store_true",
                    help="capture one gnnpre_propagate call (all K hops) in a CUDA graph and time its replays: for the "
                         "small workloads, whose steps are bound by launch latency")
    ap.add_argument("--stage", default="aggregate", choices=["aggregate", "lc"],
                    help="aggregate: the K-hop precomputation (the headline); lc: the first dense stage of an LC model "
                         "(Eq. 9) over the precomputed hops, every row once in a seeded random order")
    ap.add_argument("--hidden", type=int, default=256, help="hidden width of --stage lc")
    ap.add_argument("--lc-precision", default="tf32x3", choices=["tf32", "tf32x3"],
                    help="--stage lc: which precision the line leads with: every operand split into two tf32 numbers "
                         "(fp32-like accuracy, the like-for-like figure: the paper's arithmetic is fp32), or plain tf32 "
                         "operands; the other one is timed beside it")
    ap.add_argument("--e2e-col-slabs", type=int, default=0, help="column slabs c of the host-buffer runs (0 = the library's choice; forcing c also "
                                                                    "forces the equal-slab schedule)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="default run only: skip the compact records of configurations 1, 2, 3 (a corner) and 5")
    ap.add_argument("--c5-scale", type=int, default=2,
                    help="divisor of configuration 5's nodes and edges in the default run's streamed record")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self._stop = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                parts = [p.strip() for p in out.strip().split(",")]
                if len(parts) == 6:
                    self.rows.append(parts)
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thread.join(timeout=10)

    def summary(self):
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        sm = sorted(float(r[0]) for r in self.rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[2 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(self.rows[0][1]), "reasons": reasons,
                "samples": len(self.rows)}


def profiled_traffic(workload_name):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, or None when there is
    none for this workload or the kernel sources have changed since it was taken."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", f"k_segments_tma_{workload_name}_dram.md")
    if not os.path.exists(path):
        return None
    text = open(path).read()
    t = re.search(r"traffic_bytes_per_launch:\s*(\d+)", text)
    h = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
    if not t or not h:
        return None
    return int(t.group(1)) if kernel_source_hash() == h.group(1) else None


def kernel_source_hash():
    """sha256 over the files that hold the bulk-copy segment kernel and the pieces it shares with the others (what an
    ncu capture of it depends on)."""
    import hashlib
    cur = hashlib.sha256()
    for f in ("segments_common.cuh", "segments_tma.cuh"):
        cur.update(open(os.path.join(ROOT, "paper_2207_12000_b200", "csrc", f), "rb").read())
    return cur.hexdigest()


def profiled_traffic_lc(rows_per_launch):
    """DRAM bytes per launch of k_lc_first_layer: the committed ncu figure of a smaller case scaled by gathered
    rows (traffic is proportional to them), or None when the kernel source has changed since the capture."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", "k_lc_first_layer_c4_quarter_scale_dram.md")
    if not os.path.exists(path):
        return None
    text = open(path).read()
    t = re.search(r"traffic_bytes_per_launch:\s*(\d+)", text)
    r = re.search(r"rows_per_launch:\s*(\d+)", text)
    h = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
    if not t or not r or not h:
        return None
    src = open(os.path.join(ROOT, "paper_2207_12000_b200", "csrc", "lc_layer.cu"), "rb").read()
    if hashlib.sha256(src).hexdigest() != h.group(1):
        return None
    return int(round(int(t.group(1)) * rows_per_launch / int(r.group(1))))


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: every rank runs an independent replica, the job is as slow as the slowest."""
    if world <= 1:
        return ms
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_step: int, steps: int, world: int, total_ms: float) -> float:
    """Whole-job throughput of `world` replicas (weak scaling: per-GPU work is fixed)."""
    return world * units_per_step * steps / (total_ms * 1e-3)


def byte_model(n, m, F):
    """Algorithmic bytes of one hop.  gather: every neighbour row comes from memory once per edge;
    min: every matrix is touched once."""
    gather = 4 * m * F + 4 * n * F + 4 * m + 16 * n
    least = 8 * n * F + 4 * m + 16 * n
    return gather, least


def oracle_sample(w, g_cpu, X_cpu, target_seconds, got=None):
    """Times the CPU oracle, as it stands, on a row range of hop 1 sized for about target_seconds.  `got` maps a
    label to hop 1 as the CUDA path computed it (anything indexable by a row range that gives a numpy array):
    the rows the oracle has just computed are then compared with it, floor-free, |g - o| / (|A^| |x|)."""
    import oracle as orc
    rp, ci = g_cpu.rowptr.numpy(), g_cpu.colidx.numpy()
    n = g_cpu.n
    diag = 0 if w.op == gi.OP_SAGE else 1
    probe_rows = max(1, n // 256)
    t0 = time.perf_counter()
    orc.hop_rows_f32(w.op, w.gin_eps, rp, ci, X_cpu, np.arange(probe_rows), want_abs=bool(got))
    t_probe = time.perf_counter() - t0
    probe_edges = int(rp[probe_rows]) + diag * probe_rows
    rate = probe_edges / max(t_probe, 1e-6)
    want_edges = rate * target_seconds
    total_edges = int(rp[n]) + diag * n
    rows = n if want_edges >= total_edges else int(np.searchsorted(rp, want_edges))
    rows = max(1, min(n, rows))
    t0 = time.perf_counter()
    y, scale = orc.hop_rows_f32(w.op, w.gin_eps, rp, ci, X_cpu, np.arange(rows), want_abs=bool(got))  # |A^||X| only for the check
    t = time.perf_counter() - t0
    edges = int(rp[rows]) + diag * rows
    out = {"value": edges * X_cpu.shape[1] / t, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
           "sample": f"hop 1 of {w.name} on rows [0, {rows}) = {edges} of {total_edges} edges, {t:.2f} s"}
    if got:
        nz = scale > 0
        parity = {"rows": rows, "tolerance": 1e-5, "measure": "max |gpu - oracle| / (|A^| |X|) over the sampled rows of hop 1"}
        for label, hop1 in got.items():
            g = np.asarray(hop1[0:rows], dtype=np.float64)
            err = float((np.abs(g - y)[nz] / scale[nz]).max(initial=0.0))
            exact_zero = bool((g[~nz] == 0).all())
            parity[label] = {"max_backward_error": err, "ok": bool(err <= 1e-5 and exact_zero)}
        out["parity"] = parity
    return out, t


def run_reference(args, w):
    """The oracle as the reference arm: every step is a bounded sample of the workload on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    g = gi.make_graph(w, device=dev).to("cpu")
    X = gi.make_features(w, device=dev).cpu().numpy()
    per_step = min(args.cpu_seconds, 120.0 / max(1, args.steps + args.warmup))
    vals, ms = [], []
    base = None
    for i in range(args.warmup + args.steps):
        base, t = oracle_sample(w, g, X, per_step)
        if i >= args.warmup:
            vals.append(base["value"])
            ms.append(t * 1e3)
    value = float(np.mean(vals))
    base["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(ms)), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, g, None), "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(w, g, info):
    cfg = {"workload": f"{w.name}: {w.kind} graph, {g.n} nodes, {g.nnz} directed nnz, F={w.feat_dim}, K={w.hops}, "
                       f"op={('gcn_sym', 'sage_mean', 'gin_sum')[w.op]}",
           "l2_policy": "inputs larger than L2 (X and every hop are n*F*4 bytes each; no flush between steps)"
           if g.n * w.feat_dim * 4 > 126e6 else "L2 flushed between steps by writing a 256 MB buffer"}
    if info:
        cfg.update({"blocks": info["b"], "col_slabs": info["c"], "segment_edges": info["segment_edges"],
                    "nnz_tilde": info["nnz_tilde"]})
    return cfg


def run_lc_stage(args, w):
    """--stage lc: Y_k = act(X_k[batch] W_1) for the K precomputed hops of the workload (Eq. 9's first dense
    stage; hidden width and ReLU from the paper's settings).  A step is one call over all n rows in a seeded
    random order (one epoch's worth of mini-batches); the 4096-row mini-batch is timed beside it."""
    from paper_2207_12000_b200 import binding as B  # fails loudly if the CUDA library is missing
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("--stage lc is a single-GPU measurement")
    g = gi.make_graph(w, device="cuda")
    X = gi.make_features(w, device="cuda")
    K, F, H, n = w.hops, w.feat_dim, args.hidden, g.n
    plan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, F, gin_eps=w.gin_eps)
    hops, _ = B.gnnpre_propagate(plan, X, K)
    plan.close()
    del X
    Wt = gi.normal_matrix(H, F, w.seed + 77, device="cuda") / float(np.sqrt(F))
    order = torch.from_numpy(np.random.default_rng(w.seed).permutation(n).astype(np.int32)).cuda()
    relu_mask = (1 << K) - 2  # sigma on every term that has another layer after it (k >= 2 in Eq. 9)
    prec = B.GNNPRE_LC_TF32X3 if args.lc_precision == "tf32x3" else B.GNNPRE_LC_TF32
    Y = torch.empty((K, n, H), dtype=torch.float32, device="cuda")
    flag_check = B.gnnpre_lc_first_layer(hops, order[:4096], Wt, relu_mask=relu_mask, precision=prec)  # synchronising call: error word read
    del flag_check
    stream = torch.cuda.current_stream()

    def timed(batch, out, steps, warmup):
        for _ in range(warmup):
            B.gnnpre_lc_first_layer(hops, batch, Wt, relu_mask=relu_mask, precision=prec, out=out, check=False)
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record(stream)
        for i in range(steps):
            B.gnnpre_lc_first_layer(hops, batch, Wt, relu_mask=relu_mask, precision=prec, out=out, check=False)
            ev[i + 1].record(stream)
        torch.cuda.synchronize()
        return [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]

    with ClockSampler(torch.cuda.current_device()) as sampler:  # the same kernel runs in all three timings
        ms = timed(order, Y, args.steps, max(3, args.warmup))
        in_order = timed(None, Y, args.steps, 3)
        mini = timed(order[:4096], Y[:, :4096], 200, 5)
        t_end = time.perf_counter() + 1.5  # untimed: the same calls, long enough for the clock sampler to see the load
        while time.perf_counter() < t_end:
            timed(order, Y, 20, 0)
    clocks = sampler.summary()
    other = B.GNNPRE_LC_TF32 if prec == B.GNNPRE_LC_TF32X3 else B.GNNPRE_LC_TF32X3
    main_prec, prec = prec, other
    other_ms = float(np.mean(timed(order, Y, args.steps, 3)))  # timed() reads `prec`
    prec = main_prec
    total_ms = float(sum(ms))
    ms_step = total_ms / args.steps
    elems = K * n * H
    peak, which = measured_peaks()
    alg_bytes = 4 * K * n * (F + H) + 4 * H * F  # every gathered row read once, every output written once, the weight once
    achieved = alg_bytes / (ms_step * 1e-3) / 1e9
    line = {
        "metric": "first dense stage of an LC model: output elems/s", "value": elems / (ms_step * 1e-3), "unit": "elems/s",
        "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "tf32 inputs, f32 accumulate" if prec == B.GNNPRE_LC_TF32 else "2 x tf32 per input, f32 accumulate",
        "data": "synthetic", "stage": "lc",
        "config": {"workload": f"{w.name}: first dense stage over the {K} hops of n={n}, F={F}; hidden={H}; all rows, seeded random order",
                   "l2": "inputs and outputs larger than L2", "mini_batch_4096_ms": float(np.median(mini)),
                   "rows_in_order_ms": float(np.median(in_order)), "tflops": 2.0 * K * n * F * H / (ms_step * 1e-3) / 1e12},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": profiled_traffic_lc(K * n) if H == 256 and F == 100 and prec == B.GNNPRE_LC_TF32 else None, "peak_source": which,
                     "algorithmic_bytes_per_launch": alg_bytes},
        "gpu_launches": args.steps, "clocks": clocks, "e2e": None,
        "other_precision": {"dtype": "tf32 inputs, f32 accumulate" if other == B.GNNPRE_LC_TF32 else "2 x tf32 per input, f32 accumulate",
                            "ms_per_step": other_ms, "value": elems / (other_ms * 1e-3)},
    }
    if not args.no_cpu_baseline:
        import oracle as orc
        hop0 = gi.make_features(w).numpy()  # timing only: a seeded matrix of the hop's shape, nothing from the device
        Wt_np = gi.normal_matrix(H, F, w.seed + 77).numpy() / np.float32(np.sqrt(F))
        rows = 2048
        t0 = time.perf_counter()
        orc.lc_first_layer(hop0, order[:rows].cpu().numpy(), Wt_np, relu=True)
        t = time.perf_counter() - t0
        rows2 = int(max(rows, min(n, rows * args.cpu_seconds / max(t, 1e-6))))
        t0 = time.perf_counter()
        orc.lc_first_layer(hop0, order[:rows2].cpu().numpy(), Wt_np, relu=True)
        t = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": rows2 * H / t, "unit": "elems/s", "cores": orc.num_threads(), "kind": "oracle",
                                "sample": f"one [n, {F}] matrix, first {rows2} rows of the order, {t:.2f} s"}
    print(json.dumps(line))


_LINK = {}


def host_link_peak():
    """The host link's ceiling measured in this process: one 1 GiB pinned copy per direction, best of 3."""
    if _LINK:
        return dict(_LINK)
    pin = torch.empty(1 << 30, dtype=torch.uint8, pin_memory=True)
    devb = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    for name, dst, src in (("h2d_gbs", devb, pin), ("d2h_gbs", pin, devb)):
        best = 0.0
        for _ in range(3):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            dst.copy_(src, non_blocking=True)
            torch.cuda.synchronize()
            best = max(best, (1 << 30) / (time.perf_counter() - t0) / 1e9)
        _LINK[name] = best
    del pin, devb
    return dict(_LINK)


def link_record(stats, seconds):
    """Achieved host-link rate of a streamed call against the measured ceiling of its busier direction."""
    link = host_link_peak()
    moved = max(stats.h2d_bytes, stats.d2h_bytes)
    link["achieved_gbs"] = moved / seconds / 1e9
    link["direction"] = "d2h" if stats.d2h_bytes >= stats.h2d_bytes else "h2d"
    link["frac"] = link["achieved_gbs"] / link[link["direction"] + "_gbs"]
    return link


def time_resident(B, plan, X, K, outs, steps, warmup, flush, stream, graph=None, barrier=None, sampler_index=None):
    """Device-resident timing of `steps` gnnpre_propagate calls with CUDA events on the launching stream.
    Pass 1 times the calls as a user makes them (asynchronous): ms per step.  Pass 2 repeats them with the
    library's per-launch events on: duration of the segment kernel.  Returns a dict."""
    barrier = barrier or torch.cuda.synchronize

    def step(want_stats, start=None):
        if flush is not None:
            flush.fill_(1)  # L2 flush between iterations, outside the timed interval
        if start is not None:
            start.record(stream)
        if graph is not None and not want_stats:
            graph.replay()
            return None
        _, st = B.gnnpre_propagate(plan, X, K, outs, stream=stream, want_stats=want_stats)
        return st

    for _ in range(max(3, warmup)):
        step(False)
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    seg_ms, seg_launches, launches, st = 0.0, 0, 0, None
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    if sampler:
        sampler.__enter__()
    barrier()
    for a, b_ in ev:
        step(False, start=a)
        b_.record(stream)
    barrier()
    for a, b_ in ev2:
        st = step(True, start=a)
        b_.record(stream)
        seg_ms += st.segments_ms
        seg_launches += st.segments_launches
        launches += st.kernel_launches
    barrier()
    if sampler:
        sampler.__exit__()
    step_ms = [a.elapsed_time(b_) for a, b_ in ev]
    return {"total_ms": float(sum(step_ms)), "ms_per_step": float(sum(step_ms)) / steps,
            "seg_ms": seg_ms, "seg_launches": seg_launches, "launches": launches,
            "pass2_ms": float(sum(a.elapsed_time(b_) for a, b_ in ev2)),
            "hop_ms": [float(st.hop_ms[k]) for k in range(K)], "clocks": sampler.summary() if sampler else None}


def time_ceiling(B, plan, X, flush, stream, reps=10):
    """Average duration of the fetch-only yardstick (gnnpre_gather_ceiling: one hop's gathers, rows summed
    plainly, nothing stored), timed like a hop: CUDA events, L2 flushed before each when the hop runs flushed."""
    sink = B.gnnpre_gather_ceiling(plan, X, stream=stream)
    for _ in range(2):
        B.gnnpre_gather_ceiling(plan, X, sink, stream=stream)
    ms = []
    for _ in range(reps):
        if flush is not None:
            flush.fill_(1)
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        B.gnnpre_gather_ceiling(plan, X, sink, stream=stream)
        b_.record(stream)
        torch.cuda.synchronize()
        ms.append(a.elapsed_time(b_))
    if B.gnnpre_plan_status(plan, stream) != 0:
        raise RuntimeError("a bounded wait ran out inside the gather-ceiling kernel")
    return float(np.mean(ms))


def compact_resident_record(B, w, steps=20, blocks=None, with_cuda_graph=False):
    """One device-resident workload measured like the headline one, reported as a compact record: ms per step
    (all K hops), the segment kernel per hop, and the fetch-only yardstick beside it."""
    g = gi.make_graph(w, device="cuda")
    X = gi.make_features(w, device="cuda")
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    K, F = w.hops, w.feat_dim
    b = w.blocks if blocks is None else blocks
    plan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, F, gin_eps=w.gin_eps, force_blocks=b,
                               force_col_slabs=1 if b else 0)
    info = plan.info()
    m = info["nnz_tilde"]
    outs = [torch.empty((g.n, F), dtype=torch.float32, device="cuda") for _ in range(K)]
    small = g.n * F * 4 <= 126e6
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if small else None
    stream = torch.cuda.current_stream()
    t = time_resident(B, plan, X, K, outs, steps, 3, flush, stream)
    ceil_ms = time_ceiling(B, plan, X, flush, stream)
    seg_ms_per_hop = t["seg_ms"] / (steps * K)
    gather_b, least_b = byte_model(g.n, m, F)
    rec = {"workload": workload_config(w, g, info)["workload"], "blocks": info["b"], "segment_edges": info["segment_edges"],
           "l2": "flushed between steps" if small else "inputs larger than L2",
           "ms_per_step": t["ms_per_step"], "value": K * m * F / (t["ms_per_step"] * 1e-3), "unit": UNIT,
           "segment_kernel_ms_per_hop": seg_ms_per_hop,
           "segment_launches_per_hop": t["seg_launches"] / (steps * K),
           "gather_ceiling_ms_per_hop": ceil_ms,
           "frac_of_gather_ceiling": ceil_ms / seg_ms_per_hop if seg_ms_per_hop > 0 else None,
           "gather_model_gbs": gather_b / (seg_ms_per_hop * 1e-3) / 1e9,
           "gpu_launches_per_step": t["launches"] / steps}
    if with_cuda_graph:  # the launch-bound workload also as a replayed CUDA graph of all K hops
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            B.gnnpre_propagate(plan, X, K, outs, stream=side)
        tg = time_resident(B, plan, X, K, outs, steps, 3, flush, stream, graph=graph)
        rec["ms_per_step_cuda_graph"] = tg["ms_per_step"]
        del graph
    plan.close()
    return rec


def streamed_run(B, w, g, X_dev, args, reps, blocks, col_slabs, ld=None):
    """The same metric through the C ABI with HOST buffers: X and every hop in pinned host memory (the graph too
    for streamed workloads), copies inside the timed region.  Returns (record, hop-1 host tensor or None)."""
    K, F = w.hops, w.feat_dim
    ld = ld or F
    if X_dev.is_cuda:
        Xh = torch.zeros((g.n, ld), dtype=torch.float32, pin_memory=True)[:, :F]
        Xh.copy_(X_dev)
    else:
        Xh = X_dev  # already in pinned host memory
    outs_h = [torch.empty((g.n, ld), dtype=torch.float32, pin_memory=True)[:, :F] for _ in range(K)]
    if w.streamed:  # the graph lives in pinned host memory too
        rp, ci = g.rowptr.cpu().pin_memory(), g.colidx.cpu().pin_memory()
    else:
        rp, ci = g.rowptr, g.colidx
    plan = B.gnnpre_build_plan(rp, ci, w.op, F, gin_eps=w.gin_eps, force_blocks=blocks, force_col_slabs=col_slabs,
                               segment_edges=args.segment_edges, budget_bytes=int(args.budget_gb * 1e9),
                               operands_mem=B.GNNPRE_MEM_HOST)
    for _ in range(2):
        B.gnnpre_propagate(plan, Xh, K, outs_h)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(reps):
        _, st = B.gnnpre_propagate(plan, Xh, K, outs_h, want_stats=True)
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / reps
    info = plan.info()
    rec = {"value": K * info["nnz_tilde"] * F / dt, "unit": UNIT, "h2d_bytes_per_step": int(st.h2d_bytes),
           "d2h_bytes_per_step": int(st.d2h_bytes), "ms_per_step": dt * 1e3, "steps": reps,
           "col_slabs": info["c"], "blocks": info["b"], "structure_on_host": bool(info["structure_mem"]),
           "schedule": ("resident", "equal column slabs", "narrow-first column panels")[st.schedule],
           "upload_slabs": int(st.upload_slabs), "startup_ms": float(st.startup_ms), "drain_ms": float(st.drain_ms),
           "host_link": link_record(st, dt), "segment_edges": info["segment_edges"]}
    plan.close()
    return rec, outs_h, Xh


def c5_streamed_record(B, args):
    """Configuration 5, scaled to what the host's memory holds, as the paper's streamed setting: graph, X and
    both hop outputs in pinned host memory, default budget.  Reports the host-link fraction and checks the
    outputs it timed against the oracle on a bounded row sample (part of the CPU-baseline leg)."""
    w = gi.scaled(gi.WORKLOADS["c5"], args.c5_scale)
    g = gi.make_graph(w, device="cuda")
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    Xh = gi.normal_matrix(w.n, w.feat_dim, w.seed, device="cuda", pin=True)
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    rec, outs_h, Xh = streamed_run(B, w, g, Xh, args, reps=3, blocks=0, col_slabs=args.e2e_col_slabs)
    rec["workload"] = (f"{w.name}: rmat graph, {g.n} nodes, {g.nnz} directed nnz, F={w.feat_dim}, K={w.hops}, op=gcn_sym; "
                       "graph, X and hop outputs in pinned host memory")
    rec["scale_note"] = (f"configuration 5 at 1/{args.c5_scale} of its nodes and edges: at full size X and two hop outputs alone "
                         "are 171 GB of pinned memory, more than the host of this machine has beside the generator")
    if not args.no_cpu_baseline:
        cpu, _ = oracle_sample(w, g.to("cpu"), Xh.numpy(), min(args.cpu_seconds, 4.0), got={"streamed": outs_h[0].numpy()})
        rec["cpu_baseline"] = cpu
        rec["parity_checked"] = bool(cpu["parity"]["streamed"]["ok"])
    del outs_h, Xh
    return rec


def configs_object(B, args):
    """Compact records of the other configurations (1, 2, a corner of 3's sweep, and 5 streamed), so that one
    default run carries a measured line for each of the five.  A record that cannot be taken (say, the host has
    no room for configuration 5's pinned matrices) reports its error instead of taking the whole run down."""
    import dataclasses
    import gc

    def attempt(fn, *a, **kw):
        try:
            return fn(*a, **kw)
        except (RuntimeError, MemoryError) as err:  # GnnpreError is a RuntimeError; so are torch's allocation failures
            gc.collect()
            torch.cuda.empty_cache()
            return {"error": f"{type(err).__name__}: {err}"[:300]}

    out = {}
    out["c1"] = attempt(compact_resident_record, B, gi.WORKLOADS["c1"], steps=50, with_cuda_graph=True)
    out["c2"] = attempt(compact_resident_record, B, gi.WORKLOADS["c2"], steps=20)
    c3 = gi.WORKLOADS["c3"]
    for op, opname in ((gi.OP_GCN, "gcn"), (gi.OP_SAGE, "sage")):
        for F in (16, 128, 512):
            out[f"c3_{opname}_F{F}"] = attempt(compact_resident_record, B, dataclasses.replace(c3, op=op, feat_dim=F), steps=20)
    torch.cuda.empty_cache()
    out["c5"] = attempt(c5_streamed_record, B, args)
    return out


def main():
    args = parse()
    w = gi.scaled(gi.WORKLOADS[args.workload], args.scale_down)
    if args.feat_dim or args.op >= 0:
        import dataclasses
        w = dataclasses.replace(w, feat_dim=args.feat_dim or w.feat_dim, op=args.op if args.op >= 0 else w.op)
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.stage == "lc":
        run_lc_stage(args, w)
        return

    from paper_2207_12000_b200 import binding as B  # fails loudly if the CUDA library is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- inputs (seeded, generated on the device, resident before timing starts)
    t0 = time.perf_counter()
    g = gi.make_graph(w, device="cuda")
    X = gi.make_features(w, device="cuda")
    torch.cuda.synchronize()
    torch.cuda.empty_cache()  # the generator's temporaries go back to the driver: the library allocates with cudaMalloc
    gen_s = time.perf_counter() - t0
    K, F = w.hops, w.feat_dim
    F_total = F
    sharded = args.shard == "columns" and world > 1
    if sharded:
        from paper_2207_12000_b200.shard import column_shard
        f_lo, f_hi = column_shard(F, world, rank)
        if f_hi == f_lo:
            raise SystemExit(f"rank {rank}: more ranks than 4-column slabs of F={F}")
        X = X[:, f_lo:f_hi]  # a strided view: the library takes the leading dimension
        F = f_hi - f_lo
    blocks = w.blocks if args.blocks < 0 else args.blocks
    flags = B.GNNPRE_FLAG_LAUNCH_PER_BLOCK if args.per_block_launch else 0
    if args.no_bulk_copy:
        flags |= B.GNNPRE_FLAG_NO_BULK_COPY

    t0 = time.perf_counter()
    plan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, F, gin_eps=w.gin_eps, force_blocks=blocks,
                               force_col_slabs=1 if blocks else 0, segment_edges=args.segment_edges, flags=flags)
    torch.cuda.synchronize()
    plan_ms = (time.perf_counter() - t0) * 1e3
    info = plan.info()
    m = info["nnz_tilde"]
    if not args.ld and F % 4:
        args.ld = (F + 3) // 4 * 4  # the library wants leading dimensions that are multiples of 4 floats
    if args.ld:  # rows padded to the given leading dimension: strided views, the library takes ldx / ldo
        assert args.ld >= F and args.ld % 4 == 0 and not sharded
        Xp = torch.zeros((g.n, args.ld), dtype=torch.float32, device="cuda")
        Xp[:, :F] = X
        X = Xp[:, :F]
        del Xp
    ld = args.ld or F
    outs = [torch.empty((g.n, ld), dtype=torch.float32, device="cuda")[:, :F] for _ in range(K)]
    small = g.n * F * 4 <= 126e6
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if small else None
    stream = torch.cuda.current_stream()

    graph = None
    if args.cuda_graph:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            B.gnnpre_propagate(plan, X, K, outs, stream=side)  # first call outside the capture (one-time set-up)
        stream.wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            B.gnnpre_propagate(plan, X, K, outs, stream=side)

    # ---------------- timed region: device-resident inputs, CUDA events on the launching stream
    t = time_resident(B, plan, X, K, outs, args.steps, args.warmup, flush, stream, graph=graph, barrier=barrier,
                      sampler_index=local)
    total_ms = max_over_ranks(t["total_ms"], world, "cuda")
    units_per_step = K * m * (F_total if sharded else F)
    # replicas: every rank does the whole workload; column shards: the ranks share one workload
    value = aggregate_throughput(units_per_step, args.steps, 1 if sharded else world, total_ms)

    # ---------------- roofline of the dominant kernel (the segment kernel: one launch = one hop here)
    peak, peak_kind = measured_peaks()
    gather_b, least_b = byte_model(g.n, m, F)
    launches_per_hop = t["seg_launches"] / (args.steps * K)
    seg_launch_ms = t["seg_ms"] / max(1, t["seg_launches"])
    default_shape = (args.segment_edges == 0 and args.blocks < 0 and launches_per_hop == 1 and not args.no_bulk_copy
                     and not args.feat_dim and args.op < 0 and not args.ld and args.scale_down == 1)
    traffic = profiled_traffic(w.name) if default_shape else None
    secs = seg_launch_ms * 1e-3
    if traffic is not None:
        achieved, basis = traffic / secs / 1e9, "DRAM bytes of one launch (ncu, dram__bytes_read.sum + dram__bytes_write.sum) / kernel time"
        traffic_source = f"profiles/k_segments_tma_{w.name}_dram.md (ncu summary, kernel source hash matched)"
    else:
        achieved, basis = least_b / launches_per_hop / secs / 1e9, ("compulsory bytes of one launch (every matrix touched once: "
                                                                   "8nF + 4|E| + 16n per hop) / kernel time; no ncu capture "
                                                                   "matches these kernel sources and this workload")
        traffic_source = None
    ceil_ms = time_ceiling(B, plan, X, flush, stream) if world == 1 else None
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "frac_basis": basis, "peak_kind": f"{peak_kind} copy bandwidth (burst)", "traffic": traffic,
                "traffic_source": traffic_source,
                "kernel": "k_segments_tma (bulk-copy segment kernel)" if 68 <= F <= 128 and not args.no_bulk_copy
                          else "segment kernel (k_segments / k_segments_tma by tile width)",
                "kernel_ms_per_launch": seg_launch_ms, "launches_per_hop": launches_per_hop,
                "algorithmic_bytes_per_launch": gather_b / launches_per_hop,
                "gather_model_gbs": gather_b / launches_per_hop / secs / 1e9,
                "achieved_min_model": least_b / launches_per_hop / secs / 1e9,
                "model": "algorithmic bytes = gather model, every neighbour row fetched once per edge: 4|E|F + 4nF + 4|E| + 16n "
                         "per hop; L2 hits let gather_model_gbs exceed the DRAM peak, so frac is taken from DRAM traffic",
                "kernel_timing": "second pass over the same steps with CUDA events around every launch of the kernel",
                "kernel_share_of_step": t["seg_ms"] / t["pass2_ms"],
                "gather_ceiling_ms_per_hop": ceil_ms,
                "frac_of_gather_ceiling": None if ceil_ms is None else ceil_ms / (seg_launch_ms * launches_per_hop)}

    # ---------------- end to end through the C ABI with host buffers (copies inside the timed region)
    e2e, outs_h, Xh = None, None, None
    if not args.no_e2e and rank == 0:
        try:
            e2e, outs_h, Xh = streamed_run(B, w, g, X, args, reps=max(2, min(args.steps, 5)), blocks=blocks,
                                           col_slabs=args.e2e_col_slabs, ld=ld)
            if sharded:  # rank 0 times its own slab; the job's figure assumes the other ranks' slabs take as long
                e2e["value"] *= world
            # same bits are expected only when both plans cut the edge list the same way
            comparable = e2e["blocks"] == info["b"] and e2e["segment_edges"] == info["segment_edges"] and F <= 128
            e2e["bitwise_equal_to_resident"] = all(torch.equal(o.cpu(), h) for o, h in zip(outs, outs_h)) if comparable else None
            e2e["max_abs_diff_to_resident"] = max(float((o.cpu() - h).abs().max()) for o, h in zip(outs, outs_h))
        except RuntimeError as err:  # the library's errors and torch's allocation failures alike
            e2e = {"value": None, "unit": UNIT, "error": str(err)[:300]}

    # ---------------- the oracle on this machine's host cores, bounded sample (rank 0, one GPU only); the rows it
    # computes are compared with hop 1 of the outputs that were timed
    cpu = None
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        got = {"resident": outs[0].cpu().numpy()}
        if outs_h is not None:
            got["host_buffers"] = outs_h[0].numpy()
        cpu, _ = oracle_sample(w, g.to("cpu"), np.ascontiguousarray(X.cpu().numpy()), args.cpu_seconds, got=got)
        if e2e is not None and "host_buffers" in cpu["parity"]:
            e2e["parity_checked"] = bool(cpu["parity"]["host_buffers"]["ok"])
    del outs_h, Xh

    configs = None
    if rank == 0 and world == 1 and args.workload == "c4" and default_shape and not args.no_configs:
        plan.close()
        del outs, X, flush
        torch.cuda.empty_cache()
        configs = configs_object(B, args)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
                "scaling": "strong" if sharded else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": dict(workload_config(w, g, info), parallelism="column shards" if sharded else "replicas",
                               cuda_graph=bool(args.cuda_graph), leading_dim=ld),
                "clocks": t["clocks"], "e2e": e2e, "gpu_launches": int(t["launches"]), "roofline": roofline,
                "cpu_baseline": cpu, "plan_build_ms": plan_ms, "input_generation_s": gen_s,
                # the same metric if every step also rebuilt the plan (degrees, scales, Eq. 12, edge blocks, segments)
                "value_including_plan_build": (1 if sharded else world) * units_per_step / ((total_ms / args.steps + plan_ms) * 1e-3),
                "hop_ms": t["hop_ms"], "configs": configs}
        print(json.dumps(line), flush=True)
    if configs is None:
        plan.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
