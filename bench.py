#!/usr/bin/env python
"""Benchmark of the FluxBin decode linear stack on B200 (one JSON line on stdout).

Workload (N=1): the Llama-2-70B-shaped stack of decode linears -- 80 layers x {q, k, v, o, gate,
up, down}, 2 global bases + 1 extra base on a seeded random 5 % of the input columns, g = 128,
batch 1, fp16 activations, every linear with its own input, all 560 packed layers resident in HBM
at once (about 21 GB, far larger than L2, so every step streams the weights from HBM).  A "step" is
one forward token.  --launch says how its 560 linears are launched (replayed from a CUDA graph):
  stack   one fluxbin_plan launch for the whole step (default; the workload gives every linear its own
          input, so all 560 are independent and the persistent kernel streams them back to back)
  layer   one plan per layer (80 launches)
  group   one plan per set of linears a decoder could run together: {q,k,v} {o} {gate,up} {down} (320)
  linear  one fluxbin_linear call per linear (560)

value = algorithmic bytes moved per second over all GPUs (GB/s); us_per_layer and us_per_linear
carry the latency side of the metric.  With --gpus N the N ranks run independent replicas (the
path has no exchange step): weak scaling, no collective on the data path.

--impl reference times the CPU oracle (oracle/) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import concurrent.futures as cf
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_15602_b200 import synth  # noqa: E402

METRIC = "decode_linear_stack_effective_hbm_gbps_batch1"
UNIT = "GB/s"


def algorithmic_bytes(M, N, Kb, Ks, g, n_sal, B):
    """Bytes the method must move for one call (storage model of the paper's appendix + fp16 x, y):
    bits, row scales per (row, group, base), column scales, 16-bit salient indices, activations."""
    w = Kb * M * N // 8 + 2 * Kb * M * (N // g) + 2 * Kb * N
    if Ks > 0 and n_sal > 0:
        w += Ks * M * ((n_sal + 7) // 8) + 2 * Ks * M * (N // g) + 2 * Ks * n_sal + 2 * n_sal
    return w + 2 * B * N + 2 * B * M


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 50 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, smax, power, reasons = [], [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); smax.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            try:
                power.append(float(r[2]))
            except (ValueError, IndexError):
                pass
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons),
                # nvidia-smi's power.draw is a moving average over about a second: the largest sample of a
                # short timed region is still a lower bound of the power under load
                "power_w": max(power) if power else None}


def stack_spec(config: int, layers: int | None):
    """Linears of one layer (or set) of the workload and how many such layers a step runs.  The single-layer
    and single-set workloads (configs 0-3) are run as a rotation of independently seeded copies, enough of them
    that a step streams more than four times the L2 capacity: weights come from HBM, as in decode."""
    lins, nl = synth.config_linears(config)
    if layers is not None:
        nl = layers
    elif config < 4:
        set_bytes = sum(M * N for _, M, N in lins) * 2.43 / 8          # about 2.43 bits per weight
        nl = max(1, int(540e6 // set_bytes) + 1)
    return lins, nl


def cpu_oracle_sample(config: int, B: int, max_linears: int = 28, g: int = 128, nl: int | None = None, gpu_y=None):
    """Time the oracle as it stands on the first linears of the stack (bounded sample); returns
    (GB/s of algorithmic bytes, seconds, bytes, cores, description, agreement).  gpu_y(i) -> the fp16 outputs
    [B][M] the timed GPU run left for linear i: since the oracle's results are at hand anyway, the leg also
    reports how far the two are apart (same measures as the parity tests)."""
    import oracle
    lins, nl_default = synth.config_linears(config)
    n = min(max_linears, len(lins) * (nl or nl_default))
    tot_b, tot_t = 0, 0.0
    worst_l2, worst_rel = 0.0, 0.0
    for i in range(n):
        layer, li = divmod(i, len(lins))
        L = synth.make_config_linear(config, layer, li, g=(g or lins[li][2]))
        x = synth.make_config_activations(config, layer, li, B)
        t0 = time.perf_counter()
        want = oracle.linear_direct(L, x)
        tot_t += time.perf_counter() - t0
        tot_b += algorithmic_bytes(L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal, B)
        if gpu_y is not None:
            got = gpu_y(i).astype(np.float64)
            for b in range(B):
                rms = float(np.sqrt(np.mean(want[b] ** 2)))
                worst_l2 = max(worst_l2, float(np.linalg.norm(got[b] - want[b]) / np.linalg.norm(want[b])))
                worst_rel = max(worst_rel, float((np.abs(got[b] - want[b]) / np.maximum(np.abs(want[b]), 1e-2 * rms)).max()))
    agreement = None if gpu_y is None else {"linears": n, "max_rel_l2": worst_l2, "max_rel_err": worst_rel,
                                            "outputs": "fp16 (adds up to 2^-11 of rounding)"}
    return tot_b / tot_t / 1e9, tot_t, tot_b, oracle.num_threads(), f"first {n} linears of the stack (B={B})", agreement


def dense_fp16_gemv_context(lins, nl, B):
    """Context, not a target: a dense fp16 weight of every distinct shape of the workload through cuBLAS
    (torch.matmul, harness only), rotating over enough copies that the weights come from HBM; returns the
    time the whole stack would take at those per-shape rates and the per-shape timings."""
    import torch
    shapes = {}
    for _, M, N in lins:
        shapes[(M, N)] = shapes.get((M, N), 0) + nl
    per_shape, total_us, total_bytes = {}, 0.0, 0
    for (M, N), count in shapes.items():
        copies = max(2, int(600e6 // (2 * M * N)) + 1)               # > 4x L2 of weights in rotation
        w = [torch.randn(M, N, device="cuda", dtype=torch.float16) for _ in range(copies)]
        x = torch.randn(N, B, device="cuda", dtype=torch.float16)
        for i in range(copies):
            torch.matmul(w[i], x)
        torch.cuda.synchronize()
        reps = max(1, 60 // copies)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            for i in range(copies):
                torch.matmul(w[i], x)
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) * 1e3 / (reps * copies)
        per_shape[f"{M}x{N}"] = {"us": round(us, 2), "GBps": round(2 * M * N / us / 1e3, 1), "count": count}
        total_us += us * count
        total_bytes += 2 * M * N * count
        del w, x
    torch.cuda.empty_cache()
    return {"ms_per_step": total_us / 1e3, "dense_weight_bytes_per_step": total_bytes,
            "GBps_of_dense_bytes": total_bytes / total_us / 1e3, "per_shape": per_shape,
            "how": "torch.matmul (cuBLAS) on random fp16 weights of the same shapes, plain launches, rotating copies "
                   "larger than L2; per-shape time x count"}


def run_reference(args, rank):
    """--impl reference: the CPU oracle on the host cores, each step a bounded sample."""
    if rank != 0:
        return
    vals = []
    for i in range(args.warmup + args.steps):
        gbps, t, b, cores, sample, _ = cpu_oracle_sample(args.config, args.batch, max_linears=args.ref_linears)
        if i >= args.warmup:
            vals.append((gbps, t))
    gbps = statistics.mean(v[0] for v in vals)
    ms = statistics.mean(v[1] for v in vals) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": gbps, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config {args.config}: sample = {sample}", "batch": args.batch},
            "cpu_baseline": {"value": gbps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": gbps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, help="workload: 4 = Llama-2-70B-shaped stack")
    ap.add_argument("--layers", type=int, default=None, help="override the number of layers (profiling only)")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--fp16-tables", action="store_true",
                    help="batched launches keep their lookup tables in fp16 (fluxbin_set_table_format); no effect at batch 1")
    ap.add_argument("--g", type=int, default=128, help="columns per row-scale group; 0 = one scale per row (g = N)")
    ap.add_argument("--no-graph", action="store_true", help="plain launches instead of a CUDA graph replay")
    ap.add_argument("--launch", default="stack", choices=["linear", "group", "layer", "stack"],
                    help="linear: one fluxbin_linear call per linear; group: one plan per set of linears that "
                         "depend on nothing inside the set ({q,k,v}, {o}, {gate,up}, {down}); layer: one plan per "
                         "layer; stack: one plan for the whole stack (valid because the workload gives every "
                         "linear its own input)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the dense fp16 cuBLAS GEMV context timing")
    ap.add_argument("--ref-linears", type=int, default=7, help="linears per step of --impl reference")
    ap.add_argument("--per-linear", action="store_true", help="also print per-linear timings to stderr")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2608_15602_b200 import build as fb_build
    fb_build.build()
    from paper_2608_15602_b200 import fluxbin, layer as fb_layer

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    B = args.batch
    lins, nl = stack_spec(args.config, args.layers)
    jobs = [(layer, li) for layer in range(nl) for li in range(len(lins))]

    # ---- build the resident stack: generate (threads) -> pack on the host -> upload ----------------
    t_setup = time.perf_counter()
    def gen(job):
        layer, li = job
        return job, synth.make_config_linear(args.config, layer, li, g=(args.g or lins[li][2])), \
            synth.make_config_activations(args.config, layer, li, B)

    linears, xs_host, alg_bytes = [], [], []
    eff_flops = 0.0
    lookups = 0
    nthreads = max(1, min(16, (os.cpu_count() or 4) - 1))
    with cf.ThreadPoolExecutor(nthreads) as ex:
        window = []
        it = iter(jobs)
        for _ in range(2 * nthreads):
            j = next(it, None)
            if j is not None:
                window.append(ex.submit(gen, j))
        while window:
            job, L, x = window.pop(0).result()
            j = next(it, None)
            if j is not None:
                window.append(ex.submit(gen, j))
            lin = fb_layer.FluxBinLinear(L, fp16_tables=args.fp16_tables)
            linears.append(lin)
            xs_host.append(x)
            alg_bytes.append(algorithmic_bytes(L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal, B))
            eff_flops += 2.0 * L.M * (L.N + L.n_sal) * B
            lookups += L.Kb * L.M * (L.N // 8) + L.Ks * L.M * ((L.n_sal + 7) // 8)      # one per weight byte
            del L
    setup_s = time.perf_counter() - t_setup

    # activations / outputs: one arena each (device) + pinned host mirrors for the end-to-end leg
    n_in = sum(l.N for l in linears) * B
    n_out = sum(l.M for l in linears) * B
    x_host = torch.empty(n_in, dtype=torch.float16).pin_memory()
    y_host = torch.empty(n_out, dtype=torch.float16).pin_memory()
    off = 0
    for l, x in zip(linears, xs_host):
        x_host[off:off + B * l.N] = torch.from_numpy(x.view(np.float16).reshape(-1))
        off += B * l.N
    x_dev = torch.empty(n_in, dtype=torch.float16, device="cuda")
    y_dev = torch.empty(n_out, dtype=torch.float16, device="cuda")
    x_dev.copy_(x_host)
    ws = fb_layer.Workspace(max(l.weight.workspace_size(B) for l in linears))
    views = []
    ox = oy = 0
    for l in linears:
        views.append((l, x_dev[ox:ox + B * l.N].view(B, l.N), y_dev[oy:oy + B * l.M].view(B, l.M)))
        ox += B * l.N
        oy += B * l.M
    packed_bytes = sum(l.packed_bytes for l in linears)
    stream = torch.cuda.Stream()

    # how the linears of a step are grouped into launches
    nlin = len(lins)
    names = [n for n, _, _ in lins]
    if args.launch == "linear":
        groups = None
    elif args.launch == "group":
        dep_sets = [["q", "k", "v"], ["o"], ["gate", "up"], ["down"]] if "gate" in names else [[n] for n in names]
        groups = [[layer * nlin + names.index(n) for n in ds] for layer in range(nl) for ds in dep_sets]
    elif args.launch == "layer":
        groups = [[layer * nlin + li for li in range(nlin)] for layer in range(nl)]
    else:
        groups = [list(range(len(linears)))]
    plans = None
    if groups is not None:
        plans = [fb_layer.FluxBinPlan([views[i] for i in g]) for g in groups]
        launches_per_step = sum(p.num_launches() for p in plans)
    else:
        launches_per_step = sum(l.weight.num_launches(B) for l in linears)

    def issue_all():
        if plans is not None:
            for p in plans:
                p.run(stream=stream)
        else:
            for l, xv, yv in views:
                l.forward(xv, ws, out=yv, stream=stream)

    graph = None
    with torch.cuda.stream(stream):
        issue_all()                                   # first call per device does the one-time set-up
        stream.synchronize()
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                issue_all()

    def step():
        if graph is not None:
            graph.replay()
        else:
            issue_all()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing --------------------------------------------------------------------
    with torch.cuda.stream(stream):
        for _ in range(max(3, args.warmup)):
            step()
        barrier()
        sampler = ClockSampler(local_rank)
        sampler.start()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ev[0].record(stream)
        for i in range(args.steps):
            step()
            ev[i + 1].record(stream)
        barrier()
        clocks = sampler.stop()
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    total_ms = ev[0].elapsed_time(ev[-1])

    # ---- end to end: pinned host x -> device, the stack, y -> pinned host, every step ---------------
    # Two sets of device activation/output buffers alternate, so the copies of one step overlap the kernels
    # of its neighbours (copy-in, compute and copy-out each on a stream of their own, ordered by events);
    # every step still moves its own inputs and outputs inside the timed region.
    x_dev2, y_dev2 = torch.empty_like(x_dev), torch.empty_like(y_dev)
    views2 = []
    ox = oy = 0
    for l in linears:
        views2.append((l, x_dev2[ox:ox + B * l.N].view(B, l.N), y_dev2[oy:oy + B * l.M].view(B, l.M)))
        ox += B * l.N
        oy += B * l.M
    plans2 = [fb_layer.FluxBinPlan([views2[i] for i in g]) for g in groups] if groups is not None else None

    def issue_all2():
        if plans2 is not None:
            for p in plans2:
                p.run(stream=stream)
        else:
            for l, xv, yv in views2:
                l.forward(xv, ws, out=yv, stream=stream)

    graph2 = None
    with torch.cuda.stream(stream):
        issue_all2()
        stream.synchronize()
        if not args.no_graph:
            graph2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph2, stream=stream):
                issue_all2()
    bufs = [(x_dev, y_dev, graph, issue_all), (x_dev2, y_dev2, graph2, issue_all2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_steps(n):
        comp_done = [None, None]
        out_done = [None, None]
        for i in range(n):
            k = i & 1
            xd, yd, g, issue = bufs[k]
            if comp_done[k] is not None:
                s_in.wait_event(comp_done[k])          # the kernels of step i-2 have read this x buffer
            with torch.cuda.stream(s_in):
                xd.copy_(x_host, non_blocking=True)
                in_done = torch.cuda.Event()
                in_done.record(s_in)
            stream.wait_event(in_done)
            if out_done[k] is not None:
                stream.wait_event(out_done[k])         # step i-2's results have left this y buffer
            with torch.cuda.stream(stream):
                if g is not None:
                    g.replay()
                else:
                    issue()
                comp_done[k] = torch.cuda.Event()
                comp_done[k].record(stream)
            s_out.wait_event(comp_done[k])
            with torch.cuda.stream(s_out):
                y_host.copy_(yd, non_blocking=True)
                out_done[k] = torch.cuda.Event()
                out_done[k].record(s_out)
        for e in out_done:
            if e is not None:
                stream.wait_event(e)

    e2e_steps(2)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s_in.wait_stream(stream)
    e0.record(stream)
    s_in.wait_event(e0)
    e2e_steps(args.steps)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    # the results that reached the host are those of the device-resident steps (same inputs), from either buffer set
    y_ref = y_dev.float().cpu()
    y_got = y_host.float()
    y2_got = y_dev2.float().cpu()
    scale = float(y_ref.abs().max())
    e2e_max_diff = max(float((y_got - y_ref).abs().max()), float((y2_got - y_ref).abs().max())) / max(scale, 1e-30)
    if not (e2e_max_diff < 5e-3 and bool(torch.isfinite(y_got).all()) and scale > 0):
        raise RuntimeError(f"end-to-end outputs differ from the device-resident run: {e2e_max_diff}")

    # ---- optional per-linear timing (plain launches, rotating over the layers so L2 stays cold) -----
    per_linear = None
    if args.per_linear and rank == 0:
        per_linear = {}
        nlin = len(lins)
        with torch.cuda.stream(stream):
            for li, (name, M, N) in enumerate(lins):
                idxs = [layer * nlin + li for layer in range(nl)]
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                reps = 3
                for r in range(reps + 1):
                    if r == 1:
                        a.record(stream)
                    for i in idxs:
                        l, xv, yv = views[i]
                        l.forward(xv, ws, out=yv, stream=stream)
                b.record(stream)
                stream.synchronize()
                us = a.elapsed_time(b) * 1e3 / (reps * len(idxs))
                per_linear[f"{name}_{M}x{N}"] = {"us": round(us, 2), "GBps": round(alg_bytes[li] / us / 1e3, 1)}
        print(json.dumps({"per_linear_plain_launches": per_linear}), file=sys.stderr)

    # ---- max over ranks, aggregate ------------------------------------------------------------------
    from paper_2608_15602_b200 import dist_util
    total_ms, e2e_ms = dist_util.max_over_ranks([total_ms, e2e_ms], device="cuda")
    bytes_per_step = sum(alg_bytes)
    ms_per_step = total_ms / args.steps
    value = dist_util.replica_throughput(bytes_per_step, ms_per_step, world)
    e2e_value = dist_util.replica_throughput(bytes_per_step, e2e_ms / args.steps, world)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        peak = float(peaks["hbm_gbs"])
        achieved = bytes_per_step / (ms_per_step * 1e-3) / 1e9     # one GPU's kernels
        traffic = None
        tpath = os.path.join(ROOT, "profiles", "dram_traffic.txt")
        if os.path.exists(tpath):
            with open(tpath) as f:
                tj = json.load(f)
            # ncu DRAM bytes per algorithmic byte of the captured launch, scaled to a mean launch of this run
            traffic = tj.get("dram_bytes_per_algorithmic_byte", None)
            if traffic is not None:
                traffic = traffic * bytes_per_step / launches_per_step
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"config {args.config}: Llama-2-70B-shaped decode linear stack" if args.config == 4
                       else f"config {args.config}: {nl} independently seeded copies of the layer/set per step",
                       "layers": nl, "linears_per_step": len(linears), "batch": B,
                       "table_entries": "fp16" if (args.fp16_tables and B > 1) else "fp32",
                       "Kb": 2, "Ks": 0 if args.config == 0 else 1, "salient_frac": 0.0 if args.config == 0 else 0.05,
                       "g": args.g or "N", "packed_bytes_resident": packed_bytes, "algorithmic_bytes_per_step": bytes_per_step,
                       "l2": "inputs larger than L2 (weights streamed once per step)" if packed_bytes > 4e8
                       else "working set fits L2: L2-warm number",
                       "launch": ("cuda graph replay" if graph is not None else "plain launches") + f", {args.launch}: "
                       f"{launches_per_step} kernel launches per step",
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "us_per_layer": ms_per_step * 1e3 / nl, "us_per_linear": ms_per_step * 1e3 / len(linears),
            "frac_of_8TBps": achieved / 8000.0,
            "step_ms_min_median_max": [min(step_ms), statistics.median(step_ms), max(step_ms)],
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_source": f"{peak_kind} (torch copy, read+write; a burst figure)",
                         # the same for the fastest timed step (before the power cap pulls the clocks down)
                         "achieved_best_step": bytes_per_step / (min(step_ms) * 1e-3) / 1e9,
                         "frac_best_step": bytes_per_step / (min(step_ms) * 1e-3) / 1e9 / peak,
                         "kernel": "fluxbin_linear_kernel", "per": "mean over the launches of one step"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel() * 2),
                    "d2h_bytes_per_step": int(y_host.numel() * 2), "ms_per_step": e2e_ms / args.steps,
                    "overlap": "two buffer sets: copies of step i overlap kernels of steps i-1 / i+1",
                    "max_diff_vs_device_run": e2e_max_diff},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks, "setup_s": round(setup_s, 1),
        }
        # the paper's effective-throughput figure: 2 * M * (N + n_sal) * B flops per linear over the measured time
        line["effective_tflops"] = eff_flops / (ms_per_step * 1e-3) / 1e12
        if B > 1:
            # Batched launches are bound by shared-memory bandwidth, not HBM: every weight byte costs one table
            # lookup per chunk of vectors, an entry of 4 bytes (fp32) or 2 bytes (fp16) per vector of the chunk.
            fp16 = bool(args.fp16_tables)
            ch = 8 if fp16 else 4
            nvec = lambda nb: 1 if nb == 1 else 2 if nb == 2 else 4 if nb <= 4 else 8
            chunks = [ch] * (B // ch)
            rest = B % ch
            if rest:                                                      # the library's rule for the last chunk
                big = packed_bytes >= (128 << 20)
                first = 2 if (big and not fp16 and rest == 3) else 4 if (big and fp16 and rest in (5, 6)) else rest
                chunks += [first] + ([rest - first] if first < rest else [])
            assert len(chunks) == launches_per_step or args.launch != "stack"
            entry_bytes = sum((2 if (fp16 and nb >= 2) else 4) * nvec(nb) for nb in chunks)
            mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
            sms = torch.cuda.get_device_properties(0).multi_processor_count
            smem_peak = sms * 128 * mhz * 1e6 / 1e9                     # GB/s at 128 B/clk/SM
            smem_achieved = lookups * entry_bytes / (ms_per_step * 1e-3) / 1e9
            line["lookup_ceiling"] = {"bound": "smem", "achieved": smem_achieved, "peak": smem_peak, "unit": "GB/s",
                                      "frac": smem_achieved / smem_peak, "entry_bytes_per_weight_byte": entry_bytes,
                                      "peak_source": f"{sms} SMs x 128 B/clk at the median SM clock under load ({mhz} MHz)"}
        if not args.no_context:
            line["context_dense_fp16_gemv"] = dense_fp16_gemv_context(lins, nl, B)
        if clocks.get("power_w"):
            # board power (largest sample; see ClockSampler) x time: context only, a lower bound for short runs
            line["joules_per_step_lower_bound"] = clocks["power_w"] * ms_per_step * 1e-3
        if not args.no_cpu_baseline:
            y_timed = y_dev.cpu().numpy()                  # outputs of the device-resident steps
            y_offs = np.cumsum([0] + [B * l.M for l in linears])

            def gpu_y(i):
                return y_timed[y_offs[i]:y_offs[i + 1]].reshape(B, linears[i].M)

            gbps, tsec, nbytes, cores, sample, agreement = cpu_oracle_sample(args.config, B, g=args.g, nl=nl, gpu_y=gpu_y)
            line["cpu_baseline"] = {"value": gbps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                                    "seconds": round(tsec, 2), "gpu_vs_oracle_on_sample": agreement}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
