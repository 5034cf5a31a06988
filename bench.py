#!/usr/bin/env python
"""Benchmark of the FluxBin decode linear stack on B200 (one JSON line on stdout).

Headline workload (N=1): the Llama-2-70B-shaped stack of decode linears -- 80 layers x {q, k, v, o, gate,
up, down}, 2 global bases + 1 extra base on a seeded random 5 % of the input columns, g = 128,
batch 1, fp16 activations, every linear with its own input, all 560 packed layers resident in HBM
at once (about 21 GB, far larger than L2, so every step streams the weights from HBM).  A "step" is
one forward token.  --launch says how its 560 linears are launched (replayed from a CUDA graph):
  stack   one fluxbin_plan launch for the whole step (default; the workload gives every linear its own
          input, so all 560 are independent and the persistent kernel streams them back to back: the
          throughput of the kernel, an upper bound for a decoder)
  layer   one plan per layer (80 launches)
  group   one plan per set of linears a decoder could run together: {q,k,v} {o} {gate,up} {down} (320):
          the finest launch structure a real decoder allows; reported in the same line as `group_mode`
  linear  one fluxbin_linear call per linear (560)

value = algorithmic bytes moved per second over all GPUs (GB/s); us_per_layer and us_per_linear
carry the latency side of the metric.  With --gpus N the N ranks run independent replicas (the
path has no exchange step): weak scaling, no collective on the data path.

Beside the headline the line carries (rank 0, one GPU; --sections picks them):
  group_mode  the same stack with one launch per dependency group
  sustained   the headline launch replayed for at least two seconds under the clock sampler
  configs     the smaller workloads (one layer, hybrid layer, 7B set, 13B set) in linear / group / stack mode
              as rotations of copies larger than L2, and the batched cases of the workloads
  variants    the paper's deployed formats at the shapes of its per-operator latency table, one chained call each
  mu_sweep    sub-vector size 4 against 8 on the 7B-shaped set at batch 1, 4, 8 (the paper's sub-vector-size table)
  rc_decomp   the decomposition step (Algorithm 3) on dense matrices
  cpu_baseline, context_dense_fp16_gemv

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
L2_BYTES = 126e6
ALL_SECTIONS = ["group_mode", "sustained", "configs", "variants", "mu_sweep", "rc_decomp", "context", "cpu_baseline"]


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
    """nvidia-smi clocks and throttle reasons sampled every 20 ms while a timed region runs."""
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
                                          "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [t.strip() for t in line.split(",")]))

    def wait_for_samples(self, n: int, timeout: float = 3.0):
        """Block until the sampler has delivered n rows (nvidia-smi takes a while to print its first one)."""
        t0 = time.perf_counter()
        while self.proc is not None and len(self.rows) < n and time.perf_counter() - t0 < timeout:
            time.sleep(0.01)

    def stop(self, since: float | None = None):
        """Summary of the rows sampled after perf_counter() time `since` (all rows if None)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, smax, power, reasons = [], [], [], set()
        for ts, r in self.rows:
            if since is not None and ts < since:
                continue
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
                "sm_mhz_min": min(sm) if sm else None, "samples": len(sm), "reasons": sorted(reasons),
                # nvidia-smi's power.draw is a moving average over about a second: the largest sample of a
                # short timed region is still a lower bound of the power under load
                "power_w": max(power) if power else None}


# ---------------------------------------------------------------------------------------------------------
# resident workloads
# ---------------------------------------------------------------------------------------------------------

def rotation_copies(set_bytes: float) -> int:
    """Copies of a layer / set in rotation so that a step streams more than four times the L2 capacity."""
    return max(1, int(4.3 * L2_BYTES // set_bytes) + 1)


class Stack:
    """Packed linears resident on the device plus activation / output arenas for one batch size.

    members: list of (FluxBinLinear, canonical dims, x fp16 bits [B][N]); `names` the linears of one layer / set in
    order, `nl` how many such layers the members hold (member index = layer * len(names) + linear)."""

    def __init__(self, members, names, nl, B, fp16_tables=False, mu4=False):
        import torch
        from paper_2608_15602_b200 import fluxbin, layer as fb_layer
        self.names, self.nl, self.B, self.fp16, self.mu4 = names, nl, B, bool(fp16_tables and B > 1), bool(mu4)
        self.linears = [m[0] for m in members]
        self.dims = [m[1] for m in members]
        self._fmt_before = [l.weight.table_format() for l in self.linears]
        for l in self.linears:                      # workspaces and plans are sized after the format is set
            l.weight.set_table_format(fluxbin.TABLES_FP32_MU4 if self.mu4 else fluxbin.TABLES_FP16 if self.fp16 else fluxbin.TABLES_FP32)
        self.alg_bytes = [algorithmic_bytes(*d, B) for d in self.dims]
        self.eff_flops = sum(2.0 * d[0] * (d[1] + d[5]) * B for d in self.dims)
        self.lookups = sum(d[2] * d[0] * (d[1] // 8) + d[3] * d[0] * ((d[5] + 7) // 8) for d in self.dims)   # one per weight byte
        self.packed_bytes = sum(l.packed_bytes for l in self.linears)
        n_in = sum(l.N for l in self.linears) * B
        n_out = sum(l.M for l in self.linears) * B
        self.x_host = torch.empty(n_in, dtype=torch.float16).pin_memory()
        self.y_host = torch.empty(n_out, dtype=torch.float16).pin_memory()
        off = 0
        for l, m in zip(self.linears, members):
            self.x_host[off:off + B * l.N] = torch.from_numpy(m[2].view(np.float16).reshape(-1))
            off += B * l.N
        self.x_dev = torch.empty(n_in, dtype=torch.float16, device="cuda")
        self.y_dev = torch.empty(n_out, dtype=torch.float16, device="cuda")
        self.x_dev.copy_(self.x_host)
        self.ws = fb_layer.Workspace(max(l.weight.workspace_size(B) for l in self.linears))
        self.views = self.make_views(self.x_dev, self.y_dev)

    def make_views(self, x_dev, y_dev):
        views, ox, oy, B = [], 0, 0, self.B
        for l in self.linears:
            views.append((l, x_dev[ox:ox + B * l.N].view(B, l.N), y_dev[oy:oy + B * l.M].view(B, l.M)))
            ox += B * l.N
            oy += B * l.M
        return views

    def restore_formats(self):
        for l, f in zip(self.linears, self._fmt_before):
            l.weight.set_table_format(f)

    def groups(self, launch):
        """Member indices per launch; None = one fluxbin_linear call per member."""
        nlin, names = len(self.names), self.names
        if launch == "linear":
            return None
        if launch == "group":
            dep_sets = [["q", "k", "v"], ["o"], ["gate", "up"], ["down"]] if "gate" in names else [[n] for n in names]
            return [[layer * nlin + names.index(n) for n in ds] for layer in range(self.nl) for ds in dep_sets]
        if launch == "layer":
            return [[layer * nlin + li for li in range(nlin)] for layer in range(self.nl)]
        return [list(range(len(self.linears)))]

    def runner(self, launch, stream, views=None, graph=True):
        return Runner(self, launch, stream, views if views is not None else self.views, graph)


class Runner:
    """One step of a stack in a launch mode: plans (or plain calls) captured into a CUDA graph."""

    def __init__(self, stack, launch, stream, views, graph=True):
        import torch
        from paper_2608_15602_b200 import layer as fb_layer
        self.stack, self.launch, self.stream, self.views = stack, launch, stream, views
        groups = stack.groups(launch)
        self.plans = None if groups is None else [fb_layer.FluxBinPlan([views[i] for i in g]) for g in groups]
        if self.plans is not None:
            self.launches_per_step = sum(p.num_launches() for p in self.plans)
        else:
            self.launches_per_step = sum(l.weight.num_launches(stack.B) for l in stack.linears)
        self.graph = None
        with torch.cuda.stream(stream):
            self.issue()                                   # first call per device does the one-time set-up
            stream.synchronize()
            if graph:
                self.graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(self.graph, stream=stream):
                    self.issue()

    def issue(self):
        if self.plans is not None:
            for p in self.plans:
                p.run(stream=self.stream)
        else:
            for l, xv, yv in self.views:
                l.forward(xv, self.stack.ws, out=yv, stream=self.stream)

    def step(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.issue()

    def time(self, steps, warmup, barrier=None):
        """(total ms, per-step ms) of `steps` steps after `warmup` untimed ones, CUDA events on the launch stream."""
        import torch
        with torch.cuda.stream(self.stream):
            for _ in range(warmup):
                self.step()
            (barrier or torch.cuda.synchronize)()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
            ev[0].record(self.stream)
            for i in range(steps):
                self.step()
                ev[i + 1].record(self.stream)
            (barrier or torch.cuda.synchronize)()
        return ev[0].elapsed_time(ev[-1]), [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]


def generate_members(jobs, make, fp16_tables=False):
    """(FluxBinLinear, dims, x) per job; generation runs in a thread pool ahead of packing and upload."""
    from paper_2608_15602_b200 import layer as fb_layer
    members = []
    nthreads = max(1, min(16, (os.cpu_count() or 4) - 1))
    with cf.ThreadPoolExecutor(nthreads) as ex:
        window, it = [], iter(jobs)
        for _ in range(2 * nthreads):
            j = next(it, None)
            if j is not None:
                window.append(ex.submit(make, j))
        while window:
            L, x = window.pop(0).result()
            j = next(it, None)
            if j is not None:
                window.append(ex.submit(make, j))
            lin = fb_layer.FluxBinLinear(L, fp16_tables=fp16_tables)
            members.append((lin, (L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal), x))
            del L
    return members


def build_config_stack(config, nl, B, g=128, fp16_tables=False, mu4=False):
    """Workload `config` with nl independently seeded layers / sets (config 4: the layers of the stack)."""
    lins, _ = synth.config_linears(config)
    jobs = [(layer, li) for layer in range(nl) for li in range(len(lins))]

    def make(job):
        layer, li = job
        return synth.make_config_linear(config, layer, li, g=(g or lins[li][2])), synth.make_config_activations(config, layer, li, B)

    return Stack(generate_members(jobs, make, fp16_tables), [n for n, _, _ in lins], nl, B, fp16_tables, mu4)


def build_rotation(make_layers, names, B, fp16_tables=False, mu4=False):
    """A rotation of copies of one set of layers, enough of them that a step streams more than four times L2.
    The set is generated and packed once; the copies are device-side clones at their own addresses (what the
    memory system sees is the same as with independently seeded copies: every copy is read once per step)."""
    from paper_2608_15602_b200 import layer as fb_layer
    base = []
    for L, x in make_layers():
        lin = fb_layer.FluxBinLinear(L, fp16_tables=fp16_tables)
        base.append((lin, (L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal), x))
    set_bytes = sum(m[0].packed_bytes for m in base)
    copies = rotation_copies(set_bytes)
    members = list(base)
    for _ in range(copies - 1):
        members += [(m[0].clone(), m[1], m[2]) for m in base]
    return Stack(members, names, copies, B, fp16_tables, mu4)


def lookup_ceiling(stack, ms_per_step, launches_per_step, mhz, launch="stack"):
    """Batched launches are bound by shared-memory bandwidth, not HBM: every weight byte costs one table lookup
    per chunk of vectors, an entry of 4 bytes (fp32) or 2 bytes (fp16) per vector of the chunk."""
    import torch
    B, fp16 = stack.B, stack.fp16
    ch = 8 if fp16 else 4
    nvec = lambda nb: 1 if nb == 1 else 2 if nb == 2 else 4 if nb <= 4 else 8
    chunks = [ch] * (B // ch)
    rest = B % ch
    if rest:                                                      # the library's rule for the last chunk
        big = stack.packed_bytes >= (128 << 20)
        first = 2 if (big and not fp16 and rest == 3) else 4 if (big and fp16 and rest in (5, 6)) else rest
        chunks += [first] + ([rest - first] if first < rest else [])
    assert len(chunks) == launches_per_step or launch != "stack"
    entry_bytes = sum((2 if (fp16 and nb >= 2) else 4) * nvec(nb) for nb in chunks) * (2 if stack.mu4 else 1)   # mu = 4: two lookups per byte
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    smem_peak = sms * 128 * mhz * 1e6 / 1e9                     # GB/s at 128 B/clk/SM
    smem_achieved = stack.lookups * entry_bytes / (ms_per_step * 1e-3) / 1e9
    return {"bound": "smem", "achieved": smem_achieved, "peak": smem_peak, "unit": "GB/s",
            "frac": smem_achieved / smem_peak, "entry_bytes_per_weight_byte": entry_bytes,
            "peak_source": f"{sms} SMs x 128 B/clk at {mhz} MHz"}


# ---------------------------------------------------------------------------------------------------------
# baselines and context
# ---------------------------------------------------------------------------------------------------------

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


# ---------------------------------------------------------------------------------------------------------
# the sections beside the headline
# ---------------------------------------------------------------------------------------------------------

def summarize(stack, runner, total_ms, step_ms, steps, peak, per="linear"):
    nbytes = sum(stack.alg_bytes)
    ms = total_ms / steps
    n_lin = len(stack.linears)
    gbps = nbytes / (ms * 1e-3) / 1e9
    out = {"launch": runner.launch, "launches_per_step": runner.launches_per_step, "batch": stack.B,
           "table_entries": "fp32, mu = 4" if stack.mu4 else "fp16" if stack.fp16 else "fp32", "GBps": round(gbps, 1), "frac_of_measured_peak": round(gbps / peak, 4),
           "frac_of_8TBps": round(gbps / 8000.0, 4), "us_per_linear": round(ms * 1e3 / n_lin, 3),
           "us_per_set": round(ms * 1e3 / stack.nl, 3), "ms_per_step": round(ms, 4),
           "step_ms_min": round(min(step_ms), 4), "copies_or_layers": stack.nl,
           "packed_MB_streamed_per_step": round(stack.packed_bytes / 1e6, 1)}
    if stack.B > 1:
        lc = lookup_ceiling(stack, ms, runner.launches_per_step, 1965.0, runner.launch)
        out["lookup_ceiling_frac_at_1965MHz"] = round(lc["frac"], 4)
    return out


def section_configs(main_stack, stream, peak, steps=20, warmup=3):
    """Configs 0-3 at batch 1 in every launch mode, and the batched cases of the workloads."""
    import torch
    rows = []

    def timed(stack, launch):
        r = stack.runner(launch, stream)
        total, step_ms = r.time(steps, warmup)
        row = summarize(stack, r, total, step_ms, steps, peak)
        del r
        return row

    for config in (0, 1, 2, 3):
        lins, _ = synth.config_linears(config)
        names = [n for n, _, _ in lins]

        def make_layers(config=config, lins=lins, B=1):
            return [(synth.make_config_linear(config, 0, li), synth.make_config_activations(config, 0, li, B))
                    for li in range(len(lins))]

        st = build_rotation(make_layers, names, 1)
        for launch in (("linear", "stack") if config < 2 else ("linear", "group", "stack")):
            row = timed(st, launch)
            row["workload"] = f"config {config}"
            rows.append(row)
        del st
        torch.cuda.empty_cache()
        batches = {1: (4, 16), 3: (8,)}.get(config, ())
        for B in batches:
            for fp16 in (False, True):
                st = build_rotation(lambda: make_layers(B=B), names, B, fp16_tables=fp16)
                row = timed(st, "stack")
                row["workload"] = f"config {config}"
                rows.append(row)
                if config == 3:
                    row = timed(st, "group")
                    row["workload"] = f"config {config}"
                    rows.append(row)
                st.restore_formats()
                del st
                torch.cuda.empty_cache()
    # config 4 (the first 16 layers of the resident stack) at batch 4 and 16
    nlin = len(main_stack.names)
    nl16 = min(16, main_stack.nl)
    for B in (4, 16):
        for fp16 in (False, True):
            members = []
            for i in range(nl16 * nlin):
                layer, li = divmod(i, nlin)
                members.append((main_stack.linears[i], main_stack.dims[i], synth.make_config_activations(4, layer, li, B)))
            st = Stack(members, main_stack.names, nl16, B, fp16_tables=fp16)
            for launch in ("stack", "group"):
                row = timed(st, launch)
                row["workload"] = f"config 4, first {nl16} layers"
                rows.append(row)
            st.restore_formats()
            del st
            torch.cuda.empty_cache()
    return {"rows": rows, "how": f"CUDA-graph replay, {warmup} warm-up + {steps} timed steps each, CUDA events; configs 0-3: a step "
            "runs a rotation of device-resident copies of the layer / set at distinct addresses, more than four times L2 "
            "in total, so the weights stream from HBM; linear = one fluxbin_linear call per linear (chained on one stream), "
            "group = one plan per dependency group ({q,k,v} {o} {gate,up} {down}), stack = one plan for all copies "
            "(throughput); frac_of_measured_peak is against the measured copy rate"}


def section_variants(stream, peak, steps=10, warmup=3):
    """The paper's deployed formats (2b, 2b-s8, 2b-s16, 4b at g = 128) at the shapes of its per-operator latency
    table: one chained fluxbin_linear call per copy, copies rotating through more than L2."""
    import torch
    rows = []
    for (M, N) in ((4096, 4096), (5120, 5120), (4096, 11008), (5120, 13824)):
        for variant in ("2b", "2b-s8", "2b-s16", "4b"):
            Kb = 4 if variant == "4b" else 2
            s = {"2b": 0, "4b": 0, "2b-s8": 8, "2b-s16": 16}[variant]

            def make_layers(M=M, N=N, Kb=Kb, s=s):
                idx = synth.salient_per_group(7, 0, N, 128, s) if s else None
                return [(synth.make_linear(7, 0, M, N, Kb, 2 if s else 0, 128, idx), synth.make_activations(7, 0, 1, N))]

            st = build_rotation(make_layers, ["lin"], 1)
            for launch in ("linear", "stack"):
                r = st.runner(launch, stream)
                total, step_ms = r.time(steps, warmup)
                row = summarize(st, r, total, step_ms, steps, peak)
                rows.append({"format": f"{variant}-g128", "shape": f"{M}x{N}", "launch": launch, "us_per_call": row["us_per_linear"],
                             "GBps": row["GBps"], "frac_of_measured_peak": row["frac_of_measured_peak"],
                             "effective_tflops": round(st.eff_flops / (total / steps * 1e-3) / 1e12, 2), "copies": st.nl})
                del r
            del st
            torch.cuda.empty_cache()
    return {"rows": rows, "how": "batch 1; linear = dependent calls chained on one stream (the per-operator latency the paper's "
            "table reports, its kernels on A100: 41-252 us), stack = the same copies as one plan (throughput); effective_tflops = "
            "2 M (N + n_sal) / t as in the paper"}


def section_mu_sweep(stream, peak, steps=10, warmup=3):
    """Sub-vector size mu = 4 against mu = 8 on the LLaMA-2-7B-shaped set in the 2b-g128 format at batch 1, 4 and 8
    (the paper's sub-vector-size table): shared-memory bytes of the lookup tables a CTA holds, and throughput."""
    import torch
    lins = synth.LLAMA2_7B
    names = [n for n, _, _ in lins]
    rows = []
    for B in (1, 4, 8):
        def make_layers(B=B):
            return [(synth.make_linear(9, li, M, N, 2, 0, 128), synth.make_activations(9, li, B, N)) for li, (_, M, N) in enumerate(lins)]

        for mu in (4, 8):
            st = build_rotation(make_layers, names, B, mu4=(mu == 4))
            for launch in ("group", "stack"):
                r = st.runner(launch, stream)
                total, step_ms = r.time(steps, warmup)
                row = summarize(st, r, total, step_ms, steps, peak)
                nb = min(B, 4)                                               # vectors per launch (fp32 entries: chunks of four)
                nvec = 1 if nb == 1 else 2 if nb == 2 else 4
                rows.append({"mu": mu, "batch": B, "launch": launch, "launches_per_step": row["launches_per_step"],
                             "table_KB_per_table_set": (2 * 16 if mu == 4 else 256) * 32 * 4 * nvec // 1024,
                             "GBps": row["GBps"], "frac_of_measured_peak": row["frac_of_measured_peak"],
                             "us_per_set": row["us_per_set"], "sets_per_s": round(1e6 / row["us_per_set"], 1),
                             "lookup_ceiling_frac_at_1965MHz": row.get("lookup_ceiling_frac_at_1965MHz")})
                del r
            st.restore_formats()
            del st
            torch.cuda.empty_cache()
    return {"rows": rows, "how": "fp32 table entries, the same packed layers for both sub-vector sizes; a table set serves 256 columns "
            "(32 slots of 8 columns: mu = 8 one 256-entry table per slot, mu = 4 two 16-entry tables per slot) for the vectors of one launch "
            "(chunks of up to four); group = one plan per dependency group, stack = one plan for all copies; sets_per_s = passes over "
            "the seven linears of one decoder layer per second"}


def section_rc_decomp(shapes=((4096, 4096), (8192, 8192)), K=2, T=10, g=128):
    """fluxbin_rc_decomp (Algorithm 3) on seeded dense matrices: ms per call and the rate at which W is streamed."""
    import torch
    from paper_2608_15602_b200 import fluxbin
    rows = []
    for (M, N) in shapes:
        copies = max(1, int(3 * L2_BYTES // (4 * M * N))) + 1           # W rotates through more than L2
        Ws = [torch.from_numpy(synth.make_dense_weight(11, c, M, N, 0.05)).cuda() for c in range(copies)]
        out = {"bits": torch.empty((K, M, N // 32), dtype=torch.int32, device="cuda"),
               "row_scale": torch.empty((K, M, N // g), dtype=torch.float16, device="cuda"),
               "col_scale": torch.empty((K, N), dtype=torch.float16, device="cuda"),
               "row_scale_f32": torch.empty((K, M, N // g), dtype=torch.float32, device="cuda"),
               "col_scale_f32": torch.empty((K, N), dtype=torch.float32, device="cuda")}
        ws = torch.empty(fluxbin.rc_decomp_workspace_size(M, N, g, K), dtype=torch.uint8, device="cuda")
        stream = int(torch.cuda.current_stream().cuda_stream)

        def call(W):
            fluxbin.rc_decomp(W.data_ptr(), W.stride(0), M, N, g, K, T, 1e-8, out["bits"].data_ptr(),
                              out["row_scale"].data_ptr(), out["col_scale"].data_ptr(), out["row_scale_f32"].data_ptr(),
                              out["col_scale_f32"].data_ptr(), ws.data_ptr(), ws.numel(), stream)

        for W in Ws:
            call(W)
        torch.cuda.synchronize()
        reps = 3
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            for W in Ws:
                call(W)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / (reps * copies)
        passes = fluxbin.rc_decomp_passes(K, T)
        rows.append({"shape": f"{M}x{N}", "g": g, "K": K, "T": T, "ms_per_call": round(ms, 4), "passes_over_W": passes,
                     "us_per_pass": round(ms * 1e3 / passes, 2), "GBps_of_W": round(4.0 * M * N * passes / (ms * 1e-3) / 1e9, 1),
                     "copies": copies})
        del Ws, out, ws
        torch.cuda.empty_cache()
    return {"rows": rows, "how": "CUDA events around whole calls, matrices rotating through more than L2; every pass reads the "
            "fp32 matrix once (4 M N algorithmic bytes)"}


# ---------------------------------------------------------------------------------------------------------

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
    ap.add_argument("--mu", type=int, default=8, choices=[4, 8],
                    help="sub-vector size: 8 (default) or 4 (fluxbin_set_table_format FLUXBIN_TABLES_FP32_MU4: 16-entry tables, twice the lookups)")
    ap.add_argument("--g", type=int, default=128, help="columns per row-scale group; 0 = one scale per row (g = N)")
    ap.add_argument("--no-graph", action="store_true", help="plain launches instead of a CUDA graph replay")
    ap.add_argument("--launch", default="stack", choices=["linear", "group", "layer", "stack"],
                    help="linear: one fluxbin_linear call per linear; group: one plan per set of linears that "
                         "depend on nothing inside the set ({q,k,v}, {o}, {gate,up}, {down}); layer: one plan per "
                         "layer; stack: one plan for the whole stack (valid because the workload gives every "
                         "linear its own input)")
    ap.add_argument("--sections", default=None,
                    help="comma-separated extra sections of the line (default: all at the default workload on one GPU, "
                         f"none otherwise): {','.join(ALL_SECTIONS)}; 'none' for the headline alone")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the dense fp16 cuBLAS GEMV context timing")
    ap.add_argument("--ref-linears", type=int, default=7, help="linears per step of --impl reference")
    ap.add_argument("--rc-shape", default=None, help="MxN: run only the rc_decomp section on this shape (profiling)")
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
    from paper_2608_15602_b200 import dist_util

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    default_workload = (args.config == 4 and args.layers is None and args.batch == 1 and args.g == 128 and args.launch == "stack" and args.mu == 8)
    if args.sections is None:
        sections = list(ALL_SECTIONS) if (default_workload and world == 1) else ["context", "cpu_baseline"]
    else:
        sections = [] if args.sections == "none" else [s for s in args.sections.split(",") if s]
        unknown = [s for s in sections if s not in ALL_SECTIONS]
        if unknown:
            raise SystemExit(f"unknown sections {unknown}")
    if args.no_cpu_baseline and "cpu_baseline" in sections:
        sections.remove("cpu_baseline")
    if args.no_context and "context" in sections:
        sections.remove("context")
    if rank != 0 or world > 1:
        sections = [s for s in sections if s in ("context", "cpu_baseline")] if rank == 0 else []

    if args.rc_shape:
        M, N = (int(t) for t in args.rc_shape.lower().split("x"))
        print(json.dumps({"rc_decomp": section_rc_decomp(shapes=((M, N),))}), flush=True)
        return

    B = args.batch
    lins, nl_default = synth.config_linears(args.config)
    if args.layers is not None:
        nl = args.layers
    elif args.config < 4:
        set_bytes = sum(M * N for _, M, N in lins) * 2.43 / 8          # about 2.43 bits per weight
        nl = rotation_copies(set_bytes)
    else:
        nl = nl_default

    # ---- build the resident stack: generate (threads) -> pack on the host -> upload ----------------
    t_setup = time.perf_counter()
    stack = build_config_stack(args.config, nl, B, g=args.g, fp16_tables=args.fp16_tables, mu4=(args.mu == 4))
    setup_s = time.perf_counter() - t_setup
    stream = torch.cuda.Stream()
    runner = stack.runner(args.launch, stream, graph=not args.no_graph)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing (the sampler runs from before the warm-up: a short timed region alone
    #      would see one or two samples) ----------------------------------------------------------------
    sampler = ClockSampler(local_rank).start()
    sampler.wait_for_samples(1)
    t_load = time.perf_counter()
    total_ms, step_ms = runner.time(args.steps, max(3, args.warmup), barrier)
    clocks = sampler.stop(since=t_load)
    clocks["window"] = "warm-up steps + timed steps"

    # ---- end to end: pinned host x -> device, the stack, y -> pinned host, every step ---------------
    # Two sets of device activation/output buffers alternate, so the copies of one step overlap the kernels
    # of its neighbours (copy-in, compute and copy-out each on a stream of their own, ordered by events);
    # every step still moves its own inputs and outputs inside the timed region.
    x_dev2, y_dev2 = torch.empty_like(stack.x_dev), torch.empty_like(stack.y_dev)
    runner2 = stack.runner(args.launch, stream, views=stack.make_views(x_dev2, y_dev2), graph=not args.no_graph)
    bufs = [(stack.x_dev, stack.y_dev, runner), (x_dev2, y_dev2, runner2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    x_host, y_host = stack.x_host, stack.y_host

    def e2e_steps(n):
        comp_done = [None, None]
        out_done = [None, None]
        for i in range(n):
            k = i & 1
            xd, yd, r = bufs[k]
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
                r.step()
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
    y_ref = stack.y_dev.float().cpu()
    y_got = y_host.float()
    y2_got = y_dev2.float().cpu()
    scale = float(y_ref.abs().max())
    e2e_max_diff = max(float((y_got - y_ref).abs().max()), float((y2_got - y_ref).abs().max())) / max(scale, 1e-30)
    if not (e2e_max_diff < 5e-3 and bool(torch.isfinite(y_got).all()) and scale > 0):
        raise RuntimeError(f"end-to-end outputs differ from the device-resident run: {e2e_max_diff}")
    y_timed = stack.y_dev.cpu().numpy()                  # outputs of the device-resident steps
    del runner2, x_dev2, y_dev2, bufs

    # ---- max over ranks, aggregate ------------------------------------------------------------------
    total_ms, e2e_ms = dist_util.max_over_ranks([total_ms, e2e_ms], device="cuda")
    bytes_per_step = sum(stack.alg_bytes)
    ms_per_step = total_ms / args.steps
    value = dist_util.replica_throughput(bytes_per_step, ms_per_step, world)
    e2e_value = dist_util.replica_throughput(bytes_per_step, e2e_ms / args.steps, world)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        peak = float(peaks["hbm_gbs"])
        achieved = bytes_per_step / (ms_per_step * 1e-3) / 1e9     # one GPU's kernels
        launches_per_step = runner.launches_per_step
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
                       "layers": nl, "linears_per_step": len(stack.linears), "batch": B,
                       "table_entries": "fp32, mu = 4" if stack.mu4 else "fp16" if stack.fp16 else "fp32",
                       "Kb": 2, "Ks": 0 if args.config == 0 else 1, "salient_frac": 0.0 if args.config == 0 else 0.05,
                       "g": args.g or "N", "packed_bytes_resident": stack.packed_bytes, "algorithmic_bytes_per_step": bytes_per_step,
                       "l2": "inputs larger than L2 (weights streamed once per step)" if stack.packed_bytes > 4e8
                       else "working set fits L2: L2-warm number",
                       "launch": ("cuda graph replay" if runner.graph is not None else "plain launches") + f", {args.launch}: "
                       f"{launches_per_step} kernel launches per step"
                       + (" (all linears independent: the throughput of the kernel; see group_mode for the launch "
                          "structure a decoder allows)" if args.launch == "stack" else ""),
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "us_per_layer": ms_per_step * 1e3 / nl, "us_per_linear": ms_per_step * 1e3 / len(stack.linears),
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
        line["effective_tflops"] = stack.eff_flops / (ms_per_step * 1e-3) / 1e12
        if B > 1:
            mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
            line["lookup_ceiling"] = lookup_ceiling(stack, ms_per_step, launches_per_step, mhz, args.launch)
        if clocks.get("power_w"):
            # board power (largest sample; see ClockSampler) x time: context only, a lower bound for short runs
            line["joules_per_step_lower_bound"] = clocks["power_w"] * ms_per_step * 1e-3

        t_sections = time.perf_counter()
        if "sustained" in sections:
            # the headline launch replayed for at least two seconds: the rate the power cap allows
            n_sus = max(args.steps, int(2200.0 / ms_per_step) + 1)
            s2 = ClockSampler(local_rank).start()
            s2.wait_for_samples(1)
            t0 = time.perf_counter()
            tot, sms_ = runner.time(n_sus, 3)
            c2 = s2.stop(since=t0 + 0.5)                 # clocks once the run has settled
            tail = sms_[len(sms_) // 2:]
            ach = bytes_per_step / (statistics.mean(tail) * 1e-3) / 1e9
            line["roofline"]["sustained"] = {
                "steps": n_sus, "seconds": round(tot / 1e3, 2), "achieved": bytes_per_step / (tot / n_sus * 1e-3) / 1e9,
                "achieved_second_half": ach, "frac_second_half": ach / peak, "frac_of_8TBps_second_half": ach / 8000.0,
                "ms_per_step_second_half": statistics.mean(tail), "sm_mhz_median": c2.get("sm_mhz"), "sm_mhz_min": c2.get("sm_mhz_min"),
                "power_w_max": c2.get("power_w"), "reasons": c2.get("reasons"), "clock_samples": c2.get("samples"),
                "ms_times_ghz": statistics.mean(tail) * (c2.get("sm_mhz") or 0) / 1e3,
                "note": "same launch as the headline replayed back to back; after about half a second the board sits at its "
                        "power cap (sw_power_cap) and the SM clock settles below its maximum"}
        if "group_mode" in sections and args.launch != "group" and "gate" in stack.names:
            rg = stack.runner("group", stream)
            sg = ClockSampler(local_rank).start()
            sg.wait_for_samples(1)
            t0 = time.perf_counter()
            tot, sms_ = rg.time(args.steps, max(3, args.warmup))
            cg = sg.stop(since=t0)
            ach = bytes_per_step / (tot / args.steps * 1e-3) / 1e9
            line["group_mode"] = {"launches_per_step": rg.launches_per_step, "ms_per_step": tot / args.steps, "value": ach, "unit": UNIT,
                                  "frac": ach / peak, "frac_of_8TBps": ach / 8000.0, "us_per_launch": tot / args.steps * 1e3 / rg.launches_per_step,
                                  "step_ms_min_median_max": [min(sms_), statistics.median(sms_), max(sms_)], "sm_mhz_median": cg.get("sm_mhz"),
                                  "what": "the same resident stack, one plan per dependency group ({q,k,v} {o} {gate,up} {down}), chained on "
                                          "one stream with programmatic dependent launch, CUDA-graph replay: the launch structure of a real decoder"}
            del rg
        if "configs" in sections:
            line["configs"] = section_configs(stack, stream, peak)
        if "variants" in sections:
            line["variants"] = section_variants(stream, peak)
        if "mu_sweep" in sections:
            line["mu_sweep"] = section_mu_sweep(stream, peak)
        if "rc_decomp" in sections:
            line["rc_decomp"] = section_rc_decomp()
        if "context" in sections:
            line["context_dense_fp16_gemv"] = dense_fp16_gemv_context(lins, nl, B)
        if "cpu_baseline" in sections:
            y_offs = np.cumsum([0] + [B * l.M for l in stack.linears])

            def gpu_y(i):
                return y_timed[y_offs[i]:y_offs[i + 1]].reshape(B, stack.linears[i].M)

            gbps, tsec, nbytes, cores, sample, agreement = cpu_oracle_sample(args.config, B, g=args.g, nl=nl, gpu_y=gpu_y)
            line["cpu_baseline"] = {"value": gbps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                                    "seconds": round(tsec, 2), "gpu_vs_oracle_on_sample": agreement}
        line["sections_s"] = round(time.perf_counter() - t_sections, 1)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
