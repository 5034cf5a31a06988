"""Time (and give ncu something small to capture) one linear shape of a workload.

    python -m paper_2608_15602_b200.profile_case --config 4 --linear 4 --copies 3 --reps 5

builds `copies` distinct packed layers of that shape (different seeded layers, so together they
can exceed L2), replays a CUDA graph of one fluxbin_linear call per copy `reps` times and prints
the mean time per call from CUDA events, the algorithmic bytes and the resulting GB/s.
--variant/--shape time the paper's deployed formats (2b, 2b-s8, 2b-s16, 4b at g = 128) instead.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import build, synth


def algorithmic_bytes(L, B):
    w = L.Kb * L.M * L.N // 8 + 2 * L.Kb * L.M * (L.N // L.g) + 2 * L.Kb * L.N
    if L.Ks > 0 and L.n_sal > 0:
        w += L.Ks * L.M * ((L.n_sal + 7) // 8) + 2 * L.Ks * L.M * (L.N // L.g) + 2 * L.Ks * L.n_sal + 2 * L.n_sal
    return w + 2 * B * L.N + 2 * B * L.M


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--linear", type=int, default=4, help="index into the layer's linears (config 4: 0=q 1=k 4=gate 6=down)")
    ap.add_argument("--copies", type=int, default=3)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--fp16-tables", action="store_true", help="fp16 lookup-table entries for batched launches")
    ap.add_argument("--g", type=int, default=128)
    ap.add_argument("--variant", default=None, choices=["2b", "2b-s8", "2b-s16", "4b"],
                    help="one of the paper's deployed formats at --shape MxN instead of a workload linear: "
                         "2 or 4 global bases; s8/s16 = exactly 8/16 salient columns per group with 2 extra bases")
    ap.add_argument("--shape", default="4096x4096", help="MxN for --variant")
    args = ap.parse_args()
    build.build()
    from . import layer as fb_layer

    lins = []
    for c in range(args.copies):
        if args.variant:
            M, N = (int(t) for t in args.shape.lower().split("x"))
            Kb = 4 if args.variant == "4b" else 2
            s_per_group = {"2b": 0, "4b": 0, "2b-s8": 8, "2b-s16": 16}[args.variant]
            idx = synth.salient_per_group(7, c, N, args.g, s_per_group) if s_per_group else None
            L = synth.make_linear(7, c, M, N, Kb, 2 if s_per_group else 0, args.g, idx)
            x = synth.make_activations(7, c, args.batch, N)
        else:
            L = synth.make_config_linear(args.config, c, args.linear, g=args.g)
            x = synth.make_config_activations(args.config, c, args.linear, args.batch)
        lin = fb_layer.FluxBinLinear(L, fp16_tables=args.fp16_tables)
        xt = torch.from_numpy(x.view(np.float16)).cuda()
        y = torch.empty((args.batch, L.M), dtype=torch.float16, device="cuda")
        lins.append((lin, xt, y))
        nbytes = algorithmic_bytes(L, args.batch)
        dims = (L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal)
    ws = lins[0][0].workspace(args.batch)
    stream = torch.cuda.current_stream()
    for lin, xt, y in lins:                      # one warm-up pass
        lin.forward(xt, ws, out=y)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()                # plain launches pay Python's call overhead; replay a graph
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for lin, xt, y in lins:
                lin.forward(xt, ws, out=y, stream=side)
        graph.replay()
        side.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(side)
        for _ in range(args.reps):
            graph.replay()
        b.record(side)
        side.synchronize()
    us = a.elapsed_time(b) * 1e3 / (args.reps * len(lins))
    print(json.dumps({"dims_M_N_Kb_Ks_g_nsal": dims, "batch": args.batch, "copies": args.copies, "us_per_call": round(us, 2),
                      "algorithmic_bytes": nbytes, "GBps": round(nbytes / us / 1e3, 1),
                      "packed_bytes": lins[0][0].packed_bytes}))


if __name__ == "__main__":
    main()
