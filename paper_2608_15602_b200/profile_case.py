"""Time (and give ncu something small to capture) one linear shape of a workload.

    python -m paper_2608_15602_b200.profile_case --config 4 --linear 4 --copies 3 --reps 5

builds `copies` distinct packed layers of that shape (different seeded layers, so together they
exceed L2), runs them round-robin `reps` times with plain launches and prints the mean time per
call from CUDA events, the algorithmic bytes and the resulting GB/s.
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
    ap.add_argument("--g", type=int, default=128)
    args = ap.parse_args()
    build.build()
    from . import layer as fb_layer

    lins = []
    for c in range(args.copies):
        L = synth.make_config_linear(args.config, c, args.linear, g=args.g)
        x = synth.make_config_activations(args.config, c, args.linear, args.batch)
        lin = fb_layer.FluxBinLinear(L)
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
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.reps):
        for lin, xt, y in lins:
            lin.forward(xt, ws, out=y)
    b.record(stream)
    torch.cuda.synchronize()
    us = a.elapsed_time(b) * 1e3 / (args.reps * len(lins))
    print(json.dumps({"dims_M_N_Kb_Ks_g_nsal": dims, "batch": args.batch, "copies": args.copies, "us_per_call": round(us, 2),
                      "algorithmic_bytes": nbytes, "GBps": round(nbytes / us / 1e3, 1),
                      "packed_bytes": lins[0][0].packed_bytes}))


if __name__ == "__main__":
    main()
