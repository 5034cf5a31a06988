"""Time fluxbin_rc_decomp on one seeded dense matrix (CUDA events around the whole call, then per pass).

    python -m paper_2608_15602_b200.profile_rc_decomp --shape 4096x4096 --g 128 --K 2 --T 10

Prints one JSON line: ms per call, passes over W per call (1 initialisation + T * (K + 1)), microseconds per
pass, and the rate at which W is streamed (every pass reads the fp32 matrix once: 4*M*N algorithmic bytes; the
sign words and scales add K/32 + ... of that and are not counted)."""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import build, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="4096x4096")
    ap.add_argument("--g", type=int, default=128)
    ap.add_argument("--K", type=int, default=2)
    ap.add_argument("--T", type=int, default=10)
    ap.add_argument("--copies", type=int, default=4, help="distinct matrices rotated through (keeps W out of L2)")
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args()
    build.build()
    from . import layer
    M, N = (int(t) for t in args.shape.lower().split("x"))
    from . import fluxbin
    Ws = [torch.from_numpy(synth.make_dense_weight(11, c, M, N, 0.05)).cuda() for c in range(args.copies)]
    K, g = args.K, args.g
    out = {"bits": torch.empty((K, M, N // 32), dtype=torch.int32, device="cuda"),
           "row_scale": torch.empty((K, M, N // g), dtype=torch.float16, device="cuda"),
           "col_scale": torch.empty((K, N), dtype=torch.float16, device="cuda"),
           "row_scale_f32": torch.empty((K, M, N // g), dtype=torch.float32, device="cuda"),
           "col_scale_f32": torch.empty((K, N), dtype=torch.float32, device="cuda")}
    ws = torch.empty(fluxbin.rc_decomp_workspace_size(M, N, g, K), dtype=torch.uint8, device="cuda")
    stream = int(torch.cuda.current_stream().cuda_stream)

    def call(W):
        fluxbin.rc_decomp(W.data_ptr(), W.stride(0), M, N, g, K, args.T, 1e-8, out["bits"].data_ptr(),
                          out["row_scale"].data_ptr(), out["col_scale"].data_ptr(), out["row_scale_f32"].data_ptr(),
                          out["col_scale_f32"].data_ptr(), ws.data_ptr(), ws.numel(), stream)

    for W in Ws:
        call(W)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.reps):
        for W in Ws:
            call(W)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / (args.reps * args.copies)
    passes = 1 + args.T * (args.K + 1)
    # quality of the last result, from the device outputs
    ar = out["row_scale_f32"].double().repeat_interleave(args.g, dim=2)
    bits = out["bits"].view(torch.int32)
    shifts = torch.arange(32, device="cuda", dtype=torch.int32)
    B = (((bits.unsqueeze(-1) >> shifts) & 1).reshape(args.K, M, N).double() * 2 - 1)
    What = (ar * out["col_scale_f32"].double().unsqueeze(1) * B).sum(dim=0)
    W64 = Ws[-1].double()
    rel = float(((W64 - What) ** 2).sum() / (W64 ** 2).sum())
    print(json.dumps({"shape": [M, N], "g": args.g, "K": args.K, "T": args.T, "ms_per_call": round(ms, 4),
                      "passes_over_W": passes, "us_per_pass": round(ms * 1e3 / passes, 2),
                      "GBps_of_W": round(4.0 * M * N * passes / (ms * 1e-3) / 1e9, 1),
                      "relative_squared_error": rel}))


if __name__ == "__main__":
    main()
