"""GPU parity at the benchmark's sizes and launch configuration: a run of Llama-2-70B-shaped layers (full
8192 / 28672-wide linears, 2 + 1 bases, 5 % salient columns, g = 128, batch 1, fp16 outputs) as ONE plan --
the launch `bench.py` times, which selects the two-pairs-per-row-block kernel -- checked against the CPU oracle
on sampled linears (one of every shape, spread over the layers, every output of each) and, for all other
linears, against properties that hold at any size.
"""
import numpy as np
import pytest

import oracle
from paper_2608_15602_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

LAYERS = 8            # enough cost per CTA for the host to pick the two-pair kernel (asserted below)
REL_L2 = 1e-3
MAX_REL = 5e-3


def check_fp16(y_half, want, what):
    """fp16 output against the fp64 oracle: the fp32 tolerances plus half an fp16 ulp of rounding."""
    y = y_half.astype(np.float64)
    for b in range(want.shape[0]):
        rms = np.sqrt(np.mean(want[b] ** 2))
        l2 = np.linalg.norm(y[b] - want[b]) / np.linalg.norm(want[b])
        rel = np.abs(y[b] - want[b]) / np.maximum(np.abs(want[b]), 1e-2 * rms)
        assert l2 <= REL_L2, f"{what}: rel L2 {l2:.3e}"
        assert rel.max() <= MAX_REL + 2.0 ** -11, f"{what}: max rel {rel.max():.3e} at {rel.argmax()}"


def test_stack_plan_at_benchmark_sizes():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import layer as fb

    lins, _ = synth.config_linears(4)
    sampled = {(li * 3 + 1) % LAYERS: li for li in range(len(lins))}        # layer -> linear checked in full there
    sampled = {(layer, li) for layer, li in sampled.items()}
    assert len(sampled) == len(lins)
    members, wants, stats = [], {}, {}
    for layer in range(LAYERS):
        for li, (name, M, N) in enumerate(lins):
            L = synth.make_config_linear(4, layer, li)
            x = synth.make_config_activations(4, layer, li, 1)
            lin = fb.FluxBinLinear(L)
            members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                            torch.full((1, M), float("nan"), dtype=torch.float16, device="cuda")))
            if (layer, li) in sampled:
                wants[(layer, li)] = oracle.linear_direct(L, x)
            # expected scale of every output of this linear (the bits are independent fair signs):
            # var(y_i) = sum_k sum_j (alpha_r * alpha_c * x)^2
            xs = x.view(np.float16).astype(np.float64)[0] ** 2
            ac = L.col_scale.view(np.float16).astype(np.float64) ** 2                       # [Kb][N]
            ar = L.row_scale.view(np.float16).astype(np.float64) ** 2                       # [Kb][M][N/g]
            per_group = (ac * xs[None, :]).reshape(L.Kb, N // L.g, L.g).sum(axis=2)         # [Kb][N/g]
            stats[(layer, li)] = float(np.sqrt(np.einsum("kmg,kg->m", ar, per_group).mean()))
            del L
    plan = fb.FluxBinPlan(members)
    assert plan.pairs_per_row_block() == 2, "this many layers must select the kernel variant the benchmark times"
    assert plan.num_launches() == 1
    for rep in range(2):                     # twice: the workspace must come back zeroed
        for _, _, y in members:
            y.fill_(float("nan"))
        plan.run()
        torch.cuda.synchronize()
        for idx, (lin, _, y) in enumerate(members):
            layer, li = divmod(idx, len(lins))
            got = y.cpu().numpy()
            assert np.isfinite(got).all(), f"layer {layer} linear {li}: unwritten or non-finite outputs"
            if (layer, li) in wants:
                check_fp16(got, wants[(layer, li)], f"run {rep} layer {layer} {lins[li][0]} {lin.M}x{lin.N}")
            else:
                # any size: the root mean square of the outputs matches the scale the inputs imply (the
                # salient base adds a few per cent on top of the global bases counted here)
                rms = float(np.sqrt(np.mean(got.astype(np.float64) ** 2)))
                assert 0.9 * stats[(layer, li)] <= rms <= 1.25 * stats[(layer, li)], \
                    f"layer {layer} linear {li}: rms {rms:.4g} vs expected {stats[(layer, li)]:.4g}"
