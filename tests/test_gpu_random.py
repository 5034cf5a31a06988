"""Seeded random sweep of the GPU path against the oracle: shapes, group sizes, base counts, salient maps and batch
sizes drawn at random (single calls), and random plans long enough to reach both kernel variants."""
import numpy as np
import pytest

import oracle
from paper_2608_15602_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from test_gpu_parity import check, fb, run  # noqa: E402,F401  (same tolerances and call helper)


def random_layer(r, seed, max_m=300, max_n=1024):
    N = int(r.integers(1, max_n // 32 + 1)) * 32
    groups = [g for g in (32, 64, 96, 128, 256, 512, N) if N % g == 0]
    g = int(r.choice(groups))
    M = int(r.integers(1, max_m + 1))
    Kb = int(r.integers(1, 5))
    Ks = int(r.integers(0, 3))
    mode = int(r.integers(0, 4))
    if Ks == 0 or mode == 0:
        idx = np.zeros(0, np.int32)
    elif mode == 1:
        idx = synth.salient_random(seed, 1, N, float(r.uniform(0.01, 0.3)))
    elif mode == 2:
        idx = np.arange(N, dtype=np.int32)                                   # every column salient
    else:
        G = int(r.integers(0, N // g))                                        # all salient columns in one group
        idx = np.sort(r.choice(g, size=int(r.integers(1, g + 1)), replace=False)).astype(np.int32) + G * g
    return synth.make_linear(seed, 2, M, N, Kb, Ks, g, idx)


@pytest.mark.parametrize("case", range(24))
def test_random_single_calls(fb, case):
    r = np.random.default_rng(260815602 + 1000 + case)
    L = random_layer(r, 5000 + case)
    B = int(r.integers(1, 7))
    x = synth.make_activations(5000 + case, 3, B, L.N, outlier_frac=float(r.choice([0.0, 0.02])))
    check(run(fb, L, x), oracle.linear_direct(L, x), f"case {case}: M={L.M} N={L.N} g={L.g} Kb={L.Kb} Ks={L.Ks} n_sal={L.n_sal} B={B}")


@pytest.mark.parametrize("case", range(4))
def test_random_plans(fb, case):
    r = np.random.default_rng(260815602 + 2000 + case)
    n = int(r.choice([3, 12, 40, 90]))
    g = 128
    members, wants = [], []
    for i in range(n):
        M = int(r.integers(1, 400))
        # (N > g: a layer with a single row-scale group is a format class of its own and cannot share a plan)
        N = int(r.integers(2, 9)) * 128 * (4 if case >= 2 else 1)             # cases 2, 3: wide layers, long runs
        Ks = int(r.integers(0, 2))
        idx = synth.salient_random(7000 + case, i, N, 0.05) if Ks else np.zeros(0, np.int32)
        L = synth.make_linear(7000 + case, i, M, N, 2, Ks, g, idx)
        x = synth.make_activations(7000 + case, 100 + i, 1, N)
        lin = fb.FluxBinLinear(L)
        members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                        torch.full((1, M), float("nan"), dtype=torch.float32, device="cuda")))
        wants.append(oracle.linear_direct(L, x))
    plan = fb.FluxBinPlan(members)
    for _ in range(2):
        for _, _, y in members:
            y.fill_(float("nan"))
        plan.run()
        torch.cuda.synchronize()
        for (lin, _, y), want in zip(members, wants):
            check(y.cpu().numpy(), want, f"plan case {case} ({n} members, {plan.pairs_per_row_block()} pairs per row block) {lin.M}x{lin.N}")
