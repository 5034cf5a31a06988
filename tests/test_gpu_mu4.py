"""GPU parity of the mu = 4 launch modes (FLUXBIN_TABLES_FP32_MU4: two 16-entry tables per byte of weight bits
instead of one 256-entry table, the paper's sub-vector-size study) against the CPU oracle, element by element
through the C-ABI.  The packed layer is the one the mu = 8 path reads; only the table shape and the lookups differ,
so the results agree with the oracle within the same fp32-level bounds as the mu = 8 path (a chain of up to 32
entry adds per row-scale segment instead of 9 when four vectors share an entry: 12 more roundings)."""
import numpy as np
import pytest

import oracle
from paper_2608_15602_b200 import synth
from test_gpu_parity import check, layer_of

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

EXTRA = 12


@pytest.fixture(scope="module")
def fb():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import layer
    return layer


def mu4_linear(fb, L):
    from paper_2608_15602_b200 import fluxbin
    lin = fb.FluxBinLinear(L)
    lin.weight.set_table_format(fluxbin.TABLES_FP32_MU4)
    assert lin.weight.table_format() == fluxbin.TABLES_FP32_MU4
    return lin


def run_mu4(fb, L, x_bits, fp32=True):
    lin = mu4_linear(fb, L)
    B = x_bits.shape[0]
    xt = torch.from_numpy(x_bits.view(np.float16)).cuda()
    ws = lin.workspace(B)
    outs = []
    for rep in range(2):                                 # the second call reuses the workspace the first one left
        y = lin.forward(xt, ws, fp32_out=fp32)
        torch.cuda.synchronize()
        assert int(ws.tensor.count_nonzero()) == 0, "workspace must be left zeroed"
        outs.append(y.float().cpu().numpy())
    rtol = 1e-4 if fp32 else 2e-3
    assert np.allclose(outs[0], outs[1], rtol=rtol, atol=rtol * 0.1 * np.abs(outs[0]).max())
    return outs[0]


#          M,    N,  Kb, Ks, g,  n_sal
SHAPES = [(1, 128, 1, 0, 128, 0),
          (33, 384, 3, 2, 128, 40),          # odd number of units, two salient bases
          (100, 256, 1, 1, 256, 19),         # g = 256
          (127, 1024, 2, 1, 128, 51),        # narrow last salient pair (16 slots)
          (1000, 512, 2, 1, 512, 1),         # g = N, narrow last pair (8 slots)
          (65, 640, 2, 1, 128, 640),         # every column salient
          (600, 2048, 2, 2, 128, 128),
          (2100, 384, 2, 0, 128, 0),
          (257, 1024, 4, 0, 128, 0)]         # four bases


@pytest.mark.parametrize("M,N,Kb,Ks,g,n_sal", SHAPES)
@pytest.mark.parametrize("B", [1, 2, 3, 4, 7])
def test_small_and_ragged_shapes(fb, M, N, Kb, Ks, g, n_sal, B):
    L = layer_of(M * 5 + N + B, M, N, Kb, Ks, g, n_sal)
    x = synth.make_activations(13, M + B, B, N)
    check(run_mu4(fb, L, x), oracle.linear_direct(L, x), f"mu4 {(M, N, Kb, Ks, g, n_sal, B)}", L, x, extra_roundings=EXTRA)


def test_fp16_outputs(fb):
    L = layer_of(3, 300, 768, 2, 1, 128, 30)
    x = synth.make_activations(14, 3, 5, 768)
    want = oracle.linear_direct(L, x)
    got = run_mu4(fb, L, x, fp32=False)
    ulp = np.spacing(np.abs(want).astype(np.float16)).astype(np.float64)
    rms = np.sqrt(np.mean(want ** 2))
    assert np.all(np.abs(got - want) <= 1.01 * ulp + 5e-3 * np.maximum(np.abs(want), 1e-2 * rms))


@pytest.mark.parametrize("cfg,B", [(0, 1), (1, 1), (1, 4), (1, 8), (2, 1)])
def test_workload_layers(fb, cfg, B):
    """the 4096 x 4096, hybrid 4096 x 4096 and 11008-wide layers of the workloads (2b-g128, with and without salient columns)"""
    L = synth.make_config_linear(cfg, 0, 0)
    x = synth.make_config_activations(cfg, 0, 0, B)
    check(run_mu4(fb, L, x), oracle.linear_direct(L, x), f"config {cfg} B={B}", L, x, extra_roundings=EXTRA)


def test_longest_k_split_of_the_70b_stack(fb):
    """down of the 70B-shaped stack: 8192 x 28672, the longest K split (224 units)"""
    names = [n for n, _, _ in synth.LLAMA2_70B]
    L = synth.make_config_linear(4, 0, names.index("down"))
    x = synth.make_config_activations(4, 0, names.index("down"), 4)
    check(run_mu4(fb, L, x), oracle.linear_direct(L, x), "70B down B=4", L, x, extra_roundings=EXTRA)


def test_plan_of_mu4_members_and_gated_pair(fb):
    """q, k, v sharing x plus a gated {gate, up} pair in one persistent launch, all members with mu = 4 tables"""
    dims = [(512, 1024), (128, 1024), (128, 1024), (1408, 1024), (1408, 1024)]
    Ls = [layer_of(50 + i, M, N, 2, 1, 128, 20) for i, (M, N) in enumerate(dims)]
    lins = [mu4_linear(fb, L) for L in Ls]
    for B in (1, 3):
        x = synth.make_activations(15, B, B, 1024)
        xt = torch.from_numpy(x.view(np.float16)).cuda()
        ys = [torch.empty((B, M), dtype=torch.float32, device="cuda") for M, _ in dims]
        members = [(lin, xt, y) for lin, y in zip(lins, ys)]
        members[4] = (lins[4], xt, None)
        plan = fb.FluxBinPlan(members, gate_up=[(3, 4)])
        for rep in range(2):
            plan.run()
            torch.cuda.synchronize()
            assert int(plan.ws.tensor.count_nonzero()) == 0
            for i in range(3):
                check(ys[i].cpu().numpy(), oracle.linear_direct(Ls[i], x), f"plan member {i} B={B}", Ls[i], x, extra_roundings=EXTRA)
            g, u = oracle.linear_direct(Ls[3], x), oracle.linear_direct(Ls[4], x)
            want = g / (1.0 + np.exp(-g)) * u
            got = ys[3].cpu().numpy().astype(np.float64)
            rms = np.sqrt(np.mean(want ** 2))
            assert np.all(np.abs(got - want) <= 1e-4 * np.maximum(np.abs(want), rms))


def test_format_rules(fb):
    from paper_2608_15602_b200 import fluxbin
    # scale groups of 32 or 64 columns have no mu = 4 kernel
    for g in (32, 64):
        lin = fb.FluxBinLinear(layer_of(g, 40, 256, 2, 0, g, 0))
        with pytest.raises(fluxbin.FluxBinError):
            lin.weight.set_table_format(fluxbin.TABLES_FP32_MU4)
        assert lin.weight.table_format() == fluxbin.TABLES_FP32
    # members of a plan must agree on the format
    La, Lb = layer_of(1, 64, 256, 2, 0, 128, 0), layer_of(2, 64, 256, 2, 0, 128, 0)
    a, b = mu4_linear(fb, La), fb.FluxBinLinear(Lb)
    xt = torch.zeros((1, 256), dtype=torch.float16, device="cuda")
    ys = [torch.empty((1, 64), dtype=torch.float32, device="cuda") for _ in range(2)]
    with pytest.raises(fluxbin.FluxBinError):
        fb.FluxBinPlan([(a, xt, ys[0]), (b, xt, ys[1])])
    # back to the default format the same handle runs the mu = 8 path again
    x = synth.make_activations(16, 1, 2, 256)
    xt2 = torch.from_numpy(x.view(np.float16)).cuda()
    a.weight.set_table_format(fluxbin.TABLES_FP32)
    y = a.forward(xt2, a.workspace(2), fp32_out=True)
    torch.cuda.synchronize()
    check(y.cpu().numpy(), oracle.linear_direct(La, x), "back to mu = 8", La, x)
