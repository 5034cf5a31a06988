"""GPU parity of plans (many layers in one persistent launch) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2608_15602_b200 import synth
from test_gpu_parity import check, layer_of

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import layer
    return layer


def make_members(fb, specs, B, fp32, shared_x=False):
    members, wants = [], []
    x_shared = None
    for i, (M, N, Kb, Ks, g, n_sal) in enumerate(specs):
        L = layer_of(100 + i, M, N, Kb, Ks, g, n_sal)
        if shared_x and x_shared is not None:
            x = x_shared
        else:
            x = synth.make_activations(7, i, B, N)
            x_shared = x
        lin = fb.FluxBinLinear(L)
        xt = torch.from_numpy(x.view(np.float16)).cuda()
        yt = torch.full((B, M), float("nan"), dtype=torch.float32 if fp32 else torch.float16, device="cuda")
        members.append((lin, xt, yt))
        wants.append(oracle.linear_direct(L, x))
    return members, wants


SPECS = [(300, 1024, 2, 1, 128, 51), (33, 256, 2, 0, 128, 0), (1000, 2048, 2, 2, 128, 100), (64, 256, 3, 1, 128, 7),
         (2100, 384, 2, 1, 128, 19), (1, 128, 1, 0, 128, 0)]


@pytest.mark.parametrize("B", [1, 2, 3, 6])
@pytest.mark.parametrize("fp32", [True, False])
def test_plan_of_mixed_shapes(fb, B, fp32):
    members, wants = make_members(fb, SPECS, B, fp32)
    plan = fb.FluxBinPlan(members)
    assert plan.num_launches() == (B + 3) // 4
    for rep in range(2):                                   # second run reuses the self-cleaning workspace
        for _, _, y in members:
            y.fill_(float("nan"))
        plan.run()
        torch.cuda.synchronize()
        assert int(plan.ws.tensor.count_nonzero()) == 0, "workspace must be left zeroed"
        for (lin, _, y), want in zip(members, wants):
            got = y.float().cpu().numpy()
            if fp32:
                check(got, want, f"plan member M={lin.M} rep {rep}")
            else:
                ulp = np.spacing(np.abs(want).astype(np.float16)).astype(np.float64)
                rms = np.sqrt(np.mean(want ** 2))
                assert np.all(np.abs(got - want) <= 1.01 * ulp + 5e-3 * np.maximum(np.abs(want), 1e-2 * rms))


def test_plan_members_sharing_one_input(fb):
    """q/k/v-style: three layers reading the same activation vector."""
    specs = [(512, 1024, 2, 1, 128, 51), (128, 1024, 2, 1, 128, 51), (128, 1024, 2, 1, 128, 51)]
    members, wants = make_members(fb, specs, 1, True, shared_x=True)
    x0 = members[0][1]
    members = [(lin, x0, y) for lin, _, y in members]
    plan = fb.FluxBinPlan(members)
    plan.run()
    torch.cuda.synchronize()
    for (lin, _, y), want in zip(members, wants):
        check(y.cpu().numpy(), want, "shared input")


def test_plan_equals_single_calls_on_a_70b_layer(fb):
    """All seven linears of one Llama-2-70B-shaped layer in one plan vs. the oracle (batch 1)."""
    members, wants = [], []
    for li in range(7):
        L = synth.make_config_linear(4, 1, li)
        x = synth.make_config_activations(4, 1, li, 1)
        lin = fb.FluxBinLinear(L)
        members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                        torch.empty((1, L.M), dtype=torch.float32, device="cuda")))
        wants.append(oracle.linear_direct(L, x))
        del L
    plan = fb.FluxBinPlan(members)
    plan.run()
    torch.cuda.synchronize()
    for (lin, _, y), want in zip(members, wants):
        check(y.cpu().numpy(), want, f"70B member {lin.M}x{lin.N}")


def test_long_plan_runs_the_two_pair_kernel(fb):
    """A plan whose shares span whole couples of pairs launches the kernel variant that keeps two table sets
    resident and reduces two pairs' row sums at once (the variant the full-stack benchmark times); a short
    plan of the same members launches the one-pair variant.  Both must match the oracle on every output."""
    shapes = [(256, 4096), (250, 4096), (512, 4096), (96, 8192)]
    members, wants = [], []
    for i in range(120):
        M, N = shapes[i % len(shapes)]
        n_sal = int(round(0.05 * N))
        L = layer_of(500 + i, M, N, 2, 1, 128, n_sal)
        x = synth.make_activations(9, i, 1, N)
        lin = fb.FluxBinLinear(L)
        members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                        torch.full((1, M), float("nan"), dtype=torch.float32, device="cuda")))
        wants.append(oracle.linear_direct(L, x))
    long_plan = fb.FluxBinPlan(members)
    assert long_plan.pairs_per_row_block() == 2
    for _ in range(2):                      # twice: the workspace must come back zeroed
        for _, _, y in members:
            y.fill_(float("nan"))
        long_plan.run()
        torch.cuda.synchronize()
        for (lin, _, y), want in zip(members, wants):
            check(y.cpu().numpy(), want, f"two-pair kernel, member {lin.M}x{lin.N}")
    short_plan = fb.FluxBinPlan(members[:4])
    assert short_plan.pairs_per_row_block() == 1
    for _, _, y in members[:4]:
        y.fill_(float("nan"))
    short_plan.run()
    torch.cuda.synchronize()
    for (lin, _, y), want in zip(members[:4], wants[:4]):
        check(y.cpu().numpy(), want, f"one-pair kernel, member {lin.M}x{lin.N}")


def test_plan_rejects_mixed_scale_formats_and_bad_buffers(fb):
    from paper_2608_15602_b200 import fluxbin
    a = fb.FluxBinLinear(layer_of(1, 64, 256, 2, 0, 128, 0))
    b = fb.FluxBinLinear(layer_of(2, 64, 256, 2, 0, 64, 0))       # row-scale groups of 64: other format class
    x = torch.zeros((1, 256), dtype=torch.float16, device="cuda")
    ya = torch.zeros((1, 64), dtype=torch.float16, device="cuda")
    yb = torch.zeros((1, 64), dtype=torch.float16, device="cuda")
    tb = fluxbin.plan_table_bytes(2, 1)
    table = torch.zeros(tb, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    args = ([x.data_ptr()] * 2, [256, 256], [ya.data_ptr(), yb.data_ptr()], [64, 64], 1, False)
    st, _ = fluxbin.plan_create_status([a.weight, b.weight], *args, table.data_ptr(), tb, ws.data_ptr(), 1 << 16)
    assert st == 7
    st, _ = fluxbin.plan_create_status([a.weight, a.weight], *args, table.data_ptr(), tb - 1, ws.data_ptr(), 1 << 16)
    assert st == 5
    st, _ = fluxbin.plan_create_status([a.weight, a.weight], *args, table.data_ptr(), tb, ws.data_ptr(), 64)
    assert st == 5
    st, h = fluxbin.plan_create_status([a.weight, a.weight], *args, table.data_ptr(), tb, ws.data_ptr(), 1 << 16)
    assert st == 0
    fluxbin.library().fluxbin_plan_free(h)


@pytest.mark.parametrize("B,fp16,launches", [(3, False, 2), (7, False, 3), (5, True, 2), (6, True, 2), (13, True, 3), (7, True, 1)])
def test_large_plans_cut_a_rest_with_dead_vectors_once_more(fb, B, fp16, launches):
    """A plan that streams at least 128 MiB of packed weights runs a rest of 3 vectors (fp32 entries) as 2 + 1 and a
    rest of 5 or 6 vectors (fp16 entries) as 4 + 1 / 4 + 2; every batch row must still come out right."""
    from test_gpu_fp16_tables import check_fp16_tables
    members, cases, nbytes = [], [], 0
    for i in range(4):
        L = synth.make_config_linear(4, 1, 4)                    # 28672 x 8192: 65 MB packed each
        x = synth.make_activations(23, i, B, L.N)
        lin = fb.FluxBinLinear(L, fp16_tables=fp16)
        nbytes += lin.packed_bytes
        members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                        torch.full((B, L.M), float("nan"), dtype=torch.float32, device="cuda")))
        if i == 0:
            cases.append((L, x, oracle.linear_direct(L, x)))
    assert nbytes >= 128 << 20
    plan = fb.FluxBinPlan(members)
    assert plan.num_launches() == launches
    assert members[0][0].weight.num_launches(B) == ((B + 7) // 8 if fp16 else (B + 3) // 4), "one layer alone stays below the threshold"
    for rep in range(2):
        for _, _, y in members:
            y.fill_(float("nan"))
        plan.run()
        torch.cuda.synchronize()
        assert int(plan.ws.tensor.count_nonzero()) == 0, "workspace must be left zeroed"
        for _, _, y in members:
            assert bool(torch.isfinite(y).all()), "every batch row of every member is written"
        L, x, want = cases[0]
        got = members[0][2].cpu().numpy()
        if fp16:
            check_fp16_tables(got, want, L, x, f"B={B} rep {rep}", strict=True)
        else:
            check(got, want, f"B={B} rep {rep}")
        # the four members hold the same layer: same weights, different activations -> rows must differ between members
        assert not torch.equal(members[0][2], members[1][2])


@pytest.mark.parametrize("B,fp32", [(1, True), (1, False), (3, True), (8, False)])
def test_gated_pairs_write_silu_gate_times_up(fb, B, fp32):
    """fluxbin_plan_create_gated: y = silu(W_gate x) * (W_up x) written once by whoever completes a row tile of both
    layers, against the oracle's two results combined in fp64; an unpaired member of the same plan is unaffected and
    the workspace (both layers' accumulators, the shared tickets) comes back zeroed."""
    specs = [(11008, 4096, 2, 1, 128, 205), (11008, 4096, 2, 1, 128, 205),      # gate, up of a 7B-shaped block
             (300, 1024, 2, 1, 128, 51),                                         # an ordinary member in between
             (777, 512, 2, 0, 128, 0), (777, 512, 3, 2, 128, 40)]                # a ragged pair with different base counts
    Ls = [layer_of(500 + i, *sp) for i, sp in enumerate(specs)]
    xs = [synth.make_activations(31, 0, B, 4096), None, synth.make_activations(31, 2, B, 1024),
          synth.make_activations(31, 3, B, 512), synth.make_activations(31, 4, B, 512)]
    xs[1] = xs[0]                                                                # gate and up read the same input
    lins = [fb.FluxBinLinear(L) for L in Ls]
    xt = [torch.from_numpy(x.view(np.float16)).cuda() for x in xs]
    dt = torch.float32 if fp32 else torch.float16
    ys = [torch.full((B, L.M), float("nan"), dtype=dt, device="cuda") for L in Ls]
    gate_up = [(0, 1), (4, 3)]                                                   # second pair: member 4 gates member 3
    members = [(lins[i], xt[i], None if i in (1, 3) else ys[i]) for i in range(5)]
    plan = fb.FluxBinPlan(members, gate_up=gate_up)
    want = [oracle.linear_direct(L, x) for L, x in zip(Ls, xs)]
    silu = lambda t: t / (1.0 + np.exp(-t))
    for rep in range(2):
        for i in (0, 2, 4):
            ys[i].fill_(float("nan"))
        plan.run()
        torch.cuda.synchronize()
        assert int(plan.ws.tensor.count_nonzero()) == 0, "plan workspace must be left zeroed"
        got = [y.float().cpu().numpy() for y in ys]
        tol = dict() if fp32 else dict()
        for g, u in gate_up:
            expect = silu(want[g]) * want[u]
            if fp32:
                check(got[g], expect, f"gated pair ({g},{u}) B={B} run {rep}")
            else:
                y = got[g].astype(np.float64)
                for b in range(B):
                    rms = np.sqrt(np.mean(expect[b] ** 2))
                    assert np.linalg.norm(y[b] - expect[b]) / np.linalg.norm(expect[b]) <= 1e-3
                    assert (np.abs(y[b] - expect[b]) / np.maximum(np.abs(expect[b]), 1e-2 * rms)).max() <= 5e-3 + 2.0 ** -11
        if fp32:
            check(got[2], want[2], "unpaired member")
        assert np.isnan(ys[1].float().cpu().numpy()).all() and np.isnan(ys[3].float().cpu().numpy()).all(), "up members have no output"


def test_gated_plan_argument_errors(fb):
    from paper_2608_15602_b200 import fluxbin
    a = fb.FluxBinLinear(layer_of(1, 64, 256, 2, 0, 128, 0))
    b = fb.FluxBinLinear(layer_of(2, 64, 256, 2, 0, 128, 0))
    c = fb.FluxBinLinear(layer_of(3, 96, 256, 2, 0, 128, 0))           # another row count
    x = torch.zeros((1, 256), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 96), dtype=torch.float16, device="cuda")
    tb = fluxbin.plan_table_bytes(3, 1)
    table = torch.zeros(tb, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    ws_args = (1, False, table.data_ptr(), tb, ws.data_ptr(), 1 << 16)
    ptrs = ([x.data_ptr()] * 3, [256] * 3, [y.data_ptr(), None, y.data_ptr()], [96, 0, 96])
    W = [a.weight, b.weight, c.weight]
    assert fluxbin.plan_create_gated_status(W, *ptrs, [(0, 2)], *ws_args)[0] == 2        # 64 rows against 96
    assert fluxbin.plan_create_gated_status(W, *ptrs, [(0, 0)], *ws_args)[0] == 3        # a member with itself
    assert fluxbin.plan_create_gated_status(W, *ptrs, [(0, 1), (1, 2)], *ws_args)[0] == 3  # member 1 twice
    assert fluxbin.plan_create_gated_status(W, *ptrs, [(0, 5)], *ws_args)[0] == 3        # no such member
    assert fluxbin.plan_create_gated_status(W, *ptrs, [(1, 0)], *ws_args)[0] == 1        # the gate (member 1) has no output buffer
    st, h = fluxbin.plan_create_gated_status(W, *ptrs, [(0, 1)], *ws_args)
    assert st == 0
    fluxbin.library().fluxbin_plan_free(h)
