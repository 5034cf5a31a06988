"""GPU parity for the combinations the workloads and the paper's tables name beyond the single-layer tests:

* the Llama-2-70B-shaped plan at batch 4 and 16 (fp32 table entries, the default): two layers in one plan,
  every output and every batch row of one linear of each of the four shapes (8192 x 8192, 1024 x 8192,
  28672 x 8192 and 8192 x 28672, the longest K split) against the oracle, the rest against the scale property;
* the Llama-2-13B-shaped gate projection (13824 x 5120) at batch 8;
* the paper's deployed formats at full size (kernel tables of the appendix): 2b-s16-g128 (16 salient columns in
  every group of 128, two extra bases on them), 2b-s8-g128 and 4b-g128 at 4096 x 4096 and 4096 x 11008;
* the grouped-query shapes of the other model families the paper evaluates (Llama-3.1-8B: 1024 x 4096,
  14336 x 4096, 4096 x 14336; Qwen3-8B: 12288 x 4096) in the 2b-s8-g128 format.

All through the C-ABI, fp32 outputs, element by element, with the contract's tolerances and the fp32-level
bounds of test_gpu_parity.check.
"""
import numpy as np
import pytest

import oracle
from paper_2608_15602_b200 import synth
from test_gpu_parity import check, f16

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import layer
    return layer


def run_once(fb, L, x_bits):
    lin = fb.FluxBinLinear(L)
    B = x_bits.shape[0]
    ws = lin.workspace(B)
    y = lin.forward(torch.from_numpy(x_bits.view(np.float16)).cuda(), ws, fp32_out=True)
    torch.cuda.synchronize()
    assert int(ws.tensor.count_nonzero()) == 0, "workspace must be left zeroed"
    return y.cpu().numpy()


def variant_layer(variant, M, N, seed):
    Kb = 4 if variant == "4b" else 2
    s = {"2b": 0, "4b": 0, "2b-s8": 8, "2b-s16": 16}[variant]
    idx = synth.salient_per_group(seed, 2, N, 128, s) if s else None
    return synth.make_linear(seed, 2, M, N, Kb, 2 if s else 0, 128, idx)


@pytest.mark.parametrize("variant", ["2b-s16", "2b-s8", "4b"])
@pytest.mark.parametrize("M,N", [(4096, 4096), (4096, 11008)])
def test_deployed_formats_at_kernel_table_shapes(fb, variant, M, N):
    L = variant_layer(variant, M, N, 31)
    x = synth.make_activations(31, 3, 1, N)
    check(run_once(fb, L, x), oracle.linear_direct(L, x), f"{variant}-g128 {M}x{N}", L, x)


@pytest.mark.parametrize("M,N", [(1024, 4096), (14336, 4096), (4096, 14336), (12288, 4096)])
def test_grouped_query_shapes_of_other_model_families(fb, M, N):
    L = variant_layer("2b-s8", M, N, 32)
    x = synth.make_activations(32, 4, 1, N)
    check(run_once(fb, L, x), oracle.linear_direct(L, x), f"2b-s8-g128 {M}x{N}", L, x)


def test_llama13b_gate_batch8(fb):
    L = synth.make_config_linear(3, 0, 4)
    assert (L.M, L.N) == (13824, 5120)
    x = synth.make_config_activations(3, 0, 4, 8)
    check(run_once(fb, L, x), oracle.linear_direct(L, x), "13B gate B=8", L, x)


@pytest.mark.parametrize("B", [4, 16])
def test_llama70b_plan_batched(fb, B):
    """Two 70B-shaped layers as one plan at batch B with fp32 table entries (chunks of four vectors)."""
    lins, _ = synth.config_linears(4)
    checked = {(0, 0), (1, 1), (0, 4), (1, 6)}                 # q 8192^2, k 1024x8192, gate 28672x8192, down 8192x28672
    members, keep = [], {}
    stats = {}
    for layer in range(2):
        for li, (name, M, N) in enumerate(lins):
            L = synth.make_config_linear(4, layer, li)
            x = synth.make_config_activations(4, layer, li, B)
            lin = fb.FluxBinLinear(L)
            members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                            torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")))
            if (layer, li) in checked:
                keep[(layer, li)] = (L, x)
            else:
                xs = f16(x) ** 2
                per_group = (f16(L.col_scale)[None] ** 2 * xs[:, None, :]).reshape(B, L.Kb, N // L.g, L.g).sum(axis=3)
                stats[(layer, li)] = np.sqrt(np.einsum("kmg,bkg->bm", f16(L.row_scale) ** 2, per_group).mean(axis=1))
    plan = fb.FluxBinPlan(members)
    assert plan.num_launches() == B // 4
    for rep in range(2):                                       # twice: the workspace must come back zeroed
        for _, _, y in members:
            y.fill_(float("nan"))
        plan.run()
        torch.cuda.synchronize()
    assert int(plan.ws.tensor.count_nonzero()) == 0, "plan workspace must be left zeroed"
    for idx, (lin, _, y) in enumerate(members):
        layer, li = divmod(idx, len(lins))
        got = y.cpu().numpy()
        assert np.isfinite(got).all(), f"layer {layer} linear {li}: unwritten or non-finite outputs"
        if (layer, li) in keep:
            L, x = keep[(layer, li)]
            check(got, oracle.linear_direct(L, x), f"B={B} layer {layer} {lins[li][0]} {lin.M}x{lin.N}", L, x)
        else:
            rms = np.sqrt(np.mean(got.astype(np.float64) ** 2, axis=1))
            want = stats[(layer, li)]
            assert np.all((0.9 * want <= rms) & (rms <= 1.25 * want)), f"layer {layer} linear {li}: rms {rms} vs {want}"
