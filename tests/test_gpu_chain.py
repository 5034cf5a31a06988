"""GPU parity of one-vector calls (B = 1) of small layers against the CPU oracle, element by element through the
C-ABI: layers whose whole work is a handful of items per CTA (full and narrow last salient pairs, several salient
bases, one to many row blocks, ragged row counts, fp32 and fp16 outputs), the trailing one-vector chunk of a batched
call, and chains of dependent calls on one stream, where each launch may start (programmatic dependent launch)
while its predecessor drains but must see its output."""
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


#        M,    N,  Kb, Ks, g,  n_sal
CASES = [(1, 256, 2, 0, 128, 0),            # one row, one row block, two pairs
         (33, 384, 3, 2, 128, 40),          # odd number of units, two salient bases
         (100, 512, 1, 1, 256, 19),         # g = 256
         (257, 1024, 2, 1, 128, 51),        # narrow last pair (16 slots)
         (1000, 2048, 2, 1, 128, 8),        # narrow last pair (8 slots)
         (600, 2048, 2, 2, 128, 128),       # full last pair
         (2100, 384, 2, 0, 128, 0),         # many row blocks, three pairs, no salient branch
         (4096, 4096, 2, 1, 128, 205),      # the hybrid 4096 x 4096 layer of the workloads
         (5120, 5120, 2, 0, 128, 0),
         (3000, 4096, 4, 0, 128, 0)]        # four bases


@pytest.mark.parametrize("M,N,Kb,Ks,g,n_sal", CASES)
@pytest.mark.parametrize("fp32", [True, False])
def test_one_vector_call_matches_oracle(fb, M, N, Kb, Ks, g, n_sal, fp32):
    L = layer_of(M + N + Kb, M, N, Kb, Ks, g, n_sal)
    lin = fb.FluxBinLinear(L)
    x = synth.make_activations(17, M, 1, N)
    xt = torch.from_numpy(x.view(np.float16)).cuda()
    ws = lin.workspace(1)
    want = oracle.linear_direct(L, x)
    for rep in range(2):
        y = torch.full((1, M + 8), float("nan"), dtype=torch.float32 if fp32 else torch.float16, device="cuda")
        lin.forward(xt, ws, out=y[:, :M])
        torch.cuda.synchronize()
        got = y.float().cpu().numpy()
        assert np.isnan(got[:, M:]).all(), "nothing beyond M is written"
        assert int(ws.tensor.count_nonzero()) == 0, "the workspace stays zeroed"
        if fp32:
            check(got[:, :M], want, f"{(M, N, Kb, Ks, g, n_sal)} run {rep}", L, x)
        else:
            ulp = np.spacing(np.abs(want).astype(np.float16)).astype(np.float64)
            rms = np.sqrt(np.mean(want ** 2))
            assert np.all(np.abs(got[:, :M] - want) <= 1.01 * ulp + 5e-3 * np.maximum(np.abs(want), 1e-2 * rms))


def test_trailing_one_vector_chunk(fb):
    """B = 5 runs as a chunk of four vectors and one of a single vector."""
    L = layer_of(77, 1536, 2048, 2, 1, 128, 100)
    lin = fb.FluxBinLinear(L)
    x = synth.make_activations(18, 1, 5, 2048)
    xt = torch.from_numpy(x.view(np.float16)).cuda()
    ws = lin.workspace(5)
    want = oracle.linear_direct(L, x)
    for rep in range(2):
        y = lin.forward(xt, ws, fp32_out=True)
        torch.cuda.synchronize()
        check(y.cpu().numpy(), want, f"B=5 run {rep}", L, x)


def test_chain_of_dependent_one_vector_calls(fb):
    """y1 = L1 x, y2 = L2 y1, y3 = L3 y2, y4 = L4 y3 back to back on one stream (two kernel instantiations: scale
    groups of 128 and of 64 columns): each launch may start while its predecessor drains but must see its output."""
    dims = [(1024, 2048, 2, 128), (768, 1024, 2, 128), (1536, 768, 4, 64), (512, 1536, 2, 128)]   # (M, N, Kb, g), N of the next = M of the previous
    Ls, lins = [], []
    for i, (M, N, Kb, g) in enumerate(dims):
        L = layer_of(400 + i, M, N, Kb, 1, g, N // 20)
        Ls.append(L)
        lins.append(fb.FluxBinLinear(L))
    x0 = synth.make_activations(5, 5, 1, 2048)
    xt = torch.from_numpy(x0.view(np.float16)).cuda()
    ws = fb.Workspace(max(l.weight.workspace_size(1) for l in lins))
    for rep in range(3):
        h, outs = xt, []
        for lin in lins:
            h = lin.forward(h, ws)
            outs.append(h)
        torch.cuda.synchronize()
        cur = x0
        for L, got in zip(Ls, outs):
            want = oracle.linear_direct(L, cur)
            g = got.cpu().numpy()
            ulp = np.spacing(np.abs(want).astype(np.float16)).astype(np.float64)
            rms = np.sqrt(np.mean(want ** 2))
            assert np.all(np.abs(g.astype(np.float64) - want) <= 1.01 * ulp + 5e-3 * np.maximum(np.abs(want), 1e-2 * rms))
            cur = g.view(np.uint16)
