"""GPU parity of the fp16-table mode of batched launches (fluxbin_set_table_format) against the CPU oracle.

With fp16 entries every looked-up partial sum (Eq. 14: a signed sum of the 8 fused activations of a sub-vector)
is the fp32 value rounded once to fp16, so it carries a relative error of at most 2^-11; all sums are still
accumulated in fp32.  The tolerance follows from that arithmetic:

  * per output, rigorous:  |y - want| <= fp32 tolerance + 2^-11 * sum_k sum_G alpha_r(k,i,G) * sum_{j in G}
    |alpha_c(k,j) x_j|  (+ the same over the salient bases) -- every entry is at most the sum of the magnitudes
    of its 8 terms, the row scale multiplies the error like the value;
  * per batch row:  the rounding errors are independent and centred, at most 2^-11 and about 2^-11 / sqrt(3) of
    each entry in the root mean square, so the error of an output is a random walk over its entries:
    ||y - want||_2 <= fp32 tolerance + 2 * 2^-11 * || rss ||_2, rss_i the root-sum-square over the entries of output
    i of alpha_r * (sum of the magnitudes of the entry's 8 terms)  (the factor 2 covers outputs with only a handful
    of entries, where a walk can reach twice its root mean square);
  * layers with thousands of columns (the workloads): the entries themselves add up like a random walk too, the
    relative L2 error of a row of outputs is about 3e-4 and the fp32 path's bound of 1e-3 still holds (`strict`).
"""
import numpy as np
import pytest

import oracle
from paper_2608_15602_b200 import synth
from test_gpu_parity import MAX_REL, REL_L2, f16, layer_of

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import layer
    return layer


def entry_bounds(L, x_bits):
    """([B][M], [B][M]): per output the sum, and the root-sum-square, over its looked-up entries of alpha_r times
    the largest magnitude the entry can have (the sum of |alpha_c * x| over its 8 columns; the salient columns of
    a group form entries of their own, 8 consecutive virtual columns at most)."""
    x = f16(x_bits)[:, :L.N]
    B, G = x.shape[0], L.N // L.g
    l1, sq = np.zeros((B, L.M)), np.zeros((B, L.M))
    ar, ac = np.abs(f16(L.row_scale)).reshape(L.Kb, L.M, G), np.abs(f16(L.col_scale)).reshape(L.Kb, L.N)
    for k in range(L.Kb):
        ent = (np.abs(x) * ac[k][None, :]).reshape(B, L.N // 8, 8).sum(axis=2)             # [B][N/8] entry magnitudes
        l1 += ent.reshape(B, G, L.g // 8).sum(axis=2) @ ar[k].T
        sq += (ent ** 2).reshape(B, G, L.g // 8).sum(axis=2) @ (ar[k] ** 2).T
    if L.Ks and L.n_sal:
        idx = np.asarray(L.sal_idx, np.int64)
        sr, sc = np.abs(f16(L.sal_row_scale)).reshape(L.Ks, L.M, G), np.abs(f16(L.sal_col_scale)).reshape(L.Ks, L.n_sal)
        for k in range(L.Ks):
            terms = np.abs(x[:, idx]) * sc[k][None, :]                                     # [B][n_sal]
            per_group = np.zeros((B, G))
            np.add.at(per_group, (slice(None), idx // L.g), terms)
            l1 += per_group @ sr[k].T
            sq += (per_group ** 2) @ (sr[k] ** 2).T          # all salient columns of a group as ONE entry: an upper bound
    return l1, np.sqrt(sq)


def check_fp16_tables(y, want, L, x_bits, what="", strict=False):
    y = np.asarray(y, np.float64)
    l1, rss = entry_bounds(L, x_bits)
    for b in range(want.shape[0]):
        rms = np.sqrt(np.mean(want[b] ** 2))
        err2 = np.linalg.norm(y[b] - want[b])
        assert err2 <= REL_L2 * np.linalg.norm(want[b]) + 2.0 * 2.0 ** -11 * np.linalg.norm(rss[b]), \
            f"{what} batch row {b}: L2 error {err2:.3e} of {np.linalg.norm(want[b]):.3e}"
        if strict:
            assert err2 <= REL_L2 * np.linalg.norm(want[b]), f"{what} batch row {b}: rel L2 {err2 / np.linalg.norm(want[b]):.3e}"
        tol = MAX_REL * np.maximum(np.abs(want[b]), 1e-2 * rms) + 2.0 ** -11 * l1[b]
        bad = np.abs(y[b] - want[b]) > tol
        assert not bad.any(), f"{what} batch row {b}: {int(bad.sum())} outputs beyond the rounding bound, first {bad.argmax()}"


def run(fb, L, x_bits, fp32=True):
    lin = fb.FluxBinLinear(L, fp16_tables=True)
    B = x_bits.shape[0]
    assert lin.weight.table_format() == 1 and lin.weight.num_launches(B) == (B + 7) // 8
    xt = torch.from_numpy(x_bits.view(np.float16)).cuda()
    ws = lin.workspace(B)
    y = torch.full((B, L.M), float("nan"), dtype=torch.float32 if fp32 else torch.float16, device="cuda")
    lin.forward(xt, ws, out=y)
    torch.cuda.synchronize()
    assert int(ws.tensor.count_nonzero()) == 0, "workspace must be left zeroed"
    y2 = lin.forward(xt, ws, fp32_out=fp32)          # second call on the same workspace
    torch.cuda.synchronize()
    a, b = y.float().cpu().numpy(), y2.float().cpu().numpy()
    rtol = 1e-4 if fp32 else 2e-3
    assert np.allclose(a, b, rtol=rtol, atol=rtol * 0.1 * np.abs(a).max()), "second call on a reused workspace differs"
    return a


SMALL = [(1, 32, 1, 0, 32, 0), (5, 128, 2, 1, 32, 7), (33, 384, 3, 2, 128, 40), (100, 256, 1, 1, 256, 19),
         (127, 1024, 2, 1, 128, 51), (9, 160, 4, 3, 32, 160), (1000, 512, 2, 1, 512, 1), (31, 256, 2, 2, 64, 9),
         (600, 2048, 2, 2, 128, 128), (2100, 384, 2, 0, 128, 0)]


@pytest.mark.parametrize("M,N,Kb,Ks,g,n_sal", SMALL)
@pytest.mark.parametrize("B", [2, 3, 4, 5, 8, 9, 17])
def test_small_and_ragged_shapes(fb, M, N, Kb, Ks, g, n_sal, B):
    """Chunks of 2, 4 and 8 vectors (entries of 4, 8 and 16 bytes), ragged chunks, and a trailing chunk of one
    vector (B = 9, 17), which runs with fp32 entries."""
    L = layer_of(M * 3 + N + B, M, N, Kb, Ks, g, n_sal)
    x = synth.make_activations(13, M + B, B, N)
    check_fp16_tables(run(fb, L, x), oracle.linear_direct(L, x), L, x, f"{(M, N, Kb, Ks, g, n_sal, B)}")


@pytest.mark.parametrize("B", [2, 4, 8, 16])
def test_config1_hybrid_with_outliers(fb, B):
    L = synth.make_config_linear(1, 0, 0)
    x = synth.make_config_activations(1, 0, 0, B)
    check_fp16_tables(run(fb, L, x), oracle.linear_direct(L, x), L, x, f"config 1 B={B}", strict=True)


@pytest.mark.parametrize("g,B", [(4096, 2), (64, 4), (256, 3), (32, 8)])
def test_row_scale_formats(fb, g, B):
    L = synth.make_config_linear(1, 0, 0, g=g)
    x = synth.make_config_activations(1, 0, 0, B)
    check_fp16_tables(run(fb, L, x), oracle.linear_direct(L, x), L, x, f"g={g} B={B}", strict=True)


@pytest.mark.parametrize("li,B", [(0, 8), (6, 8), (4, 4)])
def test_llama13b_shapes(fb, li, B):
    L = synth.make_config_linear(3, 0, li)
    x = synth.make_config_activations(3, 0, li, B)
    check_fp16_tables(run(fb, L, x, fp32=False), oracle.linear_direct(L, x), L, x, f"13B linear {li} B={B}", strict=True)


def test_error_is_of_the_size_the_rounding_predicts(fb):
    """Against the fp32-table result of the same layer the fp16-table result differs by about 2^-11 / sqrt(3) of
    the root-sum-square of the terms: well above zero (the mode is really in use) and well below the bound."""
    L = synth.make_config_linear(1, 0, 0)
    B = 8
    x = synth.make_config_activations(1, 0, 0, B)
    want = oracle.linear_direct(L, x)
    got16 = run(fb, L, x)
    lin32 = fb.FluxBinLinear(L)
    assert lin32.weight.table_format() == 0 and lin32.weight.num_launches(B) == 2
    y32 = lin32.forward(torch.from_numpy(x.view(np.float16)).cuda(), lin32.workspace(B), fp32_out=True).cpu().numpy()
    for b in range(B):
        e16 = np.linalg.norm(got16[b] - want[b]) / np.linalg.norm(want[b])
        e32 = np.linalg.norm(y32[b] - want[b]) / np.linalg.norm(want[b])
        assert e32 < 2e-6, f"fp32 tables: rel L2 {e32:.3e}"
        assert 5e-5 < e16 < 6e-4, f"fp16 tables: rel L2 {e16:.3e} is not what one rounding per entry gives"


def test_single_vector_ignores_the_format(fb):
    L = synth.make_config_linear(1, 0, 0)
    x = synth.make_config_activations(1, 0, 0, 1)
    want = oracle.linear_direct(L, x)
    got = run(fb, L, x)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 2e-6


def test_plan_with_fp16_tables(fb):
    specs = [(300, 1024, 2, 1, 128, 51), (33, 256, 2, 0, 128, 0), (1000, 2048, 2, 2, 128, 100), (2100, 384, 2, 1, 128, 19)]
    for B in (4, 6, 11):
        members, cases = [], []
        for i, (M, N, Kb, Ks, g, n_sal) in enumerate(specs):
            L = layer_of(200 + i, M, N, Kb, Ks, g, n_sal)
            x = synth.make_activations(17, i, B, N)
            lin = fb.FluxBinLinear(L, fp16_tables=True)
            members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                            torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")))
            cases.append((L, x, oracle.linear_direct(L, x)))
        plan = fb.FluxBinPlan(members)
        assert plan.num_launches() == (B + 7) // 8
        for rep in range(2):
            for _, _, y in members:
                y.fill_(float("nan"))
            plan.run()
            torch.cuda.synchronize()
            assert int(plan.ws.tensor.count_nonzero()) == 0, "workspace must be left zeroed"
            for (lin, _, y), (L, x, want) in zip(members, cases):
                check_fp16_tables(y.cpu().numpy(), want, L, x, f"plan B={B} member M={lin.M} rep {rep}")


def test_long_plan_of_two_vectors_runs_the_two_pair_kernel(fb):
    """Two vectors with fp16 entries share the 4-byte table slots of the single-vector kernel, so a plan with
    enough work per CTA runs the variant that keeps two table sets resident (g = 128 and g = 64 formats)."""
    for g, shapes in ((128, [(256, 4096), (250, 4096), (512, 4096), (96, 8192)]), (64, [(300, 2048), (512, 4096)])):
        members, cases = [], []
        for i in range(120):
            M, N = shapes[i % len(shapes)]
            L = layer_of(700 + i, M, N, 2, 1, g, int(round(0.05 * N)))
            x = synth.make_activations(19, i, 2, N)
            lin = fb.FluxBinLinear(L, fp16_tables=True)
            members.append((lin, torch.from_numpy(x.view(np.float16)).cuda(),
                            torch.full((2, M), float("nan"), dtype=torch.float32, device="cuda")))
            cases.append((L, x, oracle.linear_direct(L, x)))
        plan = fb.FluxBinPlan(members)
        assert plan.pairs_per_row_block() == 2 and plan.num_launches() == 1
        for rep in range(2):                      # twice: the workspace must come back zeroed
            for _, _, y in members:
                y.fill_(float("nan"))
            plan.run()
            torch.cuda.synchronize()
            for (lin, _, y), (L, x, want) in zip(members, cases):
                check_fp16_tables(y.cpu().numpy(), want, L, x, f"two-pair kernel g={g}, member {lin.M}x{lin.N} rep {rep}", strict=True)
        short = fb.FluxBinPlan(members[:4])
        assert short.pairs_per_row_block() == 1
        for _, _, y in members[:4]:
            y.fill_(float("nan"))
        short.run()
        torch.cuda.synchronize()
        for (lin, _, y), (L, x, want) in zip(members[:4], cases[:4]):
            check_fp16_tables(y.cpu().numpy(), want, L, x, f"one-pair kernel g={g}, member {lin.M}x{lin.N}", strict=True)


def test_plan_rejects_mixed_table_formats(fb):
    from paper_2608_15602_b200 import fluxbin
    L = layer_of(5, 64, 256, 2, 0, 128, 0)
    a, b = fb.FluxBinLinear(L), fb.FluxBinLinear(L, fp16_tables=True)
    x = torch.zeros((4, 256), dtype=torch.float16, device="cuda")
    ya, yb = torch.empty((4, 64), dtype=torch.float16, device="cuda"), torch.empty((4, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(fluxbin.FluxBinError):
        fb.FluxBinPlan([(a, x, ya), (b, x, yb)])
    with pytest.raises(fluxbin.FluxBinError):
        a.weight.set_table_format(7)


@pytest.mark.parametrize("case", range(16))
def test_random_single_calls(fb, case):
    """Seeded random shapes, group sizes, base counts, salient maps (none, random, every column, one group only),
    batch sizes 2..20 and activation outliers."""
    from test_gpu_random import random_layer
    r = np.random.default_rng(260815602 + 3000 + case)
    L = random_layer(r, 9000 + case)
    B = int(r.integers(2, 21))
    x = synth.make_activations(9000 + case, 3, B, L.N, outlier_frac=float(r.choice([0.0, 0.02])))
    check_fp16_tables(run(fb, L, x), oracle.linear_direct(L, x), L, x,
                      f"case {case}: M={L.M} N={L.N} g={L.g} Kb={L.Kb} Ks={L.Ks} n_sal={L.n_sal} B={B}")


def test_entries_beyond_the_fp16_range_saturate(fb):
    """The documented limit of the mode: a table entry is a sum of 8 fused activations rounded to fp16, so with
    activations of 6e4 and column scales near 1 the entries overflow to infinity and the outputs are not finite;
    the fp32 entries of the default mode hold the same sums."""
    L = layer_of(77, 64, 256, 2, 0, 128, 0)
    L.col_scale[:] = np.float16(1.0).view(np.uint16)
    x = np.full((2, 256), np.float16(6.0e4).view(np.uint16), np.uint16)
    xt = torch.from_numpy(x.view(np.float16)).cuda()
    lin32, lin16 = fb.FluxBinLinear(L), fb.FluxBinLinear(L, fp16_tables=True)
    y32 = lin32.forward(xt, lin32.workspace(2), fp32_out=True).cpu().numpy()
    y16 = lin16.forward(xt, lin16.workspace(2), fp32_out=True).cpu().numpy()
    want = oracle.linear_direct(L, x)
    assert np.isfinite(y32).all() and np.allclose(y32, want, rtol=1e-4, atol=1e-4 * np.abs(want).max())
    assert not np.isfinite(y16).all()
