"""GPU parity: the CUDA path (through the C-ABI) against the CPU oracle, element by element.

Tolerances (fp32 accumulation, stated by the benchmark spec): relative L2 error <= 1e-3 per batch row and
max relative error <= 5e-3 per output, the per-output denominator floored at 1e-2 * rms(row) so
that outputs that cancel to ~0 do not divide by nothing.

Those two are the contract.  The fp32 path is far better than that, and a regression of two decimal digits
would still pass them, so fp32 outputs computed with fp32 table entries are also held to the level the
arithmetic implies (`check` with the layer and the activations at hand):

* per output  |y - y_ref| <= c * 2^-24 * T_i  with  T_i = sum over all terms |alpha_r * alpha_c * x|  of row i:
  every fp32 operation on the way from the terms to y_i rounds a partial sum that is at most T_i in magnitude,
  so the error is at most (roundings on the longest path) * 2^-24 * T_i.  The path: 7 adds inside a table entry
  (Eq. 14), at most 9 adds of entries inside a row-scale segment, one scale multiply-add per segment of the item
  (<= 32), then one atomic add per table set (pair) of the layer: c = 56 + number of pairs.
* per batch row with at least 64 outputs  ||y - y_ref||_2 <= 2e-5 * ||y_ref||_2: the roundings are independent,
  so the error of a row of outputs is a random walk of about sqrt(c) steps of 2^-24 relative to partial sums of
  the size of the result, measured at 1e-6 to 2e-6; 2e-5 leaves a factor of ten and is fifty times below 1e-3.
"""
import numpy as np
import pytest

import oracle
from paper_2608_15602_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL_L2 = 1e-3
MAX_REL = 5e-3
FIELDS = ["bits", "row_scale", "col_scale", "sal_idx", "sal_bits", "sal_row_scale", "sal_col_scale"]


@pytest.fixture(scope="module")
def fb():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import fluxbin, layer
    return layer


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)


TIGHT_L2 = 2e-5


def term_magnitudes(L, x_bits):
    """T[b][i] = sum of |alpha_r * alpha_c * x| over every term of output i (global and salient bases)."""
    xs = np.abs(f16(x_bits))                                                       # [B][N]
    ng = L.N // L.g
    per_group = (xs[:, None, :] * f16(L.col_scale)[None]).reshape(xs.shape[0], L.Kb, ng, L.g).sum(axis=3)   # [B][Kb][ng]
    T = np.einsum("kmg,bkg->bm", f16(L.row_scale), per_group)
    if L.Ks and L.n_sal:
        grp = L.sal_idx // L.g
        a = xs[:, None, L.sal_idx] * f16(L.sal_col_scale)[None]                      # [B][Ks][n_sal]
        per_group_s = np.zeros((xs.shape[0], L.Ks, ng))
        np.add.at(per_group_s, (slice(None), slice(None), grp), a)
        T += np.einsum("kmg,bkg->bm", f16(L.sal_row_scale), per_group_s)
    return T


def roundings_on_longest_path(L):
    pairs = (-(-L.N // 128) * L.Kb + 1) // 2
    if L.Ks and L.n_sal:
        groups = len(np.unique(L.sal_idx // L.g))
        pairs += ((((L.n_sal + 7 * groups) // 8 + 15) // 16) * L.Ks + 1) // 2        # an upper bound (per-group padding)
    return 56 + pairs


def check(y, want, what="", L=None, x=None, extra_roundings=0):
    """The contract's tolerances; with the layer and the activations given (fp32 outputs, fp32 table entries)
    also the level the fp32 arithmetic implies (see the module docstring).  extra_roundings: what a variant of the
    path adds to the longest chain of fp32 operations."""
    y = np.asarray(y, np.float64)
    for b in range(want.shape[0]):
        rms = np.sqrt(np.mean(want[b] ** 2))
        l2 = np.linalg.norm(y[b] - want[b]) / max(np.linalg.norm(want[b]), 1e-300)
        rel = np.abs(y[b] - want[b]) / np.maximum(np.abs(want[b]), 1e-2 * rms + 1e-300)
        assert l2 <= REL_L2, f"{what} batch row {b}: rel L2 {l2:.3e}"
        assert rel.max() <= MAX_REL, f"{what} batch row {b}: max rel {rel.max():.3e} at {rel.argmax()}"
    if L is not None:
        T = term_magnitudes(L, x)
        c = roundings_on_longest_path(L) + extra_roundings
        excess = np.abs(y - want) / (c * 2.0 ** -24 * T + 1e-300)
        assert excess.max() <= 1.0, f"{what}: error {excess.max():.2f} x the fp32 rounding bound at {np.unravel_index(excess.argmax(), excess.shape)}"
        if want.shape[1] >= 64:
            for b in range(want.shape[0]):
                l2 = np.linalg.norm(y[b] - want[b]) / max(np.linalg.norm(want[b]), 1e-300)
                assert l2 <= TIGHT_L2, f"{what} batch row {b}: rel L2 {l2:.3e} (fp32 level is ~2e-6)"


def run(fb, L, x_bits, fp32=True, ldx=None):
    lin = fb.FluxBinLinear(L)
    B = x_bits.shape[0]
    xt = torch.from_numpy(x_bits.view(np.float16)).cuda()
    ws = lin.workspace(B)
    y = lin.forward(xt, ws, fp32_out=fp32)
    torch.cuda.synchronize()
    assert int(ws.tensor.count_nonzero()) == 0, "workspace must be left zeroed"
    y2 = lin.forward(xt, ws, fp32_out=fp32)          # second call on the same workspace
    torch.cuda.synchronize()
    a, b = y.float().cpu().numpy(), y2.float().cpu().numpy()
    # atomics reorder fp32 sums from run to run; fp16 outputs may then round to the neighbouring value
    rtol = 1e-4 if fp32 else 2e-3
    assert np.allclose(a, b, rtol=rtol, atol=rtol * 0.1 * np.abs(a).max()), "second call on a reused workspace differs"
    return y.float().cpu().numpy() if fp32 else y.cpu().numpy()


def layer_of(seed, M, N, Kb, Ks, g, n_sal):
    idx = None
    if Ks and n_sal:
        idx = np.sort(np.random.default_rng(seed).choice(N, n_sal, replace=False)).astype(np.int32)
    return synth.make_linear(seed, 5, M, N, Kb, Ks, g, idx)


SMALL = [(1, 32, 1, 0, 32, 0), (5, 128, 2, 1, 32, 7), (33, 384, 3, 2, 128, 40), (100, 256, 1, 1, 256, 19),
         (127, 1024, 2, 1, 128, 51), (7, 96, 2, 2, 96, 50), (9, 160, 4, 3, 32, 160), (1000, 512, 2, 1, 512, 1),
         (31, 256, 2, 2, 64, 9), (65, 640, 2, 1, 128, 640), (600, 2048, 2, 2, 128, 128), (2100, 384, 2, 0, 128, 0)]


@pytest.mark.parametrize("M,N,Kb,Ks,g,n_sal", SMALL)
@pytest.mark.parametrize("B", [1, 2, 3, 4, 7])
def test_small_and_ragged_shapes(fb, M, N, Kb, Ks, g, n_sal, B):
    L = layer_of(M * 3 + N + B, M, N, Kb, Ks, g, n_sal)
    x = synth.make_activations(11, M + B, B, N)
    want = oracle.linear_direct(L, x)
    check(run(fb, L, x), want, f"{(M, N, Kb, Ks, g, n_sal, B)}", L, x)


def test_config0_full_layer(fb):
    L = synth.make_config_linear(0, 0, 0)
    x = synth.make_config_activations(0, 0, 0, 1)
    check(run(fb, L, x), oracle.linear_direct(L, x), "config 0", L, x)


@pytest.mark.parametrize("B", [1, 4, 16])
def test_config1_hybrid_with_outliers(fb, B):
    L = synth.make_config_linear(1, 0, 0)
    x = synth.make_config_activations(1, 0, 0, B)
    check(run(fb, L, x), oracle.linear_direct(L, x), f"config 1 B={B}", L, x)


@pytest.mark.parametrize("g,B", [(128, 2), (4096, 2), (32, 1), (64, 1), (64, 4), (256, 1), (256, 3)])
def test_row_scale_formats(fb, g, B):
    """g = 128 (one scale per row and group, the paper's format), g = N (one per row) and the group sizes of the
    paper's ablation (32, 64, 256): 4, 8 or 16 sub-vectors per row-scale segment in the global region."""
    L = synth.make_config_linear(1, 0, 0, g=g)
    x = synth.make_config_activations(1, 0, 0, B)
    check(run(fb, L, x), oracle.linear_direct(L, x), f"g={g} B={B}", L, x)


def test_paper_structured_salient_pattern(fb):
    """Exactly s = 8 salient columns per group of 128 with Ks = Kb = 2 (the paper's 2b-s8-g128)."""
    N, M = 2048, 1536
    idx = synth.salient_per_group(3, 1, N, 128, 8)
    L = synth.make_linear(3, 1, M, N, 2, 2, 128, idx)
    x = synth.make_activations(3, 1, 1, N)
    check(run(fb, L, x), oracle.linear_direct(L, x), "2b-s8-g128", L, x)


@pytest.mark.parametrize("li", [0, 4, 6])
def test_llama7b_shapes(fb, li):
    L = synth.make_config_linear(2, 0, li)
    x = synth.make_config_activations(2, 0, li, 1)
    check(run(fb, L, x), oracle.linear_direct(L, x), f"7B linear {li}", L, x)


@pytest.mark.parametrize("li,B", [(0, 8), (4, 1), (6, 8)])
def test_llama13b_shapes(fb, li, B):
    L = synth.make_config_linear(3, 0, li)
    x = synth.make_config_activations(3, 0, li, B)
    check(run(fb, L, x), oracle.linear_direct(L, x), f"13B linear {li} B={B}", L, x)


@pytest.mark.parametrize("li", [0, 1, 4, 6])
def test_llama70b_shapes_batch1(fb, li):
    L = synth.make_config_linear(4, 3, li)
    x = synth.make_config_activations(4, 3, li, 1)
    check(run(fb, L, x), oracle.linear_direct(L, x), f"70B linear {li}", L, x)


@pytest.mark.parametrize("B", [1, 3])
def test_widest_layer(fb, B):
    """N = 65536, the widest layer the 16-bit column indices of the packed column tables allow: 512 global units
    (the longest K split there is) and salient columns at both ends of the index range."""
    N = 65536
    idx = np.array([0, 1, 127, 128, 40000, 65407, 65408, 65534, 65535], dtype=np.int32)
    L = synth.make_linear(91, 5, 70, N, 1, 2, 128, idx)
    x = synth.make_activations(91, 6, B, N)
    check(run(fb, L, x), oracle.linear_direct(L, x), f"N = 65536, B = {B}", L, x)


def test_fp16_output_is_rounded_fp32_result(fb):
    L = synth.make_config_linear(1, 0, 0)
    x = synth.make_config_activations(1, 0, 0, 2)
    y32 = run(fb, L, x, fp32=True)
    y16 = run(fb, L, x, fp32=False).astype(np.float64)
    want = oracle.linear_direct(L, x)
    ulp = np.spacing(np.abs(want).astype(np.float16)).astype(np.float64)
    assert np.all(np.abs(y16 - want) <= ulp * 1.01 + np.abs(y32 - want))


def test_leading_dimensions_and_overwrite(fb):
    """ldx > N, ldy > M; y is fully overwritten (pre-filled with NaN) and nothing beyond M is touched."""
    L = layer_of(77, 130, 256, 2, 1, 128, 13)
    B = 3
    x = synth.make_activations(1, 2, B, 320)
    lin = fb.FluxBinLinear(L)
    xt = torch.from_numpy(x.view(np.float16)).cuda()
    out = torch.full((B, 200), float("nan"), dtype=torch.float32, device="cuda")
    ws = lin.workspace(B)
    lin.forward(xt, ws, out=out[:, :130])
    torch.cuda.synchronize()
    o = out.cpu().numpy()
    assert np.all(np.isnan(o[:, 130:]))
    check(o[:, :130], oracle.linear_direct(L, x), "strided")


def test_special_cases_on_gpu(fb):
    """Complementary bases cancel; all-ones weights give Kb*sum(x)."""
    L = layer_of(5, 64, 512, 2, 0, 128, 0)
    L.bits[1] = ~L.bits[0]
    L.row_scale[1] = L.row_scale[0]
    L.col_scale[1] = L.col_scale[0]
    x = synth.make_activations(2, 3, 1, 512)
    y = run(fb, L, x)
    bound = (np.abs(f16(x)) * f16(L.col_scale[0])).sum() * f16(L.row_scale[0]).max()
    assert np.all(np.abs(y) <= 1e-5 * bound)
    L2 = layer_of(6, 40, 256, 3, 1, 64, 9)
    L2.bits[:] = 0xFFFFFFFF
    L2.sal_bits[:] = 0xFFFFFFFF
    L2.sal_bits[:, :, -1] &= np.uint32((1 << (9 % 32)) - 1)
    one = np.float16(1.0).view(np.uint16)
    for a in (L2.row_scale, L2.col_scale, L2.sal_row_scale, L2.sal_col_scale):
        a[:] = one
    x = synth.make_activations(2, 4, 2, 256)
    xs = f16(x)
    want = 3 * xs.sum(1) + xs[:, L2.sal_idx].sum(1)
    y = run(fb, L2, x)
    assert np.allclose(y, want[:, None], rtol=1e-4, atol=1e-3)


def test_device_round_trip_bit_exact(fb):
    L = layer_of(9, 257, 1024, 2, 2, 128, 77)
    lin = fb.FluxBinLinear(L)
    U = lin.unpack()
    for f in FIELDS:
        assert np.array_equal(getattr(L, f), getattr(U, f)), f


def test_lut_identity_on_device(fb):
    """Every table entry the kernel builds equals the signed sum of its sub-vector's fused
    activations (Eq. 14) within 8 roundings of fp32."""
    from paper_2608_15602_b200 import fluxbin
    L = synth.make_config_linear(1, 0, 0)
    x = synth.make_config_activations(1, 0, 0, 1)
    lin = fb.FluxBinLinear(L)
    xt = torch.from_numpy(x.view(np.float16)).cuda()
    out = torch.empty((32, 256), dtype=torch.float32, device="cuda")
    nsets = lin.weight.num_table_sets()
    for pair in (0, 17, nsets - 1):
        cols, alpha = fluxbin.debug_tables(lin.weight, xt.data_ptr(), pair, out.data_ptr())
        torch.cuda.synchronize()
        T = out.cpu().numpy().astype(np.float64)
        a = (f16(x)[0, cols] * f16(alpha)).reshape(32, 8)
        for t in range(32):
            ref = oracle.lut_tables(a[t], 8)[0]
            tol = 8 * 2.0 ** -24 * np.abs(a[t]).sum() + 1e-30
            assert np.all(np.abs(T[t] - ref) <= tol), (pair, t)
    # the fused activations of a global table are x * alpha_c of 8 consecutive columns
    cols, alpha = fluxbin.debug_tables(lin.weight, xt.data_ptr(), 0, out.data_ptr())
    assert np.array_equal(cols[:128], np.arange(128)) and np.array_equal(alpha[:128], L.col_scale[0, :128])
    assert np.array_equal(alpha[128:], L.col_scale[1, :128])


def test_argument_errors_do_not_launch(fb):
    from paper_2608_15602_b200 import fluxbin
    L = layer_of(1, 64, 128, 2, 0, 128, 0)
    lin = fb.FluxBinLinear(L)
    x = torch.zeros((1, 128), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 64), dtype=torch.float16, device="cuda")
    ws = lin.workspace(1)
    w = lin.weight
    args = dict(d_x=x.data_ptr(), B=1, ldx=128, d_y=y.data_ptr(), y_is_fp32=False, ldy=64, d_ws=ws.tensor.data_ptr(),
                ws_bytes=ws.nbytes)
    assert fluxbin.linear_status(w, **args) == 0
    assert fluxbin.linear_status(w, **{**args, "B": 0}) == 3
    assert fluxbin.linear_status(w, **{**args, "ldx": 64}) == 3
    assert fluxbin.linear_status(w, **{**args, "ldy": 63}) == 3
    assert fluxbin.linear_status(w, **{**args, "ws_bytes": 16}) == 5
    assert fluxbin.linear_status(w, **{**args, "d_x": x.data_ptr() + 2}) == 6
    assert fluxbin.linear_status(w, **{**args, "d_y": 0}) == 1
    torch.cuda.synchronize()


def test_calls_with_another_device_current_are_rejected(fb):
    """fluxbin_linear and fluxbin_plan_create / fluxbin_plan_run compare the current device with the one that
    holds the layer and return a status instead of launching a kernel that would read another GPU's pointers.
    With one GPU in the machine the mismatch is made by rewriting the device ordinal stored in the host-side
    handle (checked through fluxbin_weight_device), never by touching a second device."""
    import ctypes
    from paper_2608_15602_b200 import fluxbin
    L = layer_of(2, 64, 128, 2, 0, 128, 0)
    lin = fb.FluxBinLinear(L)
    w = lin.weight
    x = torch.zeros((1, 128), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 64), dtype=torch.float16, device="cuda")
    ws = lin.workspace(1)
    args = dict(d_x=x.data_ptr(), B=1, ldx=128, d_y=y.data_ptr(), y_is_fp32=False, ldy=64, d_ws=ws.tensor.data_ptr(),
                ws_bytes=ws.nbytes)
    dev = w.device()
    assert dev == torch.cuda.current_device()
    # the handle is { 256-byte header copy, device pointer, byte count, int device, ... }
    field = ctypes.c_int.from_address(w.handle + 256 + 8 + 8)
    assert field.value == dev
    field.value = dev + 1
    try:
        assert w.device() == dev + 1, "the handle layout changed: this test pokes the wrong field"
        assert fluxbin.linear_status(w, **args) == 7
        assert fluxbin.linear_noalloc_status(w, x.data_ptr(), 1, 128, y.data_ptr(), False, 64) == 7
        table = torch.empty(fluxbin.plan_table_bytes(1, 1), dtype=torch.uint8, device="cuda")
        pws = fb.Workspace(fluxbin.plan_workspace_bytes([w], 1))
        st, h = fluxbin.plan_create_status([w], [x.data_ptr()], [128], [y.data_ptr()], [64], 1, False, table.data_ptr(),
                                           table.numel(), pws.tensor.data_ptr(), pws.nbytes)
        assert st == 7 and not h
    finally:
        field.value = dev
    assert fluxbin.linear_status(w, **args) == 0
    torch.cuda.synchronize()


def test_back_to_back_dependent_layers_share_a_workspace(fb):
    """y1 = L1 x, y2 = L2 y1, y3 = L3 y2 launched back to back on one stream with one workspace: each
    kernel may start while its predecessor drains (programmatic dependent launch) but must see the
    predecessor's output and a clean workspace."""
    dims = [(1024, 2048), (768, 1024), (1536, 768)]          # (M, N) chained: N of the next = M of the previous
    Ls, lins = [], []
    for i, (M, N) in enumerate(dims):
        L = layer_of(300 + i, M, N, 2, 1, 128, N // 20)
        Ls.append(L)
        lins.append(fb.FluxBinLinear(L))
    x0 = synth.make_activations(4, 4, 2, 2048)
    xt = torch.from_numpy(x0.view(np.float16)).cuda()
    ws = fb.Workspace(max(l.weight.workspace_size(2) for l in lins))
    for rep in range(3):
        h = xt
        outs = []
        for lin in lins:
            h = lin.forward(h, ws)                            # fp16 output feeds the next layer directly
            outs.append(h)
        torch.cuda.synchronize()
        cur = x0
        for L, got in zip(Ls, outs):
            want = oracle.linear_direct(L, cur)
            g = got.cpu().numpy()
            ulp = np.spacing(np.abs(want).astype(np.float16)).astype(np.float64)
            rms = np.sqrt(np.mean(want ** 2))
            assert np.all(np.abs(g.astype(np.float64) - want) <= 1.01 * ulp + 5e-3 * np.maximum(np.abs(want), 1e-2 * rms))
            cur = g.view(np.uint16)                           # the next layer's oracle input is the GPU's fp16 output
