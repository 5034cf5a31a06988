"""GPU parity of the row-column binary decomposition (fluxbin_rc_decomp, through the C-ABI) against the numpy
oracle of Algorithm 3 / Eq. 5-6.

The scales are fp32 on the GPU and fp64 in the oracle: they agree to a relative tolerance.  The signs are an
integer decision taken in floating point: both sides take it in fp32 in the same order (the oracle's
dtype=float32 mode), and where they still differ -- the scales feeding the decision differ in their last bits --
the element must be a near-tie, i.e. the GPU's choice is as good as the oracle's within rounding (several results
are correct; what is unique, the achieved error, is compared).
"""
import numpy as np
import pytest

from oracle import rc_decomp as rc
from paper_2608_15602_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import layer
    return layer


def unpack_bits(bits_i32, N):
    """[K][M][N/32] words -> [K][M][N] of +-1."""
    w = bits_i32.view(np.uint32)
    b = (w[..., None] >> np.arange(32, dtype=np.uint32)) & 1
    return np.where(b.reshape(w.shape[0], w.shape[1], N) == 1, 1.0, -1.0)


def gpu_decomp(fb, W, g, K, T, eps):
    out = fb.rc_decompose(torch.from_numpy(W).cuda(), g, K, T, eps)
    torch.cuda.synchronize()
    ar = out["row_scale_f32"].cpu().numpy().astype(np.float64)
    ac = out["col_scale_f32"].cpu().numpy().astype(np.float64)
    B = unpack_bits(out["bits"].cpu().numpy(), W.shape[1])
    return ar, ac, B, out


def recon(ar, ac, B, g):
    return np.einsum("kmn,kn,kmn->mn", np.repeat(ar, g, axis=2), ac, B)


@pytest.mark.parametrize("M,N,g,K,T", [(64, 128, 128, 1, 0), (64, 128, 128, 1, 3), (100, 256, 128, 2, 4), (37, 192, 64, 3, 3),
                                       (130, 96, 32, 4, 2), (65, 512, 256, 2, 5), (1, 128, 128, 2, 2)])
def test_matches_the_oracle(fb, M, N, g, K, T):
    W = synth.make_dense_weight(7, M * 7 + N + K, M, N, outlier_col_frac=0.05)
    eps = 1e-8
    ar, ac, B, _ = gpu_decomp(fb, W, g, K, T, eps)
    want_ar, want_ac, want_B = rc.rc_decomp_matrix(W, g, K, T, eps, dtype=np.float32)
    loss_gpu = ((W - recon(ar, ac, B, g)) ** 2).sum()
    loss_ref = ((W - recon(want_ar, want_ac, want_B, g)) ** 2).sum()
    energy = (W.astype(np.float64) ** 2).sum()
    assert abs(loss_gpu - loss_ref) <= 1e-4 * loss_ref + 1e-9 * energy, (loss_gpu, loss_ref)
    mism = (B != want_B).any(axis=0)
    assert mism.mean() <= 2e-3, f"{mism.sum()} of {mism.size} elements chose other signs"
    # where the signs agree over a whole (row, group) block and column, the scales are the same numbers
    assert np.allclose(ar, want_ar, rtol=2e-3, atol=1e-6 * np.abs(want_ar).max())
    assert np.allclose(ac, want_ac, rtol=2e-3, atol=1e-6)
    # every differing element is a near-tie under the GPU's own scales: its choice is optimal within rounding
    Mag = np.repeat(ar, g, axis=2) * ac[:, None, :]
    for i, j in np.argwhere(mism):
        errs = []
        for t in range(1 << K):
            b = np.array([1.0 if (t >> k) & 1 else -1.0 for k in range(K)])
            errs.append(abs(W[i, j] - (Mag[:, i, j] * b).sum()))
        mine = abs(W[i, j] - (Mag[:, i, j] * B[:, i, j]).sum())
        assert mine <= min(errs) + 1e-5 * (abs(W[i, j]) + np.abs(Mag[:, i, j]).sum())


def test_gpu_signs_are_optimal_for_the_gpu_scales(fb):
    """Eq. 6 on the device, element by element: no tuple beats the chosen one (beyond fp32 rounding)."""
    M, N, g, K = 96, 256, 128, 3
    W = synth.make_dense_weight(8, 1, M, N)
    ar, ac, B, _ = gpu_decomp(fb, W, g, K, 3, 1e-8)
    Mag = np.repeat(ar, g, axis=2) * ac[:, None, :]
    chosen = np.abs(W - (Mag * B).sum(axis=0))
    best = np.full(W.shape, np.inf)
    for t in range(1 << K):
        b = np.array([1.0 if (t >> k) & 1 else -1.0 for k in range(K)])[:, None, None]
        best = np.minimum(best, np.abs(W - (Mag * b).sum(axis=0)))
    assert (chosen <= best + 1e-6 * (np.abs(W) + np.abs(Mag).sum(axis=0))).all()


def test_rank_one_matrix_is_recovered(fb):
    r = np.random.default_rng(5)
    M, N = 64, 128
    a, b = np.abs(r.standard_normal(M)) + 0.1, np.abs(r.standard_normal(N)) + 0.1
    S = np.where(r.random((M, N)) < 0.5, -1.0, 1.0)
    W = (np.outer(a, b) * S).astype(np.float32)
    ar, ac, B, _ = gpu_decomp(fb, W, 128, 1, 2, 0.0)
    assert np.array_equal(B[0], S)
    assert np.allclose(recon(ar, ac, B, 128), W, rtol=1e-5, atol=1e-6)


def test_output_feeds_the_packer_and_the_linear_layer(fb):
    """Decompose on the GPU, hand the canonical arrays to fluxbin_pack, run the decode linear layer: the result is
    the product with the reconstructed matrix (computed from the fp16-rounded scales the layer stores)."""
    M, N, g, K = 256, 512, 128, 2
    W = synth.make_dense_weight(9, 2, M, N)
    _, _, B, out = gpu_decomp(fb, W, g, K, 4, 1e-8)
    rs = out["row_scale"].cpu().numpy().view(np.uint16)
    cs = out["col_scale"].cpu().numpy().view(np.uint16)
    L = synth.Linear(M, N, K, 0, g, 0, out["bits"].cpu().numpy().view(np.uint32), rs, cs, np.zeros(0, np.int32),
                     np.zeros((0, M, 0), np.uint32), np.zeros((0, M, N // g), np.uint16), np.zeros((0, 0), np.uint16))
    x = synth.make_activations(9, 3, 2, N)
    lin = fb.FluxBinLinear(L)
    y = lin.forward(torch.from_numpy(x.view(np.float16)).cuda(), lin.workspace(2), fp32_out=True)
    torch.cuda.synchronize()
    What = recon(rs.view(np.float16).astype(np.float64), cs.view(np.float16).astype(np.float64), B, g)
    want = x.view(np.float16).astype(np.float64) @ What.T
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3
    # and the decomposition is a useful approximation of W: two bases leave well under a fifth of its energy
    assert ((W - What) ** 2).sum() / (W.astype(np.float64) ** 2).sum() < 0.2


def test_argument_errors(fb):
    from paper_2608_15602_b200 import fluxbin
    W = torch.zeros((32, 128), dtype=torch.float32, device="cuda")
    bits = torch.zeros((1, 32, 4), dtype=torch.int32, device="cuda")
    rs = torch.zeros((1, 32, 1), dtype=torch.float16, device="cuda")
    cs = torch.zeros((1, 128), dtype=torch.float16, device="cuda")
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    args = [W.data_ptr(), 128, 32, 128, 128, 1, 1, 1e-8, bits.data_ptr(), rs.data_ptr(), cs.data_ptr(), None, None,
            ws.data_ptr(), ws.numel()]
    assert fluxbin.rc_decomp_status(*args) == 0
    bad = list(args); bad[0] = None
    assert fluxbin.rc_decomp_status(*bad) == 1                   # NULL
    bad = list(args); bad[4] = 96
    assert fluxbin.rc_decomp_status(*bad) == 2                   # N % g != 0: shape
    bad = list(args); bad[5] = 5
    assert fluxbin.rc_decomp_status(*bad) == 3                   # K out of range
    bad = list(args); bad[14] = 16
    assert fluxbin.rc_decomp_status(*bad) == 5                   # workspace too small
    bad = list(args); bad[0] = W.data_ptr() + 4
    assert fluxbin.rc_decomp_status(*bad) == 6                   # W not 16-byte aligned
    assert fluxbin.rc_decomp_workspace_size(32, 128, 96, 1) == 0


def test_full_size_matrix_on_sampled_groups(fb):
    """A 4096 x 4096 matrix (the size the timing is quoted on), g = 128, K = 2, T = 4: three column groups checked
    against the oracle in full; every group's error ratio must lie in the band two bases reach on this input."""
    M = N = 4096
    g, K, T = 128, 2, 4
    W = synth.make_dense_weight(10, 1, M, N, outlier_col_frac=0.05)
    ar, ac, B, _ = gpu_decomp(fb, W, g, K, T, 1e-8)
    for G in (0, 13, 31):
        cols = slice(G * g, (G + 1) * g)
        want_ar, want_ac, want_B = rc.rc_decomp(W[:, cols], K, T, 1e-8, dtype=np.float32)
        mism = (B[:, :, cols] != want_B).any(axis=0)
        assert mism.mean() <= 2e-3
        assert np.allclose(ar[:, :, G], want_ar, rtol=2e-3, atol=1e-6 * np.abs(want_ar).max())
        assert np.allclose(ac[:, cols], want_ac, rtol=2e-3, atol=1e-6)
    err = ((W - recon(ar, ac, B, g)) ** 2).reshape(M, N // g, g).sum(axis=(0, 2))
    energy = (W.astype(np.float64) ** 2).reshape(M, N // g, g).sum(axis=(0, 2))
    ratio = err / energy
    assert (ratio > 0.03).all() and (ratio < 0.15).all(), (ratio.min(), ratio.max())


def test_quantize_dense_helper(fb):
    """dense W -> decomposition -> packed layer in one call; the layer multiplies like W up to the quantisation error."""
    M, N = 512, 1024
    W = synth.make_dense_weight(12, 1, M, N)
    lin = fb.quantize_dense(torch.from_numpy(W).cuda(), g=128, K=4, T=6)
    x = synth.make_activations(12, 2, 1, N)
    y = lin.forward(torch.from_numpy(x.view(np.float16)).cuda(), lin.workspace(1), fp32_out=True)
    torch.cuda.synchronize()
    want = x.view(np.float16).astype(np.float64) @ W.astype(np.float64).T
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 0.12        # four bases leave < 1 % of W's energy


def test_hybrid_decomposition_matches_the_oracle(fb):
    """Global bases + refinement on given salient columns (Algorithm 2, steps 2-3) on the GPU against the oracle."""
    M, N, g, Kb, Ks, T = 96, 512, 128, 2, 2, 4
    W = synth.make_dense_weight(13, 1, M, N, outlier_col_frac=0.05)
    sal_idx = synth.salient_per_group(13, 2, N, g, 8)
    r = fb.hybrid_decompose(torch.from_numpy(W).cuda(), g, Kb, Ks, sal_idx, T, 1e-8)
    torch.cuda.synchronize()
    want = rc.hybrid_decomp(W, g, Kb, Ks, sal_idx, T, 1e-8, dtype=np.float32)
    B = unpack_bits(r["bits"].cpu().numpy(), N)
    sB = unpack_bits(r["sal_bits"].cpu().numpy(), len(sal_idx))
    got = rc.hybrid_reconstruct(r["row_scale_f32"].cpu().numpy().astype(np.float64), r["col_scale_f32"].cpu().numpy().astype(np.float64), B,
                                r["sal_row_scale_f32"].cpu().numpy().astype(np.float64),
                                r["sal_col_scale_f32"].cpu().numpy().astype(np.float64), sB, sal_idx, g)
    ref = rc.hybrid_reconstruct(*want, sal_idx, g)
    loss_gpu, loss_ref = ((W - got) ** 2).sum(), ((W - ref) ** 2).sum()
    assert abs(loss_gpu - loss_ref) <= 1e-3 * loss_ref
    assert ((sB != want[5]).any(axis=0)).mean() <= 5e-3
    assert np.allclose(r["sal_col_scale_f32"].cpu().numpy(), want[4], rtol=5e-3, atol=1e-5)
    assert np.allclose(r["sal_row_scale_f32"].cpu().numpy(), want[3], rtol=5e-3, atol=1e-5 * np.abs(want[3]).max())
    # the refinement helps: the error on the salient columns drops
    base = np.einsum("kmn,kn,kmn->mn", np.repeat(r["row_scale_f32"].cpu().numpy().astype(np.float64), g, axis=2),
                     r["col_scale_f32"].cpu().numpy().astype(np.float64), B)
    assert ((W[:, sal_idx] - got[:, sal_idx]) ** 2).sum() < 0.5 * ((W[:, sal_idx] - base[:, sal_idx]) ** 2).sum()


def test_quantize_dense_hybrid_layer_runs_through_the_linear_path(fb):
    M, N, g = 256, 1024, 128
    W = synth.make_dense_weight(14, 1, M, N, outlier_col_frac=0.05)
    sal_idx = synth.salient_random(14, 2, N, 0.05)                  # uneven counts per group, some groups empty
    Wt = torch.from_numpy(W).cuda()
    lin2 = fb.quantize_dense(Wt, g=g, K=2, T=6)
    linh = fb.quantize_dense(Wt, g=g, K=2, T=6, sal_idx=sal_idx, Ks=2)
    x = synth.make_activations(14, 3, 2, N)
    xt = torch.from_numpy(x.view(np.float16)).cuda()
    want = x.view(np.float16).astype(np.float64) @ W.astype(np.float64).T
    err = []
    for lin in (lin2, linh):
        y = lin.forward(xt, lin.workspace(2), fp32_out=True)
        torch.cuda.synchronize()
        err.append(np.linalg.norm(y.cpu().numpy().astype(np.float64) - want) / np.linalg.norm(want))
    assert err[1] < err[0] < 0.4            # the salient bases reduce the output error
    # and the packed hybrid layer round-trips to the arrays the decomposition produced
    got = linh.unpack()
    assert got.n_sal == len(sal_idx) and np.array_equal(got.sal_idx, sal_idx)


def test_salient_collect_gathers_the_padded_refinement(fb):
    """fluxbin_rc_salient_collect against a numpy gather of the same padded arrays: sign bits of the virtual columns,
    block row scales scattered to their groups (zero elsewhere), column scales, fp16 rounding to nearest even."""
    from paper_2608_15602_b200 import fluxbin
    rng = np.random.default_rng(5)
    M, N, g, Ks, width = 37, 1024, 128, 2, 32
    groups = np.array([0, 2, 3, 7], np.int32)                       # blocks of the padded matrix -> row-scale groups
    counts = [5, 32, 1, 17]
    sal_idx = np.concatenate([G * g + np.sort(rng.choice(g, c, replace=False)) for G, c in zip(groups, counts)]).astype(np.int32)
    n_sal, nblocks = len(sal_idx), len(groups)
    pos = np.concatenate([b * width + np.arange(c) for b, c in enumerate(counts)]).astype(np.int32)
    ncols_p = nblocks * width
    bits_p = rng.integers(0, 2 ** 32, size=(Ks, M, ncols_p // 32), dtype=np.uint64).astype(np.uint32)
    rs_p = rng.standard_normal((Ks, M, nblocks)).astype(np.float32) * 0.02
    cs_p = rng.standard_normal((Ks, ncols_p)).astype(np.float32)
    dev = lambda a: torch.from_numpy(a).cuda()
    out_bits = torch.full((Ks, M, (n_sal + 31) // 32), -1, dtype=torch.int32, device="cuda")
    out_rs = torch.full((Ks, M, N // g), 7, dtype=torch.float16, device="cuda")
    out_cs = torch.empty((Ks, n_sal), dtype=torch.float16, device="cuda")
    out_rs32 = torch.empty((Ks, M, N // g), dtype=torch.float32, device="cuda")
    out_cs32 = torch.empty((Ks, n_sal), dtype=torch.float32, device="cuda")
    t = [dev(bits_p.view(np.int32)), dev(rs_p), dev(cs_p), dev(pos), dev(groups)]
    fluxbin.rc_salient_collect(t[0].data_ptr(), t[1].data_ptr(), t[2].data_ptr(), t[3].data_ptr(), t[4].data_ptr(), M, N, g, Ks,
                               n_sal, width, nblocks, out_bits.data_ptr(), out_rs.data_ptr(), out_cs.data_ptr(),
                               out_rs32.data_ptr(), out_cs32.data_ptr())
    torch.cuda.synchronize()
    signs = (bits_p[:, :, pos // 32] >> (pos % 32).astype(np.uint32)) & 1                       # [Ks][M][n_sal]
    want_bits = np.zeros((Ks, M, (n_sal + 31) // 32), np.uint32)
    for v in range(n_sal):
        want_bits[:, :, v // 32] |= signs[:, :, v].astype(np.uint32) << np.uint32(v % 32)
    assert np.array_equal(out_bits.cpu().numpy().view(np.uint32), want_bits)
    want_rs = np.zeros((Ks, M, N // g), np.float32)
    want_rs[:, :, groups] = rs_p
    assert np.array_equal(out_rs32.cpu().numpy(), want_rs)
    assert np.array_equal(out_rs.cpu().numpy().view(np.uint16), want_rs.astype(np.float16).view(np.uint16))
    assert np.array_equal(out_cs32.cpu().numpy(), cs_p[:, pos])
    assert np.array_equal(out_cs.cpu().numpy().view(np.uint16), cs_p[:, pos].astype(np.float16).view(np.uint16))


PACK_CASES = [(1, 32, 1, 0, 32, 0), (5, 128, 2, 1, 32, 7), (33, 384, 3, 2, 128, 40), (100, 256, 1, 1, 256, 19),
              (257, 1024, 2, 1, 128, 51), (65, 640, 2, 1, 128, 640), (127, 128, 4, 4, 64, 128), (600, 2048, 2, 2, 128, 128),
              (1000, 512, 2, 1, 512, 1), (31, 256, 2, 2, 64, 9), (40, 65536, 1, 1, 128, 300)]      # last: the widest layer


@pytest.mark.parametrize("M,N,Kb,Ks,g,n_sal", PACK_CASES)
def test_pack_device_writes_the_bytes_of_pack_host(fb, M, N, Kb, Ks, g, n_sal):
    """The device packer and the host packer produce the same buffer, byte for byte (all scale formats, narrow and
    full last salient pairs, ragged row counts), and the handle it returns multiplies like the layer."""
    from paper_2608_15602_b200 import fluxbin
    from test_gpu_parity import layer_of, check
    import oracle
    L = layer_of(M + 7 * N, M, N, Kb, Ks, g, n_sal)
    want = fluxbin.pack_host(L)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int32 if a.dtype == np.uint32 else a.dtype)).cuda()
    has_sal = L.Ks > 0 and L.n_sal > 0
    arrays = [dev(L.bits), dev(L.row_scale.view(np.int16)), dev(L.col_scale.view(np.int16))]
    arrays += [dev(L.sal_idx), dev(L.sal_bits), dev(L.sal_row_scale.view(np.int16)), dev(L.sal_col_scale.view(np.int16))] if has_sal else []
    ptrs = [a.data_ptr() for a in arrays] + ([None] * 4 if not has_sal else [])
    packed = torch.full((want.size,), 0xAB, dtype=torch.uint8, device="cuda")
    ws = torch.empty(max(256, fluxbin.pack_device_workspace_size(N, g, L.n_sal)), dtype=torch.uint8, device="cuda")
    w = fluxbin.pack_device((L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal), ptrs, L.sal_idx, packed.data_ptr(), want.size, ws.data_ptr(),
                            ws.numel(), buffer=packed)
    got = packed.cpu().numpy()
    assert np.array_equal(got, want), f"first difference at byte {np.nonzero(got != want)[0][:5]}"
    lin = object.__new__(fb.FluxBinLinear)
    lin.device, lin.buffer, lin.weight, lin.M, lin.N, lin.packed_bytes = packed.device, packed, w, M, N, want.size
    x = synth.make_activations(3, M, 2, N)
    y = lin.forward(torch.from_numpy(x.view(np.float16)).cuda(), lin.workspace(2), fp32_out=True)
    torch.cuda.synchronize()
    check(y.cpu().numpy(), oracle.linear_direct(L, x), "device-packed layer", L, x)
    # argument errors are statuses
    st, _ = fluxbin.pack_device_status((L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal), ptrs, L.sal_idx, packed.data_ptr(), want.size - 1,
                                       ws.data_ptr(), ws.numel())
    assert st == 5
    st, _ = fluxbin.pack_device_status((L.M, L.N + 1, L.Kb, L.Ks, L.g, L.n_sal), ptrs, L.sal_idx, packed.data_ptr(), want.size,
                                       ws.data_ptr(), ws.numel())
    assert st == 2
