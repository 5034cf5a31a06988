"""Pins for the CPU oracle: brute force, closed forms, invariants, printed values.

Each test is chosen so that a plausible mistake in oracle/fluxbin_oracle.c (a dropped term, a
wrong sign, a transposed index, a wrong group for a row scale) fails it.
"""
import numpy as np
import pytest

import oracle
from oracle import models
from paper_2608_15602_b200 import synth
from conftest import golden_rows


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)


def h(vals):
    return np.asarray(vals, np.float32).astype(np.float16).view(np.uint16)


def tiny(seed, M, N, Kb, Ks, g, n_sal):
    if n_sal > 0 and Ks > 0:
        rng = np.random.default_rng(seed)
        idx = np.sort(rng.choice(N, size=n_sal, replace=False)).astype(np.int32)
    else:
        idx = None
    return synth.make_linear(seed, 7, M, N, Kb, Ks, g, idx)


def numpy_dense(L):
    """Independent numpy reconstruction of What (vectorised, from the definition)."""
    W = np.zeros((L.M, L.N))
    cols = np.arange(L.N)
    for k in range(L.Kb):
        B = ((L.bits[k][:, cols // 32] >> (cols % 32).astype(np.uint32)) & 1).astype(np.float64) * 2 - 1
        W += f16(L.row_scale[k])[:, cols // L.g] * f16(L.col_scale[k])[None, :] * B
    v = np.arange(L.n_sal)
    for k in range(L.Ks):
        B = ((L.sal_bits[k][:, v // 32] >> (v % 32).astype(np.uint32)) & 1).astype(np.float64) * 2 - 1
        W[:, L.sal_idx] += f16(L.sal_row_scale[k])[:, L.sal_idx // L.g] * f16(L.sal_col_scale[k])[None, :] * B
    return W


def test_half_conversion_all_patterns():
    """Every finite fp16 bit pattern converts exactly (numpy's float16 is the independent reference)."""
    allbits = np.arange(65536, dtype=np.uint16)
    ref = allbits.view(np.float16).astype(np.float64)
    got = np.array([oracle.half_to_double(int(b)) for b in allbits])
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin], ref[fin])
    assert np.all(np.signbit(got[fin]) == np.signbit(ref[fin]))
    assert np.all(np.isnan(got[np.isnan(ref)]))
    assert np.array_equal(got[np.isinf(ref)], ref[np.isinf(ref)])


SHAPES = [(M, N, g) for M in (1, 5, 33) for (N, g) in ((32, 32), (128, 32), (128, 128), (384, 128), (384, 384))]


@pytest.mark.parametrize("M,N,g", SHAPES)
@pytest.mark.parametrize("Kb,Ks,n_sal", [(1, 0, 0), (2, 0, 0), (3, 1, 1), (2, 1, 7), (2, 2, 9), (4, 1, 8), (2, 1, -1)])
def test_direct_equals_brute_force_dense(M, N, g, Kb, Ks, n_sal):
    n_sal = N if n_sal < 0 else min(n_sal, N)
    L = tiny(1000 + M + N + g + Kb, M, N, Kb, Ks, g, n_sal)
    x = synth.make_activations(5, M + N, 3, N)
    W = oracle.dense_weight(L)
    Wn = numpy_dense(L)
    assert np.allclose(W, Wn, rtol=1e-14, atol=0)
    y_dense = f16(x) @ Wn.T                       # numpy matmul on the numpy matrix
    y_dense_c = oracle.dense_linear(L, x)
    y = oracle.linear_direct(L, x)
    scale = np.abs(f16(x)) @ np.abs(Wn).T + 1e-300
    assert np.all(np.abs(y - y_dense) <= 1e-13 * scale)
    assert np.all(np.abs(y_dense_c - y_dense) <= 1e-13 * scale)


def test_one_hot_reads_back_columns():
    """x = e_j  =>  y = What[:, j]: catches transposed operands and wrong salient scatter."""
    L = tiny(3, 6, 128, 2, 2, 32, 11)
    W = numpy_dense(L)
    for j in list(range(0, 128, 13)) + [int(c) for c in L.sal_idx]:
        x = np.zeros((1, 128), np.uint16)
        x[0, j] = h([1.0])[0]
        y = oracle.linear_direct(L, x)
        assert np.allclose(y[0], W[:, j], rtol=1e-14, atol=0)


def test_all_plus_one_unit_scales_closed_form():
    """All bits 1, all scales 1  =>  y_i = Kb*sum_j x_j + Ks*sum_{j in I_sal} x_j."""
    M, N, Kb, Ks, g = 4, 256, 3, 2, 64
    L = tiny(11, M, N, Kb, Ks, g, 19)
    L.bits[:] = 0xFFFFFFFF
    L.sal_bits[:] = 0xFFFFFFFF
    one = h([1.0])[0]
    for a in (L.row_scale, L.col_scale, L.sal_row_scale, L.sal_col_scale):
        a[:] = one
    x = synth.make_activations(2, 1, 2, N)
    xs = f16(x)
    want = Kb * xs.sum(1) + Ks * xs[:, L.sal_idx].sum(1)
    for fn in (oracle.linear_direct, oracle.lut_linear):
        y = fn(L, x)
        assert np.allclose(y, want[:, None], rtol=1e-12)


def test_all_minus_one_flips_sign():
    """All bits 0 (=> -1) negates the all-ones result: pins the bit -> sign convention."""
    M, N = 3, 64
    L = tiny(12, M, N, 1, 0, 64, 0)
    L.bits[:] = 0
    L.row_scale[:] = h([1.0])[0]
    L.col_scale[:] = h([1.0])[0]
    x = synth.make_activations(2, 9, 1, N)
    assert np.allclose(oracle.linear_direct(L, x), -f16(x).sum(), rtol=1e-12)


def test_complementary_bases_cancel_exactly():
    """B2 = not B1 with equal scales => y = 0 exactly."""
    L = tiny(13, 7, 128, 2, 0, 128, 0)
    L.bits[1] = ~L.bits[0]
    L.row_scale[1] = L.row_scale[0]
    L.col_scale[1] = L.col_scale[0]
    x = synth.make_activations(2, 3, 2, 128)
    y = oracle.linear_direct(L, x)
    scale = np.abs(f16(x)) @ np.abs(numpy_dense(tiny(13, 7, 128, 2, 0, 128, 0))).T
    assert np.all(np.abs(y) <= 1e-13 * (scale + 1))


def test_row_scale_group_is_the_columns_group():
    """Setting one (row, group) scale to zero removes exactly that group's columns from that row."""
    L = tiny(14, 4, 256, 1, 0, 64, 0)
    x = synth.make_activations(2, 4, 1, 256)
    y0 = oracle.linear_direct(L, x)
    L2 = tiny(14, 4, 256, 1, 0, 64, 0)
    L2.row_scale[0, 2, 1] = 0
    y1 = oracle.linear_direct(L2, x)
    cols = np.arange(64, 128)
    B = ((L.bits[0][2, cols // 32] >> (cols % 32).astype(np.uint32)) & 1).astype(np.float64) * 2 - 1
    removed = f16(L.row_scale[0, 2, 1]) * np.sum(f16(x)[0, cols] * f16(L.col_scale[0, cols]) * B)
    d = y0 - y1
    assert abs(d[0, 2] - removed) <= 1e-12 * abs(removed)
    assert np.all(d[0, [0, 1, 3]] == 0)


def test_salient_all_columns_equals_extra_global_base():
    """sal_idx = 0..N-1 with Ks=1 is the same matrix as a (Kb+1)-base global layer."""
    M, N, g = 5, 128, 32
    idx = np.arange(N, dtype=np.int32)
    L = synth.make_linear(21, 1, M, N, 2, 1, g, idx)
    G = synth.make_linear(21, 1, M, N, 3, 0, g)
    G.bits[:2], G.row_scale[:2], G.col_scale[:2] = L.bits, L.row_scale, L.col_scale
    G.bits[2], G.row_scale[2], G.col_scale[2] = L.sal_bits[0], L.sal_row_scale[0], L.sal_col_scale[0]
    x = synth.make_activations(2, 5, 2, N)
    a, b = oracle.linear_direct(L, x), oracle.linear_direct(G, x)
    assert np.allclose(a, b, rtol=1e-12, atol=1e-14)


def test_no_salient_equals_global_only():
    L = tiny(22, 5, 128, 2, 1, 128, 0)
    assert L.Ks == 0
    x = synth.make_activations(2, 6, 1, 128)
    assert np.allclose(oracle.linear_direct(L, x), f16(x) @ numpy_dense(L).T, rtol=1e-12, atol=1e-15)


def test_batch_rows_are_independent_and_ldx_respected():
    L = tiny(23, 9, 128, 2, 1, 64, 5)
    x = synth.make_activations(2, 7, 3, 160)     # ldx = 160 > N
    y = oracle.linear_direct(L, x)
    for b in range(3):
        yb = oracle.linear_direct(L, x[b:b + 1, :128].copy())
        assert np.array_equal(y[b], yb[0])


@pytest.mark.parametrize("mu", [4, 8])
def test_lut_entries_are_signed_sums_and_obey_closed_forms(mu):
    rng = np.random.default_rng(mu)
    a = rng.standard_normal(3 * mu)
    T = oracle.lut_tables(a, mu)
    assert T.shape == (3, 1 << mu)
    for t in range(3):
        sub = a[t * mu:(t + 1) * mu]
        for p in range(1 << mu):               # the defining sum, entry by entry
            signs = np.array([1.0 if (p >> n) & 1 else -1.0 for n in range(mu)])
            assert abs(T[t, p] - np.dot(sub, signs)) <= 1e-14 * np.abs(sub).sum()
        full = (1 << mu) - 1
        assert abs(T[t, full] - sub.sum()) <= 1e-14 * np.abs(sub).sum()
        assert abs(T[t, 0] + sub.sum()) <= 1e-14 * np.abs(sub).sum()
        p = np.arange(1 << mu)
        assert np.allclose(T[t, p], -T[t, full - p], atol=1e-13)       # LUT[p] = -LUT[~p]
        assert abs(T[t].sum()) <= 1e-11
        for n in range(mu):                                            # flipping bit n moves by 2*a_n
            q = p[(p >> n) & 1 == 0]
            assert np.allclose(T[t, q | (1 << n)] - T[t, q], 2 * sub[n], atol=1e-13)


@pytest.mark.parametrize("mu", [4, 8])
@pytest.mark.parametrize("M,N,g,Kb,Ks,n_sal", [(5, 128, 32, 2, 1, 7), (33, 384, 128, 2, 2, 40), (4, 256, 256, 3, 0, 0),
                                               (6, 128, 64, 1, 1, 128), (3, 256, 64, 4, 2, 1)])
def test_lut_form_equals_direct_sum(mu, M, N, g, Kb, Ks, n_sal):
    """Eq. 13-15 (tables + lookups + VCM gather) compute the same numbers as Eq. 10."""
    L = tiny(40 + M, M, N, Kb, Ks, g, n_sal)
    x = synth.make_activations(3, M, 2, N)
    y = oracle.linear_direct(L, x)
    yl = oracle.lut_linear(L, x, mu)
    scale = np.abs(f16(x)) @ np.abs(numpy_dense(L)).T + 1e-300
    assert np.all(np.abs(y - yl) <= 1e-12 * scale)


def test_abw_matches_printed_table():
    for Kb, Ks, g, s, printed in golden_rows("abw_table6.txt"):
        got = models.abw(4096, 4096, int(Kb), int(Ks), int(g), int(s))
        assert abs(got - printed) <= 0.011, (Kb, Ks, g, s, got, printed)


def test_smem_model_matches_printed_table():
    for mu, bs, printed_kb in golden_rows("smem_table9.txt"):
        got = models.smem_bytes(int(bs), 2, 128, 64, int(mu)) / 1024
        assert abs(got - printed_kb) < 0.5


def test_effective_tflops_matches_printed_table():
    for M, N, ns, lat, printed in golden_rows("tflops_table10.txt"):
        got = models.effective_tflops(int(M), int(N), int(ns), lat * 1e-6)
        assert abs(got - printed) <= 0.006


def test_complexity_reduction_factor():
    """Lookup count is mu/Kb times smaller than the M*N multiply-adds of a dense GEMV (mu=8, Kb=2 -> 4x)."""
    build, read = models.complexity(4096, 4096, 2, 0, 0, 8)
    assert (4096 * 4096) / read == 4.0
    assert build == 2 * (4096 // 8) * 256


def test_algorithmic_bytes_consistent_with_storage_model():
    for (M, N, Kb, Ks, g, n_sal) in [(4096, 4096, 2, 0, 128, 0), (8192, 28672, 2, 1, 128, 1434), (4096, 4096, 2, 2, 128, 256)]:
        bits = models.storage_bits(M, N, Kb, Ks, g, n_sal)
        byts = models.algorithmic_bytes(M, N, Kb, Ks, g, n_sal, 0)
        pad = Ks * M * (((n_sal + 7) // 8) * 8 - n_sal) if Ks and n_sal else 0
        assert byts * 8 == bits + pad


def test_generator_is_reproducible_and_canonical():
    a = synth.make_config_linear(1, 0, 0)
    assert (a.M, a.N, a.Kb, a.Ks, a.n_sal) == (4096, 4096, 2, 1, 205)
    assert np.all(np.diff(a.sal_idx) > 0) and a.sal_idx.min() >= 0 and a.sal_idx.max() < 4096
    assert np.all(a.sal_bits[:, :, -1] >> np.uint32(205 % 32) == 0)
    b = synth.make_linear(synth.BASE_SEED + 1, 0, 64, 4096, 2, 1, 128, a.sal_idx)
    assert np.array_equal(b.col_scale, a.col_scale)
    rs = f16(a.row_scale)
    assert 0.012 < rs.mean() < 0.020 and rs.min() >= 0          # E|N(0,0.02)| = 0.01596
    cs = f16(a.col_scale)
    assert 0.99 < cs.mean() < 1.01
    frac = np.unpackbits(a.bits[:, :64].view(np.uint8)).mean()
    assert 0.49 < frac < 0.51
    x = f16(synth.make_config_activations(1, 0, 0, 4))
    assert x.shape == (4, 4096) and 1.5 < x.std() < 3.0         # 1 % channels x20 inflate the std
