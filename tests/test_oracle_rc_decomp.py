"""Pins for the row-column binary decomposition oracle (oracle/rc_decomp.py): what the paper and the mathematics
fix without reference to any implementation -- closed forms, least-squares optimality (Proposition 3.2, Eq. 5),
exhaustive optimality of the sign search (Proposition 3.3, Eq. 6), monotone descent of the alternating scheme,
fixed points, symmetries, and the textbook special case K = 1, T = 0."""
import itertools

import numpy as np
import pytest

from oracle import rc_decomp as rc


def rng(seed):
    return np.random.default_rng(260815602 + seed)


def test_k1_t0_is_the_classic_binary_code():
    """No alternating steps, one base: B = sign(X), a_c = 1, a_r = mean |X| per row (the closed form of a binary
    weight with one scale per row) -- Eq. 5 with a_c = 1."""
    X = rng(1).standard_normal((7, 24))
    ar, ac, B = rc.rc_decomp(X, 1, 0, eps=0.0)
    assert np.array_equal(B[0], np.where(X >= 0, 1.0, -1.0))
    assert np.array_equal(ac[0], np.ones(24))
    assert np.allclose(ar[0], np.abs(X).mean(axis=1), rtol=1e-15)


@pytest.mark.parametrize("axis", ["row", "col"])
def test_scale_update_is_the_least_squares_solution(axis):
    """Eq. 5 against numpy's least-squares solver, one scalar problem per row (or column)."""
    r = rng(2)
    M, n = 6, 9
    T = r.standard_normal((M, n))
    B = np.where(r.random((M, n)) < 0.5, -1.0, 1.0)
    if axis == "row":
        other = np.abs(r.standard_normal(n)) + 0.1
        got = rc._scale_update(T, other[None, :], B, 0.0)
        want = [np.linalg.lstsq((other * B[i])[:, None], T[i], rcond=None)[0][0] for i in range(M)]
    else:
        other = np.abs(r.standard_normal(M)) + 0.1
        got = rc._scale_update(T, other[:, None], B, 0.0)
        want = [np.linalg.lstsq((other * B[:, j])[:, None], T[:, j], rcond=None)[0][0] for j in range(n)]
    assert np.allclose(got, want, rtol=1e-12)


def test_epsilon_enters_the_denominator_as_printed():
    T = np.array([[2.0, -4.0]])
    B = np.array([[1.0, -1.0]])
    ac = np.array([1.0, 0.5])
    # num = 1*2 + (-0.5)(-4) = 4, den = 1 + 0.25 + eps
    assert rc._scale_update(T, ac[None, :], B, 0.75)[0] == pytest.approx(4.0 / 2.0, rel=1e-15)


@pytest.mark.parametrize("K", [1, 2, 3])
def test_sign_search_is_exhaustively_optimal(K):
    """Eq. 6 against brute force over all 2^K tuples, element by element."""
    r = rng(3 + K)
    M, n = 4, 5
    X = r.standard_normal((M, n))
    ar = np.abs(r.standard_normal((K, M))) + 0.05
    ac = np.abs(r.standard_normal((K, n))) + 0.05
    B = rc.sign_search(X, ar, ac)
    for i in range(M):
        for j in range(n):
            errs = {b: abs(X[i, j] - sum(ar[k, i] * ac[k, j] * b[k] for k in range(K)))
                    for b in itertools.product((-1.0, 1.0), repeat=K)}
            best = min(errs.values())
            assert errs[tuple(B[:, i, j])] == pytest.approx(best, abs=1e-15)


def test_sign_search_tie_goes_to_the_lowest_tuple_index():
    # X = 0 with one base: both signs give |m|; index 0 means b = -1
    B = rc.sign_search(np.zeros((1, 1)), np.ones((1, 1)), np.ones((1, 1)))
    assert B[0, 0, 0] == -1.0
    # two equal bases, X = 0: tuples (-,+) [t=2] and (+,-) [t=1] both give 0; t = 1 wins: b_1 = +1, b_2 = -1
    B = rc.sign_search(np.zeros((1, 1)), np.ones((2, 1)), np.ones((2, 1)))
    assert (B[0, 0, 0], B[1, 0, 0]) == (1.0, -1.0)


@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_every_update_is_a_descent_step(K):
    """Each of the three updates is the exact minimiser of the loss over its block of variables (eps = 0), so the
    squared error never increases along the whole run."""
    X = rng(10 + K).standard_normal((16, 32)) * 0.02
    trace = []
    rc.rc_decomp(X, K, 6, eps=0.0, trace=trace)
    losses = [l for _, l in trace]
    for (name, a), b in zip(trace[1:], losses[:-1]):
        assert a <= b * (1 + 1e-12) + 1e-30, f"{name}: {b} -> {a}"
    assert losses[-1] < losses[0]
    assert losses[-1] < (X ** 2).sum()


def test_more_bases_fit_better():
    X = rng(20).standard_normal((32, 64))
    err = []
    for K in (1, 2, 3, 4):
        ar, ac, B = rc.rc_decomp(X, K, 8)
        err.append(((X - rc.reconstruct(ar, ac, B)) ** 2).sum() / (X ** 2).sum())
    assert err[0] > err[1] > err[2] > err[3]
    assert err[0] < 0.45            # one binary base with per-row scales leaves 1 - 2/pi = 0.363 of a Gaussian's energy
    assert err[0] == pytest.approx(1 - 2 / np.pi, abs=0.06)


def test_rank_one_matrix_is_recovered_exactly():
    """X = (a b^T) . S with positive a, b: the initial signs are S, and the first column update makes
    a_r a_c^T = a b^T (a_r = a mean(b), a_c = b / mean(b))."""
    r = rng(30)
    a, b = np.abs(r.standard_normal(9)) + 0.1, np.abs(r.standard_normal(12)) + 0.1
    S = np.where(r.random((9, 12)) < 0.5, -1.0, 1.0)
    X = np.outer(a, b) * S
    ar, ac, B = rc.rc_decomp(X, 1, 1, eps=0.0)
    assert np.array_equal(B[0], S)
    assert np.allclose(np.outer(ar[0], ac[0]), np.outer(a, b), rtol=1e-13)
    assert np.allclose(ar[0], a * b.mean(), rtol=1e-13)


def test_exact_decomposition_is_a_fixed_point_of_every_update():
    """If X is exactly sum_k (a_r a_c^T) . B with well separated magnitudes, the sign search returns B and both
    scale updates return the scales."""
    r = rng(40)
    K, M, n = 3, 8, 10
    ar = (np.abs(r.standard_normal((K, M))) + 0.5) * np.array([4.0, 1.0, 0.2])[:, None]
    ac = np.abs(r.standard_normal((K, n))) * 0.1 + 1.0
    B = np.where(r.random((K, M, n)) < 0.5, -1.0, 1.0)
    X = rc.reconstruct(ar, ac, B)
    assert np.array_equal(rc.sign_search(X, ar, ac), B)
    for k in range(K):
        target = X - rc.reconstruct(np.delete(ar, k, 0), np.delete(ac, k, 0), np.delete(B, k, 0))
        assert np.allclose(rc._scale_update(target, ac[k][None, :], B[k], 0.0), ar[k], rtol=1e-12)
        assert np.allclose(rc._scale_update(target, ar[k][:, None], B[k], 0.0), ac[k], rtol=1e-12)


def test_symmetries():
    X = rng(50).standard_normal((10, 16))
    ar, ac, B = rc.rc_decomp(X, 2, 4)
    ar2, ac2, B2 = rc.rc_decomp(-X, 2, 4)                 # negation flips every sign, keeps the scales
    assert np.array_equal(B2, -B) and np.allclose(ar2, ar, rtol=1e-12) and np.allclose(ac2, ac, rtol=1e-12)
    ar3, ac3, B3 = rc.rc_decomp(3.0 * X, 2, 4, eps=0.0)   # a positive factor lands in the row scales
    ar0, ac0, B0 = rc.rc_decomp(X, 2, 4, eps=0.0)
    assert np.array_equal(B3, B0) and np.allclose(ar3, 3.0 * ar0, rtol=1e-12) and np.allclose(ac3, ac0, rtol=1e-12)


def test_fp32_sign_search_differs_only_on_near_ties():
    X = rng(60).standard_normal((64, 128)).astype(np.float32).astype(np.float64)
    ar = np.abs(rng(61).standard_normal((2, 64))) + 0.1
    ac = np.abs(rng(62).standard_normal((2, 128))) + 0.1
    B64, B32 = rc.sign_search(X, ar, ac), rc.sign_search(X, ar, ac, np.float32)
    diff = np.argwhere((B64 != B32).any(axis=0))
    assert len(diff) <= 2
    for i, j in diff:      # both choices are within fp32 rounding of the optimum
        e = lambda Bx: abs(X[i, j] - sum(ar[k, i] * ac[k, j] * Bx[k, i, j] for k in range(2)))
        assert abs(e(B64) - e(B32)) <= 1e-6 * (abs(X[i, j]) + (ar[:, i] * ac[:, j]).sum())


def test_matrix_form_decomposes_column_groups_independently():
    W = rng(70).standard_normal((12, 96))
    ar, ac, B = rc.rc_decomp_matrix(W, 32, 2, 3)
    assert ar.shape == (2, 12, 3) and ac.shape == (2, 96) and B.shape == (2, 12, 96)
    a1, c1, b1 = rc.rc_decomp(W[:, 32:64], 2, 3)
    assert np.array_equal(ar[:, :, 1], a1) and np.array_equal(ac[:, 32:64], c1) and np.array_equal(B[:, :, 32:64], b1)


def test_single_row_and_single_column_blocks():
    """Degenerate shapes: with one row every column has a scale of its own, so one column update of Eq. 5 (the sum
    over i has a single term) reproduces X exactly; with one column the row update does."""
    x = rng(80).standard_normal((1, 16))
    ar, ac, B = rc.rc_decomp(x, 1, 1, eps=0.0)
    assert np.allclose(rc.reconstruct(ar, ac, B), x, rtol=1e-13)
    assert np.allclose(ac[0], np.abs(x[0]) / np.abs(x[0]).mean(), rtol=1e-13)       # a_r = mean |x|, a_c = |x| / a_r
    y = rng(81).standard_normal((9, 1))
    ar, ac, B = rc.rc_decomp(y, 1, 0, eps=0.0)
    assert np.allclose(rc.reconstruct(ar, ac, B), y, rtol=1e-13)


def test_hybrid_refinement_only_touches_salient_columns_and_never_hurts():
    """Algorithm 2, steps 2-3: the extra bases approximate the residual on the salient columns, so the other
    columns keep the global reconstruction and the error on every salient column block does not grow."""
    r = rng(90)
    M, N, g = 24, 128, 32
    W = r.standard_normal((M, N)) * 0.02
    W[:, [3, 40, 41, 99]] *= 8.0
    sal_idx = np.array([3, 40, 41, 99, 100])
    # (a one-column salient block is fitted exactly by its first base; the second base then has a zero residual
    # and zero scales, and Eq. 5 becomes 0 / (0 + eps): this is what the stability constant is for)
    ar, ac, B, sr, sc, sB = rc.hybrid_decomp(W, g, 2, 2, sal_idx, 4, eps=1e-12)
    base = np.einsum("kmn,kn,kmn->mn", np.repeat(ar, g, axis=2), ac, B)
    full = rc.hybrid_reconstruct(ar, ac, B, sr, sc, sB, sal_idx, g)
    other = np.setdiff1d(np.arange(N), sal_idx)
    assert np.array_equal(full[:, other], base[:, other])
    for G in range(N // g):
        v = sal_idx[sal_idx // g == G]
        if len(v):
            assert ((W[:, v] - full[:, v]) ** 2).sum() <= ((W[:, v] - base[:, v]) ** 2).sum() * (1 + 1e-9)
    assert np.all(sr[:, :, 2] == 0)                      # group 2 (columns 64..95) has no salient column
    # with every column salient the refinement is a second RC_Decomp of the whole residual block
    ar2, ac2, B2, sr2, sc2, sB2 = rc.hybrid_decomp(W[:, :32], 32, 1, 1, np.arange(32), 3, eps=0.0)
    R = W[:, :32] - np.einsum("kmn,kn,kmn->mn", np.repeat(ar2, 32, axis=2), ac2, B2)
    a, c, b = rc.rc_decomp(R, 1, 3, eps=0.0)
    assert np.array_equal(sB2, b) and np.allclose(sr2[:, :, 0], a, rtol=1e-14) and np.allclose(sc2, c, rtol=1e-14)
