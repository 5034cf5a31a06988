"""CPU oracle for the row-column binary decomposition (test infrastructure only).

RC_Decomp of the paper's sub-routine listing (Algorithm 3, left column), written out in numpy fp64 in the
paper's order and notation, for ONE block X [M][n] (a column group of the weight matrix, or the gathered salient
columns of a group -- the caller applies the mask by handing over only the masked-in columns):

  residual R <- X;  for k = 1..K: init B(k), a_r(k), a_c(k) from R;  R <- R - (a_r a_c^T) . B(k)
  for iter = 1..T:
      for k = 1..K:  a_r(k) <- Eq. 5 (row form),  a_c(k) <- Eq. 5 (column form)
      {B(k)} <- Eq. 6: per element, the sign tuple that minimises |X_ij - sum_k M(k)_ij b_k| over all 2^K tuples
  reconstruct  X^ = sum_k (a_r(k) a_c(k)^T) . B(k)

Readings where the paper is silent (also listed in the design notes):
  R1  "Init ... from R": B = sign(R) with sign(0) = +1, a_c = 1, a_r by Eq. 5 (which for a_c = 1 is the mean of
      |R_ij| over the row: the classic scale of a binary code).
  R2  Eq. 5 is printed for a single base with target W.  With K >= 2 the target of base k is what the other bases
      leave: X - sum_{k' != k} (a_r(k') a_c(k')^T) . B(k')  -- the only reading under which the update is the
      least-squares minimiser the proposition claims.
  R3  epsilon: a parameter (default 1e-8), added to the denominators exactly as printed.
  R4  The enumeration order of Eq. 6's tuples decides ties: tuple index t = sum_k [b_k = +1] 2^k, lowest index wins.

`dtype=np.float32` evaluates the sign search of Eq. 6 in fp32 in a fixed order (magnitude M = a_r * a_c rounded
once, e = X - M(1) b_1 - ... subtracted one base at a time) -- the precision in which the CUDA path takes that
integer decision; everything else stays fp64.
Nothing here imports the CUDA package.
"""
from __future__ import annotations

import numpy as np


def _scale_update(T, other, B, eps, axis=None):
    """Eq. 5 for one scale vector: T [M][n] target, `other` the fixed scale vector broadcast along the summed
    axis (shape [1][n] for the row update, which sums over j = axis 1; [M][1] for the column update, which sums
    over i = axis 0), B the signs (+-1).  `axis` must be given when M = 1 or n = 1 makes the shapes ambiguous."""
    if axis is None:
        assert other.shape != (1, 1), "say which form of Eq. 5 is meant"
        axis = 1 if other.shape[0] == 1 else 0
    v = other * B                                    # (alpha_other . B) per element
    num = (v * T).sum(axis=axis)
    den = (v * v).sum(axis=axis) + eps
    return num / den


def reconstruct(ar, ac, B):
    """sum_k (a_r(k) a_c(k)^T) . B(k)  for ar [K][M], ac [K][n], B [K][M][n] in {-1,+1}."""
    return np.einsum("km,kn,kmn->mn", ar, ac, B)


def sign_search(X, ar, ac, dtype=np.float64):
    """Eq. 6: per element the tuple of signs minimising |X_ij - sum_k M(k)_ij b_k|; ties go to the lowest tuple
    index t = sum_k [b_k = +1] 2^k.  Returns B [K][M][n]."""
    K = ar.shape[0]
    Xd = X.astype(dtype)
    Mag = (ar.astype(dtype)[:, :, None] * ac.astype(dtype)[:, None, :]).astype(dtype)      # rounded once
    best_err = None
    best_t = np.zeros(X.shape, np.int64)
    for t in range(1 << K):
        e = Xd.copy()
        for k in range(K):
            e = (e - Mag[k]) if (t >> k) & 1 else (e + Mag[k])                              # one base at a time
        e = np.abs(e)
        if best_err is None:
            best_err = e
        else:
            better = e < best_err
            best_err = np.where(better, e, best_err)
            best_t = np.where(better, t, best_t)
    return np.stack([np.where((best_t >> k) & 1, 1.0, -1.0) for k in range(K)])


def rc_decomp(X, K, T, eps=1e-8, dtype=np.float64, trace=None):
    """RC_Decomp on one block.  Returns (a_r [K][M], a_c [K][n], B [K][M][n]).  `trace`, if a list, receives
    the squared Frobenius error after the initialisation and after every update (for the monotonicity pin)."""
    X = np.asarray(X, np.float64)
    M, n = X.shape
    ar = np.zeros((K, M))
    ac = np.ones((K, n))
    B = np.ones((K, M, n))
    loss = lambda: float(((X - reconstruct(ar, ac, B)) ** 2).sum())
    # greedy residual initialisation (R1)
    R = X.copy()
    for k in range(K):
        B[k] = np.where(R >= 0, 1.0, -1.0)
        ac[k] = 1.0
        ar[k] = _scale_update(R, ac[k][None, :], B[k], eps, axis=1)
        R = R - (ar[k][:, None] * ac[k][None, :]) * B[k]
    if trace is not None:
        trace.append(("init", loss()))
    # alternating optimisation
    for it in range(T):
        for k in range(K):
            target = X - reconstruct(np.delete(ar, k, 0), np.delete(ac, k, 0), np.delete(B, k, 0)) if K > 1 else X   # R2
            ar[k] = _scale_update(target, ac[k][None, :], B[k], eps, axis=1)
            if trace is not None:
                trace.append((f"row{k}", loss()))
            ac[k] = _scale_update(target, ar[k][:, None], B[k], eps, axis=0)
            if trace is not None:
                trace.append((f"col{k}", loss()))
        B = sign_search(X, ar, ac, dtype)
        if trace is not None:
            trace.append(("signs", loss()))
    return ar, ac, B


def rc_decomp_matrix(W, g, K, T, eps=1e-8, dtype=np.float64):
    """Every column group of g columns of W [M][N] decomposed on its own (the block loop of Algorithm 1 without
    the Hessian compensation).  Returns row scales [K][M][N/g], column scales [K][N], signs [K][M][N]."""
    W = np.asarray(W, np.float64)
    M, N = W.shape
    assert N % g == 0
    ar = np.zeros((K, M, N // g))
    ac = np.zeros((K, N))
    B = np.zeros((K, M, N))
    for G in range(N // g):
        a, c, b = rc_decomp(W[:, G * g:(G + 1) * g], K, T, eps, dtype)
        ar[:, :, G], ac[:, G * g:(G + 1) * g], B[:, :, G * g:(G + 1) * g] = a, c, b
    return ar, ac, B


def hybrid_decomp(W, g, Kb, Ks, sal_idx, T, eps=1e-8, dtype=np.float64):
    """The salient-aware variant (Algorithm 2 without the saliency search and the Hessian compensation, which need
    calibration data): per column group, step 2 decomposes the whole block with Kb bases, step 3 decomposes the
    residual restricted to the group's salient columns (given, ascending `sal_idx`) with Ks further bases.  The
    mask is applied by handing RC_Decomp only the masked-in columns.
    Returns the global part as rc_decomp_matrix does, plus the salient part in the layer's canonical form:
    sal_row [Ks][M][N/g] (0 for groups without salient columns), sal_col [Ks][n_sal], sal_B [Ks][M][n_sal]."""
    W = np.asarray(W, np.float64)
    M, N = W.shape
    sal_idx = np.asarray(sal_idx, np.int64)
    ar, ac, B = rc_decomp_matrix(W, g, Kb, T, eps, dtype)
    What_g = np.einsum("kmn,kn,kmn->mn", np.repeat(ar, g, axis=2), ac, B)
    R = W - What_g
    n_sal = len(sal_idx)
    sal_row = np.zeros((Ks, M, N // g))
    sal_col = np.zeros((Ks, n_sal))
    sal_B = np.ones((Ks, M, n_sal))
    for G in range(N // g):
        v = np.nonzero(sal_idx // g == G)[0]                      # virtual columns of this group
        if len(v) == 0:
            continue
        a, c, b = rc_decomp(R[:, sal_idx[v]], Ks, T, eps, dtype)
        sal_row[:, :, G], sal_col[:, v], sal_B[:, :, v] = a, c, b
    return ar, ac, B, sal_row, sal_col, sal_B


def hybrid_reconstruct(ar, ac, B, sal_row, sal_col, sal_B, sal_idx, g):
    """The matrix a hybrid decomposition stands for: the global bases plus the salient bases scattered back to
    their columns (Eq. 9)."""
    What = np.einsum("kmn,kn,kmn->mn", np.repeat(ar, g, axis=2), ac, B)
    sal_idx = np.asarray(sal_idx, np.int64)
    if len(sal_idx):
        What[:, sal_idx] += np.einsum("kmv,kv,kmv->mv", sal_row[:, :, sal_idx // g], sal_col, sal_B)
    return What
