"""Whitened sketch: approximate leverage scores in the sense of Eq. (row leverage score).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only tests and the benchmark's cpu-baseline
leg may import this module.  Plain numpy / scipy in fp64.

Alg. 1 uses ||a_j G||^2, which estimates the squared row norm of a_j, not the
leverage score ||U(j,:)||^2 of Eq. (row leverage score): the construction the
paper's footnote points to (sketch-based leverage approximation) first whitens
the rows with the triangular factor of the matrix.  This module restates that
construction for the d x d Gram matrix:

    M = A^T A + lambda I,  lambda = ridge * trace(A^T A) / d        (ridge >= 0)
    M = L L^T              (Cholesky, L lower triangular)
    W = L^{-T} G           (d x r)
    l_j = ||a_j W||^2

With G = I_d and ridge = 0, l_j = a_j (A^T A)^{-1} a_j^T = ||U(j,:)||^2 exactly
(full column rank); a Gaussian G ~ N(0, 1/r) gives an unbiased estimate of it.
The remaining steps are Alg. 1 (product and normalisation) unchanged: l^KV = l^K l^V, normalise.
Rows at or beyond a sequence's length take no part (not in M, score 0).
"""
from __future__ import annotations

import numpy as np
from scipy.linalg import solve_triangular


def bf16_to_f64(u16):
    return (np.asarray(u16, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def whitening_matrix(A, G, ridge):
    """A [n, d] fp64, G [d, r]: W = L^{-T} G with L L^T = A^T A + ridge * trace(A^T A)/d * I."""
    d = A.shape[1]
    M = A.T @ A
    M = M + (ridge * np.trace(M) / d) * np.eye(d)
    L = np.linalg.cholesky(M)
    return solve_triangular(L.T, np.asarray(G, dtype=np.float64), lower=False)


def whitened_row_scores(A, G, ridge):
    Y = A @ whitening_matrix(A, G, ridge)
    return np.sum(Y * Y, axis=1)


def score_whitened(K, V, G, ridge, seqlens=None):
    """K, V: uint16 bf16 bit patterns [B, H, n, d]; G fp32 [d, r].
    Returns (scores [B,H,n], head_sums [B,H], lK, lV) in fp64."""
    K, V = bf16_to_f64(K), bf16_to_f64(V)
    B, H, n, _ = K.shape
    scores = np.zeros((B, H, n))
    sums = np.zeros((B, H))
    lK = np.zeros((B, H, n))
    lV = np.zeros((B, H, n))
    for b in range(B):
        nb = n if seqlens is None else int(min(max(seqlens[b], 0), n))
        if nb == 0:
            continue
        for h in range(H):
            lK[b, h, :nb] = whitened_row_scores(K[b, h, :nb], G, ridge)
            lV[b, h, :nb] = whitened_row_scores(V[b, h, :nb], G, ridge)
            l = lK[b, h, :nb] * lV[b, h, :nb]                    # Alg. 1 (product step)
            sums[b, h] = l.sum()
            scores[b, h, :nb] = l / sums[b, h] if sums[b, h] > 0 else 0.0   # normalise
    return scores, sums, lK, lV
