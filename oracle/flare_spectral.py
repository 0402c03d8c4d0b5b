"""Linear-time eigenanalysis of the induced mixing matrix -- TEST INFRASTRUCTURE, not the product.

Follows the steps of the paper's Algorithm 1 (spectral-analysis appendix) in its order and notation, in
float64 numpy, for one head:
  1. A   = exp(Q K^T)                       [M, N]
  2. L_N = diag(1 / sum_m A[m, n])          [N]
  3. L_M = diag(1 / sum_n A[m, n])          [M]
  4. J   = L_M^{1/2} A L_N^{1/2}            [M, N]
  5. U Sigma^2 U^T = J J^T                  (M x M symmetric eigenproblem)
  6. eigenvalues  = Sigma^2
  7. eigenvectors = L_N^{1/2} J^T U Sigma^{-1}   [N, M]
Reading of a garbled sentence: the text once names the M x M matrix "J^T J"; J^T J is N x N, and the
algorithm's step 5 is consistent with J J^T, which is what is used here.  One global constant (the largest score) is
subtracted before exponentiation: it multiplies all of A by one factor c, L_M and L_N by 1/c, and leaves J
unchanged, so A cannot overflow.  Pinned in tests/test_oracle_pins.py against a dense eigendecomposition of W.
"""
from __future__ import annotations

import numpy as np


def gram_from_qk(Q_h, K_h, scale: float = 1.0):
    """Steps 1-4 of Algorithm 1 and the M x M matrix of step 5: Q_h [M, D], K_h [N, D] -> (J J^T [M, M], J [M, N], L_N [N])."""
    Q_h = np.asarray(Q_h, dtype=np.float64)
    K_h = np.asarray(K_h, dtype=np.float64)
    S = scale * (Q_h @ K_h.T)
    A = np.exp(S - S.max())
    L_N = 1.0 / A.sum(axis=0)
    L_M = 1.0 / A.sum(axis=1)
    J = np.sqrt(L_M)[:, None] * A * np.sqrt(L_N)[None, :]
    return J @ J.T, J, L_N


def eig_from_qk(Q_h, K_h, scale: float = 1.0):
    """Q_h [M, D], K_h [N, D] of one head -> (eigenvalues [M] descending, eigenvectors [N, M])."""
    JJt, J, L_N = gram_from_qk(Q_h, K_h, scale)
    sig2, U = np.linalg.eigh(JJt)
    order = np.argsort(sig2)[::-1]
    sig2, U = sig2[order], U[:, order]
    sigma = np.sqrt(np.clip(sig2, 0.0, None))
    safe = np.where(sigma > 0.0, sigma, 1.0)
    vecs = np.sqrt(L_N)[:, None] * (J.T @ U) / safe[None, :]
    return sig2, vecs
