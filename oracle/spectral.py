"""Graph quantities and the parameter prescription -- TEST INFRASTRUCTURE (NumPy/LAPACK).

  laplacian   Lambda = sum_{(i,j) in E} lambda^{ij} (e_i - e_j)(e_i - e_j)^T        (the Laplacian definition of Sec. 3.1)
  chi_1       sup_{|x|=1, x perp 1} 1/(x^T Lambda x) = 1 / lambda_2(Lambda)          (Eq. 2)
  chi_2       1/2 sup_{(i,j) in E} (e_i - e_j)^T Lambda^+ (e_i - e_j)                (Eq. 3)
  prescribe   eta = 1/(2 sqrt(chi_1 chi_2)), alpha = 1/2, alpha~ = 1/2 sqrt(chi_1/chi_2);
              without acceleration eta = 0, alpha = alpha~ = 1/2                     (the convergence proposition of Sec. 3.4)
"""
from __future__ import annotations

import numpy as np


def laplacian(n, edges, rates):
    L = np.zeros((n, n))
    for (i, j), lam in zip(np.asarray(edges), np.asarray(rates, dtype=np.float64)):
        L[i, i] += lam
        L[j, j] += lam
        L[i, j] -= lam
        L[j, i] -= lam
    return L


def chi1(L):
    w = np.linalg.eigvalsh(L)
    return 1.0 / w[1]


def chi2(L, edges):
    P = np.linalg.pinv(L, hermitian=True)
    best = 0.0
    for i, j in np.asarray(edges):
        r = P[i, i] + P[j, j] - 2.0 * P[i, j]
        best = max(best, r)
    return 0.5 * best


def prescribe(n, edges, rates, accelerated=True):
    """(eta, alpha, alpha_tilde, chi_1, chi_2)."""
    L = laplacian(n, edges, rates)
    c1, c2 = chi1(L), chi2(L, edges)
    if not accelerated:
        return 0.0, 0.5, 0.5, c1, c2
    return 1.0 / (2.0 * np.sqrt(c1 * c2)), 0.5, 0.5 * np.sqrt(c1 / c2), c1, c2
