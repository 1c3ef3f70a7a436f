"""ORACLE — TEST INFRASTRUCTURE ONLY.

The Global SVD form the paper compares with (Section 4.1 "Baselines", Section 4.2): one truncated SVD of a whole
region of K (or V) of one (layer, KV head) instead of one per page.  For a region X (T x d) with SVD U Sigma W^T and
rank r
    B = W_r^T          (r x d, orthonormal rows: the region's shared basis)
    A = X B^T          (T x r: one row per token; equal to U_r Sigma_r)
so that A B is the best rank-r approximation of the region (Eckart-Young-Mirsky, Section 3.2).  Pages of the region
keep their P rows of A; a page that leaves the window later is projected on the same basis, A_page = X_page B^T (the
paper computes its global baseline once, at prefill, and is silent on later tokens: this is the reading taken).

The decomposition is the plain one-sided Jacobi of page_svd.c, applied to X^T (d rows of length T) when T >= d and
to X itself otherwise.
"""
import numpy as np

from . import svd as _svd


def region_factors(X: np.ndarray, r: int):
    """X: [T, d] float64.  Returns (A [T, r], B [r, d], sigma [min(T, d)] sorted descending).
    Rows of B are the leading right singular vectors (zero rows past the region's rank), A = X B^T."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    T, d = X.shape
    k = min(r, T, d)
    if T >= d:
        W, _, sigma = _svd.page_factors(X.T[None], k)             # X^T = W (Sigma U^T): columns of W = right vectors of X
        B = W[0].T
    else:
        _, Y, sigma = _svd.page_factors(X[None], k)               # rows of Y = sigma_i w_i^T
        norms = sigma[0, :k]
        B = np.where(norms[:, None] > 0, Y[0] / np.where(norms > 0, norms, 1.0)[:, None], 0.0)
    if k < r:
        B = np.concatenate([B, np.zeros((r - k, d))])
    return X @ B.T, B, sigma[0]


def project_page(X_page: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Rows of A for tokens that join a region after its basis was fixed."""
    return np.asarray(X_page, dtype=np.float64) @ B.T
