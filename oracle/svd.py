"""ORACLE — TEST INFRASTRUCTURE ONLY.

Per-page truncated SVD factors (Eq. 2): for a page X (P x d),
    L = U_r            (P x r, orthonormal columns)
    R = Sigma_r W_r^T  (r x d)
so that L R is the best rank-r approximation of X (Eckart-Young-Mirsky,
Section 3.2).  The spec names them A (= L) and B (= R).

The decomposition itself is the fp64 one-sided Jacobi in page_svd.c.
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None

MAX_SWEEPS = 60
EPS = 1e-15


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        lib.pkvo_batch_page_svd.argtypes = [dp, ctypes.c_long, ctypes.c_int, ctypes.c_int,
                                            dp, dp, dp, ip, ip, ctypes.c_int, ctypes.c_double]
        lib.pkvo_batch_page_svd.restype = None
        lib.pkvo_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def n_threads() -> int:
    """OpenMP threads the batched SVD will use."""
    return int(_load().pkvo_max_threads())


def batch_svd(X: np.ndarray):
    """Full SVD of a stack of pages.

    X: [n, P, d] float64, P <= d.
    Returns (U [n,P,P], Y [n,P,d], sigma [n,P], order [n,P] int32) with
    X[i] = U[i] @ Y[i], rows of Y[i] mutually orthogonal, sigma = row norms of
    Y (unsorted) and order = indices of sigma in descending order (ties: lower
    index first).  Raises if any page hit the sweep cap.
    """
    X = np.ascontiguousarray(X, dtype=np.float64)
    assert X.ndim == 3
    n, P, d = X.shape
    assert P <= d, "pages are short and wide (P <= d)"
    U = np.empty((n, P, P), dtype=np.float64)
    Y = np.empty((n, P, d), dtype=np.float64)
    sigma = np.empty((n, P), dtype=np.float64)
    order = np.empty((n, P), dtype=np.int32)
    sweeps = np.empty((n,), dtype=np.int32)
    if n == 0:
        return U, Y, sigma, order
    dp = ctypes.POINTER(ctypes.c_double)
    ip = ctypes.POINTER(ctypes.c_int)
    _load().pkvo_batch_page_svd(X.ctypes.data_as(dp), n, P, d, U.ctypes.data_as(dp),
                                Y.ctypes.data_as(dp), sigma.ctypes.data_as(dp),
                                order.ctypes.data_as(ip), sweeps.ctypes.data_as(ip),
                                MAX_SWEEPS, EPS)
    if (sweeps < 0).any():
        raise RuntimeError("oracle Jacobi SVD hit the sweep cap on %d page(s)" % int((sweeps < 0).sum()))
    return U, Y, sigma, order


def page_factors(X: np.ndarray, r: int):
    """Rank-r factors of each page (Eq. 2).

    X: [n, P, d] float64.  Returns (A [n,P,r], B [n,r,d], sigma_sorted [n,P]).
    A = the r leading left singular vectors, B = A^T X = Sigma_r W_r^T.
    A rank-deficient page yields zero rows in B and still-orthonormal A.
    """
    U, Y, sigma, order = batch_svd(X)
    n, P, _ = U.shape
    assert 0 < r <= P
    top = order[:, :r]
    A = np.take_along_axis(U, top[:, None, :], axis=2)          # columns of U
    B = np.take_along_axis(Y, top[:, :, None], axis=1)          # rows of Y
    s_sorted = np.take_along_axis(sigma, order, axis=1)
    return A, B, s_sorted


def optimal_tail(sigma_sorted: np.ndarray, r: int) -> np.ndarray:
    """Eckart-Young-Mirsky: min over rank-r Xh of ||X - Xh||_F = sqrt(sum_{i>r} sigma_i^2)."""
    return np.sqrt((sigma_sorted[..., r:] ** 2).sum(axis=-1))
