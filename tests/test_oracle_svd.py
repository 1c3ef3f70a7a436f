"""Pins for the oracle's page SVD (Eq. 2): library routine, closed forms,
Eckart-Young-Mirsky optimality, invariants.  CPU only."""
import numpy as np
import pytest

from oracle import svd


def _rng(seed):
    return np.random.default_rng(seed)


@pytest.mark.parametrize("P,d", [(16, 128), (32, 128), (64, 128), (8, 8), (5, 11)])
def test_singular_values_match_library(P, d):
    X = _rng(1).standard_normal((3, P, d))
    _, _, s = svd.page_factors(X, 1)
    ref = np.linalg.svd(X, compute_uv=False)
    assert np.abs(s - ref).max() <= 1e-12 * ref.max()


def test_constructed_page_has_known_spectrum():
    # X = U diag(s) W^T with orthonormal U, W from QR of Gaussians: sigma = s exactly.
    P, d = 32, 128
    rng = _rng(2)
    U, _ = np.linalg.qr(rng.standard_normal((P, P)))
    W, _ = np.linalg.qr(rng.standard_normal((d, P)))
    s = np.array([10.0 * 0.8 ** i for i in range(P)])
    X = (U * s) @ W.T
    A, B, sig = svd.page_factors(X[None], 7)
    assert np.abs(sig[0] - s).max() <= 1e-12 * s[0]
    # leading left vectors equal U up to sign; rows of B equal s_i w_i^T up to the same sign
    for i in range(7):
        sign = np.sign(A[0][:, i] @ U[:, i])
        assert np.abs(sign * A[0][:, i] - U[:, i]).max() <= 1e-10
        assert np.abs(sign * B[0][i] - s[i] * W[:, i]).max() <= 1e-10 * s[0]


@pytest.mark.parametrize("P,r", [(16, 9), (32, 16), (64, 24), (64, 1), (64, 64)])
def test_eckart_young_tail_and_factor_format(P, r):
    d = 128
    X = _rng(3).standard_normal((2, P, d)) * np.linspace(0.5, 8, d)
    A, B, s = svd.page_factors(X, r)
    full = np.linalg.svd(X, compute_uv=False)
    for i in range(2):
        err = np.linalg.norm(X[i] - A[i] @ B[i])
        tail = np.sqrt((full[i][r:] ** 2).sum())
        assert abs(err - tail) <= 1e-12 * np.linalg.norm(X[i])
        assert abs(svd.optimal_tail(s, r)[i] - tail) <= 1e-12 * np.linalg.norm(X[i])
        # L has orthonormal columns; R R^T = diag(sigma_1^2..sigma_r^2); L R = L L^T X
        assert np.abs(A[i].T @ A[i] - np.eye(r)).max() <= 1e-13
        assert np.abs(B[i] @ B[i].T - np.diag(full[i][:r] ** 2)).max() <= 1e-11 * full[i][0] ** 2
        assert np.abs(A[i] @ B[i] - A[i] @ (A[i].T @ X[i])).max() <= 1e-12 * full[i][0]
        # sum of sigma^2 is the squared Frobenius norm
        assert abs((s[i] ** 2).sum() - (X[i] ** 2).sum()) <= 1e-12 * (X[i] ** 2).sum()


def test_full_factor_identity_and_invariants():
    X = _rng(4).standard_normal((2, 16, 40))
    U, Y, sigma, order = svd.batch_svd(X)
    for i in range(2):
        assert np.abs(U[i] @ Y[i] - X[i]).max() <= 1e-13
        assert np.abs(U[i].T @ U[i] - np.eye(16)).max() <= 1e-13
        G = Y[i] @ Y[i].T
        off = G - np.diag(np.diag(G))
        assert np.abs(off).max() <= 1e-13 * np.abs(G).max()
        assert (np.diff(sigma[i][order[i]]) <= 0).all()


def test_exact_low_rank_page_is_reproduced():
    rng = _rng(5)
    X = rng.standard_normal((64, 8)) @ rng.standard_normal((8, 128))
    for r in (8, 16):
        A, B, s = svd.page_factors(X[None], r)
        assert np.linalg.norm(X - A[0] @ B[0]) <= 1e-12 * np.linalg.norm(X)
        assert np.abs(A[0].T @ A[0] - np.eye(r)).max() <= 1e-13
    assert s[0][8:].max() <= 1e-12 * s[0][0]


def test_zero_and_rank_one_pages():
    Z = np.zeros((1, 16, 32))
    A, B, s = svd.page_factors(Z, 4)
    assert np.abs(B).max() == 0.0 and np.abs(A[0].T @ A[0] - np.eye(4)).max() <= 1e-15
    rng = _rng(6)
    u, w = rng.standard_normal(16), rng.standard_normal(32)
    X = np.outer(u, w)
    A, B, s = svd.page_factors(X[None], 1)
    assert abs(s[0][0] - np.linalg.norm(u) * np.linalg.norm(w)) <= 1e-12 * s[0][0]
    assert np.linalg.norm(X - A[0] @ B[0]) <= 1e-12 * s[0][0]


def test_gram_route_gives_the_same_truncation():
    # Section 3.3: top-r eigenvectors Q_r of X X^T and R = Q_r^T X are the truncated-SVD factors.
    X = _rng(7).standard_normal((32, 128)) * np.linspace(0.5, 8, 128)
    r = 12
    A, B, _ = svd.page_factors(X[None], r)
    lam, Q = np.linalg.eigh(X @ X.T)
    Qr = Q[:, ::-1][:, :r]
    assert np.abs(Qr @ (Qr.T @ X) - A[0] @ B[0]).max() <= 1e-10 * np.abs(X).max()


def test_ties_keep_lower_index_first():
    X = np.zeros((4, 6))
    X[0, 0] = X[1, 1] = X[2, 2] = 2.0
    X[3, 3] = 3.0
    _, _, sigma, order = svd.batch_svd(X[None])
    assert list(order[0]) == [3, 0, 1, 2]
