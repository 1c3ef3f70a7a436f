"""Pins of the oracle's Global SVD form (the comparison form of Section 4.2: one basis per region instead of one
per page) against what the mathematics fixes: a library SVD, the Eckart-Young tail, a constructed spectrum, the
page-wise factors when the region is one page, and full attention at full rank."""
import numpy as np
import pytest

from oracle import attention as att
from oracle import global_svd, svd
from oracle.cache import OracleCache, OracleConfig


@pytest.mark.parametrize("T,d,r", [(300, 128, 80), (128, 128, 16), (40, 128, 24), (200, 64, 64), (10, 128, 16)])
def test_region_factors_against_library_svd_and_eckart_young(T, d, r):
    rng = np.random.default_rng(T + r)
    X = rng.standard_normal((T, 12)) @ rng.standard_normal((12, d)) + 0.05 * rng.standard_normal((T, d))
    A, B, sigma = global_svd.region_factors(X, r)
    s_ref = np.linalg.svd(X, compute_uv=False)
    assert np.allclose(sigma, s_ref, rtol=1e-11, atol=1e-11)
    k = min(r, T, d)
    tail = np.sqrt((s_ref[k:] ** 2).sum())
    assert abs(np.linalg.norm(X - A @ B) - tail) <= 1e-10 * np.linalg.norm(X)
    assert np.abs(B[:k] @ B[:k].T - np.eye(k)).max() <= 1e-12            # orthonormal rows
    assert np.abs(B[k:]).max(initial=0.0) == 0.0                          # ranks the region does not have: zero rows
    assert np.abs(A - X @ B.T).max() == 0.0                               # A is the projection, by definition
    # A = U_r Sigma_r: its columns are orthogonal with norms sigma_i
    gram = A[:, :k].T @ A[:, :k]
    assert np.abs(gram - np.diag(s_ref[:k] ** 2)).max() <= 1e-9 * s_ref[0] ** 2


def test_constructed_spectrum_gives_the_prescribed_tail():
    rng = np.random.default_rng(3)
    T, d, r = 512, 128, 80
    U, _ = np.linalg.qr(rng.standard_normal((T, d)))
    W, _ = np.linalg.qr(rng.standard_normal((d, d)))
    s = 0.9 ** np.arange(d)
    X = (U * s) @ W.T
    A, B, sigma = global_svd.region_factors(X, r)
    assert np.allclose(sigma, s, rtol=1e-11)
    assert abs(np.linalg.norm(X - A @ B) - np.sqrt((s[r:] ** 2).sum())) <= 1e-12
    # the basis spans the r leading right singular vectors
    assert np.abs(B @ W[:, r:]).max() <= 1e-10


@pytest.mark.parametrize("P,r", [(64, 16), (32, 14), (16, 16)])
def test_a_region_of_one_page_reproduces_the_page_factors(P, r):
    rng = np.random.default_rng(P)
    X = rng.standard_normal((P, 128))
    A_g, B_g, _ = global_svd.region_factors(X, r)
    A_p, B_p, _ = svd.page_factors(X[None], r)
    assert np.abs(A_g @ B_g - A_p[0] @ B_p[0]).max() <= 1e-12 * np.abs(X).max() * 128


def _cache(global_rank, T, P=64, H=2, G=2, sink=64, recent=128, seed=0):
    cfg = OracleConfig(n_layers=1, n_kv_heads=H, n_q_heads=H * G, head_dim=128, page_size=P, rank_k=16, rank_v=16,
                       sink_tokens=sink, recent_tokens=recent, max_seqs=2, n_dense_slots=64, n_factor_slots=64,
                       global_rank=global_rank)
    rng = np.random.default_rng(seed)
    k, v = rng.standard_normal((T, H, 128)), rng.standard_normal((T, H, 128))
    c = OracleCache(cfg)
    return c, k, v, rng


def test_full_rank_global_cache_equals_vanilla_attention_and_shares_the_page_wise_state_machine():
    T = 64 * 9 + 5
    c, k, v, rng = _cache(128, T)
    pagewise, _, _, _ = _cache(0, T)
    for cache in (c, pagewise):
        cache.append_kv(0, [0], [T], k, v)
    assert c.compress_eligible_pages(0) == pagewise.compress_eligible_pages(0) == 6
    assert c.page_table(0, 0) == pagewise.page_table(0, 0)               # same eligibility, same slot numbering
    q = rng.standard_normal((1, 4, 128))
    out = c.decode_attention(0, [0], q)
    for h in range(4):
        ref = att.attention_plain(q[0, h], k[:, h // 2], v[:, h // 2], 128 ** -0.5)
        assert np.abs(out[0, h] - ref).max() <= 1e-12                    # rank d keeps the region exactly
    # page by page (Eq. 4, Eq. 5) the same numbers
    assert np.abs(c.decode_attention_pagewise(0, [0], q) - out).max() <= 1e-12


def test_pages_converted_later_are_projected_on_the_regions_basis():
    T0 = 64 * 8
    c, k, v, rng = _cache(24, T0 + 64 * 3)
    c.append_kv(0, [0], [T0], k[:T0], v[:T0])
    assert c.compress_eligible_pages(0) == 5                             # the region: pages 1..5
    basis = c.basis[(0, 0)]
    assert basis["pages"] == [1, 2, 3, 4, 5] and basis["B_k"].shape == (2, 24, 128)
    B_before = basis["B_k"].copy()
    c.append_kv(0, [0], [64 * 3], k[T0:], v[T0:])
    assert c.compress_eligible_pages(0) == 3                             # pages 6..8 leave the window
    assert np.array_equal(c.basis[(0, 0)]["B_k"], B_before)              # the basis is fixed by the first conversion
    kinds, slots, _ = c.page_table(0, 0)
    f = c.factor[slots[7]]
    for h in range(2):
        assert np.abs(f["A_k"][h] - k[64 * 7:64 * 8, h] @ B_before[h].T).max() <= 1e-12
    # region-level optimality holds for the region's own pages, stacked
    X = np.concatenate([k[64 * p:64 * (p + 1), 0] for p in range(1, 6)])
    A = np.concatenate([c.factor[slots[p]]["A_k"][0] for p in range(1, 6)])
    s = np.linalg.svd(X, compute_uv=False)
    assert abs(np.linalg.norm(X - A @ B_before[0]) - np.sqrt((s[24:] ** 2).sum())) <= 1e-10 * np.linalg.norm(X)
    c.free_seq(0)
    assert (0, 0) not in c.basis
