"""Pins for the oracle's INT4 factor quantization (Section 4.3).  CPU only."""
import numpy as np

from oracle import quant, svd
from oracle.accounting import page_storage_ratio
from oracle.bf16 import round_to_bf16
from oracle.cache import OracleCache, OracleConfig


def test_balanced_factors_keep_the_product_and_split_sigma_evenly():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((1, 32, 128)) * np.linspace(0.5, 8, 128)
    A, B, s = svd.page_factors(X, 14)
    L, R, sigma = quant.balanced_factors(A[0], B[0])
    assert np.abs(sigma - s[0][:14]).max() <= 1e-12 * s[0][0]
    assert np.abs(L @ R - A[0] @ B[0]).max() <= 1e-12 * s[0][0]
    # both factors carry sqrt(sigma): column norms of L~ and row norms of R~
    assert np.abs(np.linalg.norm(L, axis=0) - np.sqrt(sigma)).max() <= 1e-12 * np.sqrt(s[0][0])
    assert np.abs(np.linalg.norm(R, axis=1) - np.sqrt(sigma)).max() <= 1e-12 * np.sqrt(s[0][0])


def test_hand_computed_column_and_row_quantization():
    x = np.array([[7.0, -0.5, 0.0], [-3.5, 0.24, 0.0], [1.0, 0.26, 0.0]])
    codes, scale = quant.quantize(x, axis=0)                       # one scale per column
    assert scale.tolist() == [[1.0, round_to_bf16(np.array([0.5 / 7]))[0], 0.0]]
    s1 = scale[0, 1]
    assert codes[:, 0].tolist() == [7, -4, 1]                      # -3.5 ties to even (-4)
    assert codes[:, 1].tolist() == [-7, int(np.rint(0.24 / s1)), int(np.rint(0.26 / s1))]
    assert codes[:, 2].tolist() == [0, 0, 0]                       # zero column: scale 0, codes 0
    codes_r, scale_r = quant.quantize(x, axis=1)                   # one scale per row
    assert scale_r.shape == (3, 1) and scale_r[0, 0] == 1.0 and codes_r[0].tolist() == [7, 0, 0]
    deq = quant.dequantize(codes, scale)
    assert deq[0, 0] == 7.0 and deq[1, 0] == -4.0 and deq[:, 2].tolist() == [0.0, 0.0, 0.0]
    assert (deq == round_to_bf16(deq)).all()                       # dequantised values are bf16 values


def test_quantization_error_bound_and_axes():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((32, 16)) * np.logspace(-2, 2, 16)    # wildly different column magnitudes
    codes, scale = quant.quantize(x, axis=0)
    assert np.abs(codes).max() <= 7 and (np.abs(codes).max(axis=0) == 7).all()     # every column uses its full range
    err = np.abs(quant.dequantize(codes, scale) - x)
    assert (err <= 0.5 * scale * (1 + 2.0 ** -6) + 1e-300).all()  # half a step, plus the two bf16 roundings
    # row-wise on the same matrix is much worse for the small columns: the axis matters
    codes_r, scale_r = quant.quantize(x, axis=1)
    err_r = np.abs(quant.dequantize(codes_r, scale_r) - x)
    assert err_r[:, 0].mean() > 5 * err[:, 0].mean()      # (small entries all round to code 0 there)


def test_quantized_page_reconstruction_and_storage_ratio():
    rng = np.random.default_rng(2)
    K = rng.standard_normal((32, 8)) @ rng.standard_normal((8, 128)) + 0.05 * rng.standard_normal((32, 128))
    V = rng.standard_normal((32, 8)) @ rng.standard_normal((8, 128)) + 0.05 * rng.standard_normal((32, 128))
    Ak, Bk, _ = svd.page_factors(K[None], 16)
    Av, Bv, _ = svd.page_factors(V[None], 14)
    qAk, qBk, qAv, qBv = quant.quantized_page_factors(Ak[0], Bk[0], Av[0], Bv[0])
    for X, A, B, qa, qb in ((K, Ak[0], Bk[0], qAk, qBk), (V, Av[0], Bv[0], qAv, qBv)):
        e_exact = np.linalg.norm(X - A @ B)
        e_q = np.linalg.norm(X - qa @ qb)
        assert e_exact < e_q <= 0.25 * np.linalg.norm(X)           # INT4 adds error, but the page survives
    # storage: the unquantized row of the paper's table (0.588) is the page ratio diluted by 3 dense pages of
    # 512 at 16K; the INT4 row (0.187) must come out of the same dilution
    bf16_page = page_storage_ratio(16, 14, 32, 128)
    int4_page = quant.int4_page_storage_ratio(16, 14, 32, 128)
    assert abs((509 * bf16_page + 3) / 512 - 0.588) <= 5e-4
    assert abs((509 * int4_page + 3) / 512 - 0.187) <= 2e-3
    assert int4_page == (30 * 160 / 2 + 2 * (16 + 128 + 32 + 128)) / (2 * 32 * 128 * 2)


def test_cache_with_int4_factors_attends_over_dequantised_pages():
    cfg = OracleConfig(n_layers=1, n_kv_heads=1, n_q_heads=2, head_dim=16, page_size=8, rank_k=4, rank_v=3,
                       sink_tokens=8, recent_tokens=8, max_seqs=1, n_dense_slots=16, n_factor_slots=16, factor_bits=4)
    rng = np.random.default_rng(3)
    k, v = rng.standard_normal((50, 1, 16)), rng.standard_normal((50, 1, 16))
    c = OracleCache(cfg)
    c.append_kv(0, [0], [50], k, v)
    assert c.compress_eligible_pages() == 4
    q = rng.standard_normal((1, 2, 16))
    a, b = c.decode_attention(0, [0], q), c.decode_attention_pagewise(0, [0], q)
    assert np.abs(a - b).max() <= 1e-12
    f = next(iter(c.factor.values()))
    assert (f["A_k"] == round_to_bf16(f["A_k"])).all() and (f["B_v"] == round_to_bf16(f["B_v"])).all()
    # INT4 really is in effect: at most 15 distinct values per column of A_k (codes -7..7 times one scale)
    assert all(len(np.unique(f["A_k"][0][:, j])) <= 15 for j in range(4))
    assert all(len(np.unique(f["A_v"][0][i, :])) <= 15 for i in range(8))          # row-wise for L~_V
