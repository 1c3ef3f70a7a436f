"""Pins for the oracle's cache state machine (Section 3.3) and the size
formulas (Eq. 3, Section 1).  CPU only."""
import os

import numpy as np
import pytest

from oracle import accounting, attention as att
from oracle.cache import DENSE, FACTOR, OracleCache, OracleConfig, PoolExhausted, eligible_range

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.split("#")[0].strip()
        if line:
            out.append([float(x) for x in line.split()])
    return out


def test_storage_ratio_values_printed_in_paper():
    for rk, rv, P, d, val, tol in _rows("storage_ratio.txt"):
        assert abs(accounting.page_storage_ratio(int(rk), int(rv), int(P), int(d)) - val) <= tol
    # the benchmark's r=24, P=64 configuration: factor storage "~56%" of dense
    assert accounting.page_storage_ratio(24, 24, 64, 128) == 0.5625


def test_kv_size_example_printed_in_paper():
    for L, H, T, d, bpe, gib, rtol in _rows("kv_size.txt"):
        b = accounting.kv_cache_elements(int(L), int(H), int(T), int(d)) * bpe
        assert abs(b / 2 ** 30 - gib) <= rtol * gib


def test_dense_policy_fixtures():
    for T, P, S, W, n, first, last in _rows("dense_policy.txt"):
        lo, hi = eligible_range(int(T), int(P), int(S), int(W))
        assert (hi - lo, lo, hi - 1) == (int(n), int(first), int(last))


def test_eligibility_closed_form_equals_token_form():
    for P in (16, 32, 64):
        for S in (0, P, 2 * P):
            for W in (0, P, 4 * P):
                for T in range(0, 20 * P + 1, 7):
                    lo, hi = eligible_range(T, P, S, W)
                    assert list(range(lo, hi)) == accounting.eligible_pages_token_form(T, P, S, W)


def _cfg(**kw):
    base = dict(n_layers=1, n_kv_heads=2, n_q_heads=4, head_dim=16, page_size=8, rank_k=3, rank_v=2,
                sink_tokens=8, recent_tokens=16, max_seqs=2, n_dense_slots=64, n_factor_slots=64)
    base.update(kw)
    return OracleConfig(**base)


def _kv(rng, n, cfg):
    return (rng.standard_normal((n, cfg.n_kv_heads, cfg.head_dim)),
            rng.standard_normal((n, cfg.n_kv_heads, cfg.head_dim)))


def test_all_dense_cache_is_vanilla_attention():
    cfg = _cfg(recent_tokens=8 * 100)                  # window >= T: nothing is ever eligible
    rng = np.random.default_rng(0)
    c = OracleCache(cfg)
    k, v = _kv(rng, 45, cfg)
    c.append_kv(0, [0], [45], k, v)
    assert c.compress_eligible_pages() == 0
    q = rng.standard_normal((1, cfg.n_q_heads, cfg.head_dim))
    out = c.decode_attention(0, [0], q)
    for h in range(cfg.n_q_heads):
        ref = att.attention_plain(q[0, h], k[:, h // 2], v[:, h // 2], 0.25)
        assert np.abs(out[0, h] - ref).max() <= 1e-13


def test_full_rank_cache_is_vanilla_attention():
    cfg = _cfg(rank_k=8, rank_v=8)                     # r = P = min(P, d)
    rng = np.random.default_rng(1)
    c = OracleCache(cfg)
    k, v = _kv(rng, 61, cfg)
    c.append_kv(0, [1], [61], k, v)
    assert c.compress_eligible_pages() == 61 // 8 - 1 - 2
    q = rng.standard_normal((1, cfg.n_q_heads, cfg.head_dim))
    out = c.decode_attention(0, [1], q)
    for h in range(cfg.n_q_heads):
        ref = att.attention_plain(q[0, h], k[:, h // 2], v[:, h // 2], 0.25)
        assert np.abs(out[0, h] - ref).max() <= 1e-12


def test_pagewise_route_equals_plain_route_and_zero_query_mean():
    cfg = _cfg()
    rng = np.random.default_rng(2)
    c = OracleCache(cfg)
    k, v = _kv(rng, 77, cfg)
    c.append_kv(0, [0], [77], k, v)
    c.compress_eligible_pages()
    q = rng.standard_normal((1, cfg.n_q_heads, cfg.head_dim))
    a, b = c.decode_attention(0, [0], q), c.decode_attention_pagewise(0, [0], q)
    assert np.abs(a - b).max() <= 1e-12 * np.abs(a).max()
    out0 = c.decode_attention(0, [0], np.zeros_like(q))
    for h in range(cfg.n_q_heads):
        _, V_all = c.gather_kv(0, 0, h // 2)
        assert V_all.shape[0] == 77
        assert np.abs(out0[0, h] - V_all.mean(axis=0)).max() <= 1e-14


def _causal_block(Q, K, V, scale):
    """Textbook causal attention for the last len(Q) positions of a sequence of len(K) tokens, written as one
    masked score matrix (no per-query slicing): independent of how the oracle walks its pages."""
    n_q, T = Q.shape[0], K.shape[0]
    S = Q @ K.T * scale
    pos = np.arange(T)[None, :]
    own = (T - n_q + np.arange(n_q))[:, None]
    S = np.where(pos <= own, S, -np.inf)
    W = np.exp(S - S.max(axis=1, keepdims=True))
    return (W / W.sum(axis=1, keepdims=True)) @ V


def test_multi_query_attention_pins():
    rng = np.random.default_rng(21)
    # (a) all-dense cache: the textbook causal block
    cfg = _cfg(recent_tokens=8 * 100)
    c = OracleCache(cfg)
    k, v = _kv(rng, 45, cfg)
    c.append_kv(0, [0], [45], k, v)
    for q_len in (1, 3, 8, 11):
        q = rng.standard_normal((1, q_len, cfg.n_q_heads, cfg.head_dim))
        out = c.decode_attention_multi(0, [0], q)
        for h in range(cfg.n_q_heads):
            ref = _causal_block(q[0, :, h], k[:, h // 2], v[:, h // 2], 0.25)
            assert np.abs(out[0, :, h] - ref).max() <= 1e-13
    # (b) mixed cache: the last query is the single-query call; an earlier query equals the single-query call on a
    #     cache that was fed the same tokens, compressed at the same moment, and then given fewer new tokens
    cfg = _cfg()
    c = OracleCache(cfg)
    k, v = _kv(rng, 77, cfg)
    c.append_kv(0, [0], [70], k[:70], v[:70])
    c.compress_eligible_pages()
    c.append_kv(0, [0], [7], k[70:], v[70:])
    q = rng.standard_normal((1, 5, cfg.n_q_heads, cfg.head_dim))
    out = c.decode_attention_multi(0, [0], q)
    assert np.array_equal(out[:, 4], c.decode_attention(0, [0], q[:, 4]))
    c2 = OracleCache(cfg)
    c2.append_kv(0, [0], [70], k[:70], v[:70])
    c2.compress_eligible_pages()
    c2.append_kv(0, [0], [4], k[70:74], v[70:74])           # 74 tokens: what query 1 of 5 sees (77 - 5 + 1 + 1)
    assert np.abs(out[:, 1] - c2.decode_attention(0, [0], q[:, 1])).max() <= 1e-14
    # (c) the first token's own query returns its value row; zero queries give running means
    c3 = OracleCache(_cfg(recent_tokens=8 * 100))
    c3.append_kv(0, [1], [6], k[:6], v[:6])
    q = rng.standard_normal((1, 6, cfg.n_q_heads, cfg.head_dim))
    out = c3.decode_attention_multi(0, [1], q)
    for h in range(cfg.n_q_heads):
        assert np.abs(out[0, 0, h] - v[0, h // 2]).max() <= 1e-14
    out0 = c3.decode_attention_multi(0, [1], np.zeros_like(q))
    for j in range(6):
        assert np.abs(out0[0, j, 0] - v[:j + 1, 0].mean(axis=0)).max() <= 1e-14
    with pytest.raises(ValueError):
        c3.decode_attention_multi(0, [1], np.zeros((1, 7, cfg.n_q_heads, cfg.head_dim)))


def test_two_step_compression_pins():
    """compress_begin + compress_commit: back to back it is compress_eligible_pages (tables, factors, free lists);
    between the two the cache reads as before the begin; pages appended in between do not join the set."""
    rng = np.random.default_rng(31)
    cfg = _cfg(n_layers=2, max_seqs=2)
    k, v = _kv(rng, 90, cfg)

    def fed():
        c = OracleCache(cfg)
        c.append_kv(0, [0, 1], [60, 30], k, v)
        c.append_kv(1, [1], [50], k[:50], v[:50])
        return c
    a, b = fed(), fed()
    n = a.compress_eligible_pages(0)
    assert b.compress_begin(0) == n == (60 // 8 - 2 - 1)
    assert b.compress_commit(0) == n and b.pending == {}
    for s in (0, 1):
        assert a.page_table(s, 0) == b.page_table(s, 0)
    assert sorted(a.factor) == sorted(b.factor)
    for slot in a.factor:
        for name in ("A_k", "B_k", "A_v", "B_v"):
            assert np.array_equal(a.factor[slot][name], b.factor[slot][name])
    assert [a.dense_free.alloc() for _ in range(4)] == [b.dense_free.alloc() for _ in range(4)]
    assert a.factor_free.alloc() == b.factor_free.alloc()
    # in between: attention and tables as before the begin; later appends stay out of the begun set
    c = fed()
    q = rng.standard_normal((1, cfg.n_q_heads, cfg.head_dim))
    before, table = c.decode_attention(0, [0], q), c.page_table(0, 0)
    assert c.compress_begin(0) == n
    assert np.array_equal(c.decode_attention(0, [0], q), before) and c.page_table(0, 0) == table
    k2, v2 = _kv(rng, 16, cfg)
    c.append_kv(0, [0], [16], k2, v2)                          # two more pages become eligible
    assert len(c.eligible(0, 0)) == n + 2
    assert c.compress_commit() == n
    assert sum(kd == FACTOR for kd in c.page_table(0, 0)[0]) == n and len(c.eligible(0, 0)) == 2
    # the committed factors are those of the pages as they were (complete pages never change)
    d = fed()
    d.compress_eligible_pages(0)
    for p in range(1, 1 + n):
        fa, fb = c.factor[c.page_table(0, 0)[1][p]], d.factor[d.page_table(0, 0)[1][p]]
        assert np.array_equal(fa["A_k"], fb["A_k"]) and np.array_equal(fa["B_v"], fb["B_v"])
    assert c.compress_commit() == 0


def test_states_of_token_ranges_merge_to_attention_over_all_tokens():
    """A sequence split over three caches (first with the sink, middle all compressed, last with the window): the
    per-cache states merged by Eq. 5 equal Eq. 1 over the concatenated (partly reconstructed) tokens, and each
    state on its own normalises to that cache's attention with the expected log-sum-exp."""
    rng = np.random.default_rng(41)
    parts = [(_cfg(sink_tokens=8, recent_tokens=0), 50), (_cfg(sink_tokens=0, recent_tokens=0), 41),
             (_cfg(sink_tokens=0, recent_tokens=16), 37)]
    caches, Ks, Vs = [], [], []
    for cfg, T in parts:
        c = OracleCache(cfg)
        k, v = _kv(rng, T, cfg)
        c.append_kv(0, [1], [T], k, v)
        assert c.compress_eligible_pages() > 0
        caches.append(c)
    cfg = parts[0][0]
    q = rng.standard_normal((1, cfg.n_q_heads, cfg.head_dim))
    states = [c.attention_state(0, [1], q) for c in caches]
    for h in range(cfg.n_q_heads):
        K = np.concatenate([c.gather_kv(1, 0, h // 2)[0] for c in caches])
        V = np.concatenate([c.gather_kv(1, 0, h // 2)[1] for c in caches])
        assert K.shape[0] == 50 + 41 + 37
        merged = att.merge_page_states([(m[0, h], l[0, h], o[0, h]) for m, l, o in states])
        assert np.abs(merged - att.attention_plain(q[0, h], K, V, 0.25)).max() <= 1e-13
        for c, (m, l, o) in zip(caches, states):
            assert np.abs(o[0, h] / l[0, h] - c.decode_attention(0, [1], q)[0, h]).max() <= 1e-13
            s = c.gather_kv(1, 0, h // 2)[0] @ q[0, h] * 0.25
            assert abs(m[0, h] + np.log(l[0, h]) - np.log(np.exp(s).sum())) <= 1e-12


def test_output_invariant_under_slot_permutation():
    cfg = _cfg()
    rng = np.random.default_rng(3)
    k, v = _kv(rng, 70, cfg)
    q = rng.standard_normal((1, cfg.n_q_heads, cfg.head_dim))
    outs, tables = [], []
    for seed in (None, 5):
        if seed is None:
            c = OracleCache(cfg)
        else:
            pr = np.random.default_rng(seed)
            c = OracleCache(cfg, pr.permutation(64), pr.permutation(64))
        c.append_kv(0, [0], [70], k, v)
        c.compress_eligible_pages()
        outs.append(c.decode_attention(0, [0], q))
        tables.append(c.page_table(0, 0))
    assert (outs[0] == outs[1]).all()
    assert tables[0][0] == tables[1][0] and tables[0][1] != tables[1][1]


def test_state_machine_kinds_slots_and_free_list_policy():
    cfg = _cfg(n_kv_heads=1, n_q_heads=1)
    rng = np.random.default_rng(4)
    c = OracleCache(cfg, dense_slot_order=[5, 4, 3, 2, 1, 0, 6, 7], factor_slot_order=[9, 8, 7, 6])
    k, v = _kv(rng, 41, cfg)
    c.append_kv(0, [0], [41], k, v)                      # pages 0..5 (5 partial)
    kinds, slots, T = c.page_table(0, 0)
    assert (kinds, slots, T) == ([DENSE] * 6, [5, 4, 3, 2, 1, 0], 41)
    assert c.eligible(0, 0) == [1, 2]                    # n_c=5, window 2 pages -> p < 3
    assert c.compress_eligible_pages(0) == 2
    kinds, slots, _ = c.page_table(0, 0)
    assert kinds == [DENSE, FACTOR, FACTOR, DENSE, DENSE, DENSE] and slots == [5, 9, 8, 2, 1, 0]
    # released dense slots 4 then 3 are on the stack: next allocations get 3, then 4, then order resumes at 6
    k2, v2 = _kv(rng, 24, cfg)
    c.append_kv(0, [0], [24], k2, v2)                    # T=65: pages 6,7,8 opened
    assert c.page_table(0, 0)[1][6:] == [3, 4, 6]
    assert c.stats() == dict(dense_in_use=7, factor_in_use=2, pages_compressed=2)


def test_incremental_update_at_most_one_page_per_step_and_never_revisited():
    cfg = _cfg(n_kv_heads=1, n_q_heads=2)
    rng = np.random.default_rng(5)
    k, v = _kv(rng, 120, cfg)
    q = rng.standard_normal((1, 2, cfg.head_dim))
    inc = OracleCache(cfg)
    inc.append_kv(0, [0], [40], k[:40], v[:40])
    inc.compress_eligible_pages()
    seen = {}
    for t in range(40, 120):
        inc.append_kv(0, [0], [1], k[t:t + 1], v[t:t + 1])
        n = inc.compress_eligible_pages()
        assert n == (1 if (t + 1) % 8 == 0 else 0)       # only the step that fills a page converts one
        kinds, slots, _ = inc.page_table(0, 0)
        for p, (kd, s) in enumerate(zip(kinds, slots)):
            if kd == FACTOR:
                assert seen.setdefault(p, s) == s        # a factor page keeps its slot forever
    bulk = OracleCache(cfg)
    bulk.append_kv(0, [0], [120], k, v)
    bulk.compress_eligible_pages()
    assert bulk.page_table(0, 0)[0] == inc.page_table(0, 0)[0]
    a, b = inc.decode_attention(0, [0], q), bulk.decode_attention(0, [0], q)
    assert (a == b).all()                                # each page factorized once from the same rows


def test_per_layer_token_counts_and_multi_seq_append():
    cfg = _cfg(n_layers=2)
    rng = np.random.default_rng(6)
    c = OracleCache(cfg)
    k, v = _kv(rng, 30, cfg)
    c.append_kv(0, [0, 1], [10, 20], k, v)
    assert c.page_table(0, 0)[2] == 10 and c.page_table(1, 0)[2] == 20 and c.page_table(0, 1)[2] == 0
    K_all, _ = c.gather_kv(1, 0, 1)
    assert (K_all == k[10:, 1]).all()


def test_pool_exhaustion_and_empty_sequence():
    cfg = _cfg(n_dense_slots=2)
    rng = np.random.default_rng(7)
    c = OracleCache(cfg)
    k, v = _kv(rng, 17, cfg)
    with pytest.raises(PoolExhausted):
        c.append_kv(0, [0], [17], k, v)
    with pytest.raises(ValueError):
        OracleCache(_cfg()).decode_attention(0, [0], np.zeros((1, 4, 16)))


def test_free_seq_returns_slots():
    cfg = _cfg()
    rng = np.random.default_rng(8)
    c = OracleCache(cfg)
    k, v = _kv(rng, 50, cfg)
    c.append_kv(0, [0], [50], k, v)
    c.compress_eligible_pages()
    c.free_seq(0)
    assert c.stats()["dense_in_use"] == 0 and c.stats()["factor_in_use"] == 0


def test_bf16_storage_rounding_matches_library_and_hand_cases():
    import torch
    from oracle.bf16 import round_to_bf16
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-6, 6, 5000), [0.0, -0.0, 1.0, 65504.0]])
    ref = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert (round_to_bf16(x) == ref).all()
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: ties go to the even mantissa (1.0);
    # 1 + 3*2^-8 ties between 1+2^-7 (odd) and 1+2^-6 (even)
    assert round_to_bf16(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert round_to_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    assert round_to_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -20]))[0] == 1 + 2.0 ** -7


def test_storage_rounding_keeps_tables_and_perturbs_factors_by_bf16_epsilon():
    cfg = _cfg(n_kv_heads=1, n_q_heads=1)
    rng = np.random.default_rng(10)
    c = OracleCache(cfg)
    k, v = _kv(rng, 64, cfg)
    c.append_kv(0, [0], [64], k, v)
    c.compress_eligible_pages()
    before = {s: {n: a.copy() for n, a in f.items()} for s, f in c.factor.items()}
    table = c.page_table(0, 0)
    c.round_factors_to_storage_type()
    assert c.page_table(0, 0) == table
    for s, f in c.factor.items():
        for n, a in f.items():
            rel = np.abs(a - before[s][n]) / np.maximum(np.abs(before[s][n]), 1e-300)
            assert rel.max() <= 2.0 ** -8 and rel.max() > 0


def test_footprint_table_printed_in_paper_weak_pin():
    for L, H, d, P, S, W, rk, rv, raw_mib, comp_mib, steady, theory, rtol in _rows("footprint.txt"):
        L, H, d, P, S, W, rk, rv = (int(x) for x in (L, H, d, P, S, W, rk, rv))
        per_token = accounting.kv_cache_elements(L, H, 1, d) * 2
        T = round(raw_mib * 2 ** 20 / per_token)
        assert abs(T * per_token / 2 ** 20 - raw_mib) <= 0.01            # the raw figure is a whole token count
        got = accounting.hybrid_cache_bytes(T, P, S, W, rk, rv, d, L, H) / 2 ** 20
        assert abs(got - comp_mib) <= rtol * comp_mib
        assert abs(got / raw_mib - steady) <= 2e-3
        assert abs(accounting.page_storage_ratio(rk, rv, P, d) - theory) <= 1e-4
        assert abs((steady - theory) - 0.0017) <= 2e-4                   # "0.17 percentage points above"
