"""Pins for the oracle's attention (Eq. 1, Eq. 4, Eq. 5): brute force, closed
forms and special cases.  CPU only."""
import math

import numpy as np

from oracle import attention as att
from oracle import svd


def _brute_softmax_attention(q, K, V, scale):
    """Pure-Python loops, no max subtraction (tiny inputs only)."""
    T, d = len(K), len(q)
    s = [sum(q[k] * K[t][k] for k in range(d)) * scale for t in range(T)]
    e = [math.exp(x) for x in s]
    z = sum(e)
    return [sum(e[t] / z * V[t][k] for t in range(T)) for k in range(d)], [x / z for x in e]


def test_plain_attention_matches_brute_force():
    rng = np.random.default_rng(0)
    T, d = 7, 5
    q, K, V = rng.standard_normal(d), rng.standard_normal((T, d)), rng.standard_normal((T, d))
    out, w = _brute_softmax_attention(q.tolist(), K.tolist(), V.tolist(), 1 / math.sqrt(d))
    assert np.abs(att.attention_plain(q, K, V, 1 / math.sqrt(d)) - np.array(out)).max() <= 1e-14
    sw = att.softmax_weights(q, K, 1 / math.sqrt(d))
    assert np.abs(sw - np.array(w)).max() <= 1e-15 and abs(sw.sum() - 1) <= 1e-15


def test_zero_query_gives_mean_of_values():
    rng = np.random.default_rng(1)
    K, V = rng.standard_normal((33, 8)), rng.standard_normal((33, 8))
    assert np.abs(att.attention_plain(np.zeros(8), K, V, 0.3) - V.mean(axis=0)).max() <= 1e-15


def test_dominant_score_selects_that_row():
    rng = np.random.default_rng(2)
    K, V = rng.standard_normal((20, 8)) * 0.01, rng.standard_normal((20, 8))
    q = rng.standard_normal(8)
    K[11] = 500.0 * q / (q @ q)
    assert np.abs(att.attention_plain(q, K, V, 1.0) - V[11]).max() <= 1e-12


def test_hand_computed_two_token_case():
    # scores ln 1 and ln 3 -> weights 1/4, 3/4
    q = np.array([1.0, 0.0])
    K = np.array([[0.0, 5.0], [math.log(3.0), -2.0]])
    V = np.array([[4.0, 0.0], [0.0, 8.0]])
    assert np.abs(att.attention_plain(q, K, V, 1.0) - np.array([1.0, 6.0])).max() <= 1e-14


def test_factor_form_and_merge_equal_plain_definition():
    # Eq. 4 + Eq. 5 over a mix of dense and factor pages == Eq. 1 over [dense rows; A B rows]
    rng = np.random.default_rng(3)
    P, d, r = 16, 32, 5
    q = rng.standard_normal(d)
    scale = 1 / math.sqrt(d)
    states, Ks, Vs = [], [], []
    for p in range(6):
        if p in (0, 5):
            rows = P if p == 0 else 7            # a partial last page
            Kp, Vp = rng.standard_normal((rows, d)), rng.standard_normal((rows, d))
            states.append(att.page_state_dense(q, Kp, Vp, scale))
        else:
            Ak, Bk = rng.standard_normal((P, r)), rng.standard_normal((r, d))
            Av, Bv = rng.standard_normal((P, r + 1)), rng.standard_normal((r + 1, d))
            states.append(att.page_state_factor(q, Ak, Bk, Av, Bv, scale))
            Kp, Vp = Ak @ Bk, Av @ Bv
        Ks.append(Kp)
        Vs.append(Vp)
    ref = att.attention_plain(q, np.concatenate(Ks), np.concatenate(Vs), scale)
    out = att.merge_page_states(states)
    assert np.abs(out - ref).max() <= 1e-12 * np.abs(ref).max()
    # the merge is order-free and split-free (associativity of Eq. 5)
    perm = [3, 0, 5, 1, 4, 2]
    assert np.abs(att.merge_page_states([states[i] for i in perm]) - ref).max() <= 1e-12


def test_page_state_matches_brute_force_on_one_page():
    rng = np.random.default_rng(4)
    P, d, r = 4, 6, 2
    q = rng.standard_normal(d)
    Ak, Bk, Av, Bv = (rng.standard_normal(s) for s in [(P, r), (r, d), (P, r), (r, d)])
    m, l, o = att.page_state_factor(q, Ak, Bk, Av, Bv, 0.5)
    out, _ = _brute_softmax_attention(q.tolist(), (Ak @ Bk).tolist(), (Av @ Bv).tolist(), 0.5)
    assert np.abs(o / l - np.array(out)).max() <= 1e-13
    assert abs(m - ((Ak @ Bk) @ q * 0.5).max()) <= 1e-14


def test_full_rank_factors_reproduce_dense_attention():
    # r = min(P, d) = P: A B = X exactly, so factor-form attention is vanilla attention
    rng = np.random.default_rng(5)
    P, d = 16, 32
    K, V, q = rng.standard_normal((P, d)), rng.standard_normal((P, d)), rng.standard_normal(d)
    Ak, Bk, _ = svd.page_factors(K[None], P)
    Av, Bv, _ = svd.page_factors(V[None], P)
    m, l, o = att.page_state_factor(q, Ak[0], Bk[0], Av[0], Bv[0], 0.2)
    assert np.abs(o / l - att.attention_plain(q, K, V, 0.2)).max() <= 1e-12
