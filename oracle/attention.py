"""ORACLE — TEST INFRASTRUCTURE ONLY.

Single-query softmax attention in fp64.

attention_plain     Eq. 1: softmax(q K^T / sqrt(d)) V over the full (T x d)
                    key and value matrices.  Factorized pages are materialised
                    as L R first (the oracle is allowed to).
page_state_factor   Eq. 4: page-local (m_p, l_p, o_p) straight from factors,
                    contracting q with the small factors first.
page_state_dense    Section 3.3: the same state from stored K_p, V_p rows.
merge_page_states   Eq. 5: online-softmax merge of page states.

The cache state machine uses attention_plain; the page-wise routines exist to
check that the factor-form algebra and the merge equal the plain definition.
"""
import numpy as np


def attention_plain(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """q: [d]; K, V: [T, d]; returns softmax(K q * scale)^T V as [d] (Eq. 1)."""
    s = (K @ q) * scale
    w = np.exp(s - s.max())
    w = w / w.sum()
    return w @ V


def softmax_weights(q: np.ndarray, K: np.ndarray, scale: float) -> np.ndarray:
    s = (K @ q) * scale
    w = np.exp(s - s.max())
    return w / w.sum()


def page_state_factor(q, A_k, B_k, A_v, B_v, scale):
    """Eq. 4.  A_* are the paper's L (P x r), B_* the paper's R (r x d)."""
    q_t = B_k @ q                      # q R_K^T        (r_k)
    s = (A_k @ q_t) * scale            # (.) L_K^T / sqrt(d)   (P)
    m = s.max()
    e = np.exp(s - m)
    l = e.sum()
    o = (e @ A_v) @ B_v                # (exp(s-m) L_V) R_V    (d)
    return m, l, o


def page_state_dense(q, K_p, V_p, scale):
    """Page state from dense rows (valid rows only)."""
    s = (K_p @ q) * scale
    m = s.max()
    e = np.exp(s - m)
    return m, e.sum(), e @ V_p


def merge_page_states(states):
    """Eq. 5: m = max_p m_p; o = sum_p e^{m_p-m} o_p / sum_p e^{m_p-m} l_p."""
    m = max(st[0] for st in states)
    num = sum(np.exp(st[0] - m) * st[2] for st in states)
    den = sum(np.exp(st[0] - m) * st[1] for st in states)
    return num / den
