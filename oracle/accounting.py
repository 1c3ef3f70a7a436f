"""ORACLE — TEST INFRASTRUCTURE ONLY.  Size formulas printed in the paper."""


def page_storage_ratio(r_k: int, r_v: int, P: int, d: int) -> float:
    """Eq. 3: stored elements of a factorized K/V page pair over the dense pair.

    Factors hold r_k*(P+d) + r_v*(P+d) elements; the dense pair holds 2*P*d.
    """
    return (r_k + r_v) * (P + d) / (2.0 * P * d)


def kv_cache_elements(n_layers: int, n_kv_heads: int, T: int, d: int) -> int:
    """Section 1: a dense KV cache holds 2 * L * H_kv * T * d elements."""
    return 2 * n_layers * n_kv_heads * T * d


def eligible_pages_token_form(T: int, P: int, sink_tokens: int, recent_tokens: int):
    """Section 3.3 (construction + incremental update), written token by token.

    A page may be factorized when it is complete, lies wholly after the sink
    region and wholly before the last `recent_tokens` tokens' worth of completed
    pages: every token index t of page p must satisfy t >= sink_tokens and the
    page's end (p+1)*P must not exceed floor(T/P)*P - recent_tokens.
    This is the brute-force form used to pin the closed-form rule in cache.py.
    """
    out = []
    n_pages = T // P
    completed_tokens = n_pages * P
    for p in range(n_pages):
        first, last = p * P, (p + 1) * P - 1
        if first < sink_tokens:
            continue
        if last + 1 > completed_tokens - recent_tokens:
            continue
        out.append(p)
    return out


def hybrid_cache_bytes(T: int, P: int, sink_tokens: int, recent_tokens: int, r_k: int, r_v: int, d: int,
                       n_layers: int, n_kv_heads: int, bytes_per_element: int = 2) -> int:
    """Logical live footprint of the hybrid cache (Section 3.3 construction + Eq. 3): every
    factorized page holds (r_k + r_v)(P + d) elements, every other token 2 d elements, per layer
    and KV head.  Pages are factorized by the closed-form rule of cache.eligible_range."""
    n_c = T // P
    lo = sink_tokens // P
    hi = max(lo, n_c - recent_tokens // P)
    n_factor = hi - lo
    dense_tokens = T - n_factor * P
    per_head = n_factor * (r_k + r_v) * (P + d) + dense_tokens * 2 * d
    return n_layers * n_kv_heads * per_head * bytes_per_element
