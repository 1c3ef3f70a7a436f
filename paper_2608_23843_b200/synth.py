"""Seeded synthetic inputs shaped like long-context KV caches.

This module holds no arithmetic of the method itself: it only draws random
keys, values, queries and context lengths.  Both the CUDA path and the CPU
checker consume the buffers it returns.

Recipe (one definition for every workload).  Per (sequence, layer, KV head,
logical page), for K and V separately:
    U  ~ N(0,1)  [P, 8],   Wt ~ N(0,1) [8, d],   s_i = 0.7**i  (i = 0..7)
    X  = U diag(s) Wt + 0.05 * N(0,1) [P, d]
Keys are then multiplied channel-wise by c [d] with c_j = exp(Uniform[ln 0.5,
ln 8]), one vector per (layer, KV head) shared by all pages and sequences
(fixed key outlier channels).  With `outlier_prob` > 0 each token's key row is
multiplied by `outlier_gain` with that probability (sparse outlier tokens).
Everything is rounded to bf16.  Queries are N(0,1) in bf16.
"""
import math

import torch

SIGNAL_RANK = 8
DECAY = 0.7
NOISE_STD = 0.05
SCALE_LO, SCALE_HI = 0.5, 8.0


def _gen(device, *key):
    """A torch.Generator seeded from a tuple of small non-negative integers."""
    seed = 0x9E3779B97F4A7C15
    for k in key:
        seed = (seed * 6364136223846793005 + int(k) + 1442695040888963407) % (1 << 63)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def channel_scales(seed, layer, n_kv_heads, d, device="cpu"):
    """Per-channel key scales c [H_kv, d], log-uniform in [0.5, 8]."""
    g = _gen(device, seed, 1, layer)
    u = torch.rand((n_kv_heads, d), generator=g, device=device, dtype=torch.float32)
    return torch.exp(math.log(SCALE_LO) + u * (math.log(SCALE_HI) - math.log(SCALE_LO)))


def lowrank_pages(g, n, P, d, device="cpu"):
    """[n, P, d] fp32: rank-8 signal with singular-value profile 0.7**i plus N(0, 0.05) noise."""
    U = torch.randn((n, P, SIGNAL_RANK), generator=g, device=device, dtype=torch.float32)
    Wt = torch.randn((n, SIGNAL_RANK, d), generator=g, device=device, dtype=torch.float32)
    s = DECAY ** torch.arange(SIGNAL_RANK, device=device, dtype=torch.float32)
    E = torch.randn((n, P, d), generator=g, device=device, dtype=torch.float32)
    return torch.bmm(U * s, Wt) + NOISE_STD * E


def make_kv(seed, layer, seq, n_tokens, n_kv_heads, d, P, device="cpu",
            outlier_prob=0.0, outlier_gain=10.0):
    """Keys and values of one (sequence, layer): two bf16 tensors [n_tokens, H_kv, d].

    Tokens are generated page by page (the last page is cut to n_tokens)."""
    n_pages = -(-n_tokens // P)
    g = _gen(device, seed, 2, layer, seq)
    K = lowrank_pages(g, n_kv_heads * n_pages, P, d, device).view(n_kv_heads, n_pages * P, d)
    V = lowrank_pages(g, n_kv_heads * n_pages, P, d, device).view(n_kv_heads, n_pages * P, d)
    K = K * channel_scales(seed, layer, n_kv_heads, d, device)[:, None, :]
    if outlier_prob > 0.0:
        hit = torch.rand((n_kv_heads, n_pages * P, 1), generator=g, device=device) < outlier_prob
        K = torch.where(hit, K * outlier_gain, K)
    K = K[:, :n_tokens].transpose(0, 1).contiguous().to(torch.bfloat16)
    V = V[:, :n_tokens].transpose(0, 1).contiguous().to(torch.bfloat16)
    return K, V


def make_q(seed, layer, step, n_seqs, n_q_heads, d, device="cpu"):
    """Queries [n_seqs, H_q, d], N(0,1) rounded to bf16."""
    g = _gen(device, seed, 3, layer, step)
    return torch.randn((n_seqs, n_q_heads, d), generator=g, device=device,
                       dtype=torch.float32).to(torch.bfloat16)


def loguniform_lengths(seed, n, lo, hi):
    """n context lengths, floor(exp(Uniform[ln lo, ln hi])) (ragged serving batch)."""
    g = _gen("cpu", seed, 4)
    u = torch.rand((n,), generator=g, dtype=torch.float64)
    return [int(x) for x in torch.floor(torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo))))]


def slot_permutation(seed, n, which):
    """A seeded permutation of range(n): the shuffled physical page pool."""
    g = _gen("cpu", seed, 5, which)
    return torch.randperm(n, generator=g).to(torch.int32)
