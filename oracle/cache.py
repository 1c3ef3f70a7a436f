"""ORACLE — TEST INFRASTRUCTURE ONLY.

The hybrid paged KV cache of Section 3.3 as an fp64 state machine with the
same four operations as the library boundary:

    append_kv                 "Incremental Cache Update": a new K/V row goes to
                              the current dense page and takes part in attention
                              at once; a new dense slot opens at a page boundary.
    compress_eligible_pages   "Page-Wise Low-Rank KV Cache Construction": every
                              completed page outside the sink region and the
                              local window is replaced, once, by its rank-r
                              truncated-SVD factors (Eq. 2); the dense slot is
                              released; factor pages are never revisited.
    decode_attention          "Attention over Mixed KV Pages": softmax attention
                              (Eq. 1) over dense rows and reconstructed factor
                              pages, for every query head of every sequence.
    page_table                (kind, slot) of each logical page.

Readings where the paper is silent (slot allocation policy, per-layer token
counts, GQA head mapping) are written next to the code that takes them.
"""
from dataclasses import dataclass, field

import numpy as np

from . import attention as _att
from . import bf16 as _bf16
from . import global_svd as _global
from . import quant as _quant
from . import svd as _svd

DENSE, FACTOR = 0, 1


@dataclass
class OracleConfig:
    n_layers: int
    n_kv_heads: int
    n_q_heads: int
    head_dim: int
    page_size: int
    rank_k: int
    rank_v: int
    sink_tokens: int
    recent_tokens: int
    max_seqs: int
    n_dense_slots: int
    n_factor_slots: int
    softmax_scale: float = 0.0          # 0 => 1/sqrt(head_dim)  (Eq. 1)
    factor_bits: int = 16               # 4 => factors are INT4-quantized when a page is converted (Section 4.3)
    global_rank: int = 0                # > 0 => the Global SVD form (Section 4.2): one basis per (sequence, layer, KV
                                        # head), fixed by the pages of the first conversion; rank_k, rank_v unused


class PoolExhausted(RuntimeError):
    pass


class _FreeList:
    """Reading (paper only says storage is preallocated and dense slots are
    released): slots are handed out in the caller's order array; a released slot
    goes on a stack that is popped before the order array is consumed further."""

    def __init__(self, order):
        self.order = [int(x) for x in order]
        self.next = 0
        self.stack = []

    def alloc(self):
        if self.stack:
            return self.stack.pop()
        if self.next >= len(self.order):
            raise PoolExhausted()
        s = self.order[self.next]
        self.next += 1
        return s

    def release(self, s):
        self.stack.append(int(s))

    def in_use(self):
        return self.next - len(self.stack)


@dataclass
class _SeqLayer:
    n_tokens: int = 0
    kinds: list = field(default_factory=list)
    slots: list = field(default_factory=list)


def eligible_range(n_tokens: int, P: int, sink_tokens: int, recent_tokens: int):
    """Closed form of the eligibility rule: with n_c = floor(T/P) completed
    pages, n_s = S/P sink pages and n_w = W/P window pages, page p may be
    factorized iff n_s <= p < n_c - n_w.  The n_w most recently completed pages
    and the incomplete page stay dense; the paper's default dense region (one
    sink page, the most recently completed page, the current incomplete page)
    is S = W = P.  Returns (lo, hi) with hi >= lo."""
    n_c = n_tokens // P
    lo = sink_tokens // P
    hi = max(lo, n_c - recent_tokens // P)
    return lo, hi


class OracleCache:
    def __init__(self, cfg: OracleConfig, dense_slot_order=None, factor_slot_order=None):
        assert cfg.n_q_heads % cfg.n_kv_heads == 0
        assert cfg.sink_tokens % cfg.page_size == 0 and cfg.recent_tokens % cfg.page_size == 0
        assert 0 < cfg.rank_k <= cfg.page_size and 0 < cfg.rank_v <= cfg.page_size
        assert cfg.page_size <= cfg.head_dim
        self.cfg = cfg
        self.scale = cfg.softmax_scale if cfg.softmax_scale > 0 else 1.0 / np.sqrt(cfg.head_dim)
        self.dense_free = _FreeList(range(cfg.n_dense_slots) if dense_slot_order is None else dense_slot_order)
        self.factor_free = _FreeList(range(cfg.n_factor_slots) if factor_slot_order is None else factor_slot_order)
        # slot -> arrays.  A slot is one logical page of one layer, all KV heads.
        self.dense = {}      # slot -> (K [H_kv,P,d], V [H_kv,P,d]) fp64
        self.factor = {}     # slot -> dict(A_k [H,P,r_k], B_k [H,r_k,d], A_v, B_v) fp64
        self.sigma = {}      # slot -> (sigma_k [H,P], sigma_v [H,P]) sorted descending
        self.state = {}      # (seq, layer) -> _SeqLayer
        self.pages_compressed = 0
        self.pending = {}    # layer -> [(seq, page, factor slot, factors, sigma)] begun, not committed
        self.basis = {}      # Global SVD form: (seq, layer) -> dict(B_k [H,r,d], B_v [H,r,d], sigma_k, sigma_v, pages)

    # ------------------------------------------------------------------ append
    def _sl(self, seq, layer):
        assert 0 <= seq < self.cfg.max_seqs and 0 <= layer < self.cfg.n_layers
        return self.state.setdefault((seq, layer), _SeqLayer())

    def append_kv(self, layer, seq_ids, n_new, k, v):
        """k, v: [sum(n_new), H_kv, d] (values exactly representable in bf16,
        widened to fp64 by the caller).  Token counts are kept per (seq, layer):
        this call advances only `layer`'s count."""
        c = self.cfg
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        assert k.shape == v.shape == (int(sum(n_new)), c.n_kv_heads, c.head_dim)
        row = 0
        for seq, n in zip(seq_ids, n_new):
            sl = self._sl(int(seq), layer)
            for _ in range(int(n)):
                t = sl.n_tokens
                p, r = divmod(t, c.page_size)
                if r == 0:
                    slot = self.dense_free.alloc()
                    self.dense[slot] = (np.zeros((c.n_kv_heads, c.page_size, c.head_dim)),
                                        np.zeros((c.n_kv_heads, c.page_size, c.head_dim)))
                    sl.kinds.append(DENSE)
                    sl.slots.append(slot)
                Kp, Vp = self.dense[sl.slots[p]]
                Kp[:, r, :] = k[row]
                Vp[:, r, :] = v[row]
                sl.n_tokens = t + 1
                row += 1

    # ---------------------------------------------------------------- compress
    def eligible(self, seq, layer):
        sl = self.state.get((seq, layer))
        if sl is None:
            return []
        c = self.cfg
        lo, hi = eligible_range(sl.n_tokens, c.page_size, c.sink_tokens, c.recent_tokens)
        return [p for p in range(lo, hi) if sl.kinds[p] == DENSE]

    def compress_eligible_pages(self, layer=-1):
        """Processes eligible pages in ascending (seq, layer, page) order; for
        each: allocate a factor slot, factorize every KV head's K page (rank r_k)
        and V page (rank r_v), then release the dense slot.  Returns the number
        of logical pages converted."""
        c = self.cfg
        layers = range(c.n_layers) if layer < 0 else [layer]
        work = []
        for seq in range(c.max_seqs):
            for ly in layers:
                for p in self.eligible(seq, ly):
                    work.append((seq, ly, p))
        if not work:
            return 0
        factors = self._factorize(work)
        for (seq, ly, p), (f, sig) in zip(work, factors):
            fslot = self.factor_free.alloc()
            self.factor[fslot] = f
            self.sigma[fslot] = sig
            self._flip(seq, ly, p, fslot)
        self.pages_compressed += len(work)
        return len(work)

    def _factorize(self, work):
        """Rank-r factors (Eq. 2) of the listed (seq, layer, page) dense pages, every KV head: a list of
        (dict(A_k, B_k, A_v, B_v), (sigma_k, sigma_v)) in the order of `work`."""
        c = self.cfg
        if c.global_rank > 0:
            return self._factorize_global(work)
        Ks = np.stack([self.dense[self.state[(s, ly)].slots[p]][0] for s, ly, p in work])  # [n,H,P,d]
        Vs = np.stack([self.dense[self.state[(s, ly)].slots[p]][1] for s, ly, p in work])
        n, H = Ks.shape[0], c.n_kv_heads
        A_k, B_k, s_k = _svd.page_factors(Ks.reshape(n * H, c.page_size, c.head_dim), c.rank_k)
        A_v, B_v, s_v = _svd.page_factors(Vs.reshape(n * H, c.page_size, c.head_dim), c.rank_v)
        out = []
        for i in range(n):
            sel = slice(i * H, (i + 1) * H)
            f = dict(A_k=A_k[sel].copy(), B_k=B_k[sel].copy(), A_v=A_v[sel].copy(), B_v=B_v[sel].copy())
            if c.factor_bits == 4:
                for h in range(H):
                    f["A_k"][h], f["B_k"][h], f["A_v"][h], f["B_v"][h] = _quant.quantized_page_factors(
                        f["A_k"][h], f["B_k"][h], f["A_v"][h], f["B_v"][h])
            out.append((f, (s_k[sel].copy(), s_v[sel].copy())))
        return out

    def _factorize_global(self, work):
        """Global SVD form.  The pages of the first conversion of a (sequence, layer) are its region: their rows,
        stacked in page order, give the basis of every KV head (K and V separately); every page - of the region or
        converted later - stores A = X_page B^T and shares B."""
        c, r = self.cfg, self.cfg.global_rank
        H = c.n_kv_heads
        by_sl = {}
        for s, ly, p in work:
            by_sl.setdefault((s, ly), []).append(p)
        for (s, ly), pages in by_sl.items():
            if (s, ly) in self.basis:
                continue
            Kr = np.concatenate([self.dense[self.state[(s, ly)].slots[p]][0] for p in pages], axis=1)   # [H, T, d]
            Vr = np.concatenate([self.dense[self.state[(s, ly)].slots[p]][1] for p in pages], axis=1)
            fk = [_global.region_factors(Kr[h], r) for h in range(H)]
            fv = [_global.region_factors(Vr[h], r) for h in range(H)]
            self.basis[(s, ly)] = dict(B_k=np.stack([f[1] for f in fk]), B_v=np.stack([f[1] for f in fv]),
                                       sigma_k=[f[2] for f in fk], sigma_v=[f[2] for f in fv], pages=list(pages))
        out = []
        for s, ly, p in work:
            b = self.basis[(s, ly)]
            Kp, Vp = self.dense[self.state[(s, ly)].slots[p]]
            f = dict(A_k=np.stack([_global.project_page(Kp[h], b["B_k"][h]) for h in range(H)]), B_k=b["B_k"],
                     A_v=np.stack([_global.project_page(Vp[h], b["B_v"][h]) for h in range(H)]), B_v=b["B_v"])
            out.append((f, None))
        return out

    def _flip(self, seq, ly, p, fslot):
        """The page becomes a factor page; its dense slot is released."""
        sl = self.state[(seq, ly)]
        dslot = sl.slots[p]
        del self.dense[dslot]
        self.dense_free.release(dslot)
        sl.kinds[p] = FACTOR
        sl.slots[p] = fslot

    def compress_begin(self, layer):
        """First half of a two-step compression of one layer (a caller-side arrangement, not in the paper: the
        factorization may run while other work proceeds).  Picks the pages eligible now, ascending (seq, page),
        allocates their factor slots and computes their factors; the pages stay dense pages, with their dense
        slots, until compress_commit().  Returns the number of pages picked."""
        assert layer not in self.pending, "layer already has an uncommitted compression"
        c = self.cfg
        work = [(seq, layer, p) for seq in range(c.max_seqs) for p in self.eligible(seq, layer)]
        work = work[:len(self.factor_free.order) - self.factor_free.in_use()]      # as many as factor slots are left
        if not work:
            return 0
        self.pending[layer] = [(seq, p, self.factor_free.alloc(), f, sig)
                               for (seq, _, p), (f, sig) in zip(work, self._factorize(work))]
        return len(work)

    def compress_commit(self, layer=-1):
        """Second half: per pending page, in the order it was picked, the page becomes a factor page and its
        dense slot is released.  layer = -1: every layer with a pending compression, ascending."""
        done = 0
        for ly in (sorted(self.pending) if layer < 0 else [layer]):
            for seq, p, fslot, f, sig in self.pending.pop(ly, []):
                self.factor[fslot] = f
                self.sigma[fslot] = sig
                self._flip(seq, ly, p, fslot)
                done += 1
        self.pages_compressed += done
        return done

    # ------------------------------------------------------------------ attend
    def gather_kv(self, seq, layer, kv_head):
        """Stack the logical pages of one (seq, layer, kv head) into K_all,
        V_all [T, d]; factor pages are materialised as A B."""
        c = self.cfg
        sl = self.state[(seq, layer)]
        Ks, Vs = [], []
        n_pages = -(-sl.n_tokens // c.page_size)
        for p in range(n_pages):
            rows = min(c.page_size, sl.n_tokens - p * c.page_size)
            if sl.kinds[p] == DENSE:
                Kp, Vp = self.dense[sl.slots[p]]
                Ks.append(Kp[kv_head, :rows])
                Vs.append(Vp[kv_head, :rows])
            else:
                f = self.factor[sl.slots[p]]
                Ks.append(f["A_k"][kv_head] @ f["B_k"][kv_head])
                Vs.append(f["A_v"][kv_head] @ f["B_v"][kv_head])
        return np.concatenate(Ks), np.concatenate(Vs)

    def decode_attention(self, layer, seq_ids, q):
        """q: [n_seqs, H_q, d].  Query head h reads KV head h // G, G = H_q/H_kv
        (the grouped-query convention of the model runtime the paper builds on;
        the paper omits the head index).  Returns [n_seqs, H_q, d] fp64."""
        c = self.cfg
        q = np.asarray(q, dtype=np.float64)
        G = c.n_q_heads // c.n_kv_heads
        out = np.zeros((len(seq_ids), c.n_q_heads, c.head_dim))
        for i, seq in enumerate(seq_ids):
            sl = self.state.get((int(seq), layer))
            if sl is None or sl.n_tokens == 0:
                raise ValueError("attention over an empty sequence")
            for kvh in range(c.n_kv_heads):
                K_all, V_all = self.gather_kv(int(seq), layer, kvh)
                for g in range(G):
                    h = kvh * G + g
                    out[i, h] = _att.attention_plain(q[i, h], K_all, V_all, self.scale)
        return out

    def decode_attention_multi(self, layer, seq_ids, q):
        """Several queries per sequence (speculative decoding, a chunk of a
        prefill): q is [n_seqs, q_len, H_q, d] and query j belongs to the
        position T - q_len + j of its sequence, whose key and value rows are
        already in the cache.  Eq. 1 is causal: that position attends over the
        tokens 0 .. T - q_len + j, itself included.  Not spelled out in the
        paper (its Eq. 4 has one query); q_len = 1 is decode_attention().
        Returns [n_seqs, q_len, H_q, d] fp64."""
        c = self.cfg
        q = np.asarray(q, dtype=np.float64)
        n, q_len = q.shape[0], q.shape[1]
        G = c.n_q_heads // c.n_kv_heads
        out = np.zeros((n, q_len, c.n_q_heads, c.head_dim))
        for i, seq in enumerate(seq_ids):
            sl = self.state.get((int(seq), layer))
            if sl is None or sl.n_tokens < q_len:
                raise ValueError("fewer tokens in the cache than queries")
            for kvh in range(c.n_kv_heads):
                K_all, V_all = self.gather_kv(int(seq), layer, kvh)
                for j in range(q_len):
                    visible = sl.n_tokens - q_len + j + 1
                    for g in range(G):
                        h = kvh * G + g
                        out[i, j, h] = _att.attention_plain(q[i, j, h], K_all[:visible], V_all[:visible], self.scale)
        return out

    def attention_state(self, layer, seq_ids, q):
        """The softmax state of this cache's tokens for each query (the quantities Eq. 5 merges), for a sequence
        whose tokens are spread over several caches: m [n, H_q] = max_t s_t with s_t = q . k_t * scale (natural
        units), l [n, H_q] = sum_t exp(s_t - m), o [n, H_q, d] = sum_t exp(s_t - m) v_t.  Factor pages enter as A B.
        Merging the states of all caches with attention.merge_page_states gives Eq. 1 over all tokens."""
        c = self.cfg
        q = np.asarray(q, dtype=np.float64)
        G = c.n_q_heads // c.n_kv_heads
        n = len(seq_ids)
        m, l, o = np.zeros((n, c.n_q_heads)), np.zeros((n, c.n_q_heads)), np.zeros((n, c.n_q_heads, c.head_dim))
        for i, seq in enumerate(seq_ids):
            for kvh in range(c.n_kv_heads):
                K_all, V_all = self.gather_kv(int(seq), layer, kvh)
                for g in range(G):
                    h = kvh * G + g
                    m[i, h], l[i, h], o[i, h] = _att.page_state_dense(q[i, h], K_all, V_all, self.scale)
        return m, l, o

    def decode_attention_pagewise(self, layer, seq_ids, q):
        """Same result through Eq. 4 (factor pages evaluated from factors, never
        materialised) and Eq. 5 (merge).  Used to check the algebra only."""
        c = self.cfg
        q = np.asarray(q, dtype=np.float64)
        G = c.n_q_heads // c.n_kv_heads
        out = np.zeros((len(seq_ids), c.n_q_heads, c.head_dim))
        for i, seq in enumerate(seq_ids):
            sl = self.state[(int(seq), layer)]
            n_pages = -(-sl.n_tokens // c.page_size)
            for h in range(c.n_q_heads):
                kvh = h // G
                states = []
                for p in range(n_pages):
                    rows = min(c.page_size, sl.n_tokens - p * c.page_size)
                    if sl.kinds[p] == DENSE:
                        Kp, Vp = self.dense[sl.slots[p]]
                        states.append(_att.page_state_dense(q[i, h], Kp[kvh, :rows], Vp[kvh, :rows], self.scale))
                    else:
                        f = self.factor[sl.slots[p]]
                        states.append(_att.page_state_factor(q[i, h], f["A_k"][kvh], f["B_k"][kvh],
                                                             f["A_v"][kvh], f["B_v"][kvh], self.scale))
                out[i, h] = _att.merge_page_states(states)
        return out

    # ------------------------------------------------------------- bookkeeping
    def page_table(self, seq, layer):
        sl = self.state.get((seq, layer), _SeqLayer())
        return list(sl.kinds), list(sl.slots), sl.n_tokens

    def set_factors(self, slot, A_k, B_k, A_v, B_v):
        """Replace a factor slot's contents (used to evaluate attention over
        factors produced elsewhere, e.g. rounded to the storage type)."""
        self.factor[slot] = dict(A_k=np.asarray(A_k, np.float64), B_k=np.asarray(B_k, np.float64),
                                 A_v=np.asarray(A_v, np.float64), B_v=np.asarray(B_v, np.float64))

    def round_factors_to_storage_type(self):
        """Applies the storage step to every factor page: A and B rounded to
        bf16 (the type dense pages are stored in; Eq. 3 counts elements of one
        type).  Attention afterwards reads the stored values, still in fp64."""
        for slot, f in self.factor.items():
            self.factor[slot] = {k: _bf16.round_to_bf16(v) for k, v in f.items()}
        for b in self.basis.values():
            b["B_k"], b["B_v"] = _bf16.round_to_bf16(b["B_k"]), _bf16.round_to_bf16(b["B_v"])

    def free_seq(self, seq):
        """Release every slot of a sequence, layers ascending, pages ascending."""
        for ly in range(self.cfg.n_layers):
            self.basis.pop((seq, ly), None)
            sl = self.state.pop((seq, ly), None)
            if sl is None:
                continue
            for kind, slot in zip(sl.kinds, sl.slots):
                if kind == DENSE:
                    del self.dense[slot]
                    self.dense_free.release(slot)
                else:
                    del self.factor[slot]
                    self.sigma.pop(slot, None)
                    self.factor_free.release(slot)

    def stats(self):
        return dict(dense_in_use=self.dense_free.in_use(), factor_in_use=self.factor_free.in_use(),
                    pages_compressed=self.pages_compressed)
