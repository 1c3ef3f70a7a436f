"""ctypes binding of libpkv.so (see include/pkv.h): argument marshalling only.

Module-level functions carry the C names (`pkv_init_cache`, `pkv_append_kv`,
`pkv_compress_eligible_pages`, `pkv_decode_attention`, ...).  `Cache` is a
convenience wrapper that allocates the caller-owned device buffers with torch
and forwards to those functions; every computation runs in the CUDA library.
There is no CPU fallback: if the library has not been built, loading fails.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpkv.so")

PKV_OK = 0
PKV_ERR_INVALID_ARG = -1
PKV_ERR_POOL_EXHAUSTED = -2
PKV_ERR_BAD_SEQ = -3
PKV_ERR_CUDA = -4
PKV_ERR_NOT_CONVERGED = -5
PKV_ERR_UNSUPPORTED = -6
PKV_ERR_DEVICE_TIMEOUT = -7
PKV_KIND_DENSE, PKV_KIND_FACTOR = 0, 1

EXPORTS = [
    "pkv_query_sizes", "pkv_init_cache", "pkv_append_kv", "pkv_compress_eligible_pages",
    "pkv_decode_attention", "pkv_decode_attention_host", "pkv_get_page_table", "pkv_get_stats",
    "pkv_free_seq", "pkv_destroy_cache", "pkv_last_error", "pkv_read_factors", "pkv_write_factors",
    "pkv_read_dense", "pkv_get_decode_plan", "pkv_decode_attention_static_scratch", "pkv_get_decode_trace",
    "pkv_decode_attention_multi", "pkv_compress_begin", "pkv_compress_commit",
    "pkv_decode_attention_partial", "pkv_merge_attention_states",
    "pkv_get_rotation_schedule", "pkv_read_basis", "pkv_get_row_block_ranges",
]


class PkvConfig(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32), ("rank_k", ctypes.c_int32),
        ("rank_v", ctypes.c_int32), ("sink_tokens", ctypes.c_int32), ("recent_tokens", ctypes.c_int32),
        ("max_seqs", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
        ("n_dense_slots", ctypes.c_int64), ("n_factor_slots", ctypes.c_int64),
        ("softmax_scale", ctypes.c_float), ("jacobi_max_sweeps", ctypes.c_int32),
        ("jacobi_tol", ctypes.c_float), ("n_ctas", ctypes.c_int32), ("decode_variant", ctypes.c_int32),
        ("jacobi_energy_tol", ctypes.c_float), ("factor_bits", ctypes.c_int32), ("decode_overlap", ctypes.c_int32),
        ("global_rank", ctypes.c_int32),
    ]


class PkvSizes(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("dense_slot_bytes", "factor_slot_bytes", "dense_pool_bytes",
                                              "factor_pool_bytes", "meta_bytes", "workspace_bytes")]


class PkvStats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("dense_slots_in_use", "factor_slots_in_use", "pages_compressed",
                                              "page_svds_not_converged", "device_timeouts", "bad_slot_indices",
                                              "last_decode_bytes", "last_decode_units", "page_svds", "jacobi_rounds")]


class PkvError(RuntimeError):
    def __init__(self, status, message=""):
        super().__init__("pkv status %d: %s" % (status, message))
        self.status = status


_lib = None


def lib():
    """The loaded CUDA library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libpkv.so is missing: build it with `python -m paper_2608_23843_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        ip = ctypes.POINTER(ctypes.c_int32)
        L.pkv_query_sizes.argtypes = [ctypes.POINTER(PkvConfig), ctypes.POINTER(PkvSizes)]
        L.pkv_init_cache.argtypes = [ctypes.POINTER(PkvConfig), vp, vp, vp, vp, ip, ip, ctypes.POINTER(vp)]
        L.pkv_append_kv.argtypes = [vp, i32, i32, ip, ip, vp, vp, vp]
        L.pkv_compress_eligible_pages.argtypes = [vp, i32, ctypes.POINTER(i64), vp]
        L.pkv_decode_attention.argtypes = [vp, i32, i32, ip, vp, vp, vp, vp]
        L.pkv_decode_attention_static_scratch.argtypes = [vp, i32, i32, ip, vp, vp, vp, vp]
        L.pkv_decode_attention_multi.argtypes = [vp, i32, i32, ip, i32, vp, vp, vp, vp]
        L.pkv_compress_begin.argtypes = [vp, i32, vp, vp, ctypes.POINTER(i64)]
        L.pkv_decode_attention_partial.argtypes = [vp, i32, i32, ip, vp, vp, vp]
        L.pkv_merge_attention_states.argtypes = [vp, i32, i64, vp, vp, vp]
        L.pkv_compress_commit.argtypes = [vp, i32, vp, ctypes.POINTER(i64)]
        L.pkv_decode_attention_host.argtypes = [vp, i32, i32, ip, vp, vp, vp, vp, vp]
        L.pkv_get_page_table.argtypes = [vp, i32, i32, ip, ip, ip, ip]
        L.pkv_get_stats.argtypes = [vp, ctypes.POINTER(PkvStats), vp]
        L.pkv_free_seq.argtypes = [vp, i32]
        L.pkv_destroy_cache.argtypes = [vp]
        L.pkv_last_error.argtypes = [vp]
        L.pkv_last_error.restype = ctypes.c_char_p
        L.pkv_read_factors.argtypes = [vp, i64, i32, vp, vp, vp, vp, vp]
        L.pkv_write_factors.argtypes = [vp, i64, i32, vp, vp, vp, vp, vp]
        L.pkv_read_dense.argtypes = [vp, i64, i32, vp, vp, vp]
        L.pkv_read_basis.argtypes = [vp, i32, i32, i32, vp, vp, vp]
        L.pkv_get_decode_plan.argtypes = [vp, i32, ip, ip, ip, ip]
        L.pkv_get_decode_trace.argtypes = [vp, ctypes.POINTER(ctypes.c_int64), i32, vp]
        L.pkv_get_rotation_schedule.argtypes = [i32, ctypes.POINTER(ctypes.c_uint8), i64, ip, ip, ip]
        L.pkv_get_row_block_ranges.argtypes = [i64, i32, i32, i32, ip]
        for name in EXPORTS:
            if name != "pkv_last_error":
                getattr(L, name).restype = ctypes.c_int32
        _lib = L
    return _lib


_INT_ARRAYS = {}


def _ints(xs):
    """A ctypes int32 array for a sequence of ints (decode calls pass the same id list every step: remembered)."""
    if len(xs) > 4096:                                   # e.g. slot orders: built once, not worth remembering
        vals = [int(x) for x in xs]
        return (ctypes.c_int32 * len(vals))(*vals), len(vals)
    key = tuple(xs)
    hit = _INT_ARRAYS.get(key)
    if hit is None:
        vals = [int(x) for x in key]
        hit = ((ctypes.c_int32 * len(vals))(*vals), len(vals))
        if len(_INT_ARRAYS) >= 256:
            _INT_ARRAYS.clear()
        _INT_ARRAYS[key] = hit
    return hit


def _ptr(t):
    """Device (or host) address of a tensor as a plain int: ctypes converts it for a void* parameter, and building
    a c_void_p object per argument is a measurable part of a 5 us call."""
    return None if t is None else t.data_ptr()


def _stream(stream):
    if stream is None or isinstance(stream, int):
        return stream
    return stream.cuda_stream


try:                                                     # raw handle of the current stream without a Stream object (2 us less per call)
    _raw_current_stream = torch._C._cuda_getCurrentRawStream
except AttributeError:                                   # pragma: no cover
    _raw_current_stream = None


# ---- functions with the C names -------------------------------------------------
def pkv_query_sizes(cfg: PkvConfig) -> PkvSizes:
    out = PkvSizes()
    st = lib().pkv_query_sizes(ctypes.byref(cfg), ctypes.byref(out))
    if st != PKV_OK:
        raise PkvError(st, "pkv_query_sizes")
    return out


def pkv_init_cache(cfg, dense_pool, factor_pool, meta, workspace, dense_slot_order=None, factor_slot_order=None):
    """Tensors (or None for all four = dry run) -> opaque handle."""
    h = ctypes.c_void_p()
    d_ord = f_ord = None
    if dense_slot_order is not None:
        d_ord, _ = _ints(dense_slot_order)
    if factor_slot_order is not None:
        f_ord, _ = _ints(factor_slot_order)
    st = lib().pkv_init_cache(ctypes.byref(cfg), _ptr(dense_pool), _ptr(factor_pool), _ptr(meta), _ptr(workspace),
                              d_ord, f_ord, ctypes.byref(h))
    if st != PKV_OK:
        raise PkvError(st, "pkv_init_cache")
    return h


def _check(handle, st):
    if st != PKV_OK:
        raise PkvError(st, lib().pkv_last_error(handle).decode())


def pkv_append_kv(handle, layer, seq_ids, n_new, k, v, stream=None):
    ids, n = _ints(seq_ids)
    cnt, _ = _ints(n_new)
    _check(handle, lib().pkv_append_kv(handle, layer, n, ids, cnt, _ptr(k), _ptr(v), _stream(stream)))


def pkv_compress_eligible_pages(handle, layer=-1, stream=None) -> int:
    n = ctypes.c_int64(0)
    st = lib().pkv_compress_eligible_pages(handle, layer, ctypes.byref(n), _stream(stream))
    _check(handle, st)
    return int(n.value)


def pkv_compress_begin(handle, layer, main_stream=None, side_stream=None) -> int:
    """Starts factorizing the layer's eligible pages on side_stream; returns how many.  The pages stay dense until
    pkv_compress_commit.  If the factor pool runs out, PkvError carries the status and `begun` the pages begun."""
    n = ctypes.c_int64(0)
    st = lib().pkv_compress_begin(handle, layer, _stream(main_stream), _stream(side_stream), ctypes.byref(n))
    if st != PKV_OK:
        msg = lib().pkv_last_error(handle)
        e = PkvError(st, msg.decode() if msg else "")
        e.begun = int(n.value)
        raise e
    return int(n.value)


def pkv_compress_commit(handle, layer=-1, main_stream=None) -> int:
    n = ctypes.c_int64(0)
    _check(handle, lib().pkv_compress_commit(handle, layer, _stream(main_stream), ctypes.byref(n)))
    return int(n.value)


def pkv_decode_attention(handle, layer, seq_ids, q, out, out_f32=None, stream=None):
    ids, n = _ints(seq_ids)
    _check(handle, lib().pkv_decode_attention(handle, layer, n, ids, _ptr(q), _ptr(out), _ptr(out_f32), _stream(stream)))


def pkv_decode_attention_multi(handle, layer, seq_ids, q_len, q, out, out_f32=None, stream=None):
    """q, out: [n_seqs, q_len, H_q, d]; query j of a sequence belongs to its position T - q_len + j (causal)."""
    ids, n = _ints(seq_ids)
    _check(handle, lib().pkv_decode_attention_multi(handle, layer, n, ids, q_len, _ptr(q), _ptr(out), _ptr(out_f32),
                                                    _stream(stream)))


def pkv_decode_attention_partial(handle, layer, seq_ids, q, state, stream=None):
    """state: fp32 [n_seqs, H_q, d + 2] = (o unnormalised, m in base-2 units, l) over this cache's tokens."""
    ids, n = _ints(seq_ids)
    _check(handle, lib().pkv_decode_attention_partial(handle, layer, n, ids, _ptr(q), _ptr(state), _stream(stream)))


def pkv_merge_attention_states(states, n_shards, n_rows, out=None, out_f32=None, stream=None):
    """Eq. 5 over n_shards state arrays stored back to back ([n_shards, n_rows, d + 2] fp32)."""
    st = lib().pkv_merge_attention_states(_ptr(states), n_shards, n_rows, _ptr(out), _ptr(out_f32), _stream(stream))
    if st != PKV_OK:
        raise PkvError(st, "pkv_merge_attention_states")


def pkv_decode_attention_static_scratch(handle, layer, seq_ids, q, out, out_f32=None, stream=None):
    """Same result as pkv_decode_attention; the split-K scratch is a fixed array inside the library, for
    callers that cannot supply a workspace.  Shared by all calls on the device: do not overlap calls."""
    ids, n = _ints(seq_ids)
    _check(handle, lib().pkv_decode_attention_static_scratch(handle, layer, n, ids, _ptr(q), _ptr(out), _ptr(out_f32),
                                                             _stream(stream)))


def pkv_decode_attention_host(handle, layer, seq_ids, q_host, out_host, q_stage, out_stage, stream=None):
    ids, n = _ints(seq_ids)
    _check(handle, lib().pkv_decode_attention_host(handle, layer, n, ids, _ptr(q_host), _ptr(out_host),
                                                   _ptr(q_stage), _ptr(out_stage), _stream(stream)))


def pkv_get_page_table(handle, seq, layer, max_pages):
    kinds = (ctypes.c_int32 * max_pages)()
    slots = (ctypes.c_int32 * max_pages)()
    n_pages, n_tokens = ctypes.c_int32(0), ctypes.c_int32(0)
    st = lib().pkv_get_page_table(handle, seq, layer, kinds, slots, ctypes.byref(n_pages), ctypes.byref(n_tokens))
    if st != PKV_OK:
        raise PkvError(st, "pkv_get_page_table")
    n = n_pages.value
    return list(kinds[:n]), list(slots[:n]), int(n_tokens.value)


def pkv_get_stats(handle, stream=None) -> dict:
    s = PkvStats()
    _check(handle, lib().pkv_get_stats(handle, ctypes.byref(s), _stream(stream)))
    return {n: int(getattr(s, n)) for n, _ in PkvStats._fields_}


def pkv_get_decode_plan(handle, layer, n_ctas, n_seqs, n_kv_heads):
    """-> (cta_starts [(position, head, unit)] incl. end sentinel, seg_parts [(cta_first, n_parts)])."""
    starts = (ctypes.c_int32 * (3 * (n_ctas + 1)))()
    segs = (ctypes.c_int32 * (2 * n_seqs * n_kv_heads))()
    n_used, n_segs = ctypes.c_int32(0), ctypes.c_int32(0)
    st = lib().pkv_get_decode_plan(handle, layer, ctypes.byref(n_used), starts, ctypes.byref(n_segs), segs)
    if st != PKV_OK:
        raise PkvError(st, "pkv_get_decode_plan")
    return ([tuple(starts[3 * j:3 * j + 3]) for j in range(n_used.value + 1)],
            [tuple(segs[2 * s:2 * s + 2]) for s in range(n_segs.value)])


def pkv_get_decode_trace(handle, n_ctas, stream=None):
    """Per-CTA time stamps of the last decode launch (needs PKV_DECODE_TRACE=1 at init): list of 16-tuples."""
    buf = (ctypes.c_int64 * (16 * n_ctas))()
    _check(handle, lib().pkv_get_decode_trace(handle, buf, n_ctas, _stream(stream)))
    return [tuple(buf[16 * i:16 * i + 16]) for i in range(n_ctas)]


def pkv_free_seq(handle, seq):
    _check(handle, lib().pkv_free_seq(handle, seq))


def pkv_destroy_cache(handle):
    lib().pkv_destroy_cache(handle)


def pkv_read_factors(handle, slot, kv_head, A_k, B_k, A_v, B_v, stream=None):
    _check(handle, lib().pkv_read_factors(handle, slot, kv_head, _ptr(A_k), _ptr(B_k), _ptr(A_v), _ptr(B_v), _stream(stream)))


def pkv_write_factors(handle, slot, kv_head, A_k, B_k, A_v, B_v, stream=None):
    _check(handle, lib().pkv_write_factors(handle, slot, kv_head, _ptr(A_k), _ptr(B_k), _ptr(A_v), _ptr(B_v), _stream(stream)))


def pkv_get_rotation_schedule(page_size):
    """-> list of rounds, each a list of groups (tuples of member indices)."""
    buf = (ctypes.c_uint8 * 4096)()
    nr, ng, gs = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    rc = lib().pkv_get_rotation_schedule(int(page_size), buf, 4096, ctypes.byref(nr), ctypes.byref(ng), ctypes.byref(gs))
    if rc != PKV_OK:
        raise PkvError(rc, "pkv_get_rotation_schedule(%r)" % (page_size,))
    flat = list(buf[:nr.value * ng.value * gs.value])
    it = iter(flat)
    return [[tuple(next(it) for _ in range(gs.value)) for _ in range(ng.value)] for _ in range(nr.value)]


def pkv_get_row_block_ranges(n_row_blocks, longest_tokens, page_size, n_sms):
    """-> token ranges per row block of a tcgen05 row-block launch (1 = the blocks are not cut)."""
    n = ctypes.c_int32()
    rc = lib().pkv_get_row_block_ranges(int(n_row_blocks), int(longest_tokens), int(page_size), int(n_sms), ctypes.byref(n))
    if rc != PKV_OK:
        raise PkvError(rc, "pkv_get_row_block_ranges(%r, %r, %r, %r)" % (n_row_blocks, longest_tokens, page_size, n_sms))
    return n.value


def pkv_read_dense(handle, slot, kv_head, K, V, stream=None):
    _check(handle, lib().pkv_read_dense(handle, slot, kv_head, _ptr(K), _ptr(V), _stream(stream)))


def pkv_read_basis(handle, seq, layer, kv_head, B_k, B_v, stream=None):
    _check(handle, lib().pkv_read_basis(handle, seq, layer, kv_head, _ptr(B_k), _ptr(B_v), _stream(stream)))


# ---- convenience wrapper ----------------------------------------------------------
def make_config(n_layers, n_kv_heads, n_q_heads, rank, sink_tokens, recent_tokens, max_seqs, max_pages_per_seq,
                n_dense_slots, n_factor_slots, head_dim=128, page_size=64, rank_v=None, softmax_scale=0.0,
                jacobi_max_sweeps=0, jacobi_tol=0.0, n_ctas=0, decode_variant=0, decode_overlap=0,
                jacobi_energy_tol=0.0, factor_bits=0, global_rank=0) -> PkvConfig:
    return PkvConfig(n_layers, n_kv_heads, n_q_heads, head_dim, page_size, rank, rank if rank_v is None else rank_v,
                     sink_tokens, recent_tokens, max_seqs, max_pages_per_seq, n_dense_slots, n_factor_slots,
                     softmax_scale, jacobi_max_sweeps, jacobi_tol, n_ctas, decode_variant, jacobi_energy_tol, factor_bits, decode_overlap,
                     global_rank)


class Cache:
    """Owns the device buffers (torch uint8 tensors) and the library handle."""

    def __init__(self, cfg: PkvConfig, device="cuda", dense_slot_order=None, factor_slot_order=None, dry_run=False):
        self.cfg = cfg
        self.sizes = pkv_query_sizes(cfg)
        self.dry_run = dry_run
        if dry_run:
            self.dense_pool = self.factor_pool = self.meta = self.workspace = None
            self.stream = None
        else:
            self.device = torch.device(device)
            self._device_index = self.dense_pool_device_index(self.device)
            mk = lambda n: torch.empty(max(int(n), 256), dtype=torch.uint8, device=self.device)
            self.dense_pool, self.factor_pool = mk(self.sizes.dense_pool_bytes), mk(self.sizes.factor_pool_bytes)
            self.meta, self.workspace = mk(self.sizes.meta_bytes), mk(self.sizes.workspace_bytes)
        self.handle = pkv_init_cache(cfg, self.dense_pool, self.factor_pool, self.meta, self.workspace,
                                     dense_slot_order, factor_slot_order)

    @staticmethod
    def dense_pool_device_index(device):
        return device.index if device.index is not None else torch.cuda.current_device()

    def _st(self):
        if self.dry_run:
            return None
        if _raw_current_stream is not None:
            return _raw_current_stream(self._device_index)
        return torch.cuda.current_stream(self.device)

    def append_kv(self, layer, seq_ids, n_new, k=None, v=None):
        pkv_append_kv(self.handle, layer, seq_ids, n_new, k, v, self._st())

    def compress_eligible_pages(self, layer=-1):
        return pkv_compress_eligible_pages(self.handle, layer, self._st())

    def compress_begin(self, layer, side_stream=None):
        return pkv_compress_begin(self.handle, layer, self._st(), side_stream)

    def compress_commit(self, layer=-1):
        return pkv_compress_commit(self.handle, layer, self._st())

    def decode_attention(self, layer, seq_ids, q=None, out=None, out_f32=None):
        if out is None and q is not None:
            out = torch.empty_like(q)
        pkv_decode_attention(self.handle, layer, seq_ids, q, out, out_f32, self._st())
        return out

    def decode_attention_multi(self, layer, seq_ids, q_len, q=None, out=None, out_f32=None):
        if out is None and q is not None:
            out = torch.empty_like(q)
        pkv_decode_attention_multi(self.handle, layer, seq_ids, q_len, q, out, out_f32, self._st())
        return out

    def decode_attention_partial(self, layer, seq_ids, q, state=None):
        if state is None:
            state = torch.empty((q.shape[0], q.shape[1], q.shape[2] + 2), dtype=torch.float32, device=q.device)
        pkv_decode_attention_partial(self.handle, layer, seq_ids, q, state, self._st())
        return state

    def decode_attention_host(self, layer, seq_ids, q_host, out_host, q_stage, out_stage):
        pkv_decode_attention_host(self.handle, layer, seq_ids, q_host, out_host, q_stage, out_stage, self._st())

    def page_table(self, seq, layer):
        return pkv_get_page_table(self.handle, seq, layer, self.cfg.max_pages_per_seq)

    def stats(self):
        return pkv_get_stats(self.handle, self._st())

    def free_seq(self, seq):
        pkv_free_seq(self.handle, seq)

    def read_basis(self, seq, layer, kv_head):
        """Global SVD form: (B_k, B_v), each [global_rank, d] bf16."""
        c = self.cfg
        B_k = torch.empty((c.global_rank, c.head_dim), dtype=torch.bfloat16, device=self.device)
        B_v = torch.empty_like(B_k)
        pkv_read_basis(self.handle, seq, layer, kv_head, B_k, B_v, self._st())
        return B_k, B_v

    def read_factors(self, slot, kv_head):
        c = self.cfg
        mk = lambda *s: torch.empty(s, dtype=torch.bfloat16, device=self.device)
        if c.global_rank > 0:                               # only the token rows are stored per page
            A_k, A_v = mk(c.page_size, c.global_rank), mk(c.page_size, c.global_rank)
            pkv_read_factors(self.handle, slot, kv_head, A_k, None, A_v, None, self._st())
            return A_k, None, A_v, None
        A_k, B_k = mk(c.page_size, c.rank_k), mk(c.rank_k, c.head_dim)
        A_v, B_v = mk(c.page_size, c.rank_v), mk(c.rank_v, c.head_dim)
        pkv_read_factors(self.handle, slot, kv_head, A_k, B_k, A_v, B_v, self._st())
        return A_k, B_k, A_v, B_v

    def write_factors(self, slot, kv_head, A_k, B_k, A_v, B_v):
        ts = [t.to(device=self.device, dtype=torch.bfloat16).contiguous() for t in (A_k, B_k, A_v, B_v)]
        pkv_write_factors(self.handle, slot, kv_head, *ts, self._st())
        torch.cuda.current_stream(self.device).synchronize()     # keep `ts` alive until the copy kernel ran

    def read_dense(self, slot, kv_head):
        c = self.cfg
        K = torch.empty((c.page_size, c.head_dim), dtype=torch.bfloat16, device=self.device)
        V = torch.empty_like(K)
        pkv_read_dense(self.handle, slot, kv_head, K, V, self._st())
        return K, V

    def close(self):
        if self.handle is not None:
            if not self.dry_run:
                torch.cuda.synchronize(self.device)
            pkv_destroy_cache(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
