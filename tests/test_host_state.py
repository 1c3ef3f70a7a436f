"""Host logic of the CUDA library, exercised in dry-run mode (no GPU needed):
exported symbols, page tables / eligibility / slot allocation bit-exact against
the oracle's state machine, error codes, byte accounting and the decode plan."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import accounting
from oracle.cache import OracleCache, OracleConfig, PoolExhausted
from paper_2608_23843_b200 import pkv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2608_23843_b200 import build
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "pkv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(pkv_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations parsed"
    L = ctypes.CDLL(pkv.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(L, name), "libpkv.so does not export %s" % name
    assert declared == set(pkv.EXPORTS)


def _pair(seed=None, **kw):
    base = dict(n_layers=2, n_kv_heads=2, n_q_heads=8, rank=16, sink_tokens=64, recent_tokens=128,
                max_seqs=4, max_pages_per_seq=64, n_dense_slots=96, n_factor_slots=96)
    base.update(kw)
    cfg = pkv.make_config(**base)
    d_ord = f_ord = None
    if seed is not None:
        rng = np.random.default_rng(seed)
        d_ord, f_ord = rng.permutation(base["n_dense_slots"]), rng.permutation(base["n_factor_slots"])
    gpu = pkv.Cache(cfg, dry_run=True, dense_slot_order=d_ord, factor_slot_order=f_ord)
    ocfg = OracleConfig(n_layers=base["n_layers"], n_kv_heads=base["n_kv_heads"], n_q_heads=base["n_q_heads"],
                        head_dim=128, page_size=base.get("page_size", 64), rank_k=base["rank"],
                        rank_v=base.get("rank_v", base["rank"]),
                        sink_tokens=base["sink_tokens"], recent_tokens=base["recent_tokens"],
                        max_seqs=base["max_seqs"], n_dense_slots=base["n_dense_slots"],
                        n_factor_slots=base["n_factor_slots"])
    return gpu, OracleCache(ocfg, d_ord, f_ord), base


def _oracle_append(orc, layer, seqs, n_new, H):
    n = int(sum(n_new))
    z = np.zeros((n, H, 128))
    orc.append_kv(layer, seqs, n_new, z, z)


def _same_tables(gpu, orc, base):
    for s in range(base["max_seqs"]):
        for ly in range(base["n_layers"]):
            assert gpu.page_table(s, ly) == orc.page_table(s, ly), (s, ly)
    st, ost = gpu.stats(), orc.stats()
    assert st["dense_slots_in_use"] == ost["dense_in_use"]
    assert st["factor_slots_in_use"] == ost["factor_in_use"]
    assert st["pages_compressed"] == ost["pages_compressed"]


def test_tiny_config_has_13_factor_pages():
    gpu, orc, base = _pair(n_layers=1, n_kv_heads=1, n_q_heads=4, max_seqs=1)
    gpu.append_kv(0, [0], [1024])
    assert gpu.compress_eligible_pages() == 13
    kinds, slots, T = gpu.page_table(0, 0)
    assert T == 1024 and kinds == [0] + [1] * 13 + [0, 0]


@pytest.mark.parametrize("seed,shape", [(0, {}), (1, {}), (2, {}), (3, {}),
                                        (4, dict(page_size=32, rank=16, rank_v=14, sink_tokens=32, recent_tokens=32,
                                                 n_dense_slots=192, n_factor_slots=192, max_pages_per_seq=128)),
                                        (5, dict(page_size=16, rank=9, sink_tokens=16, recent_tokens=48,
                                                 n_dense_slots=384, n_factor_slots=384, max_pages_per_seq=256))])
def test_random_schedule_matches_oracle_bit_exact(seed, shape):
    gpu, orc, base = _pair(seed=seed, **shape)
    rng = np.random.default_rng(100 + seed)
    H = base["n_kv_heads"]
    for step in range(60):
        op = rng.integers(0, 10)
        if op < 6:
            layer = int(rng.integers(0, base["n_layers"]))
            k = int(rng.integers(1, base["max_seqs"] + 1))
            seqs = [int(x) for x in rng.choice(base["max_seqs"], size=k, replace=False)]
            n_new = [int(rng.choice([0, 1, 1, 1, 7, 64, 65, 200])) for _ in seqs]
            try:
                _oracle_append(orc, layer, seqs, n_new, H)
                ok = True
            except PoolExhausted:
                pytest.skip("schedule overflowed the pool")   # not expected with these sizes
            if ok:
                gpu.append_kv(layer, seqs, n_new)
        elif op < 9:
            layer = int(rng.integers(-1, base["n_layers"]))
            # the oracle factorizes zero pages here: cheap, and keeps slot numbering identical
            assert gpu.compress_eligible_pages(layer) == orc.compress_eligible_pages(layer)
        else:
            s = int(rng.integers(0, base["max_seqs"]))
            orc.free_seq(s)
            gpu.free_seq(s)
        _same_tables(gpu, orc, base)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_two_step_compression_schedule_matches_oracle_bit_exact(seed):
    """pkv_compress_begin / pkv_compress_commit interleaved with appends, one-step compressions of other layers and
    frees: page tables (kinds, slots, token counts) stay bit-equal to the oracle's two-step form after every call;
    calls that would touch a layer with a begun compression are refused and change nothing."""
    gpu, orc, base = _pair(seed=seed, n_layers=3, max_seqs=3, n_dense_slots=160, n_factor_slots=120)
    rng = np.random.default_rng(500 + seed)
    H, L = base["n_kv_heads"], base["n_layers"]
    pending = {}                                           # layer -> set of sequences with pages in flight
    for step in range(90):
        op = rng.integers(0, 12)
        layer = int(rng.integers(0, L))
        if op < 5:
            seqs = [int(x) for x in rng.choice(base["max_seqs"], size=int(rng.integers(1, 4)), replace=False)]
            n_new = [int(rng.choice([1, 1, 7, 64, 65, 200])) for _ in seqs]
            _oracle_append(orc, layer, seqs, n_new, H)
            gpu.append_kv(layer, seqs, n_new)
        elif op < 8:
            if layer in pending:
                with pytest.raises(pkv.PkvError) as e:
                    gpu.compress_begin(layer)
                assert e.value.status == pkv.PKV_ERR_UNSUPPORTED
            else:
                before = [orc.page_table(s, layer) for s in range(base["max_seqs"])]
                n = orc.compress_begin(layer)
                assert gpu.compress_begin(layer) == n
                assert before == [orc.page_table(s, layer) for s in range(base["max_seqs"])]     # nothing visible yet
                if n:
                    pending[layer] = {seq for seq, *_ in orc.pending[layer]}
        elif op < 10:
            which = int(rng.integers(-1, L))
            assert gpu.compress_commit(which) == orc.compress_commit(which)
            for ly in ([which] if which >= 0 else list(pending)):
                pending.pop(ly, None)
        elif op < 11:
            which = int(rng.integers(-1, L))
            if (which < 0 and pending) or which in pending:
                with pytest.raises(pkv.PkvError) as e:
                    gpu.compress_eligible_pages(which)
                assert e.value.status == pkv.PKV_ERR_UNSUPPORTED
            else:
                assert gpu.compress_eligible_pages(which) == orc.compress_eligible_pages(which)
        else:
            s_ = int(rng.integers(0, base["max_seqs"]))
            if any(s_ in seqs for seqs in pending.values()):
                with pytest.raises(pkv.PkvError) as e:
                    gpu.free_seq(s_)
                assert e.value.status == pkv.PKV_ERR_UNSUPPORTED
            else:
                orc.free_seq(s_)
                gpu.free_seq(s_)
        _same_tables(gpu, orc, base)
    assert gpu.compress_commit() == orc.compress_commit()
    _same_tables(gpu, orc, base)
    assert gpu.stats()["pages_compressed"] == orc.pages_compressed > 0


def test_two_step_compression_when_the_factor_pool_runs_out():
    """pkv_compress_begin with fewer free factor slots than eligible pages: the pages that got a slot are begun (and
    reported), the call returns PKV_ERR_POOL_EXHAUSTED, the commit converts exactly those, and a later begin picks up
    the rest once slots are free again.  Same tables as the oracle throughout."""
    gpu, orc, base = _pair(n_layers=1, max_seqs=2, n_dense_slots=64, n_factor_slots=5, sink_tokens=64, recent_tokens=64)
    H = base["n_kv_heads"]
    _oracle_append(orc, 0, [0, 1], [64 * 6, 64 * 7], H)
    gpu.append_kv(0, [0, 1], [64 * 6, 64 * 7])             # eligible: pages 1..4 of sequence 0, 1..5 of sequence 1
    with pytest.raises(pkv.PkvError) as e:
        gpu.compress_begin(0)
    assert e.value.status == pkv.PKV_ERR_POOL_EXHAUSTED and e.value.begun == 5
    assert orc.compress_begin(0) == 5
    _same_tables(gpu, orc, base)                            # nothing visible yet
    with pytest.raises(pkv.PkvError) as e:
        gpu.compress_begin(0)                               # still uncommitted
    assert e.value.status == pkv.PKV_ERR_UNSUPPORTED
    assert gpu.compress_commit(0) == orc.compress_commit(0) == 5
    _same_tables(gpu, orc, base)
    assert gpu.page_table(0, 0)[0][:6] == [0, 1, 1, 1, 1, 0] and gpu.page_table(1, 0)[0][:3] == [0, 1, 0]
    with pytest.raises(pkv.PkvError) as e:
        gpu.compress_begin(0)                               # no factor slot left at all
    assert e.value.status == pkv.PKV_ERR_POOL_EXHAUSTED and e.value.begun == 0
    assert gpu.compress_commit(0) == 0
    orc.free_seq(0)
    gpu.free_seq(0)                                         # four factor slots come back
    assert gpu.compress_begin(0) == orc.compress_begin(0) == 4
    assert gpu.compress_commit() == orc.compress_commit() == 4
    _same_tables(gpu, orc, base)
    assert gpu.page_table(1, 0)[0][:7] == [0, 1, 1, 1, 1, 1, 0]


def test_incremental_conversion_is_one_page_per_boundary_step():
    gpu, orc, base = _pair(n_layers=1, max_seqs=2, sink_tokens=64, recent_tokens=256)
    gpu.append_kv(0, [0, 1], [8192 // 16, 8192 // 16])
    gpu.compress_eligible_pages()
    T0 = 8192 // 16
    for t in range(T0, T0 + 130):
        gpu.append_kv(0, [0, 1], [1, 1])
        n = gpu.compress_eligible_pages(0)
        assert n == (2 if (t + 1) % 64 == 0 else 0)
    kinds, _, T = gpu.page_table(1, 0)
    lo, hi = 1, T // 64 - 4
    assert [i for i, k in enumerate(kinds) if k == 1] == list(range(lo, hi))


def test_error_codes_and_unchanged_state_on_failure():
    gpu, orc, base = _pair(n_dense_slots=3, n_factor_slots=1, n_layers=1)
    with pytest.raises(pkv.PkvError) as e:
        gpu.append_kv(0, [0], [64 * 4])
    assert e.value.status == pkv.PKV_ERR_POOL_EXHAUSTED and gpu.page_table(0, 0) == ([], [], 0)
    with pytest.raises(pkv.PkvError) as e:
        gpu.append_kv(0, [0, 0], [1, 1])
    assert e.value.status == pkv.PKV_ERR_BAD_SEQ
    with pytest.raises(pkv.PkvError) as e:
        gpu.append_kv(0, [9], [1])
    assert e.value.status == pkv.PKV_ERR_BAD_SEQ
    with pytest.raises(pkv.PkvError) as e:
        gpu.append_kv(5, [0], [1])
    assert e.value.status == pkv.PKV_ERR_INVALID_ARG
    with pytest.raises(pkv.PkvError) as e:
        gpu.decode_attention(0, [0])                                  # empty sequence
    assert e.value.status == pkv.PKV_ERR_INVALID_ARG
    gpu.append_kv(0, [0], [64 * 3])
    gpu.free_seq(0)
    gpu2, _, _ = _pair(n_dense_slots=8, n_factor_slots=1, n_layers=1, sink_tokens=0, recent_tokens=0)
    gpu2.append_kv(0, [0], [64 * 3])
    with pytest.raises(pkv.PkvError) as e:
        gpu2.compress_eligible_pages()
    assert e.value.status == pkv.PKV_ERR_POOL_EXHAUSTED
    assert gpu2.page_table(0, 0)[0] == [1, 0, 0]                      # the page converted before exhaustion stays converted


def test_misaligned_caller_pointers_are_refused_before_any_launch():
    """The kernels read k/v 16 bytes at a time and q as 32-bit words, and write out 8 and out_f32 16 bytes at a
    time: a pointer that breaks this is an argument error, not a device fault.  Checked on the host, so a dry-run
    cache (which never dereferences anything) can show it with made-up addresses."""
    gpu, _, _ = _pair(n_dense_slots=8, n_factor_slots=4, n_layers=1)
    L, h = pkv.lib(), gpu.handle
    ids, cnt = (ctypes.c_int32 * 1)(0), (ctypes.c_int32 * 1)(3)
    assert L.pkv_append_kv(h, 0, 1, ids, cnt, 0x10008, 0x20000, None) == pkv.PKV_ERR_INVALID_ARG
    assert L.pkv_append_kv(h, 0, 1, ids, cnt, 0x10000, 0x20004, None) == pkv.PKV_ERR_INVALID_ARG
    assert gpu.page_table(0, 0) == ([], [], 0)                         # nothing was appended
    assert L.pkv_append_kv(h, 0, 1, ids, cnt, 0x10000, 0x20000, None) == pkv.PKV_OK
    good = dict(q=0x1000, out=0x2000, f32=0x3000)
    for bad in (dict(q=0x1002), dict(out=0x2004), dict(f32=0x3008)):
        a = dict(good, **bad)
        st = L.pkv_decode_attention(h, 0, 1, ids, a["q"], a["out"], a["f32"], None)
        assert st == pkv.PKV_ERR_INVALID_ARG, (bad, st)
        assert L.pkv_decode_attention_multi(h, 0, 1, ids, 2, a["q"], a["out"], a["f32"], None) == pkv.PKV_ERR_INVALID_ARG
    assert L.pkv_decode_attention_partial(h, 0, 1, ids, 0x1000, 0x5004, None) == pkv.PKV_ERR_INVALID_ARG
    assert L.pkv_decode_attention(h, 0, 1, ids, good["q"], good["out"], good["f32"], None) == pkv.PKV_OK


def test_config_validation():
    ok = dict(n_layers=1, n_kv_heads=1, n_q_heads=4, rank=16, sink_tokens=64, recent_tokens=64, max_seqs=1,
              max_pages_per_seq=4, n_dense_slots=4, n_factor_slots=4)
    pkv.pkv_query_sizes(pkv.make_config(**ok))
    for bad, status in [(dict(sink_tokens=10), pkv.PKV_ERR_INVALID_ARG), (dict(recent_tokens=65), pkv.PKV_ERR_INVALID_ARG),
                        (dict(n_q_heads=3, n_kv_heads=2), pkv.PKV_ERR_INVALID_ARG), (dict(rank=0), pkv.PKV_ERR_INVALID_ARG),
                        (dict(rank=65), pkv.PKV_ERR_INVALID_ARG), (dict(rank=33), pkv.PKV_ERR_UNSUPPORTED),
                        (dict(head_dim=64, page_size=64), pkv.PKV_ERR_UNSUPPORTED), (dict(page_size=48, sink_tokens=48, recent_tokens=48), pkv.PKV_ERR_UNSUPPORTED),
                        (dict(page_size=16, rank=17, sink_tokens=16, recent_tokens=16), pkv.PKV_ERR_INVALID_ARG),
                        (dict(n_q_heads=16), pkv.PKV_ERR_UNSUPPORTED), (dict(rank=16, rank_v=8), pkv.PKV_ERR_UNSUPPORTED),
                        (dict(decode_variant=4), pkv.PKV_ERR_INVALID_ARG), (dict(decode_variant=-1), pkv.PKV_ERR_INVALID_ARG)]:
        with pytest.raises(pkv.PkvError) as e:
            pkv.pkv_query_sizes(pkv.make_config(**{**ok, **bad}))
        assert e.value.status == status, bad
    for good in (dict(rank=12), dict(rank=16, rank_v=14, page_size=32, sink_tokens=32, recent_tokens=32),
                 dict(rank=9, page_size=16, sink_tokens=16, recent_tokens=16), dict(rank=27), dict(decode_variant=2),
                 dict(decode_variant=3)):
        pkv.pkv_query_sizes(pkv.make_config(**{**ok, **good}))
    with pytest.raises(pkv.PkvError):
        pkv.Cache(pkv.make_config(**ok), dry_run=True, dense_slot_order=[0, 0, 1, 2])   # not a permutation


def test_slot_sizes_follow_storage_ratio_formula():
    for P, rk, rv in [(64, 8, 8), (64, 16, 16), (64, 24, 24), (64, 32, 32), (64, 27, 27), (32, 16, 14), (32, 16, 16),
                      (16, 9, 9)]:
        sz = pkv.pkv_query_sizes(pkv.make_config(n_layers=1, n_kv_heads=8, n_q_heads=32, rank=rk, rank_v=rv, page_size=P,
                                                 sink_tokens=P, recent_tokens=P, max_seqs=1, max_pages_per_seq=8,
                                                 n_dense_slots=8, n_factor_slots=8))
        assert sz.dense_slot_bytes == 8 * 2 * P * 128 * 2
        assert sz.factor_slot_bytes / sz.dense_slot_bytes == accounting.page_storage_ratio(rk, rv, P, 128)


def _decode_bytes(T, P, S, W, r, H_kv, H_q):
    n_pages = -(-T // P)
    lo, hi = S // P, max(S // P, T // P - W // P)
    nf = max(0, min(hi, n_pages) - min(lo, n_pages))
    dense_rows = T - nf * P
    return H_kv * (nf * 2 * (P * r + r * 128) * 2 + dense_rows * 2 * 128 * 2) + 2 * H_q * 128 * 2


def test_decode_byte_accounting_long_context_layer():
    # 64q/8kv, T=131072, r=24, 64 sink + 512 recent: 2039 factor pages + 9 dense pages per KV head
    gpu, _, _ = _pair(n_layers=1, n_kv_heads=8, n_q_heads=64, rank=24, sink_tokens=64, recent_tokens=512,
                      max_seqs=1, max_pages_per_seq=2048, n_dense_slots=2048, n_factor_slots=2048)
    gpu.append_kv(0, [0], [131072])
    assert gpu.compress_eligible_pages() == 2039
    gpu.decode_attention(0, [0])
    st = gpu.stats()
    assert st["last_decode_bytes"] == _decode_bytes(131072, 64, 64, 512, 24, 8, 64) == 303054848
    assert st["last_decode_units"] == 8 * (2039 + 9 * 2)


@pytest.mark.parametrize("lengths,rank", [([1024], 16), ([32768] * 8, 24), ([2048, 65536, 3001, 40000, 2049, 9999], 8),
                                          ([70, 64, 1, 129], 32)])
def test_decode_plan_covers_every_unit_once_and_is_balanced(lengths, rank):
    H, n = 8, len(lengths)
    gpu, _, _ = _pair(n_layers=1, n_kv_heads=H, n_q_heads=32, rank=rank, sink_tokens=64, recent_tokens=256,
                      max_seqs=n, max_pages_per_seq=1024, n_dense_slots=4096, n_factor_slots=4096)
    gpu.append_kv(0, list(range(n)), lengths)
    gpu.compress_eligible_pages()
    order = list(range(n))[::-1]                                      # batch order != sequence id order
    gpu.decode_attention(0, order)
    st = gpu.stats()
    assert st["last_decode_bytes"] == sum(_decode_bytes(lengths[s], 64, 64, 256, rank, H, 0) for s in order) + 2 * n * 32 * 256
    N = 296                                                            # dry-run default grid: 2 CTAs x 148 SMs
    starts, segs = pkv.pkv_get_decode_plan(gpu.handle, 0, N, n, H)
    nb = 2 if rank >= 24 else 4                                        # dense blocks per page
    blob, blk = 2 * (64 * rank + rank * 128) * 2, (64 // nb) * 512

    def units(s):
        kinds = gpu.page_table(s, 0)[0]
        return [("f", blob) if k == 1 else ("d", blk) for k in kinds for _ in range(1 if k == 1 else nb)]

    per_head = [units(s) for s in order]
    flat = [(i, h, u) for i in range(n) for h in range(H) for u in range(len(per_head[i]))]
    assert len(flat) == st["last_decode_units"]
    assert starts[0] == (0, 0, 0) and starts[-1] == (n, 0, 0)
    idx = {pos: j for j, pos in enumerate(flat)}
    idx[(n, 0, 0)] = len(flat)
    cuts = [idx[s] for s in starts]
    assert all(b > a for a, b in zip(cuts, cuts[1:])), "ranges must be non-empty and ordered"
    assert len(cuts) - 1 <= N
    # balance (the split weighs a unit by its bytes plus a fixed 2 KiB of per-unit overhead):
    # no CTA exceeds the mean by more than two units
    cost = [per_head[i][u][1] + 2048 for (i, h, u) in flat]
    loads = [sum(cost[a:b]) for a, b in zip(cuts, cuts[1:])]
    n_cut = max(1, min(N, len(flat) // 5))                              # at least one unit per consumer warp
    assert len(cuts) - 1 <= n_cut
    assert max(loads) <= sum(cost) / n_cut + 2 * (max(blob, blk) + 2048)
    # segment bookkeeping: CTAs that touch segment s are exactly [first, first + n_parts)
    for s in range(n * H):
        touching = [j for j, (a, b) in enumerate(zip(cuts, cuts[1:]))
                    if any(flat[x][0] * H + flat[x][1] == s for x in (a, b - 1)) or
                    (flat[a][0] * H + flat[a][1] < s < flat[b - 1][0] * H + flat[b - 1][1])]
        assert segs[s] == (touching[0], len(touching)), s


def test_multi_query_call_plan_and_argument_checks():
    """Several queries per sequence: the plan covers the sequences once and is cut into at most n_ctas / b ranges,
    b = ceil(q_len / (8 / G)) query blocks per sequence (the launch's CTAs work in groups of b on one range); the
    call is refused when a query would not see a whole factor page, when it has no token to see, when
    n_seqs * b exceeds max_seqs (partial states and tickets are counted per block), or with the scalar variant."""
    H, G = 2, 4
    lengths = [1000, 70, 5]
    kw = dict(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=16, sink_tokens=64, recent_tokens=64, max_seqs=9,
              max_pages_per_seq=32, n_dense_slots=64, n_factor_slots=64)
    gpu, _, _ = _pair(**kw)
    gpu.append_kv(0, [0, 1, 2], lengths)
    gpu.compress_eligible_pages()
    gpu.decode_attention(0, [0, 1, 2])
    base = gpu.stats()
    q_len = 5                                                  # 2 query tokens per tile -> 3 entries per sequence
    gpu.decode_attention_multi(0, [2, 0, 1], q_len)
    st = gpu.stats()
    assert st["last_decode_units"] == base["last_decode_units"]
    assert st["last_decode_bytes"] == base["last_decode_bytes"] + 2 * 3 * (q_len - 1) * H * G * 256
    starts, segs = pkv.pkv_get_decode_plan(gpu.handle, 0, 296, 3, H)
    assert starts[0] == (0, 0, 0) and starts[-1] == (3, 0, 0) and len(segs) == 3 * H
    assert len(starts) - 1 <= 296 // 3 and all(n_parts >= 1 for _, n_parts in segs)
    gpu.decode_attention(0, [2, 0, 1])                         # the same batch with one query: its own plan again
    assert gpu.stats()["last_decode_units"] == base["last_decode_units"]
    # q_len = 6 on the 5-token sequence: the first query would see nothing
    with pytest.raises(pkv.PkvError) as e:
        gpu.decode_attention_multi(0, [2], 6)
    assert e.value.status == pkv.PKV_ERR_INVALID_ARG
    gpu.decode_attention_multi(0, [2], 5)
    # sequence 0 has factor pages up to token 896 = 1000 - 104: 105 queries is the most that see them whole
    kinds = gpu.page_table(0, 0)[0]
    assert kinds.index(0, 1) * 64 == 896
    gpu.decode_attention_multi(0, [0], 8)
    with pytest.raises(pkv.PkvError) as e:
        gpu.decode_attention_multi(0, [0], 106)
    assert e.value.status == pkv.PKV_ERR_INVALID_ARG
    # 4 sequences' worth of entries do not fit max_seqs = 9 at three entries each
    gpu2, _, _ = _pair(**dict(kw, max_seqs=4))
    gpu2.append_kv(0, [0, 1], [100, 100])
    with pytest.raises(pkv.PkvError) as e:
        gpu2.decode_attention_multi(0, [0, 1], 5)
    assert e.value.status == pkv.PKV_ERR_INVALID_ARG
    gpu2.decode_attention_multi(0, [0, 1], 4)
    gpu3, _, _ = _pair(**dict(kw, decode_variant=1))
    gpu3.append_kv(0, [0], [100])
    gpu3.decode_attention_multi(0, [0], 1)
    with pytest.raises(pkv.PkvError) as e:
        gpu3.decode_attention_multi(0, [0], 2)
    assert e.value.status == pkv.PKV_ERR_UNSUPPORTED


@pytest.mark.parametrize("P", [64, 32, 16])
def test_rotation_schedule_of_the_page_svd_kernel(P):
    """The order in which the compression kernel rotates index pairs within a sweep (host-side table, no GPU):
    every round partitions the indices; a sweep contains every pair of indices (exactly once for P = 64 and 16;
    for P = 32, where no such design exists, 64 of the 496 pairs come two or three times); for P = 64 the members
    at positions {0, 2} of a round's groups fall into 32 different shared-memory banks (index mod 32), and so do
    the members at positions {1, 3}, which is what keeps the kernel's accesses conflict-free."""
    rounds = pkv.pkv_get_rotation_schedule(P)
    expect = {64: (21, 16, 4), 32: (13, 8, 4), 16: (15, 8, 2)}[P]
    assert (len(rounds), len(rounds[0]), len(rounds[0][0])) == expect
    seen = np.zeros((P, P), dtype=int)
    for groups in rounds:
        assert sorted(m for g in groups for m in g) == list(range(P))          # a partition
        for g in groups:
            for i in range(len(g)):
                for j in range(i + 1, len(g)):
                    seen[g[i], g[j]] += 1
                    seen[g[j], g[i]] += 1
        if P == 64:
            for positions in ((0, 2), (1, 3)):
                banks = sorted(g[k] % 32 for g in groups for k in positions)
                assert banks == list(range(32))
    off = seen[~np.eye(P, dtype=bool)]
    assert off.min() >= 1
    if P == 32:
        assert off.max() <= 3 and int((off > 1).sum()) // 2 == 64
    else:
        assert off.max() == 1
    with pytest.raises(pkv.PkvError):
        pkv.pkv_get_rotation_schedule(48)


@pytest.mark.parametrize("overlap", [0, 1, 2])
def test_buffers_promised_by_query_sizes_always_suffice(overlap):
    """pkv_init_cache lays its metadata and workspace out for the grid it will really launch, which may differ
    from the one pkv_query_sizes assumed; it must never need more than was promised (it refuses to start
    otherwise), whatever the batch size, head count or grid."""
    for max_seqs in (1, 8, 64, 256, 512, 2048, 4096):
        for H in (1, 8):
            for n_ctas in (0, 1, 148, 296, 512, 1000):
                cfg = pkv.make_config(n_layers=2, n_kv_heads=H, n_q_heads=H * 4, rank=24, sink_tokens=64,
                                      recent_tokens=256, max_seqs=max_seqs, max_pages_per_seq=8, n_dense_slots=64,
                                      n_factor_slots=64, n_ctas=n_ctas, decode_overlap=overlap)
                sz = pkv.pkv_query_sizes(cfg)
                assert sz.workspace_bytes > 0 and sz.meta_bytes > 0
                if overlap == 2:
                    assert sz.workspace_bytes <= (192 << 20) + 64 * 4160 * (max(512, n_ctas) + max_seqs * H)
                handle = pkv.pkv_init_cache(cfg, None, None, None, None, None, None)      # dry run: host logic only
                pkv.pkv_destroy_cache(handle)


def test_token_ranges_of_a_row_block_launch():
    """pkv_get_row_block_ranges(): the rule by which the tcgen05 row-block kernel's launch cuts row blocks into token
    ranges, pinned by hand-worked cases (148 SMs = 296 CTAs in flight; a range has at least eight pages; at most 32
    ranges per block and 512 states per launch)."""
    f = pkv.pkv_get_row_block_ranges
    assert f(64, 32768, 64, 148) == 4            # 8 sequences x 8 KV heads, 32 queries of 4 heads each: 296 // 64
    assert f(128, 32768, 64, 148) == 2           # 64 queries: two blocks per (sequence, head)
    assert f(512, 32768, 64, 148) == 1           # a 2048-position chunk fills the GPU by itself
    assert f(149, 32768, 64, 148) == 1           # more than half the CTAs in flight: no ranges
    assert f(148, 32768, 64, 148) == 2
    assert f(8, 32768, 64, 148) == 32            # one sequence: 296 // 8 = 37, capped at 32
    assert f(8, 4096, 64, 148) == 8              # 64 pages: eight pages per range
    assert f(8, 1000, 64, 148) == 2              # 16 pages
    assert f(8, 1023, 64, 148) == 2
    assert f(8, 960, 64, 148) == 1               # 15 pages: not two ranges of eight
    assert f(8, 16384, 16, 148) == 32            # 1024 pages of 16 tokens
    assert f(1, 1 << 20, 64, 1000) == 32         # a bigger GPU: 512 states bound the launch, 32 ranges the block
    assert f(20, 1 << 20, 64, 1000) == 25        # 512 // 20
    assert f(1, 64, 64, 1) == 1
    for bad in [(0, 100, 64, 148), (1, 0, 64, 148), (1, 100, 0, 148), (1, 100, 64, 0)]:
        with pytest.raises(pkv.PkvError):
            f(*bad)
