"""GPU behaviour around the edges: storage round trips, error paths that must leave the cache usable,
slot reuse, degenerate inputs, several caches and streams."""
import numpy as np
import pytest
import torch

from gpu_helpers import Pair, f64, gen_kv, rel_err
from paper_2608_23843_b200 import pkv, synth

pytestmark = pytest.mark.gpu


def _cfg(**kw):
    base = dict(n_layers=2, n_kv_heads=2, n_q_heads=8, rank=16, sink_tokens=64, recent_tokens=128, max_seqs=4,
                max_pages_per_seq=32, n_dense_slots=96, n_factor_slots=64)
    base.update(kw)
    return pkv.make_config(**base)


def test_appended_rows_read_back_exactly_across_calls_and_sequences():
    """pkv_append_kv scatter (several sequences per call, zero-length entries, page boundaries inside a
    call) followed by pkv_read_dense returns the very rows that went in."""
    cfg = _cfg()
    cache = pkv.Cache(cfg, "cuda", synth.slot_permutation(1, 96, 0).tolist(), synth.slot_permutation(1, 64, 1).tolist())
    lengths = {0: [5, 60, 0, 130], 1: [0, 64, 1, 7], 3: [200, 0, 0, 3]}
    kv = {s: gen_kv(5, 1, s, sum(l), cfg) for s, l in lengths.items()}
    pos = {s: 0 for s in lengths}
    for call in range(4):
        seqs = [3, 0, 1]
        n_new = [lengths[s][call] for s in seqs]
        k = torch.cat([kv[s][0][pos[s]:pos[s] + n] for s, n in zip(seqs, n_new)])
        v = torch.cat([kv[s][1][pos[s]:pos[s] + n] for s, n in zip(seqs, n_new)])
        cache.append_kv(1, seqs, n_new, k.cuda(), v.cuda())
        for s, n in zip(seqs, n_new):
            pos[s] += n
    for s in lengths:
        kinds, slots, T = cache.page_table(s, 1)
        assert T == sum(lengths[s]) and cache.page_table(s, 0) == ([], [], 0)
        for p, slot in enumerate(slots):
            rows = min(64, T - p * 64)
            for h in range(2):
                K, V = cache.read_dense(slot, h)
                torch.cuda.synchronize()
                assert torch.equal(K[:rows].cpu(), kv[s][0][p * 64:p * 64 + rows, h])
                assert torch.equal(V[:rows].cpu(), kv[s][1][p * 64:p * 64 + rows, h])
    cache.close()


def test_errors_leave_the_cache_usable_and_freed_slots_are_reused():
    cfg = _cfg(n_layers=1, n_dense_slots=12, n_factor_slots=7, max_seqs=3)
    pair = Pair(cfg, seed=2, oracle=False)
    k, v = gen_kv(6, 0, 0, 700, cfg)
    q = synth.make_q(6, 0, 0, 1, 8, 128)
    pair.gpu.append_kv(0, [0], [700], k.cuda(), v.cuda())          # 11 pages
    assert pair.gpu.compress_eligible_pages(0) == 7                 # pages 1..7 -> uses every factor slot
    ref, _ = pair.decode(0, [0], q)
    with pytest.raises(pkv.PkvError) as e:                          # 8 dense slots are free, 9 needed
        pair.gpu.append_kv(0, [1], [9 * 64], k[:576].cuda(), v[:576].cuda())
    assert e.value.status == pkv.PKV_ERR_POOL_EXHAUSTED and pair.gpu.page_table(1, 0) == ([], [], 0)
    pair.gpu.append_kv(0, [1], [5 * 64], k[:320].cuda(), v[:320].cuda())
    with pytest.raises(pkv.PkvError) as e:
        pair.gpu.compress_eligible_pages(0)                         # seq 1 has 2 eligible pages, no factor slot left
    assert e.value.status == pkv.PKV_ERR_POOL_EXHAUSTED
    with pytest.raises(pkv.PkvError) as e:
        pair.gpu.decode_attention(0, [2], q.cuda())                 # empty sequence
    assert e.value.status == pkv.PKV_ERR_INVALID_ARG
    again, _ = pair.decode(0, [0], q)
    assert (again == ref).all()                                     # sequence 0 is untouched by all of that
    # free sequence 0, rebuild it in the released slots: same answer
    pair.gpu.free_seq(0)
    pair.gpu.free_seq(1)
    assert pair.gpu.stats()["dense_slots_in_use"] == 0 and pair.gpu.stats()["factor_slots_in_use"] == 0
    pair.gpu.append_kv(0, [2], [700], k.cuda(), v.cuda())
    assert pair.gpu.compress_eligible_pages(0) == 7
    rebuilt, _ = pair.decode(0, [2], q)
    assert (rebuilt == ref).all()
    assert pair.gpu.stats()["device_timeouts"] == 0 and pair.gpu.stats()["bad_slot_indices"] == 0


def test_nan_sequence_does_not_disturb_its_neighbours():
    cfg = _cfg(n_layers=1, sink_tokens=0, recent_tokens=64)
    pair = Pair(cfg, seed=3, oracle=False)
    k, v = gen_kv(7, 0, 0, 500, cfg)
    bad = torch.full((300, 2, 128), float("nan"), dtype=torch.bfloat16)
    pair.gpu.append_kv(0, [0], [500], k.cuda(), v.cuda())
    q = synth.make_q(7, 0, 0, 2, 8, 128)
    pair.gpu.compress_eligible_pages(0)
    alone, _ = pair.decode(0, [0], q[:1])
    pair.gpu.append_kv(0, [1], [300], bad.cuda(), bad.cuda())
    pair.gpu.compress_eligible_pages(0)                              # NaN pages: must return, result unspecified
    both, _ = pair.decode(0, [0, 1], q)
    assert (both[0] == alone[0]).all()
    assert pair.gpu.stats()["device_timeouts"] == 0


def test_two_caches_and_a_side_stream():
    """Two caches with different shapes used alternately, one of them on a non-default stream."""
    cfg_a = _cfg(n_layers=1, rank=24)
    cfg_b = _cfg(n_layers=1, rank=16, rank_v=14, page_size=32, sink_tokens=32, recent_tokens=32, n_kv_heads=1, n_q_heads=4)
    a, b = Pair(cfg_a, seed=4), Pair(cfg_b, seed=5)
    ka, va = gen_kv(8, 0, 0, 900, cfg_a)
    kb, vb = gen_kv(9, 0, 0, 777, cfg_b)
    side = torch.cuda.Stream()
    a.append(0, [0], [ka], [va])
    with torch.cuda.stream(side):
        b.append(0, [0], [kb], [vb])
        b.compress(0)
    a.compress(0)
    qa, qb = synth.make_q(8, 0, 0, 1, 8, 128), synth.make_q(9, 0, 0, 1, 4, 128)
    for _ in range(3):
        got_a, _ = a.decode(0, [0], qa)
        with torch.cuda.stream(side):
            got_b, _ = b.decode(0, [0], qb)
    for pair, got, qq in ((a, got_a, qa), (b, got_b, qb)):
        pair.load_gpu_factors_into_oracle(0, 0)
        ref = pair.orc.decode_attention(0, [0], f64(qq))
        assert rel_err(got, ref) <= 1e-2


@pytest.mark.gpu
@pytest.mark.parametrize("overlap", [0, 1])
def test_cuda_graph_replay_sees_appends_and_rebuilt_plans(overlap):
    """Decode launches recorded into a CUDA graph read token counts, page tables and the plan when they run:
    a replay after an in-page append equals a fresh eager call; after an append that opens a page plus a
    compression, one eager call rebuilds the plan and the old graph is valid again.  Calls that cannot be
    recorded (append, compress, a decode whose plan is stale) return PKV_ERR_UNSUPPORTED during capture
    and leave the capture usable."""
    L, H, G = 2, 2, 4
    cfg = pkv.make_config(n_layers=L, n_kv_heads=H, n_q_heads=H * G, rank=16, sink_tokens=64, recent_tokens=128,
                          max_seqs=2, max_pages_per_seq=40, n_dense_slots=160, n_factor_slots=160,
                          decode_overlap=overlap)
    cache = pkv.Cache(cfg, "cuda", None, None)
    lengths = [700, 1500]
    data = [[synth.make_kv(21, ly, s, 2200, H, 128, 64, "cuda") for s in range(2)] for ly in range(L)]
    T = list(lengths)
    for ly in range(L):
        for s in range(2):
            cache.append_kv(ly, [s], [T[s]], data[ly][s][0][:T[s]], data[ly][s][1][:T[s]])
    cache.compress_eligible_pages(-1)
    ids = [1, 0]
    qs = [synth.make_q(21, ly, 0, 2, H * G, 128, "cuda") for ly in range(L)]
    outs = [torch.empty_like(q) for q in qs]

    def eager():
        res = [torch.empty_like(q) for q in qs]
        for ly in range(L):
            cache.decode_attention(ly, ids, qs[ly], res[ly])
        torch.cuda.synchronize()
        return [r.clone() for r in res]

    def grow(n):
        for ly in range(L):
            cache.append_kv(ly, [0, 1], [n, n], torch.cat([data[ly][0][0][T[0]:T[0] + n], data[ly][1][0][T[1]:T[1] + n]]),
                            torch.cat([data[ly][0][1][T[0]:T[0] + n], data[ly][1][1][T[1]:T[1] + n]]))
        T[0] += n
        T[1] += n

    ref = eager()                                           # also builds the plans outside any capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            # not recordable: must refuse without breaking the capture
            with pytest.raises(pkv.PkvError) as e1:
                cache.append_kv(0, [0], [1], data[0][0][0][:1], data[0][0][1][:1])
            assert e1.value.status == pkv.PKV_ERR_UNSUPPORTED
            with pytest.raises(pkv.PkvError) as e2:
                cache.compress_eligible_pages(-1)
            assert e2.value.status == pkv.PKV_ERR_UNSUPPORTED
            with pytest.raises(pkv.PkvError) as e3:
                cache.decode_attention(0, [0, 1], qs[0], outs[0])          # another batch order: no current plan
            assert e3.value.status == pkv.PKV_ERR_UNSUPPORTED
            for ly in range(L):
                cache.decode_attention(ly, ids, qs[ly], outs[ly])
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    torch.cuda.synchronize()
    for ly in range(L):
        assert torch.equal(outs[ly], ref[ly])
    # three tokens more, same pages (700 -> 703 and 1500 -> 1503 stay inside pages 10 and 23)
    grow(3)
    graph.replay()
    torch.cuda.synchronize()
    got = [o.clone() for o in outs]
    ref = eager()
    for ly in range(L):
        assert torch.equal(got[ly], ref[ly])
    # new pages and newly compressed pages: one eager call per layer rebuilds the plan, then the graph is valid again
    grow(130)
    cache.compress_eligible_pages(-1)
    ref = eager()
    graph.replay()
    torch.cuda.synchronize()
    for ly in range(L):
        assert torch.equal(outs[ly], ref[ly])
    assert cache.stats()["device_timeouts"] == 0
    cache.close()


@pytest.mark.gpu
def test_mode_2_launches_in_a_cuda_graph():
    """decode_overlap = 2 recorded into a graph: 70 launches over three layers (more than the 64 scratch sets, so the
    graph contains a draining launch) reproduce, in every replay and bit for bit, what a cache with decode_overlap = 0
    computes; launches outside a graph still work afterwards (as ordinary launches), also between replays."""
    L, H, G = 3, 2, 4
    kw = dict(n_layers=L, n_kv_heads=H, n_q_heads=H * G, rank=24, sink_tokens=64, recent_tokens=128, max_seqs=3,
              max_pages_per_seq=40, n_dense_slots=300, n_factor_slots=300)
    fast, slow = pkv.Cache(pkv.make_config(decode_overlap=2, **kw), "cuda"), pkv.Cache(pkv.make_config(decode_overlap=0, **kw), "cuda")
    lengths = [2100, 130, 900]
    for ly in range(L):
        for s_, T in enumerate(lengths):
            k, v = synth.make_kv(23, ly, s_, T, H, 128, 64, "cuda")
            for c in (fast, slow):
                c.append_kv(ly, [s_], [T], k, v)
    for c in (fast, slow):
        c.compress_eligible_pages(-1)
    ids = [2, 0, 1]
    n_launch = 70
    qs = [synth.make_q(23, i % L, i, 3, H * G, 128, "cuda") for i in range(n_launch)]
    ref = [torch.empty_like(q) for q in qs]
    for i in range(n_launch):
        slow.decode_attention(i % L, ids, qs[i], ref[i])
    outs = [torch.empty_like(q) for q in qs]
    for ly in range(L):
        fast.decode_attention(ly, ids, qs[ly], outs[ly])    # plans built outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(n_launch):
                fast.decode_attention(i % L, ids, qs[i], outs[i])
    torch.cuda.current_stream().wait_stream(side)
    for rep in range(3):
        for o in outs:
            o.zero_()
        graph.replay()
        if rep == 1:                                            # a launch outside the graph right behind a replay
            extra = torch.empty_like(qs[0])
            fast.decode_attention(0, ids, qs[0], extra)
        graph.replay()
        torch.cuda.synchronize()
        for i in range(n_launch):
            assert torch.equal(outs[i], ref[i]), (rep, i)
        if rep == 1:
            assert torch.equal(extra, ref[0])
    st = fast.stats()
    assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0
    fast.close()
    slow.close()


@pytest.mark.parametrize("bits", [16, 4])
def test_two_step_compression_on_a_side_stream(bits):
    """A chunked prefill with the factorization on a second stream: per chunk and layer, append the chunk, attend
    with all the chunk's positions as queries, begin the layer's compression on the side stream, and commit it one
    chunk later.  Checked: between begin and commit the cache reads as dense (kernel gate against the oracle in
    the same state); page tables equal the oracle's two-step form after every commit; at the end every factor
    page holds bit for bit the factors that the one-step call produces on a second cache fed the same tokens, and
    both caches give the same attention output bit for bit."""
    L, H, G, P, chunk, n_chunks = 2, 2, 4, 64, 192, 6
    cfg = pkv.make_config(n_layers=L, n_kv_heads=H, n_q_heads=H * G, rank=16, sink_tokens=P, recent_tokens=4 * P,
                          max_seqs=2 * (chunk // 2), max_pages_per_seq=32, n_dense_slots=160, n_factor_slots=120,
                          factor_bits=bits)
    pair = Pair(cfg, seed=9)
    sync = pkv.Cache(cfg, "cuda")                      # one-step path, its own slot numbering
    side = torch.cuda.Stream()
    seqs = [0, 1]
    kv = {(ly, s): gen_kv(9, ly, s, chunk * n_chunks, cfg, outlier_prob=0.01) for ly in range(L) for s in seqs}
    gq = torch.Generator().manual_seed(77)
    worst = 0.0
    for ci in range(n_chunks):
        lo, hi = ci * chunk, (ci + 1) * chunk
        for ly in range(L):
            if ci > 0:
                n = pair.gpu.compress_commit(ly)
                assert pair.orc.compress_commit(ly) == n
                pair.same_tables()
            ks = [kv[(ly, s)][0][lo:hi] for s in seqs]
            vs = [kv[(ly, s)][1][lo:hi] for s in seqs]
            pair.append(ly, seqs, ks, vs)
            sync.append_kv(ly, seqs, [chunk] * 2, torch.cat(ks).cuda(), torch.cat(vs).cuda())
            q = torch.randn((2, chunk, H * G, 128), generator=gq).to(torch.bfloat16)
            out32 = torch.empty(q.shape, dtype=torch.float32, device="cuda")
            out = torch.empty(q.shape, dtype=torch.bfloat16, device="cuda")
            # begin now, then attend while the side stream factorizes: the attention must still see these pages dense
            n_b = pair.gpu.compress_begin(ly, side)
            assert pair.orc.compress_begin(ly) == n_b == (0 if ci == 0 else 2 if ci == 1 else 6)
            pair.gpu.decode_attention_multi(ly, seqs, chunk, q.cuda(), out, out32)
            sync.compress_eligible_pages(ly)
            if ci in (2, n_chunks - 1) and ly == 1:
                torch.cuda.synchronize()
                saved = pair.orc.factor
                pair.orc.factor = dict(saved)
                for s in seqs:
                    pair.load_gpu_factors_into_oracle(s, ly)
                ref = pair.orc.decode_attention_multi(ly, seqs, f64(q))
                pair.orc.factor = saved
                got = f64(out32)
                for i in range(2):
                    for j in range(0, chunk, 13):
                        worst = max(worst, rel_err(got[i, j], ref[i, j]))
                        assert rel_err(got[i, j], ref[i, j]) <= (1e-2 if bits == 4 else 4e-3), (ci, i, j)
    assert pair.gpu.compress_commit() == pair.orc.compress_commit() > 0
    pair.same_tables()
    assert pair.gpu.compress_commit() == 0
    torch.cuda.synchronize()
    # logical pages of both caches: same kinds, same bytes
    for ly in range(L):
        for s in seqs:
            ka, sa, Ta = pair.gpu.page_table(s, ly)
            kb, sb, Tb = sync.page_table(s, ly)
            assert ka == kb and Ta == Tb and sum(ka) > 0
            for p, kind in enumerate(ka):
                if kind == 1:
                    for h in range(H):
                        fa, fb = pair.gpu.read_factors(sa[p], h), sync.read_factors(sb[p], h)
                        assert all(torch.equal(x, y) for x, y in zip(fa, fb)), (ly, s, p, h)
        q1 = synth.make_q(9, ly, 0, 2, H * G, 128, "cuda")
        oa, ob = torch.empty_like(q1), torch.empty_like(q1)
        pair.gpu.decode_attention(ly, seqs, q1, oa)
        sync.decode_attention(ly, seqs, q1, ob)
        torch.cuda.synchronize()
        assert torch.equal(oa, ob)
    st = pair.gpu.stats()
    assert st["device_timeouts"] == 0 and st["page_svds_not_converged"] == 0 and st["bad_slot_indices"] == 0
    print("two-step compression bits=%d: kernel gate max %.2e, %d pages" % (bits, worst, st["pages_compressed"]))
    sync.close()


@pytest.mark.gpu
@pytest.mark.parametrize("q_len,max_seqs", [(3, 4), (40, 2)])
def test_cuda_graph_replay_of_multi_query_and_state_calls(q_len, max_seqs):
    """pkv_decode_attention_multi (decode kernel with query columns at q_len = 3; row-block kernel at q_len = 40,
    forced by max_seqs) and pkv_decode_attention_partial + pkv_merge_attention_states recorded into one CUDA graph:
    replays equal eager calls, also after appends that stay inside the current pages."""
    H, G = 2, 2
    cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=16, sink_tokens=64, recent_tokens=128,
                          max_seqs=max_seqs, max_pages_per_seq=40, n_dense_slots=100, n_factor_slots=100, decode_overlap=1)
    cache = pkv.Cache(cfg, "cuda", None, None)
    T = [900, 1410]
    data = [synth.make_kv(31, 0, s, 2000, H, 128, 64, "cuda") for s in range(2)]
    for s in range(2):
        cache.append_kv(0, [s], [T[s]], data[s][0][:T[s]], data[s][1][:T[s]])
    cache.compress_eligible_pages(0)
    ids = [1, 0]
    g = torch.Generator(device="cuda").manual_seed(3)
    qm = torch.randn((2, q_len, H * G, 128), generator=g, device="cuda").to(torch.bfloat16)
    q1 = qm[:, -1].contiguous()
    out_m, out_1 = torch.empty_like(qm), torch.empty_like(q1)
    state = torch.empty((2, H * G, 130), dtype=torch.float32, device="cuda")

    def eager():
        a, b = torch.empty_like(qm), torch.empty_like(q1)
        cache.decode_attention_multi(0, ids, q_len, qm, a)
        st = cache.decode_attention_partial(0, ids, q1)
        pkv.pkv_merge_attention_states(st, 1, 2 * H * G, b, None, torch.cuda.current_stream())
        torch.cuda.synchronize()
        return a, b

    ref_m, ref_1 = eager()                                  # builds both plans outside the capture
    cache.decode_attention_multi(0, ids, q_len, qm, out_m)  # the multi-query plan is the current one again
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            cache.decode_attention_multi(0, ids, q_len, qm, out_m)
            with pytest.raises(pkv.PkvError) as e:         # one plan per layer: the single-query plan is stale now
                cache.decode_attention_partial(0, ids, q1, state)
            assert e.value.status == pkv.PKV_ERR_UNSUPPORTED
    torch.cuda.current_stream().wait_stream(side)
    for n in (0, 2):
        if n:
            cache.append_kv(0, [0, 1], [n, n], torch.cat([data[0][0][T[0]:T[0] + n], data[1][0][T[1]:T[1] + n]]),
                            torch.cat([data[0][1][T[0]:T[0] + n], data[1][1][T[1]:T[1] + n]]))
            T[0] += n
            T[1] += n
            cache.decode_attention_multi(0, ids, q_len, qm, out_m)         # same pages: nothing to rebuild
            ref_m, ref_1 = eager()
            cache.decode_attention_multi(0, ids, q_len, qm, torch.empty_like(qm))
        out_m.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out_m, ref_m)
    # the state call in a graph of its own, with its plan current
    cache.decode_attention_partial(0, ids, q1, state)
    graph2 = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph2, stream=side):
            cache.decode_attention_partial(0, ids, q1, state)
            pkv.pkv_merge_attention_states(state, 1, 2 * H * G, out_1, None, side)
    torch.cuda.current_stream().wait_stream(side)
    graph2.replay()
    torch.cuda.synchronize()
    assert torch.equal(out_1, ref_1)
    assert cache.stats()["device_timeouts"] == 0
    cache.close()


@pytest.mark.parametrize("n_ctas", [1, 6])
def test_a_bounded_wait_that_runs_out_is_reported_and_the_cache_stays_usable(monkeypatch, n_ctas):
    """Every wait inside the decode kernel gives up after a fixed number of clocks.  Here one is made to: the
    library's test hooks (read from the environment when the cache is created) shorten the limit to about a
    millisecond and make the producer of CTA 0 leave one unit of the first launch unarmed, so the consumer warp that
    waits for it finds nothing (nothing faults and nothing spins for ever: the wait ends by construction).  The call
    must return, the timeout must be counted, and the next call on the same cache must be correct again - also when
    the segment was split over several CTAs, whose merge tickets the aborted launch may have left drawn."""
    monkeypatch.setenv("PKV_TEST_WAIT_CLOCKS", "2000000")
    monkeypatch.setenv("PKV_TEST_DROP_UNIT", "3")
    H, G, T = 1, 4, 1500
    cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=16, sink_tokens=64, recent_tokens=128,
                          max_seqs=1, max_pages_per_seq=32, n_dense_slots=32, n_factor_slots=32, n_ctas=n_ctas)
    pair = Pair(cfg, seed=9)
    monkeypatch.delenv("PKV_TEST_WAIT_CLOCKS")
    monkeypatch.delenv("PKV_TEST_DROP_UNIT")
    k, v = gen_kv(9, 0, 0, T, cfg)
    pair.append(0, [0], [k], [v])
    pair.compress(0)
    q = synth.make_q(9, 0, 0, 1, H * G, 128)
    pair.decode(0, [0], q)                                   # the launch with the unarmed unit: returns, result invalid
    st = pair.gpu.stats()
    assert st["device_timeouts"] >= 1
    got, got32 = pair.decode(0, [0], q)                      # an ordinary launch on the same cache
    assert pair.gpu.stats()["device_timeouts"] == st["device_timeouts"]
    pair.load_gpu_factors_into_oracle(0, 0)
    ref = pair.orc.decode_attention(0, [0], f64(q))
    assert rel_err(got32, ref) <= 4e-3 and rel_err(got, ref) <= 1e-2
    pair.gpu.close()


@pytest.mark.gpu
def test_a_wait_that_runs_out_in_the_tcgen05_row_block_kernel(monkeypatch):
    """The same for the tcgen05 row-block kernel, whose CTAs allocate tensor memory: the copy lane of CTA 0 leaves one
    unit unarmed, the row threads' wait for it runs out, every role of the CTA leaves through the common exit (which
    gives tensor memory back), the call returns with the timeout counted, and the next call on the same cache - whose
    CTAs allocate tensor memory again - is correct."""
    monkeypatch.setenv("PKV_TEST_WAIT_CLOCKS", "4000000")
    monkeypatch.setenv("PKV_TEST_DROP_UNIT", "5")
    H, G, q_len, T = 1, 4, 64, 1500
    cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=24, sink_tokens=64, recent_tokens=128,
                          max_seqs=1, max_pages_per_seq=32, n_dense_slots=32, n_factor_slots=32)
    pair = Pair(cfg, seed=11)
    monkeypatch.delenv("PKV_TEST_WAIT_CLOCKS")
    monkeypatch.delenv("PKV_TEST_DROP_UNIT")
    k, v = gen_kv(11, 0, 0, T, cfg)
    pair.append(0, [0], [k[:T - q_len]], [v[:T - q_len]])
    pair.compress(0)
    pair.append(0, [0], [k[T - q_len:]], [v[T - q_len:]])
    g = torch.Generator().manual_seed(12)
    q = torch.randn((1, q_len, H * G, 128), generator=g).to(torch.bfloat16)
    qd = q.cuda()
    out32 = torch.empty(qd.shape, dtype=torch.float32, device="cuda")
    pair.gpu.decode_attention_multi(0, [0], q_len, qd, None, out32)       # the launch with the unarmed unit
    torch.cuda.synchronize()
    st = pair.gpu.stats()
    assert st["device_timeouts"] >= 1
    pair.gpu.decode_attention_multi(0, [0], q_len, qd, None, out32)       # an ordinary launch on the same cache
    torch.cuda.synchronize()
    assert pair.gpu.stats()["device_timeouts"] == st["device_timeouts"]
    pair.load_gpu_factors_into_oracle(0, 0)
    ref = pair.orc.decode_attention_multi(0, [0], f64(q))
    got32 = f64(out32)
    for j in range(q_len):
        assert rel_err(got32[0, j], ref[0, j]) <= 4e-3, j
    pair.gpu.close()
