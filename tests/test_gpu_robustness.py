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
