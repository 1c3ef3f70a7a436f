"""Seeded random sweep over page sizes, ranks (including ranks that are not multiples of 8 and full rank), head
counts, ragged lengths around the page boundaries, dense regions, grid sizes, launch modes and factor storage:
page tables bit-exact against the oracle's state machine, no device timeouts, no NaN, and the kernel gate (the
oracle attending over the GPU's own stored factors)."""
import random

import numpy as np
import pytest

from gpu_helpers import Pair, assert_kernel_gate_any_shape, attention_gates, entry_vmax, gen_kv, kernel_tolerances
from paper_2608_23843_b200 import pkv, synth

pytestmark = pytest.mark.gpu


def _case(rng, case):
    P = rng.choice([16, 32, 64, 64])
    tiles = rng.choice([1, 2, 3, 4]) if P >= 32 else rng.choice([1, 2])
    rk = min(P, 8 * tiles - rng.choice([0, 0, 1, 3]))
    rv = min(P, 8 * tiles - rng.choice([0, 0, 2, 5]))
    rk, rv = max(rk, 8 * (tiles - 1) + 1), max(rv, 8 * (tiles - 1) + 1)       # same number of 8-wide tiles
    H, G = rng.choice([1, 2, 4]), rng.choice([1, 2, 3, 4, 8])
    nseq = rng.choice([1, 2, 5, 9])
    lengths = [rng.choice([1, 2, P - 1, P, P + 1, 3 * P + 5, rng.randint(1, 40 * P)]) for _ in range(nseq)]
    max_pages = max(-(-t // P) for t in lengths) + 1
    cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=rk, rank_v=rv, page_size=P,
                          sink_tokens=P * rng.choice([0, 1, 2]), recent_tokens=P * rng.choice([0, 1, 4]),
                          max_seqs=nseq, max_pages_per_seq=max_pages, n_dense_slots=nseq * max_pages + 2,
                          n_factor_slots=nseq * max_pages + 2, n_ctas=rng.choice([0, 0, 1, 2, 7, 33, 148, 296]),
                          decode_overlap=rng.choice([0, 0, 1, 2]), factor_bits=rng.choice([16, 16, 4]))
    return cfg, lengths


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_configurations(seed):
    rng = random.Random(seed)
    for case in range(25):
        cfg, lengths = _case(rng, case)
        what = (seed, case, cfg.page_size, cfg.rank_k, cfg.rank_v, cfg.n_kv_heads, cfg.n_q_heads, lengths, cfg.n_ctas,
                cfg.decode_overlap, cfg.factor_bits)
        pair = Pair(cfg, seed=case)
        for s, T in enumerate(lengths):
            k, v = gen_kv(100 + case, 0, s, T, cfg)
            cut = rng.randint(0, T)
            if cut:
                pair.append(0, [s], [k[:cut]], [v[:cut]])
            if rng.random() < 0.5:
                pair.compress(0)
            if cut < T:
                pair.append(0, [s], [k[cut:]], [v[cut:]])
        pair.compress(0)
        pair.same_tables()
        order = list(range(len(lengths)))
        rng.shuffle(order)
        q = synth.make_q(100 + case, 0, 0, len(order), cfg.n_q_heads, 128)
        pair.decode(0, order, q)
        got, got32 = pair.decode(0, order, q)
        st = pair.gpu.stats()
        assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0 and st["page_svds_not_converged"] == 0, what
        assert not np.isnan(got).any() and not np.isnan(got32).any(), what
        g = attention_gates(pair, 0, order, q, got, got32)
        assert_kernel_gate_any_shape(g, what)
        pair.gpu.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_random_schedules(seed):
    """Random schedules of append (one token up to more than a page, a random subset of the sequences, every layer),
    compress, free and decode on a random layer in random batch order: page tables bit-exact against the oracle after
    every step, kernel gate at every decode, in every launch mode and with both factor formats."""
    rng = random.Random(1000 + seed)
    for case in range(5):
        P = rng.choice([16, 32, 64])
        L, H, G, nseq = rng.choice([1, 2, 3]), rng.choice([1, 2]), rng.choice([1, 4, 8]), rng.choice([2, 4])
        rk = min(P, rng.choice([8, 16, 24]) if P >= 32 else rng.choice([8, 16]))
        t_max = 14 * P
        cfg = pkv.make_config(n_layers=L, n_kv_heads=H, n_q_heads=H * G, rank=rk, page_size=P,
                              sink_tokens=P * rng.choice([0, 1]), recent_tokens=P * rng.choice([1, 2]), max_seqs=nseq,
                              max_pages_per_seq=t_max // P + 2, n_dense_slots=L * nseq * 8 + 8,
                              n_factor_slots=L * nseq * (t_max // P + 2), n_ctas=rng.choice([0, 5, 148]),
                              decode_overlap=rng.choice([0, 1, 2]), factor_bits=rng.choice([16, 16, 4]))
        what = (seed, case, P, L, H, G, nseq, rk, cfg.n_ctas, cfg.decode_overlap, cfg.factor_bits)
        pair = Pair(cfg, seed=case)
        data = {(ly, s): gen_kv(200 + case, ly, s, t_max, cfg) for ly in range(L) for s in range(nseq)}
        T = [0] * nseq
        for step in range(40):
            ids = [s for s in range(nseq) if rng.random() < 0.7]
            n_new = [min(rng.choice([1, 1, 1, 2, 5, P, P + 3]), t_max - T[s]) for s in ids]
            ids, n_new = [s for s, n in zip(ids, n_new) if n > 0], [n for n in n_new if n > 0]
            if ids:
                for ly in range(L):
                    pair.append(ly, ids, [data[(ly, s)][0][T[s]:T[s] + n] for s, n in zip(ids, n_new)],
                                [data[(ly, s)][1][T[s]:T[s] + n] for s, n in zip(ids, n_new)])
                for s, n in zip(ids, n_new):
                    T[s] += n
            if rng.random() < 0.6:
                pair.compress(rng.choice([-1] + list(range(L))))
            if rng.random() < 0.08:
                s = rng.randrange(nseq)
                pair.gpu.free_seq(s)
                pair.orc.free_seq(s)
                T[s] = 0
            live = [s for s in range(nseq) if T[s] > 0]
            if live and rng.random() < 0.7:
                ly = rng.randrange(L)
                rng.shuffle(live)
                q = synth.make_q(200 + case, ly, step, len(live), H * G, 128)
                got, got32 = pair.decode(ly, live, q)
                assert not np.isnan(got32).any(), (what, step)
                g = attention_gates(pair, ly, live, q, got, got32)
                assert_kernel_gate_any_shape(g, (what, step))
            pair.same_tables()
        st = pair.gpu.stats()
        assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0, (what, st)
        pair.gpu.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_random_schedules_with_two_step_compression_multi_query_and_states(seed):
    """The schedule test again with the other entry points mixed in: compression either in one step or begun on a
    side stream and committed some steps later; attention either for one query per sequence, for the q_len newest
    positions (kernel gate against the oracle's causal form), or as a softmax state that, merged alone, must
    reproduce the ordinary call bit for bit.  Page tables bit-exact after every step."""
    import torch
    from gpu_helpers import f64, rel_err
    rng = random.Random(3000 + seed)
    side = torch.cuda.Stream()
    for case in range(4):
        P = rng.choice([16, 32, 64])
        L, H, G, nseq = rng.choice([1, 2]), rng.choice([1, 2]), rng.choice([1, 2, 4, 8]), rng.choice([2, 3])
        rk = min(P, rng.choice([8, 16, 24]) if P >= 32 else rng.choice([8, 16]))
        t_max = 14 * P
        cfg = pkv.make_config(n_layers=L, n_kv_heads=H, n_q_heads=H * G, rank=rk, page_size=P,
                              sink_tokens=P * rng.choice([0, 1]), recent_tokens=P * rng.choice([1, 2]), max_seqs=nseq * 6,
                              max_pages_per_seq=t_max // P + 2, n_dense_slots=L * nseq * 12 + 8,
                              n_factor_slots=L * nseq * (t_max // P + 2), n_ctas=rng.choice([0, 5, 148]),
                              decode_overlap=rng.choice([0, 1, 2]), factor_bits=rng.choice([16, 16, 4]))
        what = (seed, case, P, L, H, G, nseq, rk, cfg.n_ctas, cfg.decode_overlap, cfg.factor_bits)
        pair = Pair(cfg, seed=case)
        data = {(ly, s): gen_kv(300 + case, ly, s, t_max, cfg) for ly in range(L) for s in range(nseq)}
        T = [0] * nseq
        begun = {}                                         # layer -> (step begun, sequences with pages in flight)
        for step in range(40):
            ids = [s for s in range(nseq) if rng.random() < 0.7]
            n_new = [min(rng.choice([1, 1, 1, 2, 5, P, P + 3]), t_max - T[s]) for s in ids]
            ids, n_new = [s for s, n in zip(ids, n_new) if n > 0], [n for n in n_new if n > 0]
            if ids:
                for ly in range(L):
                    pair.append(ly, ids, [data[(ly, s)][0][T[s]:T[s] + n] for s, n in zip(ids, n_new)],
                                [data[(ly, s)][1][T[s]:T[s] + n] for s, n in zip(ids, n_new)])
                for s, n in zip(ids, n_new):
                    T[s] += n
            for ly in list(begun):
                if step - begun[ly][0] >= 2 and rng.random() < 0.6:
                    assert pair.gpu.compress_commit(ly) == pair.orc.compress_commit(ly) > 0
                    del begun[ly]
            ly = rng.randrange(L)
            r = rng.random()
            if r < 0.35 and ly not in begun:
                n = pair.gpu.compress_begin(ly, side)
                assert pair.orc.compress_begin(ly) == n
                if n:
                    begun[ly] = (step, {s_ for s_, *_ in pair.orc.pending[ly]})
            elif r < 0.6 and ly not in begun:
                pair.compress(ly)
            if rng.random() < 0.06:
                s = rng.randrange(nseq)
                if not any(s in seqs for _, seqs in begun.values()):
                    pair.gpu.free_seq(s)
                    pair.orc.free_seq(s)
                    T[s] = 0
            live = [s for s in range(nseq) if T[s] > 0]
            if live and rng.random() < 0.8:
                ly = rng.randrange(L)
                rng.shuffle(live)
                mode = rng.choice(["one", "multi", "state"])
                if mode == "multi":
                    q_len = rng.choice([2, 3, 5, 8 // G + 1])

                    def fits(s):
                        kinds = pair.gpu.page_table(s, ly)[0]
                        f_end = max([p + 1 for p, kd in enumerate(kinds) if kd == 1], default=0)
                        return q_len <= T[s] and f_end * P <= T[s] - q_len + 1
                    batch = [s for s in live if fits(s)]
                    per_tile = max(1, min(q_len, 8 // G))
                    if batch and len(batch) * -(-q_len // per_tile) <= cfg.max_seqs:
                        g = torch.Generator().manual_seed(step * 17 + case)
                        q = torch.randn((len(batch), q_len, H * G, 128), generator=g).to(torch.bfloat16)
                        out32 = torch.empty(q.shape, dtype=torch.float32, device="cuda")
                        pair.gpu.decode_attention_multi(ly, batch, q_len, q.cuda(), None, out32)
                        torch.cuda.synchronize()
                        saved = pair.orc.factor
                        pair.orc.factor = dict(saved)
                        for s in batch:
                            pair.load_gpu_factors_into_oracle(s, ly)
                        ref = pair.orc.decode_attention_multi(ly, batch, f64(q))
                        vmax = [entry_vmax(pair.orc, s, ly) for s in batch]
                        pair.orc.factor = saved
                        got = f64(out32)
                        assert not np.isnan(got).any(), (what, step)
                        # the rule of the single-query gate, per batch entry and per query
                        for i in range(len(batch)):
                            tol32, _ = kernel_tolerances(float(np.abs(ref[i]).max()), vmax[i])
                            assert np.abs(got[i] - ref[i]).max() <= tol32, (what, step, i)
                            for j in range(q_len):
                                tol32, _ = kernel_tolerances(float(np.abs(ref[i, j]).max()), vmax[i])
                                assert np.abs(got[i, j] - ref[i, j]).max() <= tol32, (what, step, i, j)
                else:
                    q = synth.make_q(300 + case, ly, step, len(live), H * G, 128)
                    got, got32 = pair.decode(ly, live, q)
                    assert not np.isnan(got32).any(), (what, step)
                    if mode == "one":
                        g = attention_gates(pair, ly, live, q, got, got32)
                        assert_kernel_gate_any_shape(g, (what, step))
                    else:
                        qd = q.cuda()
                        state = pair.gpu.decode_attention_partial(ly, live, qd)
                        alone = torch.empty_like(qd)
                        pkv.pkv_merge_attention_states(state, 1, len(live) * H * G, alone, None, torch.cuda.current_stream())
                        torch.cuda.synchronize()
                        assert np.array_equal(f64(alone), got), (what, step)
            pair.same_tables()
        assert pair.gpu.compress_commit() == pair.orc.compress_commit()
        pair.same_tables()
        st = pair.gpu.stats()
        assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0, (what, st)
        pair.gpu.close()


@pytest.mark.parametrize("variant", [0, 3])
@pytest.mark.parametrize("seed", [1, 2])
def test_random_configurations_row_block_kernel(seed, variant):
    """Random shapes for the row-block kernels of pkv_decode_attention_multi (queries as tensor-core rows; variant 0:
    the tcgen05 kernel, which serves every shape, with its token ranges where the sequences are long enough; 3: the
    mma.sync kernel): page
    sizes, ranks with ragged last tiles, group sizes, query counts that leave the last block or the last 16-row
    tile partly empty, new positions spanning pages and dense blocks, sequences that consist of nothing but the
    new positions.  max_seqs is kept too small for the column route, so the row-block kernel serves every call.
    Kernel gate against the oracle's causal attention over the GPU's stored factors."""
    import torch
    from gpu_helpers import f64, rel_err
    rng = random.Random(5000 + seed)
    for case in range(10):
        P = rng.choice([16, 32, 64, 64])
        tiles = rng.choice([1, 2, 3, 4]) if P >= 32 else rng.choice([1, 2])
        rk = min(P, 8 * tiles - rng.choice([0, 0, 1, 3]))
        rv = min(P, 8 * tiles - rng.choice([0, 0, 2, 5]))
        rk, rv = max(rk, 8 * (tiles - 1) + 1), max(rv, 8 * (tiles - 1) + 1)
        H, G = rng.choice([1, 2]), rng.choice([1, 2, 3, 4, 8])
        q_len = -(-64 // G) + rng.choice([0, 0, 1, 5, 17, 64 // G])
        nseq = rng.choice([1, 2, 4])
        W = -(-q_len // P) * P + P * rng.choice([0, 1])
        lengths = [rng.choice([q_len, q_len + 1, q_len + P, 2 * P + q_len + 5, rng.randint(q_len, 30 * P)]) for _ in range(nseq)]
        max_pages = max(-(-t // P) for t in lengths) + 1
        cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=rk, rank_v=rv, page_size=P,
                              sink_tokens=P * rng.choice([0, 1, 2]), recent_tokens=W, max_seqs=nseq,
                              max_pages_per_seq=max_pages, n_dense_slots=nseq * max_pages + 2,
                              n_factor_slots=nseq * max_pages + 2, decode_overlap=rng.choice([0, 1, 2]),
                              decode_variant=variant)
        what = (seed, variant, case, P, rk, rv, H, G, q_len, lengths, W, cfg.sink_tokens)
        pair = Pair(cfg, seed=case)
        for s, T in enumerate(lengths):
            k, v = gen_kv(500 + case, 0, s, T, cfg)
            cut = T - q_len
            if cut:
                pair.append(0, [s], [k[:cut]], [v[:cut]])
                pair.compress(0)
            pair.append(0, [s], [k[cut:]], [v[cut:]])
            if rng.random() < 0.5:
                pair.compress(0)
        pair.same_tables()
        order = list(range(nseq))
        rng.shuffle(order)
        g = torch.Generator().manual_seed(case)
        q = torch.randn((nseq, q_len, H * G, 128), generator=g).to(torch.bfloat16)
        out32 = torch.empty(q.shape, dtype=torch.float32, device="cuda")
        pair.gpu.decode_attention_multi(0, order, q_len, q.cuda(), None, out32)
        torch.cuda.synchronize()
        st = pair.gpu.stats()
        assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0, (what, st)
        got = f64(out32)
        assert not np.isnan(got).any(), what
        saved = pair.orc.factor
        pair.orc.factor = dict(saved)
        for s in order:
            pair.load_gpu_factors_into_oracle(s, 0)
        ref = pair.orc.decode_attention_multi(0, order, f64(q))
        vmax = [entry_vmax(pair.orc, s, 0) for s in order]
        pair.orc.factor = saved
        # the rule of the single-query gate, per batch entry (all its queries and heads) and per query
        for i in range(nseq):
            tol32, _ = kernel_tolerances(float(np.abs(ref[i]).max()), vmax[i])
            assert np.abs(got[i] - ref[i]).max() <= tol32, (what, i)
            for j in range(q_len):
                tol32, _ = kernel_tolerances(float(np.abs(ref[i, j]).max()), vmax[i])
                assert np.abs(got[i, j] - ref[i, j]).max() <= tol32, (what, i, j)
        pair.gpu.close()
