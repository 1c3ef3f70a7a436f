"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (same cache
builder, default grid, overlapping per-layer launches).  The oracle cannot run these workloads whole,
so it checks sampled (sequence, layer, KV head) slices: heads are independent, so attention for the
query heads of one KV head needs only that head's pages.

  kernel gate      the oracle attends over the slice's pages exactly as stored on the GPU (bf16 factors
                   and dense rows read back): max-abs <= 1e-2 * ||out||_inf.  Every sequence of the batch x
                   at least three (layer, KV head) samples per workload.
  factor gate      every factor page of the sampled slices, at least 4096 page SVDs per workload:
                   ||X - A B||_F <= 1.01 * tail + 1e-3 * ||X||_F, tail from the oracle's fp64 SVD of the
                   regenerated page.  A page that misses this (tail small against ||X||, where bf16 storage of the
                   factors alone costs more than the allowance) is judged against the error of the oracle's own
                   optimal factors rounded to bf16 instead, and counted (pages_judged_by_storage_floor)
  end-to-end gate  oracle append + compress + attend on the regenerated slice (fp64 factors):
                   <= 1e-2 + 2 x (the oracle's own bf16-storage error, itself capped at 10 %)

The measured figures of every workload are appended, as one JSON object per line, to the file named by the
environment variable PKV_PARITY_RESULTS when it is set (tests/results/parity_fullsize.jsonl is such a run).
"""
import copy
import json
import os

import numpy as np
import pytest
import torch

import bench
from gpu_helpers import E2E_FLOOR_CAP, E2E_FLOOR_FACTOR, f64, kernel_tolerances, rel_err
from oracle import attention as oatt
from oracle import svd as osvd
from oracle.cache import FACTOR, OracleCache, OracleConfig
from paper_2608_23843_b200 import pkv, synth

pytestmark = pytest.mark.gpu
ATT_TOL = 1e-2
MIN_PAGE_SVDS = 4096


def record(workload, **figures):
    path = os.environ.get("PKV_PARITY_RESULTS")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(dict(workload=workload, **figures)) + "\n")


def stored_kv(cache, seq, layer, head):
    """K_all, V_all [T, d] of one (sequence, layer, KV head) exactly as the GPU stores them."""
    kinds, slots, T = cache.page_table(seq, layer)
    P = cache.cfg.page_size
    Ks, Vs, factors = [], [], {}
    for p, (kd, slot) in enumerate(zip(kinds, slots)):
        rows = min(P, T - p * P)
        if kd == FACTOR:
            A_k, B_k, A_v, B_v = [f64(t) for t in cache.read_factors(slot, head)]
            factors[p] = (A_k, B_k, A_v, B_v)
            Ks.append(A_k @ B_k)
            Vs.append(A_v @ B_v)
        else:
            K, V = cache.read_dense(slot, head)
            Ks.append(f64(K)[:rows])
            Vs.append(f64(V)[:rows])
    return np.concatenate(Ks), np.concatenate(Vs), factors


def kernel_gate(cache, cfg, layer, order, q, out, samples):
    G = cfg.n_q_heads // cfg.n_kv_heads
    scale = 1.0 / np.sqrt(cfg.head_dim)
    worst = 0.0
    for (i, head) in samples:
        K_all, V_all, _ = stored_kv(cache, order[i], layer, head)
        for g in range(G):
            h = head * G + g
            ref = oatt.attention_plain(f64(q[i, h]), K_all, V_all, scale)
            e = rel_err(f64(out[i, h]), ref)
            assert e <= ATT_TOL, (order[i], layer, h, e)
            worst = max(worst, e)
    return worst


def oracle_slice(w, rank, seq, layer, head, T, device, steps_kv=None):
    """Single-KV-head oracle cache of one slice, regenerated with the bench's generator."""
    P = w.get("page", 64)
    k, v = synth.make_kv(bench.SEED, layer, seq, T, w["n_kv_heads"], 128, P, device, w["outliers"])
    k, v = f64(k[:, head:head + 1]), f64(v[:, head:head + 1])
    G = w["n_q_heads"] // w["n_kv_heads"]
    n_pages = -(-T // P) + 16
    orc = OracleCache(OracleConfig(n_layers=1, n_kv_heads=1, n_q_heads=G, head_dim=128, page_size=P, rank_k=rank,
                                   rank_v=w.get("rank_v", rank), sink_tokens=w["sink"], recent_tokens=w["recent"], max_seqs=1,
                                   n_dense_slots=n_pages, n_factor_slots=n_pages))
    orc.append_kv(0, [0], [T], k, v)
    orc.compress_eligible_pages(0)
    return orc, k, v


def factor_gate(cache, w, rank, seq, layer, head, T, device, orc=None, k=None, v=None):
    """Every factor page (K and V) of one slice against the oracle's singular values.  Returns the oracle slice,
    the number of page SVDs checked and the worst err / bound."""
    if orc is None:
        orc, k, v = oracle_slice(w, rank, seq, layer, head, T, device)
    _, _, gpu_factors = stored_kv(cache, seq, layer, head)
    okinds, oslots, _ = orc.page_table(0, 0)
    assert sorted(gpu_factors) == [p for p, kd in enumerate(okinds) if kd == FACTOR]
    from oracle.bf16 import round_to_bf16
    worst, n, n_floor = 0.0, 0, 0
    P, rank_v = w.get("page", 64), w.get("rank_v", rank)
    for p, (A_k, B_k, A_v, B_v) in gpu_factors.items():
        sig_k, sig_v = orc.sigma[oslots[p]]
        opt = orc.factor[oslots[p]]
        for X, A, B, sig, r, oa, ob in ((k[p * P:(p + 1) * P, 0], A_k, B_k, sig_k[0], rank, opt["A_k"][0], opt["B_k"][0]),
                                        (v[p * P:(p + 1) * P, 0], A_v, B_v, sig_v[0], rank_v, opt["A_v"][0], opt["B_v"][0])):
            err = np.linalg.norm(X - A @ B)
            bound = 1.01 * float(np.sqrt((sig[r:] ** 2).sum())) + 1e-3 * np.linalg.norm(X)
            if err > bound:
                # Pages whose tail is small against ||X|| (a x10 outlier row at a high rank): storing the factors in
                # bf16 alone costs about 2.3e-3 ||X||, in quadrature with the tail, for any implementation.  The
                # yardstick is then what the oracle's own optimal factors give once rounded to the storage type.
                n_floor += 1
                bound = 1.01 * float(np.linalg.norm(X - round_to_bf16(oa) @ round_to_bf16(ob))) + 1e-3 * np.linalg.norm(X)
            assert err <= bound, (seq, layer, head, p, err, bound)
            worst = max(worst, err / bound)
            assert np.abs(A.T @ A - np.eye(r)).max() <= 1e-2
            n += 1
    return orc, n, worst, n_floor


def e2e_gate(orc, q_row, out_row, what):
    """q_row / out_row: [G, d] of the slice's query heads.  Returns (e2e, floor)."""
    qd = f64(q_row)[None]
    ref = orc.decode_attention(0, [0], qd)[0]
    rounded = copy.deepcopy(orc)
    rounded.round_factors_to_storage_type()
    floor = rel_err(rounded.decode_attention(0, [0], qd)[0], ref)
    e2e = rel_err(f64(out_row), ref)
    assert floor <= E2E_FLOOR_CAP, (what, floor)
    assert e2e <= ATT_TOL + E2E_FLOOR_FACTOR * floor, (what, e2e, floor)
    return e2e, floor


def check_slices(cache, w, rank, slices, lengths, qs, outs, device, n_e2e=1):
    """Factor gate over the listed (sequence, layer, KV head) slices and the end-to-end gate over the first n_e2e of
    them.  Returns dict(page_svds, factor_worst, e2e=[...], floor=[...])."""
    G = w["n_q_heads"] // w["n_kv_heads"]
    res = dict(page_svds=0, pages_judged_by_storage_floor=0, factor_worst=0.0, e2e=[], floor=[])
    for i, (seq, layer, head) in enumerate(slices):
        orc, n, worst, n_floor = factor_gate(cache, w, rank, seq, layer, head, lengths[seq], device)
        res["page_svds"] += n
        res["pages_judged_by_storage_floor"] += n_floor
        res["factor_worst"] = max(res["factor_worst"], worst)
        if i < n_e2e:
            e2e, floor = e2e_gate(orc, qs[layer][seq, head * G:(head + 1) * G], outs[layer][seq, head * G:(head + 1) * G],
                                  (seq, layer, head))
            res["e2e"].append(e2e)
            res["floor"].append(floor)
    return res


def _decode_all(cache, w, ids, device):
    qs = [synth.make_q(bench.SEED, layer, 0, len(ids), w["n_q_heads"], 128, device) for layer in range(w["n_layers"])]
    outs = [torch.empty_like(q) for q in qs]
    for layer in range(w["n_layers"]):
        cache.decode_attention(layer, ids, qs[layer], outs[layer])
    torch.cuda.synchronize()
    return qs, outs


def _finish(cache):
    st = cache.stats()
    assert st["device_timeouts"] == 0 and st["page_svds_not_converged"] == 0 and st["bad_slot_indices"] == 0, st
    cache.close()


def test_llama3_8b_layer_batch8_context_32k():
    """Llama-3-8B-shaped layer: 32q/8kv, batch 8, T=32768, r=24, 64 sink + 256 recent, shuffled pools."""
    w, device = bench.WORKLOADS["llama3_8b_32k_b8"], torch.device("cuda", 0)
    cfg, cache, lengths, comp = bench.build_workload(w, w["rank"], device)
    assert comp["n_page_svds"] == 64896 * w["n_layers"]
    ids = list(range(w["batch"]))
    assert cache.page_table(3, 0)[0] == [0] + [1] * 507 + [0] * 4
    qs, outs = _decode_all(cache, w, ids, device)
    # kernel gate: every sequence x three KV heads of one layer, and one more layer for two sequences
    worst = kernel_gate(cache, cfg, 0, ids, qs[0], outs[0], [(i, h) for i in ids for h in (0, 3, 7)])
    worst = max(worst, kernel_gate(cache, cfg, 2, ids, qs[2], outs[2], [(1, 5), (6, 2)]))
    res = check_slices(cache, w, w["rank"], [(5, 0, 7), (0, 0, 0), (7, 0, 3), (2, 2, 5), (4, 1, 1)], lengths, qs, outs, device, n_e2e=2)
    assert res["page_svds"] >= MIN_PAGE_SVDS
    again = torch.empty_like(outs[0])
    cache.decode_attention(0, ids, qs[0], again)
    torch.cuda.synchronize()
    assert torch.equal(again, outs[0])
    record("llama3_8b_32k_b8", kernel_gate_worst=worst, kernel_gate_slices=26, **res)
    _finish(cache)


def test_qwen3_32b_64_layers_context_128k():
    """Qwen3-32B-shaped long context: 64 layers, 64q/8kv, batch 1, T=131072, r=24, 64 sink + 512 recent."""
    w, device = bench.WORKLOADS["qwen3_32b_128k"], torch.device("cuda", 0)
    cfg, cache, lengths, comp = bench.build_workload(w, w["rank"], device)
    assert comp["n_page_svds"] == 2087936
    kinds = cache.page_table(0, 63)[0]
    assert kinds == [0] + [1] * 2039 + [0] * 8
    qs, outs = _decode_all(cache, w, [0], device)
    worst = 0.0
    samples = ((0, 0), (31, 5), (63, 7), (17, 2))
    for layer, head in samples:
        worst = max(worst, kernel_gate(cache, cfg, layer, [0], qs[layer], outs[layer], [(0, head)]))
    res = check_slices(cache, w, w["rank"], [(0, 31, 5), (0, 63, 7)], lengths, qs, outs, device, n_e2e=2)
    assert res["page_svds"] >= MIN_PAGE_SVDS
    record("qwen3_32b_128k", kernel_gate_worst=worst, kernel_gate_slices=len(samples), pages_per_s=comp["pages_per_s"], **res)
    _finish(cache)


def test_paper_default_shape_qwen3_8b_16k():
    """The paper's own setting: 36 layers, 32q/8kv, 16K context, P=32, ranks (16,14), one sink page and the
    last completed page + incomplete page dense (the context here ends with a 17-token incomplete page)."""
    w, device = bench.WORKLOADS["qwen3_8b_16k_paper_default"], torch.device("cuda", 0)
    cfg, cache, lengths, comp = bench.build_workload(w, w["rank"], device)
    assert cache.page_table(0, 35)[0] == [0] + [1] * 510 + [0, 0]
    sz = cache.sizes
    assert sz.factor_slot_bytes / sz.dense_slot_bytes == 0.5859375             # Eq. 3 at (16,14), P=32, d=128
    qs, outs = _decode_all(cache, w, [0], device)
    worst = 0.0
    samples = ((0, 0), (17, 3), (35, 7), (8, 5))
    for layer, head in samples:
        worst = max(worst, kernel_gate(cache, cfg, layer, [0], qs[layer], outs[layer], [(0, head)]))
    res = check_slices(cache, w, w["rank"], [(0, 17, 3), (0, 0, 0), (0, 35, 7), (0, 8, 5), (0, 26, 1)], lengths, qs, outs,
                       device, n_e2e=2)
    assert res["page_svds"] >= MIN_PAGE_SVDS
    record("qwen3_8b_16k_paper_default", kernel_gate_worst=worst, kernel_gate_slices=len(samples),
           pages_per_s=comp["pages_per_s"], **res)
    _finish(cache)


@pytest.mark.parametrize("variant", [0, 3])
@pytest.mark.parametrize("workload", ["prefill_chunk_llama3_8b_32k", "prefill_chunk_qwen3_8b_16k_p32", "prefill_chunk_qwen3_8b_16k_p16"])
def test_prefill_chunk_2048_positions_against_a_long_context(workload, variant):
    """The bench's prefill-chunk launches (`--workload prefill_chunk_llama3_8b_32k --q-len 2048`, and the same on the
    paper's default page shape, P = 32 with ranks (16, 14)): one sequence whose last 2048 positions are the queries,
    8192 query rows per KV head, served by the row-block kernels (variant 0: tcgen05, 512 CTAs of 128 rows; 3:
    mma.sync, 1024 CTAs of 64 rows).  Sampled query rows -
    the first and last positions of the chunk, positions on either side of page and block boundaries, a row from every
    128-row block parity - against plain attention over the pages exactly as the GPU stores them (kernel gate; the
    causal limit is part of what is checked), the two kernels against one another on every row, and a rerun bit for
    bit.  The third workload, pages of 16 tokens with ranks (8, 8), is judged by the rule for arbitrary shapes: with
    1024 units per row both kernels sit at 4.0e-3 of ||out||_inf on one sampled row (the same row, to four digits:
    the bf16 rounding of the softmax numerators, which they share)."""
    w, device = bench.WORKLOADS[workload], torch.device("cuda", 0)
    QL = 2048
    cfg, cache, lengths, comp = bench.build_workload(w, w["rank"], device, decode_variant=variant)
    T, Hq, Hkv = lengths[0], w["n_q_heads"], w["n_kv_heads"]
    G = Hq // Hkv
    g = torch.Generator(device="cpu").manual_seed(bench.SEED + 77)
    q = torch.randn((1, QL, Hq, 128), generator=g).to(torch.bfloat16).to(device)
    out32 = torch.empty(q.shape, dtype=torch.float32, device=device)
    out = torch.empty_like(q)
    cache.decode_attention_multi(0, [0], QL, q, out, out32)
    again = torch.empty_like(out32)
    cache.decode_attention_multi(0, [0], QL, q, None, again)
    torch.cuda.synchronize()
    assert torch.equal(again, out32) and not out32.isnan().any()
    scale = 1.0 / np.sqrt(cfg.head_dim)
    positions = [0, 1, 31, 32, 63, 64, 65, 127, 128, 1000, 1023, 1024, 1999, 2046, 2047]
    worst = 0.0
    for head in (0, 5):
        K_all, V_all, _ = stored_kv(cache, 0, 0, head)
        for j in positions:
            vis = T - (QL - 1 - j)
            for gq in range(G):
                h = head * G + gq
                ref = oatt.attention_plain(f64(q[0, j, h]), K_all[:vis], V_all[:vis], scale)
                e = rel_err(f64(out32[0, j, h]), ref)
                if workload.endswith("_p16"):
                    # not one of the benchmark configurations the stated 4e-3 was set for: the rule for arbitrary
                    # shapes (4e-3 of ||out||_inf or one bf16 unit of the largest value read, whichever is larger)
                    tol32, _ = kernel_tolerances(float(np.abs(ref).max()), float(np.abs(V_all[:vis]).max()))
                    assert np.abs(f64(out32[0, j, h]) - ref).max() <= tol32, (variant, head, j, gq, e)
                else:
                    assert e <= 4e-3, (variant, head, j, gq, e)
                assert rel_err(f64(out[0, j, h]), ref) <= ATT_TOL
                worst = max(worst, e)
    record(workload, decode_variant=variant, kernel_gate_worst=worst, rows_checked=2 * len(positions) * G)
    if variant == 0:
        _PREFILL_OUT[workload] = out32.cpu()
    elif workload in _PREFILL_OUT:
        a, b = _PREFILL_OUT.pop(workload).double().numpy(), out32.cpu().double().numpy()
        # every row of the launch: the two kernels differ by summation order and by where p and w are rounded
        err = np.abs(a - b).max(axis=-1) / np.abs(b).max(axis=-1)
        assert err.max() <= 8e-3, err.max()          # both are within 4e-3 of the same reference
        print("tcgen05 vs mma.sync over %d rows: worst %.2e, mean %.2e" % (err.size, err.max(), err.mean()))
        record(workload, tcgen05_vs_mma_sync_worst_row=float(err.max()), rows=int(err.size))
    _finish(cache)


_PREFILL_OUT = {}


@pytest.mark.parametrize("q_len", [16, 64])
def test_a_few_dozen_new_positions_per_sequence_at_full_size(q_len):
    """The bench's `--workload llama3_8b_32k_b8 --q-len 16 / 64` launches: 8 sequences of 32K, 64 / 128 row blocks of 128
    rows (half filled at q_len 16), which the tcgen05 kernel cuts into 4 / 2 token ranges of 128 / 256 units each and
    merges by Eq. 5.  Sampled rows of every sequence against plain attention over the pages as the GPU stores them
    (kernel gate), and a rerun bit for bit."""
    w, device = bench.WORKLOADS["llama3_8b_32k_b8"], torch.device("cuda", 0)
    cfg, cache, lengths, comp = bench.build_workload(w, w["rank"], device)
    B, Hq, Hkv = w["batch"], w["n_q_heads"], w["n_kv_heads"]
    G = Hq // Hkv
    ids = list(range(B))
    g = torch.Generator(device="cpu").manual_seed(bench.SEED + 78)
    q = torch.randn((B, q_len, Hq, 128), generator=g).to(torch.bfloat16).to(device)
    out32 = torch.empty(q.shape, dtype=torch.float32, device=device)
    out = torch.empty_like(q)
    cache.decode_attention_multi(0, ids, q_len, q, out, out32)
    again = torch.empty_like(out32)
    cache.decode_attention_multi(0, ids, q_len, q, None, again)
    torch.cuda.synchronize()
    st = cache.stats()
    assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0
    assert torch.equal(again, out32) and not out32.isnan().any()
    scale = 1.0 / np.sqrt(cfg.head_dim)
    worst = 0.0
    for i in ids:
        head = (3 * i + 1) % Hkv
        K_all, V_all, _ = stored_kv(cache, i, 0, head)
        for j in sorted({0, 1, q_len // 2, q_len - 1}):
            vis = lengths[i] - (q_len - 1 - j)
            for gq in range(G):
                h = head * G + gq
                ref = oatt.attention_plain(f64(q[i, j, h]), K_all[:vis], V_all[:vis], scale)
                e = rel_err(f64(out32[i, j, h]), ref)
                assert e <= 4e-3, (i, head, j, gq, e)
                assert rel_err(f64(out[i, j, h]), ref) <= ATT_TOL
                worst = max(worst, e)
    record("llama3_8b_32k_b8", q_len=q_len, kernel_gate_worst=worst, rows_checked=B * 4 * G)
    _finish(cache)


@pytest.mark.parametrize("rank", [8, 16, 24, 32])
def test_ragged_serving_batch_rank_sweep(rank):
    """Ragged serving batch: 64 requests, lengths log-uniform in [2048, 65536], 2% outlier key tokens (x10)."""
    w, device = bench.WORKLOADS["ragged_b64"], torch.device("cuda", 0)
    cfg, cache, lengths, comp = bench.build_workload(w, rank, device)
    ids = list(range(w["batch"]))
    qs, outs = _decode_all(cache, w, ids, device)
    # kernel gate: every sequence, three KV heads in rotation
    worst = kernel_gate(cache, cfg, 0, ids, qs[0], outs[0], [(i, (i + j) % 8) for i in ids for j in (0, 3, 6)])
    # factor and end-to-end gates: the shortest and the longest sequence, then further long ones until enough pages
    by_len = sorted(ids, key=lambda i: lengths[i])
    slices, n = [(by_len[0], 0, 1), (by_len[-1], 0, 6)], 0
    for rank_pos, i in enumerate(reversed(by_len[:-1])):
        if sum(2 * max(0, lengths[s] // 64 - 5) for s, _, _ in slices) >= MIN_PAGE_SVDS:
            break
        slices.append((i, 0, rank_pos % 8))
    res = check_slices(cache, w, rank, slices, lengths, qs, outs, device, n_e2e=2)
    assert res["page_svds"] >= MIN_PAGE_SVDS
    assert any(t % 64 for t in lengths)                     # partial last pages are present
    record("ragged_b64", rank=rank, kernel_gate_worst=worst, kernel_gate_slices=3 * len(ids), **res)
    _finish(cache)


def test_incremental_compression_during_decoding():
    """Incremental compression during decoding: batch 32, prompts of 8192 tokens prefilled and compressed, then
    512 steps of append -> attend -> compress; a page per (sequence, KV head, K|V) leaves the 256-token window
    every 64 steps.  Page tables are checked bit-exact against the oracle's state machine at every step; the
    kernel gate runs at sampled steps over every sequence; one slice is followed end to end by a single-head
    oracle; at the end the factor gate covers sixteen slices (pages factorized at the prefill and during the
    steps alike)."""
    device = torch.device("cuda", 0)
    H, Hq, B, T0, steps, rank = 8, 32, 32, 8192, 512, 24
    n_pages = (T0 + steps) // 64 + 1
    cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=Hq, rank=rank, sink_tokens=64, recent_tokens=256,
                          max_seqs=B, max_pages_per_seq=n_pages, n_dense_slots=B * (T0 // 64 + 2),
                          n_factor_slots=B * n_pages)
    d_ord = synth.slot_permutation(3, cfg.n_dense_slots, 0).tolist()
    f_ord = synth.slot_permutation(3, cfg.n_factor_slots, 1).tolist()
    cache = pkv.Cache(cfg, device, d_ord, f_ord)
    mirror = OracleCache(OracleConfig(n_layers=1, n_kv_heads=1, n_q_heads=1, head_dim=128, page_size=64, rank_k=rank,
                                      rank_v=rank, sink_tokens=64, recent_tokens=256, max_seqs=B,
                                      n_dense_slots=cfg.n_dense_slots, n_factor_slots=cfg.n_factor_slots), d_ord, f_ord)
    ids = list(range(B))
    kv = [synth.make_kv(3, 0, s, T0 + steps, H, 128, 64, device) for s in ids]
    cache.append_kv(0, ids, [T0] * B, torch.cat([k[:T0] for k, _ in kv]), torch.cat([v[:T0] for _, v in kv]))
    assert cache.compress_eligible_pages(0) == B * 123
    # the oracle state machine with zero data mirrors slot numbering (cheap: zero pages converge at once)
    z = np.zeros((B * T0, 1, 128))
    mirror.append_kv(0, ids, [T0] * B, z, z)
    mirror.compress_eligible_pages(0)
    seq_s, head_s, G = 11, 2, Hq // H
    orc = OracleCache(OracleConfig(n_layers=1, n_kv_heads=1, n_q_heads=G, head_dim=128, page_size=64, rank_k=rank,
                                   rank_v=rank, sink_tokens=64, recent_tokens=256, max_seqs=1, n_dense_slots=n_pages,
                                   n_factor_slots=n_pages))
    ks, vs = f64(kv[seq_s][0][:, head_s:head_s + 1]), f64(kv[seq_s][1][:, head_s:head_s + 1])
    orc.append_kv(0, [0], [T0], ks[:T0], vs[:T0])
    orc.compress_eligible_pages(0)
    z1 = np.zeros((B, 1, 128))
    n_events = 0
    worst, e2es, floors = 0.0, [], []
    for t in range(steps):
        knew = torch.cat([k[T0 + t:T0 + t + 1] for k, _ in kv])
        vnew = torch.cat([v[T0 + t:T0 + t + 1] for _, v in kv])
        cache.append_kv(0, ids, [1] * B, knew, vnew)
        mirror.append_kv(0, ids, [1] * B, z1, z1)
        orc.append_kv(0, [0], [1], ks[T0 + t:T0 + t + 1], vs[T0 + t:T0 + t + 1])
        if t + 1 in (1, 64, 65, 512):
            q = synth.make_q(3, 0, t, B, Hq, 128, device)
            out = cache.decode_attention(0, ids, q)
            torch.cuda.synchronize()
            worst = max(worst, kernel_gate(cache, cfg, 0, ids, q, out, [(seq_s, head_s)] + [(i, (i + t) % H) for i in ids]))
            e2e, floor = e2e_gate(orc, q[seq_s, head_s * G:(head_s + 1) * G], out[seq_s, head_s * G:(head_s + 1) * G], t)
            e2es.append(e2e)
            floors.append(floor)
        n = cache.compress_eligible_pages(0)
        assert n == mirror.compress_eligible_pages(0) == (B if (T0 + t + 1) % 64 == 0 else 0)
        orc.compress_eligible_pages(0)
        n_events += n > 0
    assert n_events == 8
    for s in (0, seq_s, B - 1):
        assert cache.page_table(s, 0) == mirror.page_table(s, 0)
    assert cache.page_table(seq_s, 0)[0] == orc.page_table(0, 0)[0]
    # factor gate: the slice followed step by step, then fifteen more (their oracle factorizes the final context in
    # one go: every page is factorized once, from the same rows, whenever that happens)
    wl = dict(n_kv_heads=H, n_q_heads=Hq, sink=64, recent=256)
    _, n_svds, fworst, n_floor = factor_gate(cache, wl, rank, seq_s, 0, head_s, T0 + steps, device, orc=orc, k=ks, v=vs)
    for i in range(15):
        s, h = (2 * i + 1) % B, i % H
        kk, vv = f64(kv[s][0][:, h:h + 1]), f64(kv[s][1][:, h:h + 1])
        o2 = OracleCache(OracleConfig(n_layers=1, n_kv_heads=1, n_q_heads=G, head_dim=128, page_size=64, rank_k=rank,
                                      rank_v=rank, sink_tokens=64, recent_tokens=256, max_seqs=1, n_dense_slots=n_pages,
                                      n_factor_slots=n_pages))
        o2.append_kv(0, [0], [T0 + steps], kk, vv)
        o2.compress_eligible_pages(0)
        _, n, fw, nf = factor_gate(cache, wl, rank, s, 0, h, T0 + steps, device, orc=o2, k=kk, v=vv)
        n_svds, fworst, n_floor = n_svds + n, max(fworst, fw), n_floor + nf
    assert n_svds >= MIN_PAGE_SVDS
    record("serving_b32_8k (512 steps)", kernel_gate_worst=worst, kernel_gate_slices=4 * (B + 1), page_svds=n_svds,
           pages_judged_by_storage_floor=n_floor, factor_worst=fworst, e2e=e2es, floor=floors, steps_checked=[1, 64, 65, 512])
    _finish(cache)
