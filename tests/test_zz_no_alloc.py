"""pkv_decode_attention_static_scratch: the decode call for callers that cannot hand the library a
scratch workspace (a serving process that forbids device allocation after start-up, a plug-in with
no allocator of its own).  It must give what pkv_decode_attention gives; its scratch is one array
inside the library that every call shares and that keeps the previous call's contents, so the
check runs twice in a row, with a different batch the second time.  This file sorts last on
purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

from paper_2608_23843_b200 import pkv, synth

pytestmark = pytest.mark.gpu

ATT_TOL = 1e-2          # the attention tolerance used throughout the GPU tests: max-abs <= 1e-2 * ||out||_inf


def _cache(n_ctas=0):
    H, G = 2, 4
    lengths = [4096 + 19, 900, 2500]
    cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=24, sink_tokens=64, recent_tokens=256,
                          max_seqs=len(lengths), max_pages_per_seq=80, n_dense_slots=160, n_factor_slots=120,
                          n_ctas=n_ctas)
    cache = pkv.Cache(cfg, "cuda")
    for s, T in enumerate(lengths):
        k, v = synth.make_kv(21, 0, s, T, H, 128, 64, "cpu")
        cache.append_kv(0, [s], [T], k.cuda(), v.cuda())
    cache.compress_eligible_pages(0)
    return cache, H * G


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    cache, Hq = _cache()
    for call, order in enumerate([[0, 1, 2], [2, 0]]):
        q = synth.make_q(21, 0, call, len(order), Hq, 128, "cuda")
        ref = torch.empty_like(q)
        ref32 = torch.empty(q.shape, dtype=torch.float32, device="cuda")
        pkv.pkv_decode_attention(cache.handle, 0, order, q, ref, ref32, torch.cuda.current_stream())
        got = torch.full_like(q, float("nan"))
        got32 = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
        pkv.pkv_decode_attention_static_scratch(cache.handle, 0, order, q, got, got32, torch.cuda.current_stream())
        torch.cuda.synchronize()
        # the plan of this batch splits segments over many CTAs, so the scratch really is in use
        _, segs = pkv.pkv_get_decode_plan(cache.handle, 0, 512, len(order), 2)
        assert max(n for _, n in segs) > 1
        for a, b in ((got, ref), (got32, ref32)):
            a, b = a.double().cpu().numpy(), b.double().cpu().numpy()
            assert np.isfinite(a).all()
            assert np.abs(a - b).max() <= ATT_TOL * np.abs(b).max(), (call, np.abs(a - b).max())
    st = cache.stats()
    assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0
    cache.close()


def test_static_scratch_rejects_calls_beyond_its_capacity():
    cache, Hq = _cache(n_ctas=1100)              # 1100 CTAs + segments exceed the 1024 partial states
    q = synth.make_q(21, 0, 0, 1, Hq, 128, "cuda")
    out = torch.empty_like(q)
    with pytest.raises(pkv.PkvError) as e:
        pkv.pkv_decode_attention_static_scratch(cache.handle, 0, [0], q, out, None, torch.cuda.current_stream())
    assert e.value.status == pkv.PKV_ERR_INVALID_ARG and "1024" in str(e.value)
    pkv.pkv_decode_attention(cache.handle, 0, [0], q, out, None, torch.cuda.current_stream())   # the workspace path still works
    torch.cuda.synchronize()
    cache.close()
