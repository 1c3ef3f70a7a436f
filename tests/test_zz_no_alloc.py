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

def _cache(n_ctas=0, decode_overlap=0):
    H, G = 2, 4
    lengths = [4096 + 19, 900, 2500]
    cfg = pkv.make_config(n_layers=1, n_kv_heads=H, n_q_heads=H * G, rank=24, sink_tokens=64, recent_tokens=256,
                          max_seqs=len(lengths), max_pages_per_seq=80, n_dense_slots=160, n_factor_slots=120,
                          n_ctas=n_ctas, decode_overlap=decode_overlap)
    cache = pkv.Cache(cfg, "cuda")
    for s, T in enumerate(lengths):
        k, v = synth.make_kv(21, 0, s, T, H, 128, 64, "cpu")
        cache.append_kv(0, [s], [T], k.cuda(), v.cuda())
    cache.compress_eligible_pages(0)
    return cache, H * G


@pytest.mark.parametrize("decode_overlap", [0, 2])
def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row(decode_overlap):
    """Same plan, same kernels, same order of the cross-CTA sum: the two entry points must agree bit for bit,
    whatever the cache's launch mode."""
    cache, Hq = _cache(decode_overlap=decode_overlap)
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
        assert np.isfinite(got32.cpu().numpy()).all()
        assert torch.equal(got, ref) and torch.equal(got32, ref32), (call, (got32 - ref32).abs().max().item())
        # the call keeps the same books as pkv_decode_attention
        st = cache.stats()
        assert st["last_decode_units"] > 0 and st["last_decode_bytes"] > 2 * q.numel() * 2
    st = cache.stats()
    assert st["device_timeouts"] == 0 and st["bad_slot_indices"] == 0
    cache.close()


def test_static_scratch_call_is_refused_inside_a_capture_when_the_plan_is_stale():
    """The plan is uploaded through a staging ring whose contents a graph replay would not see again: like
    pkv_decode_attention, the call refuses to be recorded while its plan needs rebuilding, and can be recorded
    (nothing asserted about the graph itself) once the plan is current."""
    cache, Hq = _cache()
    q = synth.make_q(21, 0, 0, 2, Hq, 128, "cuda")
    out = torch.empty_like(q)
    pkv.pkv_decode_attention_static_scratch(cache.handle, 0, [0, 1], q, out, None, torch.cuda.current_stream())
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            with pytest.raises(pkv.PkvError) as e:           # another batch: plan not current
                pkv.pkv_decode_attention_static_scratch(cache.handle, 0, [2, 1], q, out, None, side)
            assert e.value.status == pkv.PKV_ERR_UNSUPPORTED
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
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
