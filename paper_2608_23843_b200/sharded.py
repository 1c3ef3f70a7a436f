"""Sequence-sharded decode attention: every rank's cache holds a contiguous token range of each sequence.

Each rank computes the softmax state of its own tokens (pkv_decode_attention_partial), the states are
all-gathered (one [n_seqs, H_q, d + 2] fp32 array per rank: 16.6 KB per sequence for 32 query heads), and every
rank applies Eq. 5 to the gathered array (pkv_merge_attention_states).  Shards are summed in rank order, so all
ranks hold the same bits.  The gather is a plain torch.distributed collective on the caller's process group (NCCL
for CUDA tensors); nothing here reads a peer's memory directly.
"""
import torch
import torch.distributed as dist

from . import pkv


def gather_states(state, group=None, out=None):
    """state: [rows..., d + 2] on every rank -> [world, rows..., d + 2], index = rank in `group` (into `out` if given)."""
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    if world == 1:
        return state.unsqueeze(0) if state.is_contiguous() else state.unsqueeze(0).contiguous()
    if out is None:
        out = torch.empty((world,) + tuple(state.shape), dtype=state.dtype, device=state.device)
    dist.all_gather_into_tensor(out.view(world * state.shape[0], *state.shape[1:]), state.contiguous(), group=group)
    return out


def sequence_sharded_decode(cache, layer, seq_ids, q, out=None, out_f32=None, group=None, state=None, gathered=None):
    """q: bf16 [n_seqs, H_q, d], the same on every rank.  Returns out (bf16 [n_seqs, H_q, d]): attention over the
    tokens of all ranks' caches.  Every rank's cache must hold at least one token of every listed sequence.
    state / gathered: optional preallocated fp32 [n_seqs, H_q, d + 2] and [world, n_seqs, H_q, d + 2].  With
    decode_overlap = 2 consecutive calls' kernels run concurrently, so calls in flight need buffers of their own."""
    state = cache.decode_attention_partial(layer, seq_ids, q, state)
    states = gather_states(state, group, gathered)
    if out is None:
        out = torch.empty_like(q)
    n_rows = q.shape[0] * q.shape[1]
    pkv.pkv_merge_attention_states(states, states.shape[0], n_rows, out, out_f32,
                                   torch.cuda.current_stream(q.device))
    return out
