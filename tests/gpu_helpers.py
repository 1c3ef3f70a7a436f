"""Shared plumbing for the GPU parity tests: build the CUDA cache and the fp64
oracle cache from the same seeded bf16 inputs."""
import numpy as np
import torch

from oracle.cache import FACTOR, OracleCache, OracleConfig
from paper_2608_23843_b200 import pkv, synth


def f64(t):
    """Exact widening of a bf16/fp32 tensor to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_config(cfg: pkv.PkvConfig) -> OracleConfig:
    return OracleConfig(n_layers=cfg.n_layers, n_kv_heads=cfg.n_kv_heads, n_q_heads=cfg.n_q_heads,
                        head_dim=cfg.head_dim, page_size=cfg.page_size, rank_k=cfg.rank_k, rank_v=cfg.rank_v,
                        sink_tokens=cfg.sink_tokens, recent_tokens=cfg.recent_tokens, max_seqs=cfg.max_seqs,
                        n_dense_slots=cfg.n_dense_slots, n_factor_slots=cfg.n_factor_slots,
                        softmax_scale=cfg.softmax_scale, factor_bits=4 if cfg.factor_bits == 4 else 16)


class Pair:
    """A CUDA cache and an oracle cache fed identically."""

    def __init__(self, cfg, seed=0, shuffle=True, oracle=True):
        self.cfg, self.seed = cfg, seed
        d_ord = f_ord = None
        if shuffle:
            d_ord = synth.slot_permutation(seed, cfg.n_dense_slots, 0).tolist()
            f_ord = synth.slot_permutation(seed, cfg.n_factor_slots, 1).tolist()
        self.gpu = pkv.Cache(cfg, "cuda", d_ord, f_ord)
        self.orc = OracleCache(oracle_config(cfg), d_ord, f_ord) if oracle else None

    def append(self, layer, seq_ids, k_list, v_list):
        """k_list[i], v_list[i]: bf16 CPU tensors [n_i, H_kv, d] for seq_ids[i]."""
        n_new = [int(k.shape[0]) for k in k_list]
        k, v = torch.cat(k_list), torch.cat(v_list)
        self.gpu.append_kv(layer, seq_ids, n_new, k.cuda(), v.cuda())
        if self.orc is not None:
            self.orc.append_kv(layer, seq_ids, n_new, f64(k), f64(v))

    def compress(self, layer=-1):
        n = self.gpu.compress_eligible_pages(layer)
        if self.orc is not None:
            assert self.orc.compress_eligible_pages(layer) == n
        return n

    def decode(self, layer, seq_ids, q):
        """q: bf16 CPU tensor [n, H_q, d] -> (gpu bf16 out, gpu fp32 out) as float64 numpy."""
        qd = q.cuda()
        out = torch.empty_like(qd)
        out32 = torch.empty(qd.shape, dtype=torch.float32, device="cuda")
        self.gpu.decode_attention(layer, seq_ids, qd, out, out32)
        torch.cuda.synchronize()
        return f64(out), f64(out32)

    def same_tables(self):
        for s in range(self.cfg.max_seqs):
            for ly in range(self.cfg.n_layers):
                assert self.gpu.page_table(s, ly) == self.orc.page_table(s, ly), (s, ly)

    def load_gpu_factors_into_oracle(self, seq, layer):
        """Kernel gate: make the oracle attend over the GPU's own bf16 factors."""
        kinds, slots, _ = self.gpu.page_table(seq, layer)
        for kd, slot in zip(kinds, slots):
            if kd != FACTOR:
                continue
            parts = [self.gpu.read_factors(slot, h) for h in range(self.cfg.n_kv_heads)]
            torch.cuda.synchronize()
            self.orc.set_factors(slot, *[np.stack([f64(p[i]) for p in parts]) for i in range(4)])

    def dense_page_gpu(self, slot, head):
        K, V = self.gpu.read_dense(slot, head)
        torch.cuda.synchronize()
        return f64(K), f64(V)


def attention_gates(pair, layer, order, q, got, got32):
    """The three attention comparisons of one decode call, each max-abs error over ||ref||_inf
    per batch entry:
      kernel   GPU vs oracle attending over the GPU's own stored (bf16) factors
      e2e      GPU vs oracle with its own unrounded fp64 factors
      floor    oracle with its factors rounded to the bf16 storage type vs the same oracle unrounded:
               the error that storing factors in bf16 causes on its own, for any implementation
    """
    import copy
    qd = f64(q)
    ref = pair.orc.decode_attention(layer, order, qd)
    rounded = copy.deepcopy(pair.orc)
    rounded.round_factors_to_storage_type()
    ref_rounded = rounded.decode_attention(layer, order, qd)
    saved = pair.orc.factor
    pair.orc.factor = dict(saved)
    for s in order:
        pair.load_gpu_factors_into_oracle(s, layer)
    ref_kernel = pair.orc.decode_attention(layer, order, qd)
    pair.orc.factor = saved
    n = len(order)
    return dict(kernel=[rel_err(got32[i], ref_kernel[i]) for i in range(n)],
                kernel_bf16=[rel_err(got[i], ref_kernel[i]) for i in range(n)],
                e2e=[rel_err(got[i], ref[i]) for i in range(n)],
                floor=[rel_err(ref_rounded[i], ref[i]) for i in range(n)])


def assert_attention_gates(g, tol=1e-2, kernel_f32_tol=4e-3):
    for i in range(len(g["e2e"])):
        assert g["kernel"][i] <= kernel_f32_tol, ("kernel gate (fp32 out)", i, g["kernel"][i])
        assert g["kernel_bf16"][i] <= tol, ("kernel gate", i, g["kernel_bf16"][i])
        assert g["e2e"][i] <= tol + 3.0 * g["floor"][i], ("end-to-end gate", i, g["e2e"][i], g["floor"][i])


def gen_kv(seed, layer, seq, n_tokens, cfg, outlier_prob=0.0):
    return synth.make_kv(seed, layer, seq, n_tokens, cfg.n_kv_heads, cfg.head_dim, cfg.page_size,
                         "cpu", outlier_prob)


def rel_err(got, ref):
    """max-abs error over ||ref||_inf, per (sequence, head) row block."""
    return float(np.abs(got - ref).max() / np.abs(ref).max())
