#!/usr/bin/env python
"""Benchmark of the PuzzleKV decode hot path on B200.

One "step" = one full decode step of the workload: pkv_decode_attention for
every layer (mixed dense/factor attention over the whole context).  Inputs are
seeded synthetic caches (19 GB for the default workload, far larger than L2),
resident in HBM before the timed region.  Also reported: achieved HBM GB/s and
roofline fraction of the decode kernel, page-SVD throughput of the prefill
compression, the same step through host buffers (e2e), and the fp64 oracle
timed on this machine's host cores on a bounded sample.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOADS = {
    # Qwen3-32B-shaped long context (the headline workload): 64 layers, one 128K-token sequence
    "qwen3_32b_128k": dict(n_layers=64, n_kv_heads=8, n_q_heads=64, batch=1, T=131072, rank=24,
                           sink=64, recent=512, ragged=False, outliers=0.0),
    # Llama-3-8B-shaped decode layer, batch 8, 32K tokens each
    # (four independent layers of that shape are built and a step decodes one of them in turn, so that
    # overlapping launches never stream the same bytes and cannot feed each other through L2)
    "llama3_8b_32k_b8": dict(n_layers=4, layers_per_step=1, n_kv_heads=8, n_q_heads=32, batch=8, T=32768, rank=24,
                             sink=64, recent=256, ragged=False, outliers=0.0),
    # ragged serving batch: 64 requests of 2K..64K tokens, outlier key tokens (rank chosen with --rank)
    "ragged_b64": dict(n_layers=2, layers_per_step=1, n_kv_heads=8, n_q_heads=32, batch=64, T=(2048, 65536), rank=24,
                       sink=64, recent=256, ragged=True, outliers=0.02),
    # The paper's own setting: Qwen3-8B shape (36 layers, 32q/8kv), 16K context, P=32, ranks (16,14),
    # one sink page, last completed page + incomplete page dense
    "qwen3_8b_16k_paper_default": dict(n_layers=36, n_kv_heads=8, n_q_heads=32, batch=1, T=16384 + 17, rank=16,
                                       rank_v=14, page=32, sink=32, recent=32, ragged=False, outliers=0.0),
    # serving loop: incremental compression during decoding.  Prompts are prefilled and compressed; a step is append (one token per
    # sequence) -> decode -> compress_eligible, so every 64th step factorizes one page per (sequence, KV head, K|V)
    "serving_b32_8k": dict(n_layers=1, n_kv_heads=8, n_q_heads=32, batch=32, T=8192, rank=24, sink=64, recent=256,
                           ragged=False, outliers=0.0, serving=True),
    # A chunk of a prefill on the Llama-3-8B shape: one sequence of 32K tokens whose newest 2048 positions (inside a
    # dense window of that size) are the queries.  Use with --q-len 2048 (pkv_decode_attention_multi).
    "prefill_chunk_llama3_8b_32k": dict(n_layers=2, layers_per_step=1, n_kv_heads=8, n_q_heads=32, batch=1, T=32768,
                                        rank=24, sink=64, recent=2048, ragged=False, outliers=0.0),
    # The same with the paper's default page shape (Section 4.1: P = 32, ranks (16, 14)) on the Qwen3-8B layer shape.
    "prefill_chunk_qwen3_8b_16k_p32": dict(n_layers=2, layers_per_step=1, n_kv_heads=8, n_q_heads=32, batch=1, T=16384,
                                           rank=16, rank_v=14, page=32, sink=32, recent=2048, ragged=False, outliers=0.0),
    # ... and with the smallest page of the paper's page-size ablation (P = 16) at the same rank per token (8, 8)
    "prefill_chunk_qwen3_8b_16k_p16": dict(n_layers=2, layers_per_step=1, n_kv_heads=8, n_q_heads=32, batch=1, T=16384,
                                           rank=8, rank_v=8, page=16, sink=16, recent=2048, ragged=False, outliers=0.0),
    # tiny single decode step (L2-resident; latency only)
    "tiny": dict(n_layers=1, n_kv_heads=1, n_q_heads=4, batch=1, T=1024, rank=16, sink=64, recent=128,
                 ragged=False, outliers=0.0),
}
SEED = 0
# DRAM bytes (read + write) per algorithmic byte of a decode launch, from the ncu capture summarised in
# profiles/decode_tc_kernel_r24_llama3_8b_32k_b8.md: (608.78 MB read + 3.38 MB written) / 608.70 MB.  Every
# unit is fetched once, so traffic scales with the units a launch processes.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = (608.780544e6 + 3.382016e6) / 608698368.0
# the same for INT4 factors (profiles/decode_tc_kernel_int4_r24_llama3_8b_32k_b8.md): (183.74 MB + 3.96 MB) / 182.46 MB
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE_INT4 = (183.737856e6 + 3.961344e6) / 182461440.0


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s)"


def _tensor_peak():
    """Dense bf16 tensor throughput in TFLOP/s (the burst figure: kernels here are timed in short regions)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops)"
    return 1590.0, "fallback (1.59 PFLOP/s)"


class ClockSampler:
    """Samples SM clocks and throttle reasons (read-only NVML queries from a thread; nvidia-smi if NVML cannot be
    loaded) while the timed region runs.  The sampler is started ahead of time, every sample is stamped, and the
    summary uses the samples that fell between begin() and end(): the timed region of a short workload lasts only
    tens of milliseconds."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        self.index, self.rows, self.proc, self.nvml = index, [], None, None
        self.t_begin = self.t_end = None
        self.stop_flag = False
        self.sm_max = None

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            return pynvml, pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            return pynvml, pynvml.nvmlDeviceGetHandleByIndex(self.index)

    def start(self):
        try:
            self.nvml, self.handle = self._nvml_handle()
            self.sm_max = float(self.nvml.nvmlDeviceGetMaxClockInfo(self.handle, self.nvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "10"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _poll(self):
        n = self.nvml
        masks = [n.nvmlClocksEventReasonHwSlowdown, n.nvmlClocksEventReasonHwThermalSlowdown,
                 n.nvmlClocksEventReasonSwThermalSlowdown, n.nvmlClocksEventReasonSwPowerCap]
        while not self.stop_flag:
            try:
                sm = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                why = n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                self.rows.append((time.perf_counter(), sm, [bool(why & m) for m in masks]))
            except Exception:
                pass
            time.sleep(0.002)

    def _read(self):
        for line in self.proc.stdout:
            r = [x.strip() for x in line.split(",")]
            if len(r) >= 6 and r[0].replace(".", "").isdigit():
                if r[1].replace(".", "").isdigit():
                    self.sm_max = float(r[1])
                self.rows.append((time.perf_counter(), float(r[0]), [r[2 + i].startswith("Active") for i in range(4)]))

    def median_mhz(self, spans):
        """Median SM clock of the samples stamped inside any of the (t0, t1) wall-clock spans, or None."""
        sm = [r[1] for r in list(self.rows) if any(t0 <= r[0] <= t1 for t0, t1 in spans)]
        return statistics.median(sm) if sm else None

    def begin(self):
        """Call right before the timed region (waits, briefly, until the sampler is alive)."""
        if self.nvml is not None or self.proc is not None:
            t0 = time.perf_counter()
            while not self.rows and time.perf_counter() - t0 < 2.0:
                time.sleep(0.002)
        self.t_begin = time.perf_counter()

    def end(self):
        self.t_end = time.perf_counter()

    def stop(self):
        if self.nvml is None and self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source (NVML, nvidia-smi) available"], "samples": 0}
        if self.t_end is None:
            self.end()
        time.sleep(0.02)
        self.stop_flag = True
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        t0 = self.t_begin if self.t_begin is not None else 0.0
        rows = list(self.rows)
        inside = [r for r in rows if t0 <= r[0] <= self.t_end + 0.005]
        note = None
        if not inside and rows:
            mid = 0.5 * (t0 + self.t_end)
            inside = sorted(rows, key=lambda r: abs(r[0] - mid))[:3]
            note = "no sample fell inside the timed region: the three nearest"
        sm = [r[1] for r in inside]
        reasons = sorted({self.NAMES[i] for r in inside for i in range(4) if r[2][i]})
        out = {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.sm_max, "reasons": reasons,
               "samples": len(sm), "source": "nvml" if self.nvml is not None else "nvidia-smi"}
        if note:
            out["note"] = note
        return out


def build_workload(w, rank, device, overlap=2, n_ctas=0, factor_bits=16, grow=0, keep_kv=False, plan_entries_per_seq=1,
                   decode_variant=0, global_rank=0):
    """Allocate the cache, generate each (layer, sequence) on the GPU, append and compress layer by layer.
    grow: tokens every sequence may still gain afterwards (sizes the pools and page tables); keep_kv: also
    return the generated K/V of layer 0 including those `grow` tokens (serving loop)."""
    import torch
    from paper_2608_23843_b200 import pkv, synth
    P = w.get("page", 64)
    if w["ragged"]:
        lengths = synth.loguniform_lengths(SEED, w["batch"], *w["T"])
    else:
        lengths = [w["T"]] * w["batch"]
    pages = [-(-(t + grow) // P) for t in lengths]
    n_sink, n_win = w["sink"] // P, w["recent"] // P
    n_factor = [max(0, (t + grow) // P - n_win - n_sink) for t in lengths]
    L = w["n_layers"]
    n_factor_slots = L * sum(n_factor) + 1
    # dense slots: what stays dense in every layer plus one layer's worth of transient pages
    n_dense_slots = sum(pages) + L * sum(p - f for p, f in zip(pages, n_factor)) + 8
    cfg = pkv.make_config(n_layers=L, n_kv_heads=w["n_kv_heads"], n_q_heads=w["n_q_heads"], rank=rank,
                          rank_v=w.get("rank_v", rank), page_size=P,
                          sink_tokens=w["sink"], recent_tokens=w["recent"], max_seqs=w["batch"] * plan_entries_per_seq,
                          max_pages_per_seq=max(pages), n_dense_slots=n_dense_slots, n_factor_slots=n_factor_slots,
                          decode_overlap=overlap, n_ctas=n_ctas, factor_bits=factor_bits,
                          decode_variant=decode_variant, global_rank=global_rank)
    cache = pkv.Cache(cfg, device, synth.slot_permutation(SEED, n_dense_slots, 0).tolist(),
                      synth.slot_permutation(SEED, n_factor_slots, 1).tolist())
    ids = list(range(w["batch"]))
    svd_ms, n_svds = 0.0, 0
    kept = []
    spans = []                                            # wall-clock spans of the compression calls (for the clock samples)
    for layer in range(L):
        for s in ids:
            k, v = synth.make_kv(SEED, layer, s, lengths[s] + grow, w["n_kv_heads"], 128, P, device, w["outliers"])
            cache.append_kv(layer, [s], [lengths[s]], k[:lengths[s]], v[:lengths[s]])
            if keep_kv and layer == 0:
                kept.append((k[lengths[s]:].clone(), v[lengths[s]:].clone()))
            del k, v
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0.record()
        n = cache.compress_eligible_pages(layer)
        e1.record()
        torch.cuda.synchronize()
        spans.append((t0, time.perf_counter()))
        svd_ms += e0.elapsed_time(e1)
        n_svds += n * w["n_kv_heads"] * 2
    st = cache.stats()
    comp = dict(pages_per_s=(n_svds / (svd_ms * 1e-3) if svd_ms > 0 else None), n_page_svds=n_svds, svd_ms=svd_ms,
                spans=spans, jacobi_rounds=st["jacobi_rounds"], page_svds_counted=st["page_svds"],
                not_converged=st["page_svds_not_converged"], page=P, rank=rank, rank_v=w.get("rank_v", rank),
                global_rank=global_rank)
    if keep_kv:
        comp["new_k"] = torch.stack([k for k, _ in kept], 1).contiguous()      # [grow][batch][H_kv][d]
        comp["new_v"] = torch.stack([v for _, v in kept], 1).contiguous()
    return cfg, cache, lengths, comp


N_SMS, FP32_LANES_PER_SM = 148, 128


def hbm_roofline(kernel, bytes_per_launch, launch_us, factor_bits):
    """Roofline record of the decode kernel (bound: HBM).  achieved = algorithmic bytes per launch / average launch
    duration.  The peak is the measured copy bandwidth: a STREAM-style copy reads and writes, this kernel only
    reads, so a fraction a little above 1 is possible and is flagged; `frac_of_8tbs` is the same figure against the
    nominal 8 TB/s.  `traffic` scales the DRAM bytes ncu counted on the llama3_8b_32k_b8 launch (every unit is read
    once, so traffic grows with the units processed); it is not a capture of this workload."""
    peak, peak_src = _peaks()
    achieved = bytes_per_launch / (launch_us * 1e-6) / 1e9
    ratio = NCU_TRAFFIC_PER_ALGORITHMIC_BYTE_INT4 if factor_bits == 4 else NCU_TRAFFIC_PER_ALGORITHMIC_BYTE
    rec = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
           "frac_of_8tbs": achieved / 8000.0, "peak_source": peak_src,
           "peak_kind": "read+write copy bandwidth (not an upper bound for a read-only stream)",
           "traffic": bytes_per_launch * ratio,
           "traffic_source": "ncu dram__bytes_read+write of this kernel captured on the llama3_8b_32k_b8 launch "
                             "(%.4f DRAM bytes per algorithmic byte), scaled by this launch's algorithmic bytes" % ratio,
           "launch_us": launch_us, "algorithmic_bytes_per_launch": bytes_per_launch}
    if rec["frac"] > 1.0:
        rec["note"] = "above 1.0 of the copy-based peak: the kernel reads only; see frac_of_8tbs"
    return rec


def compress_record(comp, sampler):
    """Throughput of the page-SVD kernel against the bound that applies to it: plain fp32 FMAs (the Gram matrix and
    the projection are 7 % of the work; the rest is 4 x 4 rotations in shared memory, no tensor-core shape).
    Flops per page SVD, counted from what the algorithm needs with the measured number of rotation rounds:
      Gram matrix, one triangle      P^2 d
      per round, page size 64 / 32   16 P^2   (G' = M^T G M on one triangle: 8 P^2; Q^T' = M^T Q^T: 8 P^2)
      per round, page size 16        8 P^2    (2 x 2 rotations)
      B = A^T X                      2 r P d
    Peak = SMs x 128 FMA lanes x 2 x SM clock sampled while the kernel ran (the maximum clock if no sample fell
    inside)."""
    n = comp["page_svds_counted"]
    if not n or not comp["pages_per_s"] or comp.get("global_rank"):
        return None
    P, d = comp["page"], 128
    rounds = comp["jacobi_rounds"] / n
    per_sweep = {64: 21, 32: 13, 16: 15}[P]
    per_round = (16 if P >= 32 else 8) * P * P
    r_mean = 0.5 * (comp["rank"] + comp["rank_v"])
    flops = P * P * d + rounds * per_round + 2 * r_mean * P * d
    mhz = sampler.median_mhz(comp["spans"]) if sampler is not None else None
    clock_src = "sampled during the compression launches"
    if mhz is None:
        mhz, clock_src = (sampler.sm_max if sampler is not None and sampler.sm_max else 1965.0), "maximum SM clock (no sample fell inside)"
    peak = N_SMS * FP32_LANES_PER_SM * 2 * mhz * 1e6 / 1e12
    achieved = comp["pages_per_s"] * flops / 1e12
    return {"pages_per_s": comp["pages_per_s"], "page_svds": n, "rounds_per_page": rounds,
            "sweeps_per_page": rounds / per_sweep, "not_converged": comp["not_converged"],
            "flops_per_page": flops, "bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
            "frac": achieved / peak, "sm_mhz": mhz, "clock_source": clock_src,
            "peak_source": "148 SMs x 128 fp32 FMA lanes x 2 x SM clock"}


def run_serving(args, w, rank, device, world, rk, local):
    """Serving loop: `steps` iterations of append (one token per sequence) -> decode -> compress on one
    layer, timed as a whole and call by call with CUDA events on the launching stream."""
    import torch
    from paper_2608_23843_b200 import synth
    B, Hq, P = w["batch"], w["n_q_heads"], w.get("page", 64)
    warm = max(3, args.warmup)
    total = warm + 2 * args.steps + 3           # device-resident pass, host-buffer pass, warm-ups
    sampler = ClockSampler(local)
    sampler.start()                                       # ahead of the cache build: its compression launches are sampled too
    cfg, cache, lengths, comp = build_workload(w, rank, device, 0, args.n_ctas, args.factor_bits, grow=total, keep_kv=True)
    ids = list(range(B))
    new_k, new_v = comp["new_k"], comp["new_v"]
    qs = [synth.make_q(SEED, 0, t, B, Hq, 128, device) for t in range(8)]
    out = torch.empty_like(qs[0])
    cursor = [0]
    events = []

    side = torch.cuda.Stream() if args.two_step > 0 else None
    begun_at = [None]

    def compress_step(t):
        """One-step: factorize what left the window now, on this stream.  Two-step (--two-step K): start it on a side
        stream and make the pages factor pages K steps later (they stay dense, and readable, meanwhile)."""
        if side is None:
            return cache.compress_eligible_pages(0)
        if begun_at[0] is not None and t - begun_at[0] >= args.two_step:
            cache.compress_commit(0)
            begun_at[0] = None
        n = 0
        if begun_at[0] is None:
            n = cache.compress_begin(0, side)
            if n:
                begun_at[0] = t
        return n

    def step(record):
        t = cursor[0]
        cursor[0] += 1
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if record else None
        if record:
            ev[0].record()
        cache.append_kv(0, ids, [1] * B, new_k[t], new_v[t])
        if record:
            ev[1].record()
        cache.decode_attention(0, ids, qs[t % 8], out)
        if record:
            ev[2].record()
        n = compress_step(t)
        if record:
            ev[3].record()
            events.append((ev, n))

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warm):
        step(False)
    cache.decode_attention(0, ids, qs[0], out)
    bytes_per_step = cache.stats()["last_decode_bytes"]
    barrier()
    sampler.begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step(True)
    e1.record()
    barrier()
    sampler.end()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    app = [ev[0].elapsed_time(ev[1]) * 1e3 for ev, _ in events]
    att = [ev[1].elapsed_time(ev[2]) * 1e3 for ev, _ in events]
    cmp_all = [(ev[2].elapsed_time(ev[3]) * 1e3, n) for ev, n in events]
    cmp_event = [(us, n) for us, n in cmp_all if n > 0]

    def pct(xs, p):
        xs = sorted(xs)
        return xs[min(len(xs) - 1, int(p * len(xs)))] if xs else None

    # end to end: the step's new K/V rows and q come from pinned host memory, the result goes back to it
    hk, hv = new_k.cpu().pin_memory(), new_v.cpu().pin_memory()
    hq = [q.cpu().pin_memory() for q in qs]
    hout = torch.empty_like(hq[0]).pin_memory()
    dk, dv = torch.empty_like(new_k[0]), torch.empty_like(new_v[0])
    q_stage, out_stage = torch.empty_like(qs[0]), torch.empty_like(qs[0])

    def step_host():
        t = cursor[0]
        cursor[0] += 1
        dk.copy_(hk[t], non_blocking=True)
        dv.copy_(hv[t], non_blocking=True)
        cache.append_kv(0, ids, [1] * B, dk, dv)
        cache.decode_attention_host(0, ids, hq[t % 8], hout, q_stage, out_stage)
        compress_step(t)
        torch.cuda.current_stream().synchronize()

    for _ in range(3):
        step_host()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step_host()
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / args.steps
    st = cache.stats()
    if st["device_timeouts"] or st["bad_slot_indices"] or out.float().isnan().any().item():
        raise SystemExit("decode produced timeouts or NaNs: %r" % st)
    att_mean = statistics.mean(att)
    ms, e2e_ms, att_mean = max_over_ranks([ms, e2e_ms, att_mean], world, device)
    if rk == 0:
        n_event_svds = sum(n for _, n in cmp_event) * w["n_kv_heads"] * 2
        step_bytes = 2 * B * w["n_kv_heads"] * 128 * 2 + 2 * B * Hq * 128 * 2
        line = {
            "metric": "decode_us_per_step", "value": ms * 1e3, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": dict(_config_dict(args, w, rank),
                step="append (1 token per sequence) + decode + compress_eligible on one layer" if args.two_step <= 0 else
                     "append (1 token per sequence) + decode + compress_commit %d steps after compress_begin on a side stream" % args.two_step,
                overlap="0"),
            "append_us": {"mean": statistics.mean(app), "p99": pct(app, 0.99)},
            "attention_us": {"mean": statistics.mean(att), "p99": pct(att, 0.99)},
            "compress_us": {"mean_no_event": statistics.mean([us for us, n in cmp_all if n == 0] or [0.0]),
                            "mean_event": statistics.mean([us for us, _ in cmp_event]) if cmp_event else None,
                            "event_steps": len(cmp_event),
                            "pages_per_s_event": (n_event_svds / (sum(us for us, _ in cmp_event) * 1e-6)) if cmp_event else None},
            "step_us_p99": pct([a + b + c for a, b, (c, _) in zip(app, att, cmp_all)], 0.99),
            "algorithmic_bytes_per_step": bytes_per_step,
            "pages_factorized_per_s": comp["pages_per_s"], "page_svds_timed": comp["n_page_svds"],
            "compress": compress_record(comp, sampler),
            "roofline": hbm_roofline("decode_tc_kernel<P=%d, rank tiles=%d>" % (P, (rank + 7) // 8), bytes_per_step,
                                     att_mean, args.factor_bits),
            "e2e": {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": step_bytes - B * Hq * 128 * 2,
                    "d2h_bytes_per_step": B * Hq * 128 * 2},
            "gpu_launches": args.steps * 2 + len(cmp_event), "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            o = oracle_sample(w, rank, 3, args.factor_bits)
            line["cpu_baseline"] = {"value": o["decode_s"] * 1e6 * o["slices_per_step"], "unit": "us",
                                    "cores": o["cores"], "kind": "oracle", "sample": o["sample"] + " (attention only)",
                                    "pages_per_s": o["pages_per_s"]}
        print(json.dumps(line))
    cache.close()


def oracle_sample(w, rank, steps, factor_bits=16):
    """The fp64 oracle, as it stands, on one (layer 0, KV head 0) slice of sequence 0: page SVDs and
    one decode call for the G query heads of that KV head.  Returns seconds per decode and pages/s."""
    import torch
    from oracle import svd as osvd
    from oracle.cache import OracleCache, OracleConfig
    from paper_2608_23843_b200 import synth
    G = w["n_q_heads"] // w["n_kv_heads"]
    T = synth.loguniform_lengths(SEED, w["batch"], *w["T"])[0] if w["ragged"] else w["T"]
    P = w.get("page", 64)
    k, v = synth.make_kv(SEED, 0, 0, T, w["n_kv_heads"], 128, P, "cpu", w["outliers"])
    k, v = k[:, :1].to(torch.float64).numpy(), v[:, :1].to(torch.float64).numpy()
    n_pages = -(-T // P)
    orc = OracleCache(OracleConfig(n_layers=1, n_kv_heads=1, n_q_heads=G, head_dim=128, page_size=P, rank_k=rank,
                                   rank_v=w.get("rank_v", rank), sink_tokens=w["sink"], recent_tokens=w["recent"], max_seqs=1,
                                   n_dense_slots=n_pages, n_factor_slots=n_pages, factor_bits=factor_bits))
    orc.append_kv(0, [0], [T], k, v)
    t0 = time.perf_counter()
    n = orc.compress_eligible_pages(0)
    t_svd = time.perf_counter() - t0
    q = synth.make_q(SEED, 0, 0, 1, w["n_q_heads"], 128)[:, :G].to(torch.float64).numpy()
    times = []
    for _ in range(max(1, steps)):
        t0 = time.perf_counter()
        orc.decode_attention(0, [0], q)
        times.append(time.perf_counter() - t0)
    slices_per_step = w.get("layers_per_step", w["n_layers"]) * w["n_kv_heads"] * w["batch"]
    return dict(decode_s=statistics.median(times), slices_per_step=slices_per_step,
                pages_per_s=(2 * n / t_svd if t_svd > 0 else None), cores=osvd.n_threads(), T=T,
                sample="sequence 0, layer 0, KV head 0 (1/%d of a step): %d page SVDs + %d-head decode over %d tokens; "
                       "us/step extrapolated linearly in slices" % (slices_per_step, 2 * n, G, T))


def run_reference(args, w, rank):
    rank0 = int(os.environ.get("RANK", "0")) == 0
    if os.environ.get("PKV_BENCH_RANK_MARKER"):           # lets a test see that every rank was started
        print("rank %s of %s present" % (os.environ.get("RANK", "0"), os.environ.get("WORLD_SIZE", "1")), file=sys.stderr)
    if not rank0:
        return
    o = oracle_sample(w, rank, args.steps + args.warmup, args.factor_bits)
    us = o["decode_s"] * 1e6 * o["slices_per_step"]
    line = {"impl": "reference", "metric": "decode_us_per_step", "value": us, "unit": "us", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": _config_dict(args, w, rank),
            "cpu_baseline": {"value": us, "unit": "us", "cores": o["cores"], "kind": "oracle", "sample": o["sample"],
                             "pages_per_s": o["pages_per_s"]},
            "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def _config_dict(args, w, rank):
    return {"workload": args.workload, "n_layers": w["n_layers"], "layers_per_step": w.get("layers_per_step", w["n_layers"]), "n_q_heads": w["n_q_heads"],
            "n_kv_heads": w["n_kv_heads"], "head_dim": 128, "batch": w["batch"], "context": w["T"],
            "queries_per_sequence": args.q_len,
            "page_size": w.get("page", 64), "rank": rank, "rank_v": w.get("rank_v", rank), "factor_bits": args.factor_bits,
            "global_rank": getattr(args, "global_rank", 0), "sink_tokens": w["sink"], "recent_tokens": w["recent"],
            "l2": "inputs larger than L2 (no flush)" if args.workload != "tiny" else "L2-resident (latency only)",
            "overlap": ["0: each launch waits for the previous one",
                        "1: consecutive per-layer launches overlap (programmatic dependent launch) and complete in order",
                        "2: per-layer launches overlap freely (programmatic dependent launch, rotating split-K scratch, "
                        "a draining launch every 63); valid here because queries are prepared in advance and no "
                        "launch in the step writes the cache"][args.overlap],
            "launch": "one CUDA graph replay per step (%d per-layer launches)" % w.get("layers_per_step", w["n_layers"]) if args.graph else "host launch per layer",
            "parallelism": ("sequence-sharded x%d (per layer: local softmax states, all-gather, Eq. 5 merge)" % args.gpus
                            if getattr(args, "seq_sharded", False) else "replicas x%d" % args.gpus)}


def max_over_ranks(values, world, device="cpu"):
    """Element-wise max of a list of floats over all ranks (identity when world == 1)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def row_block_flops(w, rank, lengths, q_len):
    """Algorithmic FLOPs of one pkv_decode_attention_multi launch served by a row-block kernel: query rows x (factor
    pages x 2 (d r_k + r_k P + P r_v + r_v d) + dense tokens x 4 d); the causal triangle among the new positions is
    counted in full."""
    P_, rv_ = w.get("page", 64), w.get("rank_v", rank)
    flops = 0
    for T_ in lengths:
        nf_ = max(0, T_ // P_ - w["recent"] // P_ - w["sink"] // P_)
        flops += q_len * w["n_q_heads"] * (nf_ * 2 * (128 * rank + rank * P_ + P_ * rv_ + rv_ * 128) + (T_ - nf_ * P_) * 4 * 128)
    return flops


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="qwen3_32b_128k", choices=sorted(WORKLOADS))
    ap.add_argument("--rank", type=int, default=0, help="override the workload's rank (8, 16, 24, 32)")
    ap.add_argument("--impl", default="pkv", choices=["pkv", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-standalone", action="store_true",
                    help="skip the second measurement with decode_overlap = 0 (the `standalone` record)")
    ap.add_argument("--overlap", type=int, default=2, choices=[0, 1, 2],
                    help="decode_overlap mode of the cache: 0 = every launch waits for the previous one, 1 = launches "
                         "overlap but complete in order, 2 = launches never wait for one another (default)")
    ap.add_argument("--n-ctas", type=int, default=0, help="decode grid size (0 = library default)")
    ap.add_argument("--factor-bits", type=int, default=16, choices=[4, 16], help="factor storage: bf16 or INT4 (paper, Section 4.3)")
    ap.add_argument("--global-rank", type=int, default=0, choices=[0, 64, 80, 96],
                    help="the Global SVD form the paper compares with (Section 4.2): one basis of this rank per (sequence, layer, "
                         "KV head) instead of page-wise factors")
    ap.add_argument("--q-len", type=int, default=1,
                    help="queries per sequence and step (1 = decoding; more = a speculative-decoding or chunked-prefill step "
                         "over the newest positions, pkv_decode_attention_multi)")
    ap.add_argument("--two-step", type=int, default=0,
                    help="serving loop only: factorize on a side stream (pkv_compress_begin) and commit K steps later, "
                         "instead of the one-step call inside the step")
    ap.add_argument("--seq-sharded", action="store_true",
                    help="strong scaling of one step: every rank's cache holds 1/N of each sequence's tokens (rank 0 the "
                         "sink, the last rank the dense window); per layer each rank computes its softmax state, the states "
                         "are all-gathered (NCCL) and merged by Eq. 5.  Not the default: the driver's scaling runs are replicas")
    ap.add_argument("--decode-variant", type=int, default=0, choices=[0, 2, 3],
                    help="2 = pkv_decode_attention_multi never uses its row-block kernels; 3 = its row-block kernel is the mma.sync one (comparisons)")
    ap.add_argument("--graph", action="store_true",
                    help="replay one CUDA graph per step instead of launching every layer from the host")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # launched plainly: start one rank per GPU ourselves (what the torchrun command line would do)
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    w = WORKLOADS[args.workload]
    rank = args.rank or w["rank"]
    if args.impl == "reference":
        if args.q_len != 1:
            raise SystemExit("--impl reference times the single-query path only")
        run_reference(args, w, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2608_23843_b200 import pkv, synth
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rk = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
        print("bench.py: rank %d of %d on cuda:%d (%s)" % (rk, world, local, torch.cuda.get_device_name(local)), file=sys.stderr)
    pkv.lib()                                             # fail loudly if the CUDA library is missing

    if w.get("serving"):
        run_serving(args, w, rank, device, world, rk, local)
        if world > 1:
            dist.destroy_process_group()
        return
    if args.seq_sharded:
        if w["ragged"] or w.get("serving") or args.q_len != 1 or args.graph or w["T"] % (w.get("page", 64) * world):
            raise SystemExit("--seq-sharded needs a uniform, non-serving workload whose context divides into whole pages per rank")
        w = dict(w, T=w["T"] // world, sink=w["sink"] if rk == 0 else 0, recent=w["recent"] if rk == world - 1 else 0)
    QL = args.q_len
    per_tile = max(1, min(QL, 8 // (w["n_q_heads"] // w["n_kv_heads"])))
    sampler = ClockSampler(local)
    sampler.start()                                       # ahead of the cache build: its compression launches are sampled too
    cfg, cache, lengths, comp = build_workload(w, rank, device, args.overlap, args.n_ctas, args.factor_bits,
                                               plan_entries_per_seq=-(-QL // per_tile), decode_variant=args.decode_variant,
                                               global_rank=args.global_rank)
    ids = list(range(w["batch"]))
    L, Hq = w["n_layers"], w["n_q_heads"]
    if QL == 1:
        qs = [synth.make_q(SEED, layer, 0, w["batch"], Hq, 128, device) for layer in range(L)]
    else:
        if QL > w["recent"] or w.get("serving") or args.graph:
            raise SystemExit("--q-len must not exceed the workload's dense window; not with the serving loop or --graph")
        qs = [synth.make_q(SEED, layer, 0, w["batch"] * QL, Hq, 128, device).view(w["batch"], QL, Hq, 128) for layer in range(L)]
    outs = [torch.empty_like(q) for q in qs]

    if args.seq_sharded:
        from paper_2608_23843_b200 import sharded
        sh_state = [torch.empty((w["batch"], Hq, 130), dtype=torch.float32, device=device) for _ in range(L)]
        sh_all = [torch.empty((world, w["batch"], Hq, 130), dtype=torch.float32, device=device) for _ in range(L)]

    def attend(layer, q, out):
        if args.seq_sharded:
            sharded.sequence_sharded_decode(cache, layer, ids, q, out, state=sh_state[layer], gathered=sh_all[layer])
        elif QL == 1:
            cache.decode_attention(layer, ids, q, out)
        else:
            cache.decode_attention_multi(layer, ids, QL, q, out)

    lps = w.get("layers_per_step", L)
    cursor = [0]

    def step():
        for _ in range(lps):
            layer = cursor[0] % L
            cursor[0] += 1
            attend(layer, qs[layer], outs[layer])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    eager_step = step
    if args.graph:
        # one CUDA graph of the step's per-layer launches (plans are cached on the device, so the
        # captured launches read current page tables and token counts at replay time)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            step()
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        step = graph.replay
        for _ in range(3):
            step()
    bytes_per_step = 0
    for layer in range(lps):                              # algorithmic bytes, from the library's own accounting
        attend(layer, qs[layer], outs[layer])
        bytes_per_step += cache.stats()["last_decode_bytes"]
    barrier()
    sampler.begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    sampler.end()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    # average duration of one decode-kernel launch over the timed region: the region holds nothing but
    # steps * L back-to-back launches of that kernel, so this includes the gaps between launches
    launch_ms = ms / lps

    # end to end: queries and results in pinned host memory, copies inside the timed region
    q_host = [q.cpu().pin_memory() for q in qs]
    out_host = [torch.empty_like(q).pin_memory() for q in q_host]
    q_stage, out_stage = torch.empty_like(qs[0]), torch.empty_like(qs[0])

    def step_host():
        for _ in range(lps):
            layer = cursor[0] % L
            cursor[0] += 1
            if QL == 1 and not args.seq_sharded:
                cache.decode_attention_host(layer, ids, q_host[layer], out_host[layer], q_stage, out_stage)
            else:                                         # no host-buffer variant of the multi-query call: copy around it
                q_stage.copy_(q_host[layer], non_blocking=True)
                attend(layer, q_stage, out_stage)
                out_host[layer].copy_(out_stage, non_blocking=True)
        torch.cuda.current_stream().synchronize()        # the caller reads the result on the host

    for _ in range(3):
        step_host()
    barrier()
    t0 = time.perf_counter()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record()
    for _ in range(args.steps):
        step_host()
    h1.record()
    barrier()
    e2e_ms = max(h0.elapsed_time(h1), (time.perf_counter() - t0) * 1e3) / args.steps
    st = cache.stats()
    if st["device_timeouts"] or st["bad_slot_indices"] or (outs[0].float().isnan().any().item()):
        raise SystemExit("decode produced timeouts or NaNs: %r" % st)

    # Several new positions per sequence on the same cache (pkv_decode_attention_multi, served by the tcgen05 row-block
    # kernel): a sub-record of the default line, so that one run also carries the tensor-bound kernel's figure.
    multi = None
    MQ = 64
    if (QL == 1 and not args.seq_sharded and not args.graph and not args.no_standalone and not args.global_rank
            and args.factor_bits == 16 and args.decode_variant == 0 and not w["ragged"] and w["recent"] >= MQ
            and MQ * (Hq // w["n_kv_heads"]) >= 64 and min(lengths) > w["recent"] + w["sink"]):
        mq_q = [synth.make_q(SEED + 1, layer, 0, w["batch"] * MQ, Hq, 128, device).view(w["batch"], MQ, Hq, 128) for layer in range(min(L, 2))]
        mq_out = torch.empty_like(mq_q[0])
        mq_steps = max(2, min(args.steps, 5))

        def mq_step():
            for layer in range(lps):
                cache.decode_attention_multi(layer % L, ids, MQ, mq_q[layer % len(mq_q)], mq_out)
        for _ in range(3):
            mq_step()
        barrier()
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m0.record()
        for _ in range(mq_steps):
            mq_step()
        m1.record()
        barrier()
        mq_ms = m0.elapsed_time(m1) / mq_steps
        st = cache.stats()
        if st["device_timeouts"] or st["bad_slot_indices"] or mq_out.float().isnan().any().item():
            raise SystemExit("multi-query decode produced timeouts or NaNs: %r" % st)
        multi = (mq_ms, mq_steps)

    # The same step with every launch standing alone (decode_overlap = 0: a launch starts computing only when the
    # kernel before it has finished, as in a decoder whose queries come from the layer before): a second cache of
    # the same workload, timed the same way in this run.
    standalone_ms = None
    if args.overlap != 0 and QL == 1 and not args.seq_sharded and not args.graph and not args.no_standalone:
        cache.close()
        cache = None
        torch.cuda.empty_cache()
        _, cache, _, _ = build_workload(w, rank, device, 0, args.n_ctas, args.factor_bits, decode_variant=args.decode_variant,
                                        global_rank=args.global_rank)
        for _ in range(max(3, args.warmup)):
            eager_step()
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(args.steps):
            eager_step()
        s1.record()
        barrier()
        standalone_ms = s0.elapsed_time(s1) / args.steps
        st = cache.stats()
        if st["device_timeouts"] or st["bad_slot_indices"]:
            raise SystemExit("decode produced timeouts: %r" % st)

    ms, e2e_ms, launch_ms = max_over_ranks([ms, e2e_ms, launch_ms], world, device)
    if standalone_ms is not None:
        standalone_ms = max_over_ranks([standalone_ms], world, device)[0]
    if multi is not None:
        multi = (max_over_ranks([multi[0]], world, device)[0], multi[1])

    if rk == 0:
        bytes_per_launch = bytes_per_step / lps
        qbytes = sum(q.numel() * 2 for q in qs[:lps])
        line = {
            "metric": "decode_us_per_step", "value": ms * 1e3, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": False,
            "scaling": "strong" if args.seq_sharded else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": _config_dict(args, w, rank),
            "hbm_gbs": bytes_per_step / (ms * 1e-3) / 1e9 * world,
            "frac_of_8tbs": bytes_per_step / (ms * 1e-3) / 8e12,
            "algorithmic_bytes_per_step": bytes_per_step,
            "pages_factorized_per_s": comp["pages_per_s"], "page_svds_timed": comp["n_page_svds"],
            "compress": compress_record(comp, sampler),
            "roofline": hbm_roofline("decode_tc_kernel<P=%d, rank tiles=%d%s>" % (w.get("page", 64), ((args.global_rank or rank) + 7) // 8,
                                                                                 ", Global SVD form" if args.global_rank else ""),
                                     bytes_per_launch, launch_ms * 1e3, args.factor_bits),
            "e2e": {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": qbytes, "d2h_bytes_per_step": qbytes},
            "gpu_launches": lps * args.steps * (2 if args.seq_sharded else 1), "clocks": clocks,
        }
        if standalone_ms is not None:
            r0 = hbm_roofline(line["roofline"]["kernel"], bytes_per_launch, standalone_ms * 1e3 / lps, args.factor_bits)
            line["standalone"] = {"mode": "decode_overlap=0: each launch waits for the kernel before it before it reads q "
                                          "or writes anything (cache pages are prefetched into shared memory meanwhile)",
                                  "value": standalone_ms * 1e3, "unit": "us", "steps": args.steps,
                                  "hbm_gbs": bytes_per_step / (standalone_ms * 1e-3) / 1e9 * world,
                                  "frac_of_8tbs": r0["frac_of_8tbs"], "frac": r0["frac"], "launch_us": r0["launch_us"],
                                  "gpu_launches": lps * args.steps}
        if multi is not None:
            mq_ms = multi[0]
            fl = row_block_flops(w, rank, lengths, MQ)
            tpeak, tsrc = _tensor_peak()
            n_blocks = w["batch"] * w["n_kv_heads"] * -(-(MQ * (Hq // w["n_kv_heads"])) // 128)
            ns = pkv.pkv_get_row_block_ranges(n_blocks, max(lengths), w.get("page", 64),
                                              torch.cuda.get_device_properties(device).multi_processor_count)
            tach = fl * lps / (mq_ms * 1e-3) / 1e12
            line["multi_query"] = {"queries_per_sequence": MQ, "value": mq_ms * 1e3, "unit": "us", "steps": multi[1],
                                   "launch_us": mq_ms * 1e3 / lps, "bound": "tensor", "achieved": tach, "peak": tpeak,
                                   "frac": tach / tpeak, "peak_source": tsrc, "kernel_unit": "TFLOP/s",
                                   "kernel": "block_umma_kernel (tcgen05, 128 query rows per CTA) + rowblock_merge_kernel"
                                             if ns >= 2 else "block_umma_kernel (tcgen05, 128 query rows per CTA)",
                                   "row_blocks": n_blocks, "token_ranges_per_row_block": ns,
                                   "algorithmic_flops_per_launch": fl,
                                   "gpu_launches": lps * multi[1] * (2 if ns >= 2 else 1)}
        P_, Gq = w.get("page", 64), Hq // w["n_kv_heads"]
        rows = QL * Gq
        rv_ = w.get("rank_v", rank)
        # the library's own rule (row_block_umma_supported): the tcgen05 kernel for bf16 factors unless decode_variant 3
        # pins the mma.sync kernel
        umma = args.decode_variant == 0
        # (and its rule for the route: row blocks from 64 query rows per KV head on; the mma.sync kernel only if they fill the GPU)
        if QL > 1 and args.decode_variant in (0, 3) and args.factor_bits != 4 and rows >= 64 and (
                umma or w["batch"] * w["n_kv_heads"] * -(-rows // 64) >= 128):
            # Served by the row-block kernel, whose bound is the tensor pipe, not HBM.
            flops = row_block_flops(w, rank, lengths, QL)
            tpeak, tsrc = _tensor_peak()
            tach = flops / (launch_ms * 1e-3) / 1e12
            line["roofline"] = {"bound": "tensor",
                                "kernel": (("block_umma_kernel<P=%d, rank tiles=%%d> (tcgen05, 128 query rows per CTA)" % P_) if umma else
                                           "block_tc_kernel<P=%d, rank tiles=%%d> (mma.sync, 64 query rows per CTA)" % P_) % ((rank + 7) // 8),
                                "achieved": tach, "peak": tpeak, "unit": "TFLOP/s", "frac": tach / tpeak,
                                "peak_source": tsrc + ("; the products are small (N = 32 to 128 per instruction, four dependent products per "
                                                       "page through the row threads): ncu shows the tensor pipe about 30 % busy" if umma else
                                                       "; ncu showed the mma.sync pipe 50 % busy at this rate"),
                                "traffic": None, "launch_us": launch_ms * 1e3, "algorithmic_flops_per_launch": flops}
            if umma:
                # (row blocks cut into token ranges: a second, merging launch follows)
                n_blocks = w["batch"] * w["n_kv_heads"] * -(-rows // 128)
                sms = torch.cuda.get_device_properties(device).multi_processor_count
                ns = pkv.pkv_get_row_block_ranges(n_blocks, max(lengths), P_, sms)
                line["roofline"]["token_ranges_per_row_block"] = ns
                if ns >= 2:
                    line["gpu_launches"] *= 2
        if not args.no_cpu_baseline and world == 1 and QL == 1 and not args.global_rank:
            o = oracle_sample(w, rank, 3, args.factor_bits)
            line["cpu_baseline"] = {"value": o["decode_s"] * 1e6 * o["slices_per_step"], "unit": "us",
                                    "cores": o["cores"], "kind": "oracle", "sample": o["sample"],
                                    "pages_per_s": o["pages_per_s"]}
        print(json.dumps(line))
    cache.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
