#!/usr/bin/env python
"""Benchmark of the H1B-KV decode hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: append
the new token's K/V to every layer's compressed cache (Eq. 2, Eq. 4), then decode
attention over every layer's cache (Eq. 3, Eq. 5). Workload at 1 GPU: the 7B
shape (32 layers x 32 heads, d = 128, m = 128), one sequence, 8192-token context.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0). With N > 1 (launched by torch.distributed.run)
every rank runs its own sequence on its own GPU: independent units, no
collective on the data path, weak scaling.

`--impl reference` times the fp64 CPU oracle, as it stands, on the host cores,
on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode-attn tokens/s (7B shape, 8k ctx): append 1 token + decode attention over 32 layers"
UNIT = "tokens/s"
INV_TAU = 16.0
# DRAM traffic of one decode_split_kernel launch (dram__bytes_read.sum + dram__bytes_write.sum, one ncu capture)
# per algorithmic byte: 817.9 MB moved for 805.9 MB needed at 8198 cached tokens of the default workload. Traffic
# grows in proportion to the cached tokens, so the bench scales it to the context it actually ran; the line says
# where the ratio was taken (`traffic_ratio_measured_at`), so that a stale one shows.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.0148
NCU_TRAFFIC_MEASURED_AT = {"workload": "c2_7b_8k", "tokens": 8198, "dram_bytes": 817.87e6, "algorithmic_bytes": 805.93e6,
                           "kernel": "decode_split_kernel<4,1,4,0,0>"}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) while a region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(get(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                break
            time.sleep(0.002)

    def mark(self):
        """The timed region starts here: samples taken before it (warm-up, also under load) are kept apart."""
        self.marked_at = len(self.samples)

    def stop(self, ms_per_step=None):
        self._stop_evt.set()
        if self.ident is not None:                  # started
            self.join(timeout=2)
        at = getattr(self, "marked_at", 0)
        timed = self.samples[at:] or self.samples   # a very short timed region may have caught no sample of its own
        med = float(np.median(timed)) if timed else None
        out = {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
               "samples": len(self.samples), "samples_in_timed_region": len(self.samples) - at}
        if med is not None and ms_per_step is not None:
            out["ms_per_step_x_sm_mhz"] = ms_per_step * med     # clock-normalised time: comparable from box to box
        return out


def gpu_index() -> int:
    """Physical index of the device this rank uses (for NVML)."""
    local = int(os.environ.get("LOCAL_RANK", "0"))
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        ids = [x for x in vis.split(",") if x.strip()]
        try:
            return int(ids[local])
        except Exception:
            return local
    return local


# --------------------------------------------------------------------------- ours
def run_ours(args):
    import torch

    import h1b_synth
    from paper_2510_05529_b200 import binding

    from paper_2510_05529_b200 import dist as pdist
    rank, world, local = pdist.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    pdist.init("nccl", torch.device("cuda", local))
    dev = torch.device("cuda", local)
    w = h1b_synth.WORKLOADS[args.workload]
    if args.sketch_bits or args.group_size:           # the paper's ablation axes (Table V) as throughput variants
        w = h1b_synth.scaled(w, sketch_bits=args.sketch_bits or w.sketch_bits, group_size=args.group_size or w.group_size,
                             name="%s[m=%d,G=%d]" % (w.name, args.sketch_bits or w.sketch_bits, args.group_size or w.group_size))
    if args.fp16_values:                              # Table V's "1-bit keys only" row: values stay fp16
        w = h1b_synth.scaled(w, name=w.name + "[fp16 values]")
    if args.q_heads or args.kv_heads:                 # another head-group shape on the same workload (variant)
        w = h1b_synth.scaled(w, n_q_heads=args.q_heads or w.n_q_heads, n_kv_heads=args.kv_heads or w.n_kv_heads,
                             name="%s[%d/%d heads]" % (w.name, args.q_heads or w.n_q_heads, args.kv_heads or w.n_kv_heads))
    if args.layers:                                   # fewer layers of the same shape: small enough for a profiler capture
        w = h1b_synth.scaled(w, n_layers=args.layers, name="%s[%d layers]" % (w.name, args.layers))
    if args.rope:                                     # rotary embedding fused into the append and the query sketch
        w = h1b_synth.scaled(w, name=w.name + "[rope]")
    if args.workload == "c5_prefill":
        return run_prefill(args, w, pdist, rank, world, local)
    # --shard heads: the ranks split the KV heads (and their query heads) of the SAME sequences between them: every
    # (layer, sequence, KV head) is independent, so there is still no collective on the data path; the job then
    # produces w.batch tokens per step however many ranks there are (strong scaling). Every rank draws the inputs
    # of the whole model from the same seeds and keeps its own heads' slice.
    shard = None
    w_full = w
    if args.shard == "heads" and world > 1:
        try:
            shard = pdist.shard_heads(w.n_q_heads, w.n_kv_heads, rank, world, w.head_dim)
        except ValueError as e:
            raise SystemExit("--shard heads: %s" % e)
        w = h1b_synth.scaled(w, n_q_heads=shard.n_q, n_kv_heads=shard.n_kv,
                             name=w.name + "[1/%d of the heads per rank]" % world)
    shard_heads = shard is not None
    job_ranks = 1 if shard_heads else world           # how many ranks' tokens add up
    steps, warmup = args.steps, args.warmup
    Tq = max(1, args.query_tokens)                    # > 1: a step appends Tq tokens and attends for all of them at once
    if Tq > 1:
        w = h1b_synth.scaled(w, name=w.name + "[Tq=%d]" % Tq)
    total_steps = (3 * (steps + warmup) + 16) * Tq   # device-resident run, the host-buffer run, the per-layer graph run
    lens0 = h1b_synth.lengths(w) - 1                  # the first step decodes exactly the workload's context
    page_tokens = max(0, args.page_tokens)
    pages_per_seq = (w.context - 1 + total_steps + page_tokens - 1) // page_tokens if page_tokens else 0
    if page_tokens:
        w = h1b_synth.scaled(w, name=w.name + "[pages of %d tokens]" % page_tokens)
    cfg = binding.make_config(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.sketch_bits, w.group_size,
                              max_batch=w.batch, max_seq=w.context - 1 + total_steps, device=local,
                              fp16_values=args.fp16_values, page_tokens=page_tokens, n_pages=pages_per_seq * w.batch,
                              rope=args.rope)
    # replicas: each rank is its own sequence set (different seeds per rank); head shards: one model's inputs on
    # every rank, each keeping its heads
    wr = w_full if shard_heads else h1b_synth.scaled(w, index=w.index + 10 * rank)

    def kv_rows(l, n, stream=0):
        K, V = h1b_synth.kv_rows(wr, l, n, device=str(dev), stream=stream)
        if shard_heads:
            K, V = (pdist.take_heads(t, shard.kv_begin, shard.n_kv) for t in (K, V))
        return K, V

    def queries(l, stream=0):
        q = h1b_synth.queries(wr, l, device=str(dev), stream=stream)
        return pdist.take_heads(q, shard.q_begin, shard.n_q) if shard_heads else q

    Rt = np.stack([h1b_synth.projection(h1b_synth.layer_seed(wr, l, 99), w.head_dim, w.sketch_bits)
                   for l in range(w.n_layers)])
    cache = binding.H1BCache(cfg, Rt=Rt)
    if args.rope:
        cache.h1b_set_rope_table(h1b_synth.rope_table(w.context - 1 + total_steps, w.head_dim // 2))
    if page_tokens:                                   # every sequence gets a seeded, scattered set of pool pages
        perm = np.random.default_rng(7 + rank).permutation(pages_per_seq * w.batch)
        for b in range(w.batch):
            cache.h1b_set_block_table(b, perm[b * pages_per_seq:(b + 1) * pages_per_seq])
    for l in range(w.n_layers):                       # prefill, one layer at a time
        K, V = kv_rows(l, w.context - 1)
        cache.h1b_append_kv(K.unsqueeze(0), V.unsqueeze(0), layer_begin=l, n_new=lens0)
        del K, V
    torch.cuda.synchronize()
    # per-step inputs: a pool of new tokens and queries, resident in HBM
    pool = 16
    kn = [torch.stack([kv_rows(l, 1, stream=100 + i)[0] for l in range(w.n_layers)]) for i in range(pool)]
    vn = [torch.stack([kv_rows(l, 1, stream=100 + i)[1] for l in range(w.n_layers)]) for i in range(pool)]
    qn = [torch.stack([queries(l, stream=i) for l in range(w.n_layers)]) for i in range(pool)]
    out = torch.empty((w.n_layers, w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    if Tq > 1:                                        # Tq new tokens per sequence and their Tq queries
        kq = torch.cat([kn[i] for i in range(Tq)], dim=2).contiguous()            # [L, B, Tq, Hkv, d]
        vq = torch.cat([vn[i] for i in range(Tq)], dim=2).contiguous()
        qq = torch.stack([qn[i] for i in range(Tq)], dim=2).contiguous()          # [L, B, Tq, Hq, d]
        outq = torch.empty(qq.shape, dtype=torch.float32, device=dev)

    def step(i):                                      # append the new token to all layers + decode: three launches
        if Tq > 1:
            cache.h1b_append_kv(kq, vq)
            cache.h1b_decode_attention_multi(qq, INV_TAU, out=outq)
        else:
            cache.h1b_decode_step(kn[i % pool], vn[i % pool], qn[i % pool], INV_TAU, out=out)

    def barrier():
        pdist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(gpu_index())
    sampler.start()                                   # from the warm-up on: the clocks under load, also for short runs
    for i in range(warmup):
        step(i)
    barrier()
    launches0 = cache.h1b_launch_count()
    cache.h1b_set_profiling(True)
    cache.h1b_read_profile()
    sampler.mark()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    len_first = cache.h1b_get_lengths(0)[:w.batch].astype(np.int64) + Tq
    ctx_first = int(len_first.max())
    barrier()
    ev0.record(stream)
    for i in range(steps):
        step(warmup + i)
    ev1.record(stream)
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop(ms_total / steps)
    launches = cache.h1b_launch_count() - launches0
    kern_ms, kern_n = cache.h1b_read_profile()
    cache.h1b_set_profiling(False)
    cache.h1b_poll_status()
    len_last = cache.h1b_get_lengths(0)[:w.batch].astype(np.int64)
    ctx_last = int(len_last.max())

    # end to end through the host-buffer entry point: pinned host inputs, H2D and D2H inside the timed region
    # (the several-query-tokens variant has no host-buffer entry point: its e2e repeats nothing and stays null)
    if Tq > 1:
        args.no_layer_sequential = True
    # k, v and q of a step back to back in one pinned buffer: the library then moves them with one copy
    kh, vh, qh = [], [], []
    for i in range(pool):
        nk, nq = kn[i].numel(), qn[i].numel()
        buf = torch.empty(2 * nk + nq, dtype=torch.float16).pin_memory()
        kh.append(buf[:nk].view(kn[i].shape)); vh.append(buf[nk:2 * nk].view(vn[i].shape)); qh.append(buf[2 * nk:].view(qn[i].shape))
        kh[i].copy_(kn[i]); vh[i].copy_(vn[i]); qh[i].copy_(qn[i])
    oh = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    for i in range(min(warmup, 8) if Tq == 1 else 0):
        cache.h1b_decode_step_host(kh[i % pool], vh[i % pool], qh[i % pool], INV_TAU, oh)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps if Tq == 1 else 0):
        cache.h1b_decode_step_host(kh[i % pool], vh[i % pool], qh[i % pool], INV_TAU, oh)
    e1.record(stream)
    barrier()
    e2e_ms_total = e0.elapsed_time(e1)

    # layer-sequential: one (append + attention) call per layer, the order a model that runs its layers one
    # after the other imposes, recorded once into a CUDA graph (3 kernels per layer) and replayed
    seq_ms_total = None
    if not args.no_layer_sequential:
        pdist.barrier()
        cache.h1b_sync_lengths()
        ks, vs, qs = kn[0].clone(), vn[0].clone(), qn[0].clone()

        def per_layer():
            for l in range(w.n_layers):
                cache.h1b_decode_step_layers(l, ks[l:l + 1], vs[l:l + 1], qs[l:l + 1], INV_TAU, out=out[l:l + 1])

        per_layer()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):   # other threads (NCCL's watchdog) may call CUDA
            per_layer()
        for i in range(min(warmup, 8)):
            graph.replay()
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for i in range(steps):
            graph.replay()
        g1.record(stream)
        barrier()
        seq_ms_total = g0.elapsed_time(g1)
        cache.h1b_sync_lengths()
        cache.h1b_poll_status()

    ms_total, e2e_ms_total = pdist.max_over_ranks([ms_total, e2e_ms_total], dev)     # slowest rank
    if seq_ms_total is not None:
        seq_ms_total = pdist.max_over_ranks([seq_ms_total], dev)[0]
    ms_per_step = ms_total / steps
    value = pdist.whole_job_rate(w.batch * Tq, job_ranks, ms_per_step * 1e-3)
    e2e_value = pdist.whole_job_rate(w.batch, job_ranks, e2e_ms_total / steps * 1e-3) if Tq == 1 else None

    # roofline of the dominant kernel (split-K decode attention), per launch
    entry = binding.h1b_entry_bytes(cfg)
    tokens_mean = float((0.5 * (len_first + len_last)).sum())         # cached tokens over the batch, mean over the run
    token_heads = w.n_layers * w.n_kv_heads * tokens_mean
    alg_bytes = token_heads * entry + w.n_layers * w.batch * Tq * w.n_q_heads * (w.sketch_bits // 8)
    peak, peak_kind = measured_peaks()
    kern_ms_avg = kern_ms / max(kern_n, 1)
    achieved = alg_bytes / (kern_ms_avg * 1e-3) / 1e9 if kern_n else None
    roofline = {"bound": "hbm", "kernel": "decode_split_kernel", "achieved": achieved, "peak": peak,
                "peak_kind": peak_kind + " (MEASURED_PEAKS.json hbm_gbs)" if peak_kind == "measured" else "fallback",
                "unit": "GB/s", "frac": (achieved / peak) if achieved else None,
                "frac_of_8tbs_nominal": (achieved / 8000.0) if achieved else None,
                # the capture is of the default configuration's kernel; variants have no captured traffic
                "traffic": (NCU_TRAFFIC_PER_ALGORITHMIC_BYTE * alg_bytes) if w.name == "c2_7b_8k" else None,
                "traffic_source": "ncu capture at 8198 tokens, scaled by algorithmic bytes" if w.name == "c2_7b_8k" else None,
                "traffic_ratio_measured_at": NCU_TRAFFIC_MEASURED_AT if w.name == "c2_7b_8k" else None,
                "alg_bytes_per_launch": alg_bytes,
                "kernel_ms_avg": kern_ms_avg, "kernel_launches_timed": kern_n,
                "step_gbs": alg_bytes / (ms_per_step * 1e-3) / 1e9}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if shard_heads else "weak", "vs_baseline": None,
        "dtype": "u32 xor+popcount (scores), f32 (softmax), f16 x f16 -> f32 mma (P.V on 4-bit codes)", "data": "synthetic",
        "config": {"workload": "%s: %d layers x %d/%d heads, d=%d, m=%d, batch %d per GPU, %s; fp16 K/V ~ N(0,1)%s, one "
                               "projection per layer" % (w.name, w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim,
                                                         w.sketch_bits, w.batch, w.notes,
                                                         " with 1% outlier channels x8" if w.outlier_frac else ""),
                   "ctx_first": ctx_first, "ctx_last": ctx_last, "inv_tau": INV_TAU,
                   "cache_bytes": int(token_heads * entry),
                   "l2": "working set (%.0f MB per step) is larger than L2; nothing is flushed" % (alg_bytes / 1e6)},
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": (e2e_ms_total / steps) if Tq == 1 else None,
                "h2d_bytes_per_step": int(sum(x[0].numel() * 2 for x in (kh, vh, qh))),
                "d2h_bytes_per_step": int(oh.numel() * 4)},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
    }
    if seq_ms_total is not None:                      # not the headline: the same step issued layer by layer
        line["layer_sequential"] = {"value": pdist.whole_job_rate(w.batch, job_ranks, seq_ms_total / steps * 1e-3), "unit": UNIT,
                                    "ms_per_step": seq_ms_total / steps, "launches_per_step": 3 * w.n_layers,
                                    "how": "h1b_decode_step_layers once per layer, one CUDA graph per step, replayed"}
    if args.check and rank == 0:                      # after all timing: the cache just timed against the oracle
        line["check"] = check_against_oracle(cache, w, wr, Rt, lens0, kv_rows, dev)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        if w.name == "c2_7b_8k":
            line["cpu_baseline"] = cpu_baseline(sample_layers=1, steps=5, warmup=1)
        elif args.workload in ("c3_7b_batched", "c4_gqa_32k", "c6_60m_8k") and not (args.fp16_values or args.rope or Tq > 1):
            line["cpu_baseline"] = cpu_baseline(steps=1, warmup=0, sample=OracleSample(1, w, sample_batch=min(w.batch, 2)))
    cache.close()
    pdist.finish()
    if rank == 0:
        print(json.dumps(line))


def run_prefill(args, w, pdist, rank, world, local):
    """c5: a step is the compression of an 8192-token prompt into all layers' caches (h1b_append_kv)."""
    import torch

    import h1b_synth
    from paper_2510_05529_b200 import binding
    dev = torch.device("cuda", local)
    cfg = binding.make_config(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.sketch_bits, w.group_size,
                              max_batch=w.batch, max_seq=w.context, device=local, fp16_values=args.fp16_values,
                              rope=args.rope)
    cache = binding.H1BCache(cfg, seed=11 + rank)
    if args.rope:
        cache.h1b_set_rope_table(h1b_synth.rope_table(w.context, w.head_dim // 2))
    K = torch.stack([h1b_synth.kv_rows(w, l, w.context, device=str(dev))[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, w.context, device=str(dev))[1] for l in range(w.n_layers)])
    stream = torch.cuda.current_stream()
    times = []
    launches0 = 0
    sampler = ClockSampler(gpu_index())
    sampler.start()
    for i in range(args.warmup + args.steps):
        if i == args.warmup:
            launches0 = cache.h1b_launch_count()
            sampler.mark()
        cache.h1b_reset(-1)                           # synchronous, outside the timed call
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pdist.barrier(); torch.cuda.synchronize()
        e0.record(stream)
        cache.h1b_append_kv(K, V)
        e1.record(stream)
        torch.cuda.synchronize()
        if i >= args.warmup:
            times.append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    cache.h1b_poll_status()
    launches = cache.h1b_launch_count() - launches0
    prompt_attention = None
    if args.prompt_attention:
        # attention for every token of the prompt over the cache just built (blocks of 16 query tokens, causal)
        q = torch.stack([h1b_synth.normal_fp16(h1b_synth.layer_seed(w, l, 7), (w.batch, w.context, w.n_q_heads, w.head_dim),
                                               device=str(dev)) for l in range(w.n_layers)])
        out = torch.empty(q.shape, dtype=torch.float32, device=dev)
        n_pa = max(1, min(args.steps, 3))
        l0 = cache.h1b_launch_count()
        cache.h1b_prefill_attention(q, INV_TAU, out=out)                # warm-up
        torch.cuda.synchronize()
        per_call = cache.h1b_launch_count() - l0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_pa):
            cache.h1b_prefill_attention(q, INV_TAU, out=out)
        e1.record(stream)
        torch.cuda.synchronize()
        cache.h1b_poll_status()
        pa_ms = pdist.max_over_ranks([e0.elapsed_time(e1) / n_pa], dev)[0]
        prompt_attention = {"value": pdist.whole_job_rate(w.batch * w.context, world, pa_ms * 1e-3), "unit": UNIT,
                            "ms_per_call": pa_ms, "calls": n_pa, "gpu_launches_per_call": int(per_call),
                            "how": "h1b_prefill_attention over all %d prompt tokens, %d layers at once" % (w.context, w.n_layers)}
        del q, out
    ms = pdist.max_over_ranks([float(np.mean(times))], dev)[0]
    rows = w.n_layers * w.batch * w.context * w.n_kv_heads
    alg_bytes = rows * (2 * w.head_dim * 2 + binding.h1b_entry_bytes(cfg))       # fp16 K and V in, packed entry out
    peak, peak_kind = measured_peaks()
    line = {"metric": "prefill compression tokens/s (7B shape, 8192-token prompt into 32 layers' caches)",
            "value": pdist.whole_job_rate(w.batch * w.context, world, ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16 x f16 -> f32 (projection), f32 (quantiser)",
            "data": "synthetic", "config": {"workload": "%s: %s" % (w.name, w.notes), "l2": "5.1 GB per step, larger than L2"},
            "gpu_launches": int(launches), "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "prefill_kernel (keys, tcgen05) beside prefill_values_kernel (values), one call",
                         "achieved": alg_bytes / (ms * 1e-3) / 1e9,
                         "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": alg_bytes / (ms * 1e-3) / 1e9 / peak,
                         "alg_bytes_per_launch": alg_bytes, "traffic": None,
                         "tensor_tflops": rows * w.head_dim * w.sketch_bits * 2 * 2 / (ms * 1e-3) / 1e12}}
    line["clocks"]["ms_per_step_x_sm_mhz"] = ms * clocks["sm_mhz"] if clocks.get("sm_mhz") else None
    if prompt_attention:
        line["prompt_attention"] = prompt_attention
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not (args.fp16_values or args.rope):
        line["cpu_baseline"] = prefill_cpu_baseline(w)
    cache.close()
    pdist.finish()
    if rank == 0:
        print(json.dumps(line))


# --------------------------------------------------------------------------- oracle on host cores
class OracleSample:
    """The fp64 oracle, as it stands, on a bounded sample of a decode workload: `sample_layers` of its layers and
    `sample_batch` of its sequences (all heads, every cached token of those). One decode step = compress the new
    token (Eq. 2, Eq. 4) and attend over the cached history (Eq. 2 on q, Eq. 3, Eq. 5). The history is compressed
    once, untimed. The timed figure is scaled to the whole workload (layers and sequences are independent units)."""

    def __init__(self, sample_layers: int = 1, w=None, sample_batch: int | None = None):
        import torch

        import h1b_synth
        import oracle
        self.oracle, self.w = oracle, (w or h1b_synth.WORKLOADS["c2_7b_8k"])
        w, T = self.w, self.w.context
        self.sample_batch = B = min(w.batch, sample_batch or w.batch)
        self.lens = h1b_synth.lengths(w)[:B].copy()
        self.layers = []
        for l in range(sample_layers):
            Rt = h1b_synth.projection(h1b_synth.layer_seed(w, l, 99), w.head_dim, w.sketch_bits)
            K, V = h1b_synth.kv_rows(w, l, T, batch=B)
            q = h1b_synth.queries(w, l, batch=B)
            Kb = K.view(dtype=torch.int16).numpy().view(np.uint16)
            Vb = V.view(dtype=torch.int16).numpy().view(np.uint16)
            qb = q.view(dtype=torch.int16).numpy().view(np.uint16)
            # the whole layer is compressed once; each timed step recompresses every sequence's newest token
            cache = oracle.compress(Kb, Vb, Rt, w.group_size)
            new_k = np.stack([Kb[b, self.lens[b] - 1:self.lens[b]] for b in range(B)])
            new_v = np.stack([Vb[b, self.lens[b] - 1:self.lens[b]] for b in range(B)])
            self.layers.append((Rt, new_k, new_v, qb, cache))

    def step(self) -> float:
        """Seconds for one decode step over the sampled layers and sequences."""
        o, w = self.oracle, self.w
        t0 = time.perf_counter()
        for Rt, k_new, v_new, qb, cache in self.layers:
            new = o.compress(k_new, v_new, Rt, w.group_size)
            for dst, src in zip(cache, new):
                for b in range(self.sample_batch):
                    dst[b, :, self.lens[b] - 1:self.lens[b]] = src[b]
            o.decode_cached(cache, self.lens, qb, Rt, INV_TAU, w.group_size)
        return time.perf_counter() - t0

    @property
    def scale(self) -> float:
        """Whole workload over the sample (independent units: layers x sequences)."""
        return (self.w.n_layers / len(self.layers)) * (self.w.batch / self.sample_batch)

    def describe(self, n_timed: int):
        w = self.w
        return ("%s: %d of %d layers, %d of %d sequences (%d KV heads x %s cached tokens each), mean of %d timed step(s), "
                "scaled to the whole workload (extrapolated); history compressed once outside the timed region"
                % (w.name, len(self.layers), w.n_layers, self.sample_batch, w.batch, w.n_kv_heads,
                   "/".join(str(int(x)) for x in self.lens), n_timed))


def cpu_baseline(sample_layers: int = 1, steps: int = 3, warmup: int = 1, sample: OracleSample | None = None):
    s = sample or OracleSample(sample_layers)
    for _ in range(warmup):
        s.step()
    times = [s.step() for _ in range(max(1, steps))]
    step_s = float(np.mean(times)) * s.scale
    cores = s.oracle.threads()
    out = {"value": s.w.batch / step_s, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": s.describe(len(times)), "ms_per_step": step_s * 1e3}
    if cores > 1 and sample is None:                    # the same sample once more on a single thread
        s.oracle.set_threads(1)
        try:
            one_s = s.step() * s.scale
        finally:
            s.oracle.set_threads(cores)
        out["one_thread"] = {"value": s.w.batch / one_s, "unit": UNIT, "ms_per_step": one_s * 1e3, "sample": "one timed step"}
    return out


def prefill_cpu_baseline(w, sample_tokens: int = 256):
    """The oracle's compression (Eq. 2, Eq. 4) of `sample_tokens` prompt tokens of one layer (all KV heads), scaled to
    the whole prompt and all layers."""
    import torch

    import h1b_synth
    import oracle
    Rt = h1b_synth.projection(h1b_synth.layer_seed(w, 0, 99), w.head_dim, w.sketch_bits)
    K, V = h1b_synth.kv_rows(w, 0, sample_tokens)
    Kb = K.view(dtype=torch.int16).numpy().view(np.uint16)
    Vb = V.view(dtype=torch.int16).numpy().view(np.uint16)
    oracle.compress(Kb[:, :8], Vb[:, :8], Rt, w.group_size)             # warm-up
    t0 = time.perf_counter()
    oracle.compress(Kb, Vb, Rt, w.group_size)
    dt = time.perf_counter() - t0
    step_s = dt * (w.context / sample_tokens) * w.n_layers
    return {"value": w.batch * w.context / step_s, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "%s: %d of %d prompt tokens of 1 of %d layers (all %d KV heads), one timed pass, scaled to the whole "
                      "prompt (extrapolated)" % (w.name, sample_tokens, w.context, w.n_layers, w.n_kv_heads),
            "ms_per_step": step_s * 1e3}


def check_against_oracle(cache, w, wr, Rt, lens0, kv_rows, dev, units: int = 3):
    """Opt-in leg, after all timing: three seeded (layer, sequence, KV head) units of the cache that was just timed.
    Their prompt part is compared with the oracle's compression of the same rows (decision flips inside the 1e-5
    boundary windows are counted, one outside fails), and one more decode over everything they now hold is compared
    with the oracle's Eq. 3 + Eq. 5 on the exported cache (integer scores bit for bit)."""
    import torch

    import h1b_synth
    tests_dir = os.path.join(ROOT, "tests")
    if tests_dir not in sys.path:
        sys.path.insert(0, tests_dir)
    import h1b_testlib as tl
    rng = np.random.default_rng(20251005)
    gq = w.n_q_heads // w.n_kv_heads
    q = torch.stack([h1b_synth.normal_fp16(h1b_synth.layer_seed(wr, l, 31), (w.batch, w.n_q_heads, w.head_dim), str(dev))
                     for l in range(w.n_layers)])
    out = cache.h1b_decode_attention(q, INV_TAU).cpu().numpy()
    cache.h1b_poll_status()
    res = {"units": [], "flips_inside": 0, "flips_outside": 0, "max_abs": 0.0, "max_rel": 0.0}
    for _ in range(units):
        l, b, g = int(rng.integers(w.n_layers)), int(rng.integers(w.batch)), int(rng.integers(w.n_kv_heads))
        n0 = int(lens0[b])
        K, V = kv_rows(l, w.context - 1)                     # the same draw as the prompt the cache was filled with
        st = tl.append_parity(cache, l, b, g, tl.f16_bits(K[b, :n0, g]), tl.f16_bits(V[b, :n0, g]), Rt[l])   # raises on a flip outside
        res["flips_inside"] += st["bit_flips_in"] + st["code_flips_in"] + st["scale_flips_in"]
        n = int(cache.h1b_get_lengths(l)[b])
        for hh in range(gq):
            h = g * gq + hh
            ref, qf = tl.oracle_from_export(cache, l, b, h, q[l, b, h].contiguous(), n, INV_TAU, Rt[l])
            res["flips_inside"] += qf
            err = np.abs(out[l, b, h].astype(np.float64) - ref)
            big = np.abs(ref) >= 1e-3
            res["max_abs"] = max(res["max_abs"], float(err.max()))
            if big.any():
                res["max_rel"] = max(res["max_rel"], float((err[big] / np.abs(ref[big])).max()))
        res["units"].append([l, b, g])
        del K, V
    res["within_tolerance"] = bool(res["max_abs"] <= tl.MAX_ABS and res["max_rel"] <= tl.MAX_REL)
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    t0 = time.perf_counter()
    steps = max(1, min(args.steps, 20))
    base = cpu_baseline(sample_layers=1, steps=steps, warmup=max(1, min(args.warmup, 3)))
    v = base["value"]
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": world,
            "steps": steps, "warmup": max(1, min(args.warmup, 3)), "ms_per_step": 1e3 / v, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "c2_7b_8k (bounded sample of it per step, see cpu_baseline.sample)"},
            "cpu_baseline": base,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": time.perf_counter() - t0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=30)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--check", action="store_true",
                    help="after all timing: three seeded units of the timed cache against the oracle (flip counts, errors)")
    ap.add_argument("--sketch-bits", type=int, default=0, help="override m (64, 128, 256, 512)")
    ap.add_argument("--group-size", type=int, default=0, help="override G (32, or 128 = one scale per value vector)")
    ap.add_argument("--no-layer-sequential", action="store_true", help="skip the per-layer CUDA-graph measurement")
    ap.add_argument("--query-tokens", type=int, default=1,
                    help="> 1: each step appends this many tokens per sequence and attends for all of them (variant)")
    ap.add_argument("--shard", default="sequences", choices=["sequences", "heads"],
                    help="with N > 1 ranks: 'sequences' (default) = one independent sequence set per rank, weak scaling; "
                         "'heads' = the ranks split the heads of the same sequences, strong scaling")
    ap.add_argument("--page-tokens", type=int, default=0,
                    help="> 0: a paged cache with pages of this many tokens, scattered over the pool (variant)")
    ap.add_argument("--prompt-attention", action="store_true",
                    help="c5_prefill: also time attention for every prompt token over the compressed cache (variant)")
    ap.add_argument("--q-heads", type=int, default=0, help="override the number of query heads (variant)")
    ap.add_argument("--kv-heads", type=int, default=0, help="override the number of KV heads (variant)")
    ap.add_argument("--layers", type=int, default=0, help="> 0: only this many layers of the workload's shape (variant)")
    ap.add_argument("--rope", action="store_true",
                    help="rotate keys and queries (rotary position embedding) inside the append and the query sketch (variant)")
    ap.add_argument("--fp16-values", action="store_true", help="keep values in fp16 (the 1-bit-keys-only ablation row)")
    ap.add_argument("--workload", default="c2_7b_8k",
                    choices=["c2_7b_8k", "c3_7b_batched", "c4_gqa_32k", "c5_prefill", "c6_60m_8k"],
                    help="default: the configuration the metric is quoted on; the others are variants and parity cases")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
