#!/usr/bin/env python
"""Benchmark of the SKVQ decode hot path on B200.

A "step" is one decode step over the whole batch: append one new token per sequence (one token
slides out of the fp16 window and is quantized) and run decode attention over
[packed quantized prefix || fp16 window].  The default workload is configuration 1
(Llama-2-7B-shaped, batch 8, 32 heads, context 32768, 2-bit K/V, group 128, window 128).

  python bench.py --gpus N --steps K --warmup W             (our CUDA path; under torchrun for N > 1)
  python bench.py --impl reference ...                      (the CPU oracle on a bounded sample)
  python bench.py --config 3                                (another configuration, 0..4)

Prints ONE JSON line.  `value` is context tokens per second with inputs resident in HBM; `e2e` is the
same metric through the host-buffer C-ABI call (host->device copies of k/v/q and the device->host
read of out inside the timed region).  The cache is larger than L2 for configurations 1-4, so
successive steps stream from HBM; configuration 0 (11 MB) flushes L2 between steps.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_context_tokens_per_s"
UNIT = "tokens/s"
PREFILL_CHUNK = 32768
L2_BYTES = 126 * 1024 * 1024
# DRAM bytes (read + write) per launch of the partition kernel from ncu captures, keyed by configuration;
# absent (None) where no capture exists for the current kernel.
NCU_TRAFFIC_BYTES = {1: 632.6e6, 2: 412.8e6, 4: 2551.9e6}      # reduced-batch ncu captures scaled by tokens streamed


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier copy-bandwidth measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.index, self.samples, self._stop, self._t = gpu_id, [], threading.Event(), None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                self.samples.append([x.strip() for x in out.strip().split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=10)

    def summary(self):
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            if len(s) < 6:
                continue
            try:
                mhz.append(float(s[0]))
                mx = float(s[1])
            except ValueError:
                continue
            for n, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


def build_gpu_cache(w, extra_tokens, torch, binding):
    """Prefill the cache with the library's own quantize_append, chunk by chunk; returns
    (cache, prefill_ms, prefill_bytes) where prefill_ms only covers the append kernels."""
    lengths = w.lengths()
    max_tokens = int(lengths.max()) + extra_tokens
    cache = binding.SkvqCache.for_workload(w, max_tokens)
    moved = 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    Lmax = int(lengths.max())
    # host staging of one chunk stays near 1 GiB per tensor whatever the batch size
    chunk = max(256, min(PREFILL_CHUNK, (1 << 30) // (w.batch * w.n_kv_heads * w.head_dim * 2) // 256 * 256))
    timed = None
    for t0 in range(0, Lmax, chunk):
        t1 = min(t0 + chunk, Lmax)
        n_b = np.clip(lengths - t0, 0, t1 - t0).astype(np.int32)
        k = np.zeros((w.batch, t1 - t0, w.n_kv_heads, w.head_dim), np.float16)
        v = np.zeros_like(k)
        for b in range(w.batch):
            if n_b[b]:
                k[b, :n_b[b]] = w.tokens("k", b, t0, t0 + int(n_b[b]))
                v[b, :n_b[b]] = w.tokens("v", b, t0, t0 + int(n_b[b]))
        dk, dv, dn = torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(n_b).cuda()
        cache.append(dk, dv, dn)
        torch.cuda.synchronize()
        if t0 == 0:
            # time the quantize of this first chunk on a scratch cache of the same shape: once to warm up (clocks,
            # instruction cache), then three times from empty; the figure is the best of the three
            tmp = binding.SkvqCache.for_workload(w, t1 + 64)
            best = None
            for rep in range(4):
                tmp.lengths.zero_()
                torch.cuda.synchronize()
                e0.record()
                tmp.append(dk, dv, dn)
                e1.record()
                torch.cuda.synchronize()
                if rep:
                    best = e0.elapsed_time(e1) if best is None else min(best, e0.elapsed_time(e1))
            timed = (best, int(n_b.sum()) * w.n_kv_heads * w.head_dim * 2 * 2)
            del tmp
        moved += int(n_b.sum()) * w.n_kv_heads * w.head_dim * 2 * 2
        del dk, dv
    # scale the timed chunk to the whole prefill (the work per token does not depend on the position)
    ms = timed[0] * moved / timed[1]
    return cache, ms, moved


def oracle_sample(w, n_seq, n_kv=None):
    """The CPU oracle's cache for the first n_seq sequences (full context) and the first n_kv KV heads
    (default all) of the workload: a slice of the very same inputs."""
    from oracle import skvq_oracle as orc
    n_kv = w.n_kv_heads if n_kv is None else n_kv
    rep = w.n_q_heads // w.n_kv_heads
    lengths = w.lengths()[:n_seq]
    a = w.alphas()[:n_kv]
    rk, rv = w.reorder_index("k")[:n_kv], w.reorder_index("v")[:n_kv]
    cap = int(lengths.max()) + 4096

    def new(batch):
        return orc.OracleCache(batch, n_kv * rep, n_kv, w.head_dim, w.k_bits, w.v_bits, w.group_size, w.window,
                               cap, rk, rv, a, a, n_sink=w.n_sink, meta_fp8=w.meta_fp8)
    oc = new(n_seq)
    for b in range(n_seq):
        one = new(1)
        L = int(lengths[b])
        one.append(np.ascontiguousarray(w.tokens("k", b, 0, L)[None, :, :n_kv]),
                   np.ascontiguousarray(w.tokens("v", b, 0, L)[None, :, :n_kv]))
        for name in ("k_codes", "v_codes", "k_meta", "v_meta", "k_win", "v_win", "k_sink", "v_sink"):
            getattr(oc, name)[b] = getattr(one, name)[0]
        oc.lengths[b] = L
    return oc


def time_oracle(w, steps, warmup, budget_s):
    """Decode steps (append one token + attention) of the oracle, as it stands, on a bounded sample of
    the workload: the first sequences at full context (all KV heads), or, when one sequence alone is too
    much, sequence 0 with its first KV heads, sized so that the timed steps take about budget_s of CPU
    time.  Tokens are the context tokens of the (sequence, head) units actually processed, expressed in
    whole-workload terms (a unit counts for 1 / Hkv of its sequence's tokens)."""
    from oracle import skvq_oracle as orc
    rep = w.n_q_heads // w.n_kv_heads
    lengths = w.lengths()
    # calibrate on one KV head of sequence 0
    oc = oracle_sample(w, 1, 1)
    q = w.query(0)[:1, :rep]
    t0 = time.perf_counter()
    oc.attention(q, w.sm_scale)
    per_unit = max(time.perf_counter() - t0, 1e-4) * float(lengths.mean()) / float(lengths[0])
    threads = orc.num_threads()
    per_step_budget = budget_s / max(steps, 1)
    units = max(1, int(per_step_budget / per_unit * min(threads, w.n_kv_heads * rep)))
    if units >= w.n_kv_heads:
        n_seq, n_kv = int(min(w.batch, units // w.n_kv_heads)), w.n_kv_heads
    else:
        n_seq, n_kv = 1, units
    oc = oracle_sample(w, n_seq, n_kv)
    times, tokens = [], 0.0
    for s in range(warmup + steps):
        kn = np.ascontiguousarray(w.new_token("k", s)[:n_seq, :, :n_kv])
        vn = np.ascontiguousarray(w.new_token("v", s)[:n_seq, :, :n_kv])
        q = np.ascontiguousarray(w.query(s)[:n_seq, :n_kv * rep])
        t0 = time.perf_counter()
        oc.append(kn, vn)
        oc.attention(q, w.sm_scale)
        dt = time.perf_counter() - t0
        if s >= warmup:
            times.append(dt)
            tokens += float(lengths[:n_seq].sum() + n_seq * (s + 1)) * n_kv / float(w.n_kv_heads)
    total = sum(times)
    return {"value": tokens / total, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"sequences 0..{n_seq - 1} of {w.batch} at full context, KV heads 0..{n_kv - 1} of {w.n_kv_heads} "
                      f"with their query heads, {steps} decode steps (append one token + attention), {total:.2f} s "
                      f"of CPU time; a (sequence, KV head) unit counts for 1/{w.n_kv_heads} of its sequence's tokens"}, \
        total / len(times)


def run_reference(args, w, rank):
    if rank != 0:
        return
    base, ms = time_oracle(w, args.steps, args.warmup, 120.0)
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"configs[{args.config}] {w.name}", "sample": base["sample"]},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (small profiling cases)")
    ap.add_argument("--context", type=int, default=0, help="override the context length (small profiling cases)")
    ap.add_argument("--q-heads", type=int, default=0, help="override the number of query heads (other grouped-query ratios)")
    ap.add_argument("--meta-fp8", action="store_true",
                    help="scale and zero point stored in FP8 E4M3 instead of fp16 (Sec. 4.1; 2.5 bits per element at g32)")
    ap.add_argument("--sinks", type=int, default=0,
                    help="attention sinks: first positions kept fp16 (Sec. 3.2 filter rule; the paper's experiments use 5)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2405_06219_b200 import sharding, workloads
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w0 = workloads.configs()[args.config]
    if args.batch:
        w0 = w0.scaled(batch=args.batch)
    if args.context:
        w0 = w0.scaled(context=args.context, ragged=None)
    if args.sinks:
        w0 = w0.scaled(n_sink=args.sinks)
    if args.q_heads:
        w0 = w0.scaled(n_q_heads=args.q_heads)
    if args.meta_fp8:
        w0 = w0.scaled(meta_fp8=True)

    if args.impl == "reference":
        run_reference(args, w0, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2405_06219_b200 import binding, build
    build.build_library()
    binding.lib()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SKVQ path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    w = sharding.rank_workload(w0, rank, world)
    n_steps_total = 4 * (args.warmup + args.steps) + 8      # warm-up, three passes of the steps, the end-to-end pass
    cache, prefill_ms, prefill_in = build_gpu_cache(w, n_steps_total + 64, torch, binding)
    lengths0 = w.lengths()
    hint = int(lengths0.max()) + n_steps_total
    alg_bytes = workloads.algorithmic_bytes(w, lengths0)
    part_bytes = workloads.partition_kernel_bytes(w, lengths0)
    flush = None
    if cache.nbytes() < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

    # -- parity re-check on the benchmark's own cache (sampled sequence), before timing
    parity = None
    if not args.no_parity and rank == 0:
        oc = oracle_sample(w, 1)
        lq = max(int(lengths0[0]) - w.window, 0)
        ns = min(w.n_sink, lq)      # sink rows: fp16 copies instead of codes

        def meta_bits(t):           # fp16 bit patterns, or one E4M3 byte per parameter (the oracle keeps each in a uint16)
            a = t[0, :, ns:lq].cpu().numpy()
            return a.astype(np.uint16) if w.meta_fp8 else a.view(np.uint16)
        exact = bool(np.array_equal(cache.k_codes[0, :, ns:lq].cpu().numpy(), oc.k_codes[0, :, ns:lq]) and
                     np.array_equal(cache.v_codes[0, :, ns:lq].cpu().numpy(), oc.v_codes[0, :, ns:lq]) and
                     np.array_equal(meta_bits(cache.k_meta), oc.k_meta.view(np.uint16)[0, :, ns:lq]) and
                     np.array_equal(meta_bits(cache.v_meta), oc.v_meta.view(np.uint16)[0, :, ns:lq]) and
                     np.array_equal(cache.k_sink[0, :, :ns].cpu().numpy().view(np.uint16), oc.k_sink.view(np.uint16)[0, :, :ns]) and
                     np.array_equal(cache.v_sink[0, :, :ns].cpu().numpy().view(np.uint16), oc.v_sink.view(np.uint16)[0, :, :ns]))
        q = w.query(10_000)
        out = cache.attention(torch.from_numpy(q).cuda(), w.sm_scale, hint, n_splits=args.splits)
        torch.cuda.synchronize()
        want = oc.attention(q[:1], w.sm_scale)
        err = float(np.abs(out[:1].cpu().numpy().astype(np.float64) - want).max())
        parity = {"sequence": 0, "cache_bit_exact": exact, "attention_max_abs_err": err, "tolerance": 2e-3}
        if not exact or err > 2e-3:
            raise SystemExit(f"parity failure on the benchmark inputs: {parity}")
        del oc

    # -- per-step inputs, resident in HBM before timing
    n_in = args.warmup + args.steps
    k_new = torch.from_numpy(np.stack([w.new_token("k", s) for s in range(n_in)])).cuda()
    v_new = torch.from_numpy(np.stack([w.new_token("v", s) for s in range(n_in)])).cuda()
    q_all = torch.from_numpy(np.stack([w.query(s) for s in range(n_in)])).cuda()
    out = torch.empty_like(q_all[0])
    ev_k = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]

    for a, b in ev_k:      # torch creates its events lazily: record once so the handles exist before the library re-records them
        a.record()
        b.record()
    torch.cuda.synchronize()
    args_plain = cache.attn_args(w.sm_scale, hint, args.splits)
    args_timed = [cache.attn_args(w.sm_scale, hint, args.splits, a, b) for a, b in ev_k]

    ev_call = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]

    def step(i, attn_args, ev=None):
        cache.append(k_new[i], v_new[i])
        if ev is not None:
            ev[0].record()
        binding.skvq_decode_attention(cache.cfg, cache.struct, q_all[i], out, attn_args)
        if ev is not None:
            ev[1].record()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i, args_plain)
    barrier()
    launches0 = binding.skvq_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        gpu_id = str(local_rank)
    with ClockSampler(gpu_id) as clocks:
        if flush is None:
            e0.record()
            for i in range(args.steps):
                step(args.warmup + i, args_plain)      # nothing but the calls: an event between two calls would
            e1.record()                                # keep the dependent launches from overlapping
            barrier()
            elapsed_ms = e0.elapsed_time(e1)
        else:   # small cache: flush L2 before every step and time each step on its own
            per = []
            for i in range(args.steps):
                flush.fill_(i & 1)
                e0.record()
                step(args.warmup + i, args_plain)
                e1.record()
                torch.cuda.synchronize()
                per.append(e0.elapsed_time(e1))
            barrier()
            elapsed_ms = sum(per)
        launches = binding.skvq_launch_count() - launches0
        # the same steps again with the library's own events around the partition kernel (an event between
        # the two kernels keeps the merge kernel from overlapping the partition kernel's tail, so this pass
        # measures the dominant kernel alone and the pass above measures the step as a user runs it)
        for i in range(args.steps):
            if flush is not None:
                flush.fill_(i & 1)
            step(args.warmup + i, args_timed[i])
        torch.cuda.synchronize()
        # and once more with events around the attention call (partition + merge)
        for i in range(args.steps):
            if flush is not None:
                flush.fill_(i & 1)
            step(args.warmup + i, args_plain, ev_call[i])
        torch.cuda.synchronize()
        # keep the same kernels running (untimed) until the sampler has seen them under load
        t_end = time.perf_counter() + 3.0
        while len(clocks.samples) < 4 and time.perf_counter() < t_end:
            binding.skvq_decode_attention(cache.cfg, cache.struct, q_all[0], out, args_plain)
            torch.cuda.synchronize()
    kern_ms = [a.elapsed_time(b) for a, b in ev_k]
    call_ms = [a.elapsed_time(b) for a, b in ev_call]
    tokens_per_step = float(lengths0.sum()) + w.batch * (args.warmup + (args.steps + 1) / 2.0)
    job_ms, job_tokens = sharding.reduce_job(elapsed_ms, tokens_per_step * args.steps,
                                             device=torch.device("cuda", local_rank) if world > 1 else None)
    value = job_tokens / (job_ms * 1e-3)

    # -- end to end through the host-buffer entry point
    # a step's k, v and q lie back to back in one pinned buffer, as a serving loop would stage them: one copy per step
    kv_el, q_el = w.batch * w.n_kv_heads * w.head_dim, w.batch * w.n_q_heads * w.head_dim
    hin = torch.empty((n_in, 2 * kv_el + q_el), dtype=torch.float16).pin_memory()
    for s in range(n_in):
        hin[s, :kv_el] = torch.from_numpy(w.new_token("k", 5000 + s).reshape(-1))
        hin[s, kv_el:2 * kv_el] = torch.from_numpy(w.new_token("v", 5000 + s).reshape(-1))
        hin[s, 2 * kv_el:] = torch.from_numpy(w.query(5000 + s).reshape(-1))
    hk, hv, hq = hin[:, :kv_el], hin[:, kv_el:2 * kv_el], hin[:, 2 * kv_el:]
    hout = torch.empty(tuple(q_all[0].shape), dtype=torch.float16).pin_memory()
    staging = torch.empty(binding.skvq_step_staging_size(cache.cfg), dtype=torch.uint8, device="cuda")
    a = cache.attn_args(w.sm_scale, hint, args.splits)

    def host_step(i):
        binding.skvq_decode_step_host(cache.cfg, cache.struct, hk[i], hv[i], hq[i], hout, staging, a)
        torch.cuda.synchronize()      # the caller reads hout every step

    for i in range(args.warmup):
        host_step(i)
    barrier()
    e0.record()
    for i in range(args.steps):
        host_step(args.warmup + i)
    e1.record()
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), 0.0)
    if int(cache.status[0].item()) != 0:      # capacity overflow or a copy that never completed: the numbers would be void
        raise SystemExit(f"the cache's status word is {int(cache.status[0].item())} after the timed passes")
    # lengths at the end-to-end pass: warm-up and three passes of the steps are already in the cache
    e2e_tokens = (float(lengths0.sum()) + w.batch * (2 * args.warmup + 3 * args.steps + (args.steps + 1) / 2.0)) * args.steps
    e2e_ms, e2e_tokens = sharding.reduce_job(e2e_ms, e2e_tokens,
                                             device=torch.device("cuda", local_rank) if world > 1 else None)
    kv_bytes = w.batch * w.n_kv_heads * w.head_dim * 2
    qo_bytes = w.batch * w.n_q_heads * w.head_dim * 2

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peak()
    kavg_ms = sum(kern_ms) / len(kern_ms)
    achieved = part_bytes / (kavg_ms * 1e-3) / 1e9
    cavg_ms = sum(call_ms) / len(call_ms)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": job_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"configs[{args.config}] {w.name}", "batch": w.batch, "n_q_heads": w.n_q_heads,
                   "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "context": int(lengths0.max()),
                   "window": w.window, "k_bits": w.k_bits, "v_bits": w.v_bits, "group_size": w.group_size,
                   "alpha": w.alpha, "n_sink": w.n_sink, "meta_fp8": bool(w.meta_fp8), "step": "append 1 token/sequence + decode attention",
                   "cache_bytes": cache.nbytes(),
                   "l2": "cache larger than L2, streamed every step" if flush is None else "L2 flushed between steps",
                   "parallelism": f"replica per GPU x{world}" if world > 1 else "single GPU"},
        "clocks": clocks.summary(),
        "e2e": {"value": e2e_tokens / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 2 * kv_bytes + qo_bytes,
                "d2h_bytes_per_step": qo_bytes, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode-attention partition kernel", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                     "frac_of_nominal_8000": achieved / 8000.0,
                     "algorithmic_bytes_per_launch": part_bytes, "kernel_ms_avg": kavg_ms,
                     "kernel_ms_min": min(kern_ms), "traffic": NCU_TRAFFIC_BYTES.get(args.config) if not (args.batch or args.context or args.sinks or args.q_heads or args.meta_fp8) else None,
                     "whole_call": {"what": "partition + merge kernels, all algorithmic bytes (codes, scale/zero, "
                                            "fp16 window, q, out)", "algorithmic_bytes": alg_bytes, "ms_avg": cavg_ms,
                                    "achieved": alg_bytes / (cavg_ms * 1e-3) / 1e9,
                                    "frac": alg_bytes / (cavg_ms * 1e-3) / 1e9 / peak}},
        "prefill_quantize": {"ms": prefill_ms, "bytes_in": prefill_in,
                             "gbs_in": prefill_in / (prefill_ms * 1e-3) / 1e9 if prefill_ms > 0 else None,
                             "how": "quantize_append of the first prefill chunk into an empty scratch cache, best of 3 "
                                    "after one warm-up, scaled to all prefilled tokens by bytes"},
        "parity": parity,
    }
    if not args.no_cpu_baseline:
        line["cpu_baseline"], _ = time_oracle(w, 3, 1, 20.0)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
