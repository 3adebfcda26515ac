#!/usr/bin/env python
"""Benchmark of the SKVQ decode hot path on B200.

A "step" is one decode step over the whole batch: append one new token per sequence (one token
slides out of the fp16 window and is quantized) and run decode attention over
[packed quantized prefix || fp16 window].

  python bench.py --gpus N --steps K --warmup W     (the CUDA path; under torchrun for N > 1)
  python bench.py --impl reference ...              (the CPU oracle on a bounded sample)
  python bench.py --config 2                        (one configuration, 0..4, on its own)

With no --config the line is about configuration 3 (one sequence of 1,048,576 tokens, 32 heads, 2-bit K/V,
group 128: the longest context and one of the two configurations the bandwidth target is stated on), and, on one
GPU, an `other_configs` object carries the same measurements for configurations 2 (128k, grouped-query, group 32:
the other target configuration), 1 and 4.

Prints ONE JSON line.  `value` is context tokens per second with inputs resident in HBM; `e2e` is the
same metric through the host-buffer C-ABI call (host->device copies of k/v/q and the device->host
read of out inside the timed region).  The K timed steps are repeated as whole passes until at least
half a second of device time has gone by; `ms_per_step` is the median pass, min and max are reported beside it.
The cache is larger than L2 for configurations 1-4, so successive steps stream from HBM; configuration 0
(11 MB) flushes L2 between steps.
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
DEFAULT_CONFIG = 3
OTHER_CONFIGS = (2, 1, 4)
PREFILL_CHUNK = 32768
L2_BYTES = 126 * 1024 * 1024
MIN_TIMED_MS = 500.0          # the timed passes of the headline configuration cover at least this much device time
MIN_TIMED_MS_OTHER = 300.0
MAX_TIMED_STEPS = 4096        # ... but never more steps than this (each step appends a token to the cache)
MAX_E2E_STEPS = 1024
# DRAM bytes (read + write) per launch of the partition kernel from ncu captures of reduced cases, scaled to the full
# configuration by the tokens streamed (traffic is proportional to them); None where the kernel has changed since.
NCU_TRAFFIC_BYTES = {1: 609.2e6, 2: 409.7e6, 3: 2445.6e6, 4: 2548.7e6}
NCU_TRAFFIC_SOURCE = {
    1: "same kernel as configuration 3 (partition_mma_kernel<128,2,2>): its capture's DRAM bytes / algorithmic bytes = 1.0124, times this configuration's algorithmic bytes",
    2: "ncu capture of configuration 2 at batch 2 (profiles/partition_gqa_K2V2_g32_r4_config2_batch2.md), scaled x 2 by the tokens streamed",
    3: "ncu capture of configuration 3 at a 131072-token context (profiles/partition_mma_K2V2_g128_config3_context128k.md), scaled x 8.006 by the tokens streamed",
    4: "ncu capture of configuration 4 at batch 16 (profiles/partition_mma_K4V4_g64_and_merge_config4_batch16.md), scaled x 4.014 by the tokens streamed",
}

def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier copy-bandwidth measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, gpu_id: str):
        self.index, self.samples, self._stop, self._t = gpu_id, [], threading.Event(), None

    def _run(self):
        while not self._stop.is_set():
            try:
                t = time.perf_counter()
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                self.samples.append((t, time.perf_counter(), [x.strip() for x in out.strip().split(",")]))
            except Exception:
                pass
            self._stop.wait(0.05)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=10)

    def summary(self, windows=None):
        """Median SM clock and the throttle reasons over the samples taken inside the given (t0, t1) host-time
        windows (all samples when none is given or none falls inside)."""
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

        def inside(s):      # the query overlapped a timed pass
            return any(s[1] >= a and s[0] <= b for a, b in windows)
        chosen = [s for s in self.samples if windows and inside(s)]
        scope = "samples taken between the start of the first timed pass and the end of the last"
        if not chosen:
            chosen, scope = self.samples, "whole run (no sample fell inside a timed pass)"
        mhz, mx, reasons, watts = [], None, set(), []
        for _, _, s in chosen:
            if len(s) < 6:
                continue
            try:
                mhz.append(float(s[0]))
                mx = float(s[1])
                if len(s) > 6:
                    watts.append(float(s[6]))
            except ValueError:
                continue
            for n, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz), "scope": scope, "sm_mhz_min": min(mhz) if mhz else None,
                "power_w": statistics.median(watts) if watts else None}


# ---------------------------------------------------------------------------------------------- the oracle's sample
def new_oracle_cache(w, n_seq, n_kv, cap):
    from oracle import skvq_oracle as orc
    rep = w.n_q_heads // w.n_kv_heads
    a = w.alphas()[:n_kv]
    return orc.OracleCache(n_seq, n_kv * rep, n_kv, w.head_dim, w.k_bits, w.v_bits, w.group_size, w.window, cap,
                           w.reorder_index("k")[:n_kv], w.reorder_index("v")[:n_kv], a, a, n_sink=w.n_sink,
                           meta_fp8=w.meta_fp8)


def plan_oracle_sample(w, steps, budget_s):
    """How much of the workload the CPU oracle can redo in about budget_s seconds of `steps` decode steps: the first
    n_seq sequences at full context with all KV heads, or, when one sequence alone is too much, sequence 0 with its
    first n_kv KV heads.  The oracle's speed is calibrated on a short context of the same shape (one KV head)."""
    from oracle import skvq_oracle as orc
    rep = w.n_q_heads // w.n_kv_heads
    cal = w.scaled(batch=1, context=16384, ragged=None, n_kv_heads=1, n_q_heads=rep)
    oc = new_oracle_cache(cal, 1, 1, cal.context + 64)
    oc.append(cal.prefill("k"), cal.prefill("v"))
    q = cal.query(0)
    oc.attention(q, cal.sm_scale)
    t0 = time.perf_counter()
    oc.attention(q, cal.sm_scale)
    per_token = max(time.perf_counter() - t0, 1e-5) / cal.context          # seconds per token of one KV head, one thread
    lengths = w.lengths()
    threads = orc.num_threads()
    per_unit = per_token * float(lengths.mean())
    units = max(1, int(budget_s / max(steps, 1) / per_unit * min(threads, w.n_kv_heads * rep)))
    if units >= w.n_kv_heads:
        return int(min(w.batch, units // w.n_kv_heads)), w.n_kv_heads
    return 1, units


def fill_caches(w, torch, cache, oc, n_seq, n_kv, time_prefill=False, binding=None):
    """Generates the workload chunk by chunk (once) and appends every chunk to the GPU cache (if any) through the
    library's own quantize_append and, for the first n_seq sequences and n_kv KV heads, to the oracle's cache (if
    any).  Returns (prefill_ms, prefill_bytes): the append kernels' time for all prefilled tokens, scaled from the
    first chunk, which is timed on a scratch cache (None unless time_prefill)."""
    lengths = w.lengths()
    Lmax = int(lengths.max())
    need = Lmax if cache is not None else int(lengths[:n_seq].max())
    n_gen = w.batch if cache is not None else n_seq
    # host staging of one chunk stays near 1 GiB per tensor whatever the batch size
    chunk = max(256, min(PREFILL_CHUNK, (1 << 30) // (n_gen * w.n_kv_heads * w.head_dim * 2) // 256 * 256))
    timed, moved = None, 0
    for t0 in range(0, need, chunk):
        t1 = min(t0 + chunk, need)
        n_b = np.clip(lengths[:n_gen] - t0, 0, t1 - t0).astype(np.int32)
        k = np.zeros((n_gen, t1 - t0, w.n_kv_heads, w.head_dim), np.float16)
        v = np.zeros_like(k)
        for b in range(n_gen):
            if n_b[b]:
                k[b, :n_b[b]] = w.tokens("k", b, t0, t0 + int(n_b[b]))
                v[b, :n_b[b]] = w.tokens("v", b, t0, t0 + int(n_b[b]))
        if oc is not None and n_b[:n_seq].any():
            oc.append(np.ascontiguousarray(k[:n_seq, :, :n_kv]), np.ascontiguousarray(v[:n_seq, :, :n_kv]), n_b[:n_seq])
        if cache is not None:
            dk, dv, dn = torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(n_b).cuda()
            cache.append(dk, dv, dn)
            torch.cuda.synchronize()
            if t0 == 0 and time_prefill:
                # the quantize of this first chunk on a scratch cache of the same shape: once to warm up (clocks,
                # instruction cache), then three times from empty; the figure is the best of the three
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                tmp = binding.SkvqCache.for_workload(w, t1 + 64)
                best = None
                for rep_i in range(4):
                    tmp.lengths.zero_()
                    torch.cuda.synchronize()
                    e0.record()
                    tmp.append(dk, dv, dn)
                    e1.record()
                    torch.cuda.synchronize()
                    if rep_i:
                        best = e0.elapsed_time(e1) if best is None else min(best, e0.elapsed_time(e1))
                timed = (best, int(n_b.sum()) * w.n_kv_heads * w.head_dim * 2 * 2)
                del tmp
            del dk, dv
        moved += int(n_b.sum()) * w.n_kv_heads * w.head_dim * 2 * 2
    if timed is None:
        return None, moved
    # the work per token does not depend on the position: scale the timed chunk to the whole prefill
    return timed[0] * moved / timed[1], moved


def oracle_steps(w, oc, n_seq, n_kv, steps, warmup, first_step=0):
    """Decode steps (append one token + attention) of the oracle, as it stands, on its sample.  Tokens are the context
    tokens of the (sequence, head) units actually processed, expressed in whole-workload terms (a unit counts for
    1 / Hkv of its sequence's tokens)."""
    from oracle import skvq_oracle as orc
    rep = w.n_q_heads // w.n_kv_heads
    times, tokens = [], 0.0
    for s in range(warmup + steps):
        kn = np.ascontiguousarray(w.new_token("k", first_step + s)[:n_seq, :, :n_kv])
        vn = np.ascontiguousarray(w.new_token("v", first_step + s)[:n_seq, :, :n_kv])
        q = np.ascontiguousarray(w.query(first_step + s)[:n_seq, :n_kv * rep])
        t0 = time.perf_counter()
        oc.append(kn, vn)
        oc.attention(q, w.sm_scale)
        dt = time.perf_counter() - t0
        if s >= warmup:
            times.append(dt)
            tokens += float(oc.lengths.sum()) * n_kv / float(w.n_kv_heads)
    total = sum(times)
    return {"value": tokens / total, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"sequences 0..{n_seq - 1} of {w.batch} at full context, KV heads 0..{n_kv - 1} of {w.n_kv_heads} "
                      f"with their query heads, {steps} decode steps (append one token + attention), {total:.2f} s "
                      f"of CPU time; a (sequence, KV head) unit counts for 1/{w.n_kv_heads} of its sequence's tokens"}, \
        total / len(times)


def run_reference(args, cfg_i, w, rank):
    if rank != 0:
        return
    n_seq, n_kv = plan_oracle_sample(w, args.steps + args.warmup, 120.0)
    oc = new_oracle_cache(w, n_seq, n_kv, int(w.lengths()[:n_seq].max()) + args.steps + args.warmup + 64)
    fill_caches(w, None, None, oc, n_seq, n_kv)
    base, ms = oracle_steps(w, oc, n_seq, n_kv, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"configs[{cfg_i}] {w.name}", "sample": base["sample"]},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------- one configuration
def run_config(cfg_i, w0, args, env, main):
    """Builds configuration cfg_i on this rank's GPU, checks it against the oracle on a sample, times it.  `main` adds
    the end-to-end pass and the CPU baseline.  Returns the record (rank 0) or None."""
    torch, dist, binding, sharding, workloads = env["torch"], env["dist"], env["binding"], env["sharding"], env["workloads"]
    rank, world, local_rank, clocks = env["rank"], env["world"], env["local_rank"], env["clocks"]
    w = sharding.rank_workload(w0, rank, world)
    K, W_ = args.steps, args.warmup
    extra = 3 * W_ + MAX_TIMED_STEPS + MAX_E2E_STEPS + 5 * K + 64      # every step of every pass appends a token
    lengths0 = w.lengths()
    dev = torch.device("cuda", local_rank) if world > 1 else None

    # -- caches: the GPU's through the library's prefill, the oracle's sample from the same generated chunks
    want_oracle = rank == 0 and not args.no_parity
    if want_oracle:
        if main and not args.no_cpu_baseline:
            n_seq, n_kv = plan_oracle_sample(w, 4, 20.0)
        else:
            n_seq, n_kv = 1, w.n_kv_heads
        oc = new_oracle_cache(w, n_seq, n_kv, int(lengths0[:n_seq].max()) + 64)
    else:
        oc, n_seq, n_kv = None, 0, 0
    cache = binding.SkvqCache.for_workload(w, int(lengths0.max()) + extra)
    prefill_ms, prefill_in = fill_caches(w, torch, cache, oc, n_seq, n_kv, time_prefill=True, binding=binding)
    hint = int(lengths0.max()) + extra
    alg_bytes = workloads.algorithmic_bytes(w, lengths0)
    part_bytes = workloads.partition_kernel_bytes(w, lengths0)
    flush = None
    if cache.nbytes() < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

    # -- parity on the benchmark's own cache (the oracle's sample), before timing
    parity = None
    if oc is not None:
        rep = w.n_q_heads // w.n_kv_heads
        exact = True
        for b in range(n_seq):
            lq = max(int(lengths0[b]) - w.window, 0)
            ns = min(w.n_sink, lq)      # sink rows: fp16 copies instead of codes

            def meta_bits(t):           # fp16 bit patterns, or one E4M3 byte per parameter (the oracle keeps each in a uint16)
                a = t[b, :n_kv, ns:lq].cpu().numpy()
                return a.astype(np.uint16) if w.meta_fp8 else a.view(np.uint16)
            exact = exact and bool(
                np.array_equal(cache.k_codes[b, :n_kv, ns:lq].cpu().numpy(), oc.k_codes[b, :, ns:lq]) and
                np.array_equal(cache.v_codes[b, :n_kv, ns:lq].cpu().numpy(), oc.v_codes[b, :, ns:lq]) and
                np.array_equal(meta_bits(cache.k_meta), oc.k_meta.view(np.uint16)[b, :, ns:lq]) and
                np.array_equal(meta_bits(cache.v_meta), oc.v_meta.view(np.uint16)[b, :, ns:lq]) and
                np.array_equal(cache.k_sink[b, :n_kv, :ns].cpu().numpy().view(np.uint16), oc.k_sink.view(np.uint16)[b, :, :ns]) and
                np.array_equal(cache.v_sink[b, :n_kv, :ns].cpu().numpy().view(np.uint16), oc.v_sink.view(np.uint16)[b, :, :ns]))
        q = w.query(10_000)
        out = cache.attention(torch.from_numpy(q).cuda(), w.sm_scale, hint, n_splits=args.splits)
        torch.cuda.synchronize()
        want = oc.attention(np.ascontiguousarray(q[:n_seq, :n_kv * rep]), w.sm_scale)
        err = float(np.abs(out[:n_seq, :n_kv * rep].cpu().numpy().astype(np.float64) - want).max())
        parity = {"sample": f"sequences 0..{n_seq - 1}, KV heads 0..{n_kv - 1} with their query heads, full context",
                  "cache_bit_exact": exact, "attention_max_abs_err": err, "tolerance": 2e-3}
        if not exact or err > 2e-3:
            raise SystemExit(f"parity failure on the benchmark inputs (configuration {cfg_i}): {parity}")

    # -- per-step inputs, resident in HBM before timing (the same K inputs serve every pass)
    n_in = W_ + K
    k_new = torch.from_numpy(np.stack([w.new_token("k", s) for s in range(n_in)])).cuda()
    v_new = torch.from_numpy(np.stack([w.new_token("v", s) for s in range(n_in)])).cuda()
    q_all = torch.from_numpy(np.stack([w.query(s) for s in range(n_in)])).cuda()
    out = torch.empty_like(q_all[0])
    ev_k = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in ev_k:      # torch creates its events lazily: record once so the handles exist before the library re-records them
        a.record()
        b.record()
    torch.cuda.synchronize()
    args_plain = cache.attn_args(w.sm_scale, hint, args.splits)
    args_timed = [cache.attn_args(w.sm_scale, hint, args.splits, a, b) for a, b in ev_k]
    ev_call = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    state = {"appended": 0}      # decode steps the cache has taken so far

    def step(i, attn_args, ev=None):
        cache.append(k_new[i], v_new[i])
        if ev is not None:
            ev[0].record()
        binding.skvq_decode_attention(cache.cfg, cache.struct, q_all[i], out, attn_args)
        if ev is not None:
            ev[1].record()
        state["appended"] += 1

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def pass_tokens(n_steps, appended_before):      # context tokens attended over n_steps consecutive steps
        return n_steps * (float(lengths0.sum()) + w.batch * appended_before) + w.batch * n_steps * (n_steps + 1) / 2.0

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def one_pass():
        """K steps back to back with nothing else on the stream (an event between two calls would keep the
        dependent launches from overlapping); with a small cache, L2 is flushed before every step instead and
        the steps are timed one by one."""
        barrier()
        t_host0 = time.perf_counter()
        if flush is None:
            e0.record()
            for i in range(K):
                step(W_ + i, args_plain)
            e1.record()
            barrier()
            ms = e0.elapsed_time(e1)
        else:
            ms = 0.0
            for i in range(K):
                flush.fill_(i & 1)
                e0.record()
                step(W_ + i, args_plain)
                e1.record()
                torch.cuda.synchronize()
                ms += e0.elapsed_time(e1)
            barrier()
        return ms, (t_host0, time.perf_counter())

    for i in range(W_):
        step(i, args_plain)
    barrier()
    launches0 = binding.skvq_launch_count()
    first_ms, win = one_pass()
    launches = binding.skvq_launch_count() - launches0
    pass_ms, windows, pass_tok = [first_ms], [win], [pass_tokens(K, state["appended"] - K)]
    goal = (MIN_TIMED_MS if main else MIN_TIMED_MS_OTHER) if args.min_timed_ms < 0 else args.min_timed_ms
    est = sharding.reduce_max(first_ms, dev)
    n_pass = int(min(max(1, -(-goal // max(est, 1e-3))), max(1, MAX_TIMED_STEPS // K)))
    for _ in range(n_pass - 1):
        before = state["appended"]
        ms, win = one_pass()
        pass_ms.append(ms)
        windows.append(win)
        pass_tok.append(pass_tokens(K, before))
    # the same steps again with the library's own events around the partition kernel (an event between the two
    # kernels keeps the merge kernel from overlapping the partition kernel's tail, so this pass measures the
    # dominant kernel alone and the passes above measure the step as a user runs it)
    for i in range(K):
        if flush is not None:
            flush.fill_(i & 1)
        step(W_ + i, args_timed[i])
    torch.cuda.synchronize()
    # and once more with events around the attention call (partition + merge)
    for i in range(K):
        if flush is not None:
            flush.fill_(i & 1)
        step(W_ + i, args_plain, ev_call[i])
    torch.cuda.synchronize()
    kern_ms = [a.elapsed_time(b) for a, b in ev_k]
    call_ms = [a.elapsed_time(b) for a, b in ev_call]
    pass_ms = sharding.reduce_max_list(pass_ms, dev)                  # every pass: the slowest rank
    job_tokens = sharding.reduce_sum(sum(pass_tok) / len(pass_tok), dev)      # per pass, whole job
    med_ms = statistics.median(pass_ms)
    value = job_tokens / (med_ms * 1e-3)

    # -- end to end through the host-buffer entry point (headline configuration only)
    e2e = None
    if main:
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

        def host_step(i):
            binding.skvq_decode_step_host(cache.cfg, cache.struct, hk[i], hv[i], hq[i], hout, staging, args_plain)
            torch.cuda.synchronize()      # the caller reads hout every step
            state["appended"] += 1

        for i in range(W_):
            host_step(i)
        e2e_ms, e2e_tok = [], []
        n_e2e = int(min(max(1, -(-(goal / 2) // max(est * 1.3, 1e-3))), max(1, MAX_E2E_STEPS // K)))
        for _ in range(n_e2e):
            before = state["appended"]
            barrier()
            e0.record()
            for i in range(K):
                host_step(W_ + i)
            e1.record()
            barrier()
            e2e_ms.append(e0.elapsed_time(e1))
            e2e_tok.append(pass_tokens(K, before))
        e2e_ms = sharding.reduce_max_list(e2e_ms, dev)
        e2e_tokens = sharding.reduce_sum(sum(e2e_tok) / len(e2e_tok), dev)
        kv_bytes = w.batch * w.n_kv_heads * w.head_dim * 2
        qo_bytes = w.batch * w.n_q_heads * w.head_dim * 2
        em = statistics.median(e2e_ms)
        e2e = {"value": e2e_tokens / (em * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 2 * kv_bytes + qo_bytes,
               "d2h_bytes_per_step": qo_bytes, "ms_per_step": em / K, "passes": len(e2e_ms),
               "ms_per_step_min": min(e2e_ms) / K, "ms_per_step_max": max(e2e_ms) / K,
               "what": "skvq_decode_step_host: pinned host k/v/q -> device, append, attention, out -> host, "
                       "synchronize, every step"}
    if int(cache.status[0].item()) != 0:      # capacity overflow or a copy that never completed: the numbers would be void
        raise SystemExit(f"the cache's status word is {int(cache.status[0].item())} after the timed passes")
    if rank != 0:
        return None

    peak, peak_src = measured_peak()
    kavg_ms = sum(kern_ms) / len(kern_ms)
    achieved = part_bytes / (kavg_ms * 1e-3) / 1e9
    cavg_ms = sum(call_ms) / len(call_ms)
    plain = not (args.batch or args.context or args.sinks or args.q_heads or args.meta_fp8 or args.splits or args.k_bits or args.v_bits)
    rec = {
        "workload": f"configs[{cfg_i}] {w.name}",
        "config": {"workload": f"configs[{cfg_i}] {w.name}", "batch": w.batch, "n_q_heads": w.n_q_heads,
                   "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "context": int(lengths0.max()),
                   "context_mean": float(lengths0.mean()), "window": w.window, "k_bits": w.k_bits, "v_bits": w.v_bits,
                   "group_size": w.group_size, "alpha": w.alpha, "n_sink": w.n_sink, "meta_fp8": bool(w.meta_fp8),
                   "step": "append 1 token/sequence + decode attention", "cache_bytes": cache.nbytes(),
                   "l2": "cache larger than L2, streamed every step" if flush is None else "L2 flushed between steps",
                   "parallelism": f"replica per GPU x{world}" if world > 1 else "single GPU"},
        "value": value, "unit": UNIT, "steps": K, "passes": len(pass_ms),
        "ms_per_step": med_ms / K, "ms_per_step_min": min(pass_ms) / K, "ms_per_step_max": max(pass_ms) / K,
        "timed_ms_total": sum(pass_ms), "pass_ms_per_step": [round(x / K, 5) for x in pass_ms],
        "step_bytes_per_s_gb": alg_bytes / (med_ms / K * 1e-3) / 1e9,
        "clocks": clocks.summary([(windows[0][0], windows[-1][1])]),      # the passes run back to back: one window
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode-attention partition kernel", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                     "frac_of_nominal_8000": achieved / 8000.0,
                     "algorithmic_bytes_per_launch": part_bytes, "kernel_ms_avg": kavg_ms,
                     "kernel_ms_min": min(kern_ms), "kernel_ms_median": statistics.median(kern_ms),
                     "traffic": NCU_TRAFFIC_BYTES.get(cfg_i) if plain else None,
                     "traffic_source": NCU_TRAFFIC_SOURCE.get(cfg_i) if plain else None,
                     "whole_call": {"what": "partition + merge kernels, all algorithmic bytes (codes, scale/zero, "
                                            "fp16 window, q, out)", "algorithmic_bytes": alg_bytes, "ms_avg": cavg_ms,
                                    "achieved": alg_bytes / (cavg_ms * 1e-3) / 1e9,
                                    "frac": alg_bytes / (cavg_ms * 1e-3) / 1e9 / peak,
                                    "frac_of_nominal_8000": alg_bytes / (cavg_ms * 1e-3) / 1e9 / 8000.0}},
        "prefill_quantize": {"ms": prefill_ms, "bytes_in": prefill_in,
                             "gbs_in": prefill_in / (prefill_ms * 1e-3) / 1e9 if prefill_ms else None,
                             "how": "quantize_append of the first prefill chunk into an empty scratch cache, best of 3 "
                                    "after one warm-up, scaled to all prefilled tokens by bytes"},
        "parity": parity,
    }
    if e2e is not None:
        rec["e2e"] = e2e
    if main and oc is not None and not args.no_cpu_baseline:
        rec["cpu_baseline"], _ = oracle_steps(w, oc, n_seq, n_kv, 3, 1)
    del cache, oc
    torch.cuda.empty_cache()
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=-1,
                    help="run this configuration alone (0..4); default: configuration 3, with 2, 1 and 4 beside it on one GPU")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (small profiling cases)")
    ap.add_argument("--context", type=int, default=0, help="override the context length (small profiling cases)")
    ap.add_argument("--q-heads", type=int, default=0, help="override the number of query heads (other grouped-query ratios)")
    ap.add_argument("--k-bits", type=int, default=0, help="override the key code width (2, 3, 4)")
    ap.add_argument("--v-bits", type=int, default=0, help="override the value code width (2, 3, 4; 15 = three-level '1.5-bit' codes)")
    ap.add_argument("--meta-fp8", action="store_true",
                    help="scale and zero point stored in FP8 E4M3 instead of fp16 (Sec. 4.1; 2.5 bits per element at g32)")
    ap.add_argument("--sinks", type=int, default=0,
                    help="attention sinks: first positions kept fp16 (Sec. 3.2 filter rule; the paper's experiments use 5)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="headline configuration only")
    ap.add_argument("--min-timed-ms", type=float, default=-1.0,
                    help="device time the timed passes must cover (default 500 ms, 300 ms for the other configurations); "
                         "0 = one pass, for profiler captures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    args.steps = max(args.steps, 1)

    from paper_2405_06219_b200 import sharding, workloads
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg_i = DEFAULT_CONFIG if args.config < 0 else args.config

    def shaped(i):
        w0 = workloads.configs()[i]
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
        if args.k_bits:
            w0 = w0.scaled(k_bits=args.k_bits)
        if args.v_bits:
            w0 = w0.scaled(v_bits=args.v_bits)
        return w0

    if args.impl == "reference":
        run_reference(args, cfg_i, shaped(cfg_i), rank)
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
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        gpu_id = str(local_rank)
    others = [] if (args.config >= 0 or args.no_others or world > 1 or args.batch or args.context or args.q_heads or args.k_bits or args.v_bits) \
        else list(OTHER_CONFIGS)
    with ClockSampler(gpu_id) as clocks:
        env = {"torch": torch, "dist": dist, "binding": binding, "sharding": sharding, "workloads": workloads,
               "rank": rank, "world": world, "local_rank": local_rank, "clocks": clocks}
        rec = run_config(cfg_i, shaped(cfg_i), args, env, main=True)
        other_recs = {}
        for i in others:
            r = run_config(i, shaped(i), args, env, main=False)
            if r is not None:
                other_recs[f"configs[{i}]"] = r
    if rank == 0:
        line = {
            "metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": rec["ms_per_step"], "ms_per_step_min": rec["ms_per_step_min"],
            "ms_per_step_max": rec["ms_per_step_max"], "passes": rec["passes"], "timed_ms_total": rec["timed_ms_total"],
            "pass_ms_per_step": rec["pass_ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": rec["config"], "clocks": rec["clocks"], "e2e": rec.get("e2e"), "gpu_launches": rec["gpu_launches"],
            "roofline": rec["roofline"], "prefill_quantize": rec["prefill_quantize"], "parity": rec["parity"],
        }
        if "cpu_baseline" in rec:
            line["cpu_baseline"] = rec["cpu_baseline"]
        if other_recs:
            for r in other_recs.values():
                r.pop("config", None)
            line["other_configs"] = other_recs
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
