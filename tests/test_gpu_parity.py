"""GPU parity: the CUDA library against the CPU oracle through the C ABI.

Quantized codes, scales/zeros, window contents and lengths must be bit-exact; the fp16 attention
output must be within 2e-3 (max-abs) of the oracle's fp64 attention over the same cache.
"""
import numpy as np
import pytest
import torch

from helpers import ATTN_TOL, assert_cache_bit_exact, oracle_cache_for
from paper_2405_06219_b200 import binding as B
from paper_2405_06219_b200 import build, workloads

pytestmark = pytest.mark.gpu
CF = workloads.configs()


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build_library()
    B.lib()


def small(i, **kw):
    return CF[i].scaled(**kw)


def both_caches(w, max_tokens):
    return B.SkvqCache.for_workload(w, max_tokens), oracle_cache_for(w, max_tokens)


def dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def attention_both(gpu, ora, w, step=0, n_splits=0):
    q = w.query(step)
    hint = int(ora.lengths.max())
    out = gpu.attention(dev(q), w.sm_scale, hint, n_splits=n_splits)
    torch.cuda.synchronize()
    want = ora.attention(q, w.sm_scale)
    return out.cpu().numpy().astype(np.float64), want


# ------------------------------------------------------------------ quantize_append, bit-exact
@pytest.mark.parametrize("cfg_i,kw,n", [
    (0, dict(context=700), 700),                      # 2-bit, g128, MHA: several tiles and a ragged tail
    (2, dict(context=900, batch=2), 900),             # g32 GQA
    (4, dict(context=1000, batch=3, ragged=None), 1000),   # 4-bit g64, window 256
    (0, dict(context=100), 100),                      # shorter than the window: nothing quantized
    (0, dict(context=128), 128),                      # exactly the window
    (0, dict(context=129), 129),                      # one token slides out
    (0, dict(context=300, window=0), 300),            # no window at all
    (1, dict(context=2100, batch=2, n_kv_heads=4, n_q_heads=4, k_bits=4, v_bits=2, group_size=64), 2100),  # mixed widths
])
def test_prefill_quantize_bit_exact(cfg_i, kw, n):
    w = small(cfg_i, **kw)
    gpu, ora = both_caches(w, n + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    gpu.append(dev(k), dev(v))
    assert ora.append(k, v) == 0
    assert_cache_bit_exact(gpu, ora)
    assert int(gpu.status[0].item()) == 0


def test_chunked_and_single_token_appends_bit_exact():
    w = small(2, context=700, batch=2)
    gpu, ora = both_caches(w, 800)
    k, v = w.prefill("k", 700), w.prefill("v", 700)
    t = 0
    for step in (1, 1, 5, 130, 127, 1, 1, 300, 64, 70):
        gpu.append(dev(k[:, t:t + step]), dev(v[:, t:t + step]))
        ora.append(k[:, t:t + step], v[:, t:t + step])
        t += step
        assert_cache_bit_exact(gpu, ora)
    assert t == 700
    for s in range(40):                                                # decode-style single tokens
        kn, vn = w.new_token("k", s), w.new_token("v", s)
        gpu.append(dev(kn), dev(vn))
        ora.append(kn, vn)
    assert_cache_bit_exact(gpu, ora)
    bulk = oracle_cache_for(w, 800)
    bulk.append(np.concatenate([k] + [w.new_token("k", s) for s in range(40)], 1),
                np.concatenate([v] + [w.new_token("v", s) for s in range(40)], 1))
    assert_cache_bit_exact(gpu, bulk)


@pytest.mark.parametrize("cfg_i,kw,chunks", [
    (1, dict(context=5000, batch=2, n_q_heads=4, n_kv_heads=4), (37, 3000, 64, 1500, 399)),                # g128: runs of more than 8 tiles, a 64-row tail
    (4, dict(context=3000, batch=2, ragged=None, n_q_heads=4, n_kv_heads=4), (1000, 1, 1300, 699)),        # 4-bit g64, window 256
    (2, dict(context=2600, batch=1, meta_fp8=True, n_sink=5), (700, 1900)),                                 # g32, FP8 parameters, sinks
    (2, dict(context=2100, batch=2, group_size=64, group_bounds=(0, 96, 128)), (1100, 1000)),               # two groups of unequal width
    (4, dict(context=1700, batch=1, ragged=None, n_q_heads=4, n_kv_heads=4, k_bits=4, v_bits=2, group_size=32,
             group_bounds=(0, 32, 64, 96, 128)), (900, 800)),                                               # mixed widths, boundaries given but equal
    (1, dict(context=2500, batch=2, n_q_heads=4, n_kv_heads=4, k_bits=3, v_bits=3, group_size=64), (1300, 70, 1130)),  # 3-bit streams closed up from 4-bit fields
    (2, dict(context=2300, batch=2, k_bits=3, v_bits=15, group_size=64, group_bounds=(0, 32, 128)), (1000, 1300)),     # three-level values: base-3 bytes, a code handed across the row's halves
    (1, dict(context=1900, batch=1, n_q_heads=4, n_kv_heads=4, v_bits=15, meta_fp8=True), (900, 1000)),
])
def test_bulk_appends_on_top_of_existing_tokens_bit_exact(cfg_i, kw, chunks):
    """The tile kernel of bulk appends: chunks that start at any length, several CTA runs, ragged per-sequence counts."""
    w = small(cfg_i, **kw)
    n = sum(chunks)
    gpu, ora = both_caches(w, n + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    t = 0
    for step in chunks:
        gpu.append(dev(k[:, t:t + step]), dev(v[:, t:t + step]))
        ora.append(k[:, t:t + step], v[:, t:t + step])
        t += step
        assert_cache_bit_exact(gpu, ora)
    assert int(gpu.status[0].item()) == 0
    # the same tokens with per-sequence counts: sequence b takes only part of the chunk
    gpu2, ora2 = both_caches(w, n + 64)
    counts = np.array([n - 517 * b for b in range(w.batch)], np.int32)
    gpu2.append(dev(k), dev(v), dev(counts))
    ora2.append(k, v, counts)
    assert_cache_bit_exact(gpu2, ora2)
    got, want = attention_both(gpu2, ora2, w)
    assert np.abs(got - want).max() <= ATTN_TOL


def test_ragged_append_and_overflow_flag():
    w = small(4, context=600, batch=4, ragged=None)
    gpu, ora = both_caches(w, 640)
    k, v = w.prefill("k", 600), w.prefill("v", 600)
    n = np.array([600, 0, 257, 13], np.int32)
    gpu.append(dev(k), dev(v), dev(n))
    ora.append(k, v, n)
    assert_cache_bit_exact(gpu, ora)
    # second ragged round; sequence 0 would exceed max_tokens = 640 and must stay untouched
    n2 = np.array([41, 300, 0, 41], np.int32)
    gpu.append(dev(k[:, :300]), dev(v[:, :300]), dev(n2))
    assert ora.append(k[:, :300], v[:, :300], n2) == -1
    assert_cache_bit_exact(gpu, ora)
    assert ora.lengths.tolist() == [600, 300, 257, 54]
    assert int(gpu.status[0].item()) & B.SKVQ_STATUS_OVERFLOW


# ------------------------------------------------------------------ decode attention, <= 2e-3
@pytest.mark.parametrize("cfg_i,kw,n", [
    (0, dict(), 4096),                                               # configuration 0 in full
    (1, dict(context=3000, batch=2), 3000),
    (2, dict(context=5000, batch=2), 5000),                          # GQA 4:1, g32
    (3, dict(context=9000, n_q_heads=4, n_kv_heads=4), 9000),
    (4, dict(context=1500, batch=3, ragged=None), 1500),             # 4-bit g64 W256
    (0, dict(context=100), 100), (0, dict(context=128), 128), (0, dict(context=129), 129),
    (0, dict(context=1), 1), (0, dict(context=500, window=0), 500),
    (2, dict(context=777, batch=1, n_q_heads=16, n_kv_heads=2), 777),   # 8 query heads per KV head
    (2, dict(context=3000, batch=1, n_q_heads=8, n_kv_heads=4), 3000),                    # 2 heads per KV head, g32
    (1, dict(context=3000, batch=1, n_q_heads=8, n_kv_heads=2), 3000),                    # 4 heads per KV head, g128
    (1, dict(context=2500, batch=2, n_q_heads=4, n_kv_heads=4, group_size=32), 2500),     # MHA with fine groups
    (1, dict(context=2500, batch=1, n_q_heads=8, n_kv_heads=4, group_size=64), 2500),     # 2 heads per KV head, g64
    (2, dict(context=4160, batch=1, n_q_heads=4, n_kv_heads=1, group_size=64), 4160),     # 4 heads per KV head, g64, full tiles only
    (4, dict(context=2777, batch=2, ragged=None, n_q_heads=4, n_kv_heads=4, k_bits=4, v_bits=2), 2777),     # mixed widths
    (4, dict(context=2777, batch=2, ragged=None, n_q_heads=4, n_kv_heads=4, k_bits=2, v_bits=4, group_size=128), 2777),
    (4, dict(context=3100, batch=1, ragged=None, n_q_heads=4, n_kv_heads=4, group_size=128, window=128), 3100),   # 4-bit, one group
    (4, dict(context=2000, batch=1, ragged=None, n_q_heads=8, n_kv_heads=4), 2000),      # 4-bit with 2 heads per KV head: tcgen05 kernel
    (2, dict(context=5300, batch=2, ragged=None, n_q_heads=12, n_kv_heads=4), 5300),     # 3 heads per KV head, g32: tcgen05 kernel
    (1, dict(context=70000, batch=1, n_q_heads=6, n_kv_heads=2), 70000),                 # 3 heads per KV head, g128, many tiles per CTA
    (2, dict(context=1000, batch=33, ragged=(1, 1000), n_q_heads=3, n_kv_heads=1, group_size=64), 1000),   # 3 heads, g64, plan kernel, short and empty prefixes
    (2, dict(context=6000, batch=1, n_q_heads=64, n_kv_heads=8), 6000),                  # 8 heads per KV head: two tcgen05 launches
    (1, dict(context=3500, batch=2, n_q_heads=10, n_kv_heads=2), 3500),                  # 5 heads per KV head, g128: 4 + 1
])
def test_attention_matches_oracle(cfg_i, kw, n):
    w = small(cfg_i, **kw)
    gpu, ora = both_caches(w, n + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    gpu.append(dev(k), dev(v))
    ora.append(k, v)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w)
    assert np.abs(got - want).max() <= ATTN_TOL


# ------------------------------------------------------------------ attention sinks (Sec. 3.2 filter rules)
@pytest.mark.parametrize("cfg_i,kw,n", [
    (1, dict(context=3000, batch=2, n_kv_heads=4, n_q_heads=4, n_sink=5), 3000),              # integer kernel, 5 sinks as in the paper
    (2, dict(context=2900, batch=1, n_sink=5), 2900),                                         # grouped-query kernel
    (4, dict(context=1400, batch=2, ragged=None, n_kv_heads=4, n_q_heads=4, n_sink=64), 1400),   # 4-bit, a whole tile of sinks
    (2, dict(context=800, batch=1, n_q_heads=16, n_kv_heads=2, n_sink=7), 800),               # 8 heads per KV head: two tcgen05 launches
    (2, dict(context=900, batch=2, ragged=None, n_sink=64), 900),                             # grouped-query kernel, first tile all sinks
    (2, dict(context=700, batch=1, n_q_heads=16, n_kv_heads=2, n_sink=64), 700),              # 8 heads per KV head (two tcgen05 launches), first tile all sinks
    (2, dict(context=1900, batch=1, n_q_heads=6, n_kv_heads=2, n_sink=9), 1900),              # tcgen05 kernel (3 heads per KV head)
    (0, dict(context=130, n_sink=5), 130),                                                    # fewer tokens out of the window than sinks
    (0, dict(context=300, window=0, n_sink=3), 300),
])
def test_sinks_stay_fp16_and_attention_matches_oracle(cfg_i, kw, n):
    w = small(cfg_i, **kw)
    gpu, ora = both_caches(w, n + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    cut = n // 3
    gpu.append(dev(k[:, :cut]), dev(v[:, :cut]))                      # in two pieces: sinks leave the window in either call
    gpu.append(dev(k[:, cut:]), dev(v[:, cut:]))
    ora.append(k, v)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w)
    assert np.abs(got - want).max() <= ATTN_TOL
    for s in range(6):                                                # decode steps: single-token appends
        kn, vn = w.new_token("k", s), w.new_token("v", s)
        gpu.append(dev(kn), dev(vn))
        ora.append(kn, vn)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w, step=1)
    assert np.abs(got - want).max() <= ATTN_TOL


# ------------------------------------------------------------------ FP8 E4M3 scale and zero point (Sec. 4.1)
@pytest.mark.parametrize("cfg_i,kw,n", [
    (2, dict(context=3000, batch=2, meta_fp8=True), 3000),                                     # 2-bit g32, 4 heads per KV head: 2.5 bits
    (1, dict(context=2500, batch=2, n_q_heads=4, n_kv_heads=4, meta_fp8=True), 2500),          # one head per KV head, g128
    (1, dict(context=2100, batch=1, n_q_heads=16, n_kv_heads=2, group_size=64, meta_fp8=True, n_sink=5), 2100),   # 8 heads, g64, sinks
    (4, dict(context=1300, batch=2, ragged=None, n_q_heads=4, n_kv_heads=4, meta_fp8=True), 1300),   # 4-bit g64, integer kernel
    (4, dict(context=1100, batch=1, ragged=None, n_q_heads=8, n_kv_heads=4, meta_fp8=True), 1100),   # 4-bit, 2 heads per KV head: tcgen05 kernel
    (2, dict(context=1500, batch=1, n_q_heads=24, meta_fp8=True), 1500),                             # 3 heads per KV head: tcgen05 kernel
    (4, dict(context=1500, batch=1, ragged=None, n_q_heads=4, n_kv_heads=4, k_bits=4, v_bits=2, group_size=128, meta_fp8=True), 1500),   # mixed widths
    (0, dict(context=200, meta_fp8=True), 200),
])
def test_fp8_parameters_bit_exact_cache_and_attention(cfg_i, kw, n):
    w = small(cfg_i, **kw)
    gpu, ora = both_caches(w, n + 64)
    assert gpu.k_meta.dtype == torch.uint8 and gpu.k_meta.shape[-2:] == (128 // w.group_size, 2)      # two bytes per (token, group)
    k, v = w.prefill("k", n), w.prefill("v", n)
    cut = (n * 2) // 3
    gpu.append(dev(k[:, :cut]), dev(v[:, :cut]))                      # bulk tiles, ragged ends, evictions from the ring
    gpu.append(dev(k[:, cut:]), dev(v[:, cut:]))
    ora.append(k, v)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w)
    assert np.abs(got - want).max() <= ATTN_TOL
    for s in range(5):                                                # decode steps: single-token appends
        kn, vn = w.new_token("k", s), w.new_token("v", s)
        gpu.append(dev(kn), dev(vn))
        ora.append(kn, vn)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w, step=1)
    assert np.abs(got - want).max() <= ATTN_TOL


def test_attention_ragged_batch_with_empty_sequence():
    w = small(4, context=2000, batch=6, ragged=None)
    gpu, ora = both_caches(w, 2048)
    k, v = w.prefill("k", 2000), w.prefill("v", 2000)
    n = np.array([2000, 0, 256, 257, 1024, 3], np.int32)
    gpu.append(dev(k), dev(v), dev(n))
    ora.append(k, v, n)
    got, want = attention_both(gpu, ora, w)
    assert np.abs(got - want).max() <= ATTN_TOL
    assert not got[1].any()


@pytest.mark.parametrize("n_splits", [1, 2, 3, 7, 64])
def test_split_count_does_not_change_the_result(n_splits):
    w = small(2, context=6000, batch=1)
    gpu, ora = both_caches(w, 6016)
    k, v = w.prefill("k", 6000), w.prefill("v", 6000)
    gpu.append(dev(k), dev(v))
    ora.append(k, v)
    got, want = attention_both(gpu, ora, w, n_splits=n_splits)
    assert np.abs(got - want).max() <= ATTN_TOL


def test_decode_loop_append_then_attend():
    """Steady-state decoding: each step appends one token (one slides out of the window) and attends."""
    w = small(3, context=1000, n_q_heads=8, n_kv_heads=8)
    gpu, ora = both_caches(w, 1100)
    k, v = w.prefill("k", 1000), w.prefill("v", 1000)
    gpu.append(dev(k), dev(v))
    ora.append(k, v)
    for s in range(20):
        kn, vn = w.new_token("k", s), w.new_token("v", s)
        gpu.append(dev(kn), dev(vn))
        ora.append(kn, vn)
        got, want = attention_both(gpu, ora, w, step=s)
        assert np.abs(got - want).max() <= ATTN_TOL
    assert_cache_bit_exact(gpu, ora)


@pytest.mark.parametrize("cfg_i,kw", [
    (0, dict(context=300, n_q_heads=2, n_kv_heads=2)),                       # one or two partition CTAs: room for the merge CTAs beside them
    (2, dict(context=400, batch=2, n_q_heads=8, n_kv_heads=2)),              # grouped-query kernel
    (2, dict(context=700, batch=1, n_q_heads=6, n_kv_heads=2)),              # tcgen05 kernel
    (4, dict(context=600, batch=40, ragged=(1, 600), n_q_heads=2, n_kv_heads=2)),   # plan kernel in the chain, 4-bit
])
def test_back_to_back_steps_without_synchronisation(cfg_i, kw):
    """Many decode steps (append one token, attend) enqueued with no host synchronisation in between, on contexts so
    short that only a few partition CTAs exist and merge CTAs can be resident beside them: every step's output must
    see that step's appended token in the window and that step's lengths (the kernels of a step are chained with
    programmatic dependent launches, so this is the ordering guarantee of the chain)."""
    w = small(cfg_i, **kw)
    n_steps = 48
    lengths = w.lengths()
    n = int(lengths.max())
    gpu, ora = both_caches(w, n + n_steps + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    gpu.append(dev(k), dev(v), dev(lengths))
    ora.append(k, v, lengths)
    kn = [w.new_token("k", s) for s in range(n_steps)]
    vn = [w.new_token("v", s) for s in range(n_steps)]
    qs = [w.query(s) for s in range(n_steps)]
    dk, dv, dq = dev(np.stack(kn)), dev(np.stack(vn)), dev(np.stack(qs))
    outs = torch.zeros_like(dq)
    args = gpu.attn_args(w.sm_scale, n + n_steps)
    torch.cuda.synchronize()
    for s in range(n_steps):
        gpu.append(dk[s], dv[s])
        B.skvq_decode_attention(gpu.cfg, gpu.struct, dq[s], outs[s], args)
    torch.cuda.synchronize()
    got = outs.cpu().numpy().astype(np.float64)
    for s in range(n_steps):
        ora.append(kn[s], vn[s])
        want = ora.attention(qs[s], w.sm_scale)
        assert np.abs(got[s] - want).max() <= ATTN_TOL, f"step {s}"
    assert_cache_bit_exact(gpu, ora)


@pytest.mark.parametrize("cfg_i,kw", [(1, dict(context=3000, batch=2, n_q_heads=4, n_kv_heads=4)),       # integer kernel
                                       (2, dict(context=2500, batch=2)),                                 # grouped-query kernel
                                       (2, dict(context=2500, batch=1, n_q_heads=24))])                  # tcgen05 kernel
def test_decode_step_replays_from_a_cuda_graph(cfg_i, kw):
    """The calls only enqueue work and read the lengths on the device, so one captured decode step (append one
    token, attend) can be replayed with new inputs in the same buffers."""
    w = small(cfg_i, **kw)
    n = w.context
    gpu, ora = both_caches(w, n + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    gpu.append(dev(k), dev(v))
    ora.append(k, v)
    k_in, v_in, q_in = dev(w.new_token("k", 0)), dev(w.new_token("v", 0)), dev(w.query(0))
    out = torch.empty_like(q_in)
    args = gpu.attn_args(w.sm_scale, n + 64)                          # workspace allocated before the capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                                     # one eager step first: kernels get configured
        gpu.append(k_in, v_in)
        B.skvq_decode_attention(gpu.cfg, gpu.struct, q_in, out, args)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    ora.append(w.new_token("k", 0), w.new_token("v", 0))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        gpu.append(k_in, v_in)
        B.skvq_decode_attention(gpu.cfg, gpu.struct, q_in, out, args)
    for s in range(1, 6):
        kn, vn, q = w.new_token("k", s), w.new_token("v", s), w.query(s)
        k_in.copy_(dev(kn)); v_in.copy_(dev(vn)); q_in.copy_(dev(q))
        graph.replay()
        torch.cuda.synchronize()
        ora.append(kn, vn)
        want = ora.attention(q, w.sm_scale)
        assert np.abs(out.cpu().numpy().astype(np.float64) - want).max() <= ATTN_TOL
    assert_cache_bit_exact(gpu, ora)


@pytest.mark.parametrize("pinned", [True, False])
def test_host_buffer_decode_step(pinned):
    """Page-locked and pageable host buffers alike."""
    w = small(1, context=2000, batch=2)
    gpu, ora = both_caches(w, 2100)
    k, v = w.prefill("k", 2000), w.prefill("v", 2000)
    gpu.append(dev(k), dev(v))
    ora.append(k, v)
    kn, vn, q = w.new_token("k", 0), w.new_token("v", 0), w.query(5)
    hk, hv, hq = (torch.from_numpy(np.ascontiguousarray(x)) for x in (kn, vn, q))
    hout = torch.zeros(q.shape, dtype=torch.float16)
    if pinned:      # one pinned buffer, k, v and q back to back: a single copy
        hin = torch.cat([hk.reshape(-1), hv.reshape(-1), hq.reshape(-1)]).pin_memory()
        hk, hv, hq = hin[:hk.numel()], hin[hk.numel():2 * hk.numel()], hin[2 * hk.numel():]
        hout = hout.pin_memory()
    staging = torch.empty(B.skvq_step_staging_size(gpu.cfg), dtype=torch.uint8, device="cuda")
    before = B.skvq_launch_count()
    B.skvq_decode_step_host(gpu.cfg, gpu.struct, hk, hv, hq, hout, staging, gpu.attn_args(w.sm_scale, 2001))
    torch.cuda.synchronize()
    assert B.skvq_launch_count() - before >= 3
    ora.append(kn, vn)
    want = ora.attention(q, w.sm_scale)
    assert np.abs(hout.numpy().astype(np.float64) - want).max() <= ATTN_TOL
    assert_cache_bit_exact(gpu, ora)


def test_adversarial_values_stay_bit_exact():
    """Constant groups (h = 0), zeros of both signs, tiny and large magnitudes, exact rounding ties."""
    w = small(2, context=400, batch=1)
    gpu, ora = both_caches(w, 512)
    rng = np.random.default_rng(5)
    k = w.prefill("k", 400).copy()
    v = w.prefill("v", 400).copy()
    k[0, 0:40] = np.float16(1.25)                       # constant rows
    k[0, 40:60] = np.float16(0.0)
    k[0, 60:80, :, ::2] = np.float16(-0.0)
    v[0, 0:50] = (rng.integers(0, 4, (50, 8, 128)) * 0.5 - 1.0).astype(np.float16)     # exact levels
    v[0, 50:100] = (rng.integers(0, 7, (50, 8, 128)) * 0.25 - 0.75).astype(np.float16)  # half-way ties
    v[0, 100:120] = (rng.standard_normal((20, 8, 128)) * 1e-6).astype(np.float16)      # subnormal range
    k[0, 100:120] = np.clip(rng.standard_normal((20, 8, 128)) * 2e4, -6e4, 6e4).astype(np.float16)   # near the fp16 maximum
    gpu.append(dev(k), dev(v))
    ora.append(k, v)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w)
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= ATTN_TOL


# ------------------------------------------------------------------ groups of unequal width (split_groups of Algorithm 1) and 3-bit codes
@pytest.mark.parametrize("cfg_i,kw,n", [
    (1, dict(context=2300, batch=2, n_q_heads=4, n_kv_heads=4, group_size=64, group_bounds=(0, 32, 128)), 2300),    # one head per KV head
    (2, dict(context=1900, batch=1, group_size=64, group_bounds=(0, 96, 128)), 1900),                              # 4 heads per KV head
    (4, dict(context=1200, batch=2, ragged=None, n_q_heads=4, n_kv_heads=4, group_bounds=(0, 32, 128)), 1200),     # 4-bit, window 256
    (2, dict(context=1500, batch=1, group_size=64, group_bounds=(0, 32, 128), meta_fp8=True, n_sink=5), 1500),     # FP8 parameters, sinks
    (1, dict(context=2100, batch=1, n_q_heads=4, n_kv_heads=4, k_bits=3, v_bits=3, group_size=64), 2100),          # 3-bit, the setting of Sec. 4.3
    (2, dict(context=1700, batch=2, k_bits=3, v_bits=2), 1700),                                                    # 3-bit keys, 2-bit values, g32, GQA
    (4, dict(context=1300, batch=1, ragged=None, n_q_heads=8, n_kv_heads=4, k_bits=4, v_bits=3, group_bounds=(0, 96, 128)), 1300),
    (0, dict(context=700, k_bits=3, v_bits=3, meta_fp8=True), 700),
    (2, dict(context=2600, batch=1, n_q_heads=24, group_size=64, group_bounds=(0, 96, 128)), 2600),               # 3 heads per KV head, unequal groups
    (2, dict(context=1400, batch=2, n_q_heads=40, group_size=64, group_bounds=(0, 32, 128), k_bits=3, v_bits=4), 1400),   # 5 heads: two launches, 3-bit keys, 4-bit values
    (4, dict(context=2300, batch=2, ragged=None, n_q_heads=8, n_kv_heads=2, group_size=32), 2300),               # 4-bit, 4 heads per KV head, group 32
    (4, dict(context=1900, batch=1, ragged=None, n_q_heads=4, n_kv_heads=4, group_size=32, k_bits=4, v_bits=2), 1900),   # 4-bit keys, 2-bit values, group 32, one head per KV head
    (1, dict(context=70000, batch=1, n_q_heads=2, n_kv_heads=1, k_bits=3, v_bits=3), 70000),                     # 3-bit, many tiles per CTA: the int32 value sums fold on their own
    # three-level ("1.5-bit") values, the K2 V1.5 setting of the abstract and Sec. 4.2: 26-byte rows, five base-3 digits per byte
    (1, dict(context=2200, batch=2, n_q_heads=4, n_kv_heads=4, v_bits=15), 2200),                                 # group 128, one head per KV head
    (2, dict(context=1800, batch=2, v_bits=15, n_sink=5), 1800),                                                  # group 32, 4 heads per KV head, sinks
    (2, dict(context=1500, batch=1, v_bits=15, group_size=64, group_bounds=(0, 96, 128), meta_fp8=True), 1500),   # unequal groups, FP8 parameters
    (4, dict(context=1300, batch=3, ragged=None, n_q_heads=12, n_kv_heads=2, k_bits=4, v_bits=15), 1300),         # 4-bit keys, 6 heads per KV head: two launches
    (1, dict(context=40000, batch=1, n_q_heads=2, n_kv_heads=1, k_bits=3, v_bits=15, group_size=64), 40000),      # 3-bit keys, many tiles per CTA
])
def test_unequal_groups_and_three_bit_codes_bit_exact_cache_and_attention(cfg_i, kw, n):
    w = small(cfg_i, **kw)
    gpu, ora = both_caches(w, n + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    cut = (n * 3) // 5
    gpu.append(dev(k[:, :cut]), dev(v[:, :cut]))                      # bulk-sized pieces, ragged ends, evictions from the ring
    gpu.append(dev(k[:, cut:]), dev(v[:, cut:]))
    ora.append(k, v)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w)
    assert np.abs(got - want).max() <= ATTN_TOL
    for s in range(5):                                                # decode steps: single-token appends
        kn, vn = w.new_token("k", s), w.new_token("v", s)
        gpu.append(dev(kn), dev(vn))
        ora.append(kn, vn)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w, step=1, n_splits=3)
    assert np.abs(got - want).max() <= ATTN_TOL
    assert int(gpu.status[0].item()) == 0


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_widths_groups_windows_and_chunkings(seed):
    """A seeded sweep over the options of the cache: group size and boundaries, code widths (2, 3, 4 bits, three-level
    values), KV heads and query heads per KV head, batch, window, sinks, FP8 parameters, and how the tokens arrive."""
    rng = np.random.default_rng(seed)
    for _ in range(12):
        G = int(rng.choice([32, 64, 128]))
        ng = 128 // G
        kw = dict(batch=int(rng.choice([1, 2, 3])), ragged=None, n_kv_heads=int(rng.choice([1, 2, 3, 5])), k_bits=int(rng.choice([2, 3, 4])),
                  v_bits=int(rng.choice([2, 3, 4, 15])), group_size=G, window=int(rng.choice([0, 64, 128, 256])),
                  n_sink=int(rng.choice([0, 0, 5])), meta_fp8=bool(rng.random() < 0.3))
        kw["n_q_heads"] = kw["n_kv_heads"] * int(rng.choice([1, 2, 4]))
        if ng >= 2 and rng.random() < 0.4:
            cuts = sorted(rng.choice(np.arange(1, 4), size=ng - 1, replace=False).tolist())
            kw["group_bounds"] = tuple([0] + [32 * c for c in cuts] + [128])
        chunks = [int(x) for x in rng.integers(1, 1500, size=int(rng.integers(1, 5)))]
        n = sum(chunks)
        w = small(1, context=n, **kw)
        gpu, ora = both_caches(w, n + 64)
        k, v = w.prefill("k", n), w.prefill("v", n)
        t = 0
        for step in chunks:
            gpu.append(dev(k[:, t:t + step]), dev(v[:, t:t + step]))
            ora.append(k[:, t:t + step], v[:, t:t + step])
            t += step
        assert_cache_bit_exact(gpu, ora)
        assert int(gpu.status[0].item()) == 0, (kw, chunks)
        got, want = attention_both(gpu, ora, w)
        assert np.abs(got - want).max() <= ATTN_TOL, (kw, chunks)


def test_calibrated_reorder_groups_and_clip_factors_through_the_library():
    """The offline calibrator's arrays (per-head reorder index, boundaries that differ between heads and between keys
    and values, per-group clip factors) fed to the library and to the oracle alike."""
    from oracle import skvq_oracle as orc
    from paper_2405_06219_b200 import calibrate as cal
    w = small(2, context=1600, batch=2, n_kv_heads=4, n_q_heads=8, group_size=64)
    k, v = w.prefill("k", 1600), w.prefill("v", 1600)
    q_cal = np.stack([w.query(100 + s)[0] for s in range(3)])
    res = cal.calibrate(q_cal, k[0, :384], v[0, :384], n_groups=2, k_bits=2, v_bits=2, sm_scale=w.sm_scale, grid=[0.8, 0.9, 1.0])
    assert len({tuple(b) for b in res["bounds_k"].tolist()} | {tuple(b) for b in res["bounds_v"].tolist()}) >= 2
    gpu = B.SkvqCache(w.batch, w.n_q_heads, w.n_kv_heads, 128, 2, 2, 64, w.window, 1700, res["reorder_k"], res["reorder_v"],
                      res["alpha_k"], res["alpha_v"], bounds_k=res["bounds_k"], bounds_v=res["bounds_v"])
    ora = orc.OracleCache(w.batch, w.n_q_heads, w.n_kv_heads, 128, 2, 2, 64, w.window, 1700, res["reorder_k"], res["reorder_v"],
                          res["alpha_k"], res["alpha_v"], bounds_k=res["bounds_k"], bounds_v=res["bounds_v"])
    gpu.append(dev(k), dev(v))
    ora.append(k, v)
    assert_cache_bit_exact(gpu, ora)
    got, want = attention_both(gpu, ora, w)
    assert np.abs(got - want).max() <= ATTN_TOL
