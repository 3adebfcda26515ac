"""skvq_decode_attention_noalloc: the decode-attention variant for callers that may not allocate.

A serving engine that gave all spare HBM to its KV cache has no workspace to lend and cannot call
cudaMalloc in its decode loop; this entry point keeps the split partials in an array inside the library
instead.  It must return what skvq_decode_attention returns.  The file name sorts last on purpose: the
entry point shares one device array between all calls, so it runs after every other test has had its turn,
and it must also pass when run alone in a fresh process.
"""
import ctypes

import numpy as np
import pytest
import torch

from helpers import ATTN_TOL, oracle_cache_for
from paper_2405_06219_b200 import binding as B
from paper_2405_06219_b200 import build, workloads


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.lib()


def test_shapes_beyond_the_builtin_array_are_refused_before_any_launch(lib):
    """Host-side check (no GPU needed): 4 x 32 heads x 4001 parts x 528 B is far beyond 8 MiB."""
    c = B.SkvqConfig(4, 32, 8, 128, 2, 2, 32, 128, 1 << 20)
    assert B.skvq_workspace_size(c, 1 << 20, 4000) > B.SKVQ_NOALLOC_SCRATCH_BYTES
    fake = B.SkvqCacheStruct(*([0x1000] * 11), None, None, None)
    before = B.skvq_launch_count()
    rc = lib.skvq_decode_attention_noalloc(ctypes.byref(c), ctypes.byref(fake), 0x1000, 0x1000, 0.1, 1 << 20, 4000,
                                           None)
    assert rc == B.SKVQ_ERR_SCRATCH_LIMIT
    assert "scratch" in B.skvq_strerror(rc)
    assert B.skvq_launch_count() == before


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_workspace_entry_point(lib):
    w = workloads.configs()[2].scaled(context=5000, batch=2)      # GQA, group 32, several splits + window part
    gpu = B.SkvqCache.for_workload(w, 5064)
    ora = oracle_cache_for(w, 5064)
    k, v = w.prefill("k", 5000), w.prefill("v", 5000)
    gpu.append(torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda())
    ora.append(k, v)
    for call, n_splits in enumerate((0, 5)):                      # second call reuses the array with another layout
        q = w.query(call)
        dq = torch.from_numpy(q).cuda()
        want = gpu.attention(dq, w.sm_scale, 5000, n_splits=n_splits)
        got = torch.full_like(dq, float("nan"))
        B.skvq_decode_attention_noalloc(gpu.cfg, gpu.struct, dq, got, w.sm_scale, 5000, n_splits)
        torch.cuda.synchronize()
        g, r = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert np.abs(g - r).max() <= ATTN_TOL
        assert np.abs(g - ora.attention(q, w.sm_scale)).max() <= ATTN_TOL


@pytest.mark.gpu
def test_large_batch_keeps_its_partition_table_in_the_builtin_array(lib):
    """More than 32 sequences: the plan kernel writes the partition header and the per-CTA table in front of the
    partials, so these live in the library's array too.  Ragged, short contexts, some without a quantized prefix."""
    w = workloads.configs()[4].scaled(batch=48, context=1500, ragged=(1, 1500), n_q_heads=4, n_kv_heads=4)
    lengths = w.lengths()
    n = int(lengths.max())
    gpu = B.SkvqCache.for_workload(w, n + 64)
    ora = oracle_cache_for(w, n + 64)
    k, v = w.prefill("k", n), w.prefill("v", n)
    gpu.append(torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(lengths).cuda())
    ora.append(k, v, lengths)
    for call in range(2):
        q = w.query(call)
        dq = torch.from_numpy(q).cuda()
        want = gpu.attention(dq, w.sm_scale, n)
        got = torch.full_like(dq, float("nan"))
        B.skvq_decode_attention_noalloc(gpu.cfg, gpu.struct, dq, got, w.sm_scale, n, 0)
        torch.cuda.synchronize()
        g, r = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert np.abs(g - r).max() <= ATTN_TOL
        assert np.abs(g - ora.attention(q, w.sm_scale)).max() <= ATTN_TOL


@pytest.mark.gpu
def test_stream_ordered_calls_share_the_array_without_a_host_sync(lib):
    """Two calls enqueued back to back on one stream, different queries and different split counts: the second call's
    kernels are launched behind the first call's merge and reuse the array with another layout.  Stream order is all
    a caller has to provide; both outputs must match the workspace entry point."""
    w = workloads.configs()[2].scaled(context=4000, batch=2)
    gpu = B.SkvqCache.for_workload(w, 4064)
    k, v = w.prefill("k", 4000), w.prefill("v", 4000)
    gpu.append(torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda())
    q0, q1 = torch.from_numpy(w.query(7)).cuda(), torch.from_numpy(w.query(8)).cuda()
    want0 = gpu.attention(q0, w.sm_scale, 4000, n_splits=0)
    want1 = gpu.attention(q1, w.sm_scale, 4000, n_splits=3)
    got0, got1 = torch.full_like(q0, float("nan")), torch.full_like(q1, float("nan"))
    torch.cuda.synchronize()
    for _ in range(8):      # several rounds, nothing but the calls on the stream
        B.skvq_decode_attention_noalloc(gpu.cfg, gpu.struct, q0, got0, w.sm_scale, 4000, 0)
        B.skvq_decode_attention_noalloc(gpu.cfg, gpu.struct, q1, got1, w.sm_scale, 4000, 3)
    torch.cuda.synchronize()
    for got, want in ((got0, want0), (got1, want1)):
        g, r = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert np.abs(g - r).max() <= ATTN_TOL
