"""The debugging build (-DSKVQ_CHECKED): same entry points, every row / slot / partial index compared with its buffer
before use.  No memory checker runs with these tests, so this build stands in for one: the decode path of several
shapes must give the oracle's results with the bounds bit of the status word still clear."""
import numpy as np
import pytest
import torch

from helpers import ATTN_TOL, assert_cache_bit_exact, oracle_cache_for
from paper_2405_06219_b200 import binding as B
from paper_2405_06219_b200 import build, workloads

pytestmark = pytest.mark.gpu
CF = workloads.configs()


@pytest.fixture(scope="module", autouse=True)
def checked_library():
    build.build_library()
    path = build.build_library(checked=True)
    B.use_library(path)
    try:
        yield B.lib()
    finally:
        B.use_library(None)
        B.lib()


def test_checked_library_exports_the_same_entry_points(checked_library):
    for n in B.EXPORTS:
        assert hasattr(checked_library, n), n


@pytest.mark.parametrize("cfg_i,kw,lens", [
    (1, dict(context=2100, batch=2, n_q_heads=4, n_kv_heads=4), [2100, 333]),                       # integer kernel, ragged
    (2, dict(context=1800, batch=2, n_sink=5), [1800, 1800]),                                       # grouped-query kernel, sinks
    (4, dict(context=900, batch=40, ragged=(1, 900), n_q_heads=2, n_kv_heads=2), None),             # plan kernel, 4-bit, window 256
    (2, dict(context=1000, batch=1, n_q_heads=24, meta_fp8=True), [1000]),                          # tcgen05 kernel
    (1, dict(context=900, batch=1, n_q_heads=4, n_kv_heads=4, k_bits=3, v_bits=3, group_size=64, group_bounds=(0, 32, 128)), [900]),   # tcgen05 kernel: 3-bit streams, groups of unequal width
])
def test_decode_path_stays_in_bounds(cfg_i, kw, lens):
    w = CF[cfg_i].scaled(**kw)
    lengths = w.lengths() if lens is None else np.array(lens, np.int32)
    n = int(lengths.max())
    gpu = B.SkvqCache.for_workload(w, n + 80)
    ora = oracle_cache_for(w, n + 80)
    k, v = w.prefill("k", n), w.prefill("v", n)
    gpu.append(torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), torch.from_numpy(lengths).cuda())
    ora.append(k, v, lengths)
    for s in range(6):
        kn, vn, q = w.new_token("k", s), w.new_token("v", s), w.query(s)
        gpu.append(torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda())
        ora.append(kn, vn)
        out = gpu.attention(torch.from_numpy(q).cuda(), w.sm_scale, n + 6, n_splits=(0, 3)[s & 1])
        torch.cuda.synchronize()
        assert np.abs(out.cpu().numpy().astype(np.float64) - ora.attention(q, w.sm_scale)).max() <= ATTN_TOL
    assert_cache_bit_exact(gpu, ora)
    assert int(gpu.status[0].item()) == 0          # neither SKVQ_STATUS_BOUNDS nor any other bit
