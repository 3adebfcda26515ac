"""The offline calibrator (reorder index, group boundaries, clip factors): host logic, checked on the CPU.

Its pieces are pinned against things it does not compute itself: constructed clusters whose k-means solution is
known, the CPU oracle's quantizer for the quantize-dequantize model its objective uses, and a brute-force
evaluation of Eq. 3 through the oracle's cache for the clip-factor search.
"""
import numpy as np
import pytest

from oracle import skvq_oracle as orc
from paper_2405_06219_b200 import calibrate as cal
from paper_2405_06219_b200 import workloads

D = 128


def test_kmeans_finds_separated_clusters_and_orders_them():
    rng = np.random.default_rng(0)
    v = np.concatenate([1.0 + 0.01 * rng.standard_normal(90), 10.0 + 0.1 * rng.standard_normal(30), 100.0 + rng.standard_normal(8)])
    perm = rng.permutation(v.size)
    label = cal.kmeans_1d(v[perm], 3)
    want = np.concatenate([np.zeros(90), np.ones(30), np.full(8, 2)]).astype(np.int64)[perm]
    assert np.array_equal(label, want)
    assert np.array_equal(cal.kmeans_1d(v, 1), np.zeros(v.size, np.int64))


def test_round_bounds_follow_cluster_sizes_on_the_granule_grid():
    assert cal.round_bounds([64, 64], 128).tolist() == [0, 64, 128]
    assert cal.round_bounds([120, 8], 128).tolist() == [0, 96, 128]          # 120 -> 128 would leave the last group empty
    assert cal.round_bounds([5, 123], 128).tolist() == [0, 32, 128]          # 5 -> 0 would leave the first group empty
    assert cal.round_bounds([30, 34, 30, 34], 128).tolist() == [0, 32, 64, 96, 128]
    assert cal.round_bounds([100, 20, 8], 128).tolist() == [0, 64, 96, 128]  # 100 -> 96, but two more groups need a granule each
    b = cal.round_bounds([40, 50, 38], 128)
    assert b[0] == 0 and b[-1] == 128 and np.all(np.diff(b) >= 32) and np.all(b % 32 == 0)


def test_outlier_channels_end_up_together_in_the_last_group():
    w = workloads.configs()[2].scaled(context=512, batch=1)                  # 8 outlier channels per KV head, scaled x20
    k = w.tokens("k", 0, 0, 512)
    sigma = w.key_sigma()
    for h in range(2):
        idx, bounds = cal.reorder_and_groups(k[:, h], 2)
        assert sorted(idx.tolist()) == list(range(D))                        # a permutation
        assert bounds.tolist() == [0, 96, 128]                               # a narrow group of wide-range channels at the end
        outliers = set(np.argsort(sigma[h])[-8:].tolist())
        assert outliers <= set(idx[96:].tolist())
        f = cal.channel_feature(k[:, h])
        assert np.all(np.diff(f[idx]) >= 0)                                  # stored order = ascending range


@pytest.mark.parametrize("bits,bounds,alpha", [(2, [0, 128], [0.9]), (2, [0, 96, 128], [0.85, 1.0]), (4, [0, 32, 64, 128], [1.0, 0.9, 0.8]),
                                               (3, [0, 64, 128], [0.95, 0.7])])
def test_fake_quant_is_the_cache_quantizer(bits, bounds, alpha):
    """The calibrator's quantize-dequantize model equals dequant(quantize(.)) of the CPU oracle, value for value."""
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((200, D)) * np.exp(rng.standard_normal(D))).astype(np.float16)
    x[:5] = 0.5                                                              # constant rows: h = 0
    got = cal.fake_quant(x, np.asarray(bounds), np.asarray(alpha), bits)
    ident = np.arange(D, dtype=np.int32)
    codes, meta = orc.quantize_rows(x, ident, np.asarray(alpha, np.float32), bits, D // (len(bounds) - 1) if D % (len(bounds) - 1) == 0 else D,
                                    bounds=bounds)
    want = orc.dequant_rows(codes, meta, bits, D, bounds=bounds)
    assert np.array_equal(got, want)


def test_alpha_search_minimises_eq3_as_evaluated_through_the_oracle():
    """One group per row, keys only searched against a fixed value setting: the chosen alpha is the grid point with the
    smallest attention-output error when the whole path (append with that alpha, fp64 attention) is redone by the oracle."""
    w = workloads.configs()[0].scaled(context=384)
    k, v = w.tokens("k", 0, 0, 384)[:, 0], w.tokens("v", 0, 0, 384)[:, 0]
    q = np.stack([w.query(s)[0, 0] for s in range(6)])
    ident = np.arange(D, dtype=np.int32)
    grid = [0.7, 0.8, 0.9, 1.0]
    ak, av, before, after = cal.search_alpha(q, k, v, ident, ident, np.array([0, D]), np.array([0, D]), 2, 2, w.sm_scale, grid=grid)
    assert after <= before

    def oracle_mse(a_k, a_v):
        full = orc.OracleCache(1, 1, 1, D, 2, 2, D, 384, 512, ident[None], ident[None], np.ones((1, 1), np.float32), np.ones((1, 1), np.float32))
        full.append(k[None, :, None], v[None, :, None])                     # window covers everything: full precision
        quant = orc.OracleCache(1, 1, 1, D, 2, 2, D, 0, 512, ident[None], ident[None], np.full((1, 1), a_k, np.float32),
                                np.full((1, 1), a_v, np.float32))
        quant.append(k[None, :, None], v[None, :, None])                    # no window: everything quantized
        err = 0.0
        for qi in q:
            d = quant.attention(qi[None, None], w.sm_scale) - full.attention(qi[None, None], w.sm_scale)
            err += float((d ** 2).mean())
        return err / len(q)

    # keys: alpha_v fixed at 1 while alpha_k was searched (the search does keys first)
    errs = [oracle_mse(a, 1.0) for a in grid]
    assert float(ak[0]) == pytest.approx(grid[int(np.argmin(errs))])
    errs_v = [oracle_mse(float(ak[0]), a) for a in grid]
    assert float(av[0]) == pytest.approx(grid[int(np.argmin(errs_v))])
    assert after == pytest.approx(min(errs_v), rel=1e-9)


def test_calibrated_inputs_beat_identity_order_equal_groups_no_clipping():
    """Direction of the paper's ablation (Sec. 4.3): reorder + clipping lowers the attention-output error of 2-bit keys
    with outlier channels."""
    w = workloads.configs()[2].scaled(context=512, batch=1, n_kv_heads=2, n_q_heads=8)
    k, v = w.tokens("k", 0, 0, 512), w.tokens("v", 0, 0, 512)
    q = np.stack([w.query(s)[0] for s in range(4)])
    res = cal.calibrate(q, k, v, n_groups=2, k_bits=2, v_bits=2, sm_scale=w.sm_scale, grid=[0.8, 0.9, 1.0])
    assert res["reorder_k"].shape == (2, D) and res["bounds_k"].shape == (2, 3) and res["alpha_k"].shape == (2, 2)
    assert np.all(res["mse_after"] <= res["mse_before"])
    ident = np.arange(D, dtype=np.int32)
    for h in range(2):
        qh = q[:, 4 * h:4 * h + 4].reshape(-1, D)
        _, _, plain, _ = cal.search_alpha(qh, k[:, h], v[:, h], ident, ident, np.array([0, 64, 128]), np.array([0, 64, 128]), 2, 2,
                                          w.sm_scale, grid=[1.0])
        assert res["mse_after"][h] < plain
