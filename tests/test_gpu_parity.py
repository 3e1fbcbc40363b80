"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, bit for bit."""
import numpy as np
import pytest

import oracle
import rr_inputs
from paper_2405_11425_b200 import binding as rr
from paper_2405_11425_b200 import build as rr_build

pytestmark = pytest.mark.gpu
MiB = 1 << 20


@pytest.fixture(scope="module")
def dev():
    import torch
    rr_build.build()
    torch.cuda.set_device(0)

    class Dev:
        pass

    d = Dev()
    d.torch = torch
    d.scratch = torch.zeros(rr.rr_scratch_bytes(), dtype=torch.uint8, device="cuda")
    info = rr.rr_device_info(d.scratch)
    d.info = info
    d.nsm = info["nsm_prop"]
    d.buf_bytes = 1 << 30
    d.buf = torch.empty(d.buf_bytes, dtype=torch.uint8, device="cuda")
    assert d.buf.data_ptr() % 512 == 0
    rr.rr_fill(d.buf, d.buf_bytes // 4)
    torch.cuda.synchronize()
    return d


def _out(dev, n):
    return dev.torch.full((n, 2), 0x5EADBEEF, dtype=dev.torch.int32, device="cuda")


def _np(t):
    return t.cpu().numpy().view(np.uint32)


def test_device_facts(dev):
    i = dev.info
    assert i["cc_major"] == 10
    assert i["nsm_reg"] == i["nsm_prop"] <= rr.RR_MAX_SM
    assert i["theoretical_gbps"] > 1000 and i["total_bytes"] > 100 << 30
    assert rr.rr_device_info()["nsm_reg"] == 0          # no scratch: nothing launched, not read


@pytest.mark.parametrize("n_words", [0, 1, 3, 4, 5, 127, 1023, 1024, (1 << 20) + 3, 37 * 148 * 2048 + 2])
def test_fill_matches_oracle_small(dev, n_words):
    t = dev.torch.full((n_words + 8,), 0x25A5A5A5, dtype=dev.torch.int32, device="cuda")
    rr.rr_fill(t, n_words)
    got = _np(t)
    assert np.array_equal(got[:n_words], oracle.fill(0, n_words))
    assert np.all(got[n_words:] == 0x25A5A5A5)          # nothing written past the end


def test_fill_1gib_sampled_and_folded(dev):
    words = dev.buf.view(dev.torch.int32)
    n = dev.buf_bytes // 4
    rng = np.random.default_rng(0)
    for start in [0, n - 4096] + [int(x) for x in rng.integers(0, n - 4096, 16)]:
        got = _np(words[start:start + 4096])
        assert np.array_equal(got, oracle.fill(start, 4096))


def test_cfg0_all_warps_bit_exact(dev):
    c = rr_inputs.CFG0
    out = _out(dev, c.n_warps)
    p = rr.ReadParams(dev.buf, c.region_bytes, W=c.W, mode=rr.RR_MODE_LOGICAL, n_warps=c.n_warps,
                      reads_per_warp=c.reads_per_warp, seed=c.seed)
    res = rr.rr_random_read(p, out, dev.scratch)
    expect = oracle.read_logical(c.region_bytes, c.W, c.n_warps, c.reads_per_warp, c.seed)
    assert np.array_equal(_np(out), expect)
    assert res.bytes == c.n_warps * c.reads_per_warp * 128
    assert res.status == 0 and res.blocks_run > 0 and res.gbps > 0


@pytest.mark.parametrize("W", [1, 2, 4])
@pytest.mark.parametrize("unroll", [0, 2, 4, 8, 16])
def test_logical_widths_unrolls_ragged_reads(dev, W, unroll):
    region = 777 * MiB + 384            # not a power of two, tail shorter than a line
    for reads, first in [(0, 0), (1, 0), (7, 3), (31, 0), (32, 1), (33, 0), (40, 100), (100, 7),
                         (64, 0), (96, 5)]:
        n_warps = 300
        out = _out(dev, n_warps)
        p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=n_warps,
                          reads_per_warp=reads, first_read=first, seed=11, unroll=unroll)
        rr.rr_random_read(p, out, dev.scratch)
        expect = oracle.read_logical(region, W, n_warps, reads, 11, first_read=first)
        assert np.array_equal(_np(out), expect), (W, unroll, reads, first)


@pytest.mark.parametrize("W", [1, 2, 4])
def test_checked_variant_is_clean_and_equal(dev, W):
    region = 64 * MiB + 128
    out = _out(dev, 500)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=500,
                      reads_per_warp=45, seed=5, variant=rr.RR_VARIANT_LDG_CHECKED)
    res = rr.rr_random_read(p, out, dev.scratch)
    assert res.violations == 0
    assert np.array_equal(_np(out), oracle.read_logical(region, W, 500, 45, 5))


def test_tiny_region_of_one_line(dev):
    out = _out(dev, 40)
    p = rr.ReadParams(dev.buf, 128, W=1, mode=rr.RR_MODE_LOGICAL, n_warps=40, reads_per_warp=9,
                      seed=2, variant=rr.RR_VARIANT_LDG_CHECKED)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_logical(128, 1, 40, 9, 2))


@pytest.mark.parametrize("W", [1, 2, 4])
def test_stride_mode(dev, W):
    V, R = 256, 64
    region = V * R * 128 * W
    out = _out(dev, V)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=V, reads_per_warp=R,
                      index_mode=rr.RR_INDEX_STRIDE)
    rr.rr_random_read(p, out, dev.scratch)
    got = _np(out)
    assert np.array_equal(got, oracle.read_logical(region, W, V, R, 0,
                                                   index_mode=oracle.INDEX_STRIDE))
    words = oracle.fill(0, region // 4)                 # every line exactly once
    assert int(np.bitwise_xor.reduce(got[:, 0])) == int(np.bitwise_xor.reduce(words))


@pytest.mark.parametrize("wps", [1, 8, 32])
@pytest.mark.parametrize("W", [1, 2])
def test_per_sm_ungrouped(dev, wps, W):
    region = 1000 * MiB
    out = _out(dev, dev.nsm * wps)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_PER_SM, warps_per_sm=wps,
                      reads_per_warp=70, first_read=256, seed=7)
    res = rr.rr_random_read(p, out, dev.scratch)
    assert res.sms_covered == dev.nsm and res.blocks_run == dev.nsm
    assert res.bytes == dev.nsm * wps * 70 * 128 * W
    assert np.array_equal(_np(out), oracle.read_per_sm(region, W, dev.nsm, wps, 70, 7,
                                                       first_read=256))


def test_per_sm_grouped_windows_and_inactive_sms(dev):
    region = dev.buf_bytes
    G = 9
    groups = rr_inputs.synthetic_group_map(dev.nsm, G, seed=4, inactive_frac=0.1)
    windows, cov = rr.rr_make_windows(region, 1, region // 5, G)
    windows[3] = (1000, 777)                      # an odd window
    out = _out(dev, dev.nsm * 16)
    p = rr.ReadParams(dev.buf, region, W=1, mode=rr.RR_MODE_PER_SM, warps_per_sm=16,
                      reads_per_warp=50, seed=23, group_of_sm=groups, windows=windows)
    res = rr.rr_random_read(p, out, dev.scratch)
    active = int((groups != 0xFFFF).sum())
    assert res.sms_covered == active and res.bytes == active * 16 * 50 * 128
    expect = oracle.read_per_sm(region, 1, dev.nsm, 16, 50, 23, group_of_sm=groups,
                                windows=windows)
    assert np.array_equal(_np(out), expect)
    # asynchronous form + report give the same
    out2 = _out(dev, dev.nsm * 16)
    assert rr.rr_random_read(p, out2, dev.scratch, timed=False) is None
    rep = rr.rr_read_report(p, dev.scratch)
    assert np.array_equal(_np(out2), expect) and rep.sms_covered == active
    assert rep.seconds_device > 0


def test_single_whole_window_equals_ungrouped_on_gpu(dev):
    region = 512 * MiB
    L = region // 256
    a, b = _out(dev, dev.nsm * 4), _out(dev, dev.nsm * 4)
    pa = rr.ReadParams(dev.buf, region, W=2, warps_per_sm=4, reads_per_warp=33, seed=9)
    pb = rr.ReadParams(dev.buf, region, W=2, warps_per_sm=4, reads_per_warp=33, seed=9,
                       group_of_sm=np.zeros(dev.nsm, np.uint16), windows=[[0, L]])
    rr.rr_random_read(pa, a, dev.scratch)
    rr.rr_random_read(pb, b, dev.scratch)
    assert np.array_equal(_np(a), _np(b))


def test_nsm_mismatch_is_rejected(dev):
    out = _out(dev, 8)
    p = rr.ReadParams(dev.buf, 1 << 20, warps_per_sm=1, nsm=dev.nsm - 1, reads_per_warp=1)
    with pytest.raises(rr.RRError) as e:
        rr.rr_random_read(p, out, dev.scratch)
    assert e.value.code == rr.RR_ERR_ARG


@pytest.mark.parametrize("wps", [4, 32])
def test_probe_pair_checksums_and_rates(dev, wps):
    region = dev.buf_bytes
    total = 2 * wps * 200
    for a, b in [(0, 1), (3, dev.nsm - 1), (dev.nsm - 1, 2), (5, 5)]:
        out = _out(dev, 2 * wps)
        res = rr.rr_probe_pair(dev.buf, region, a, b, total, wps, 5, out, dev.scratch)
        got = _np(out)
        full = oracle.read_per_sm(region, 1, dev.nsm, wps, total // 2 // wps, 5)
        assert np.array_equal(got[:wps], full[a * wps:(a + 1) * wps])
        if a != b:
            assert np.array_equal(got[wps:], full[b * wps:(b + 1) * wps])
            extra = res.bytes - total * 128            # what a faster SM read while waiting
            assert extra >= 0 and extra % (32 * 128) == 0 and extra <= total * 128
            assert res.sms_covered == 2
        else:
            assert not got[wps:].any() and res.bytes == total * 64 and res.sms_covered == 1
        assert res.gbps > 0 and res.seconds_device > 0


def test_probe_matrix_is_symmetric_and_positive(dev):
    wps = 8
    scratch = dev.torch.zeros(rr.rr_probe_matrix_scratch_bytes(dev.nsm), dtype=dev.torch.uint8,
                              device="cuda")
    out = _out(dev, 2 * wps)
    T, stats, ov = rr.rr_probe_matrix(dev.buf, dev.buf_bytes, 2 * wps * 256, wps, 5, 1, dev.nsm,
                                      out, scratch, with_overlaps=True)
    assert T.shape == (dev.nsm, dev.nsm) and np.array_equal(T, T.T)
    assert np.isfinite(T).all() and (T > 0).all()
    # the overlap rule: every pair either ran side by side for 98 % of its measurement or is
    # counted, and the count agrees with the per-pair matrix
    assert np.array_equal(ov, ov.T) and (np.diag(ov) == 1).all()
    low = int((ov[np.triu_indices(dev.nsm, 1)] < np.float32(0.98)).sum())
    assert stats["pairs_below_goal"] == low
    assert stats["overlap_min"] >= 0.98 or low > 0
    assert abs(stats["overlap_min"] - float(ov.min())) < 1e-6
    assert stats["reruns"] >= low                      # each of them was measured again at least once


@pytest.mark.parametrize("W", [1, 2])
def test_overlapping_windows_policy_on_gpu(dev, W):
    """Policy 2: evenly spaced windows that overlap; warps of different groups may share lines."""
    region = dev.buf_bytes
    G = 7
    groups = rr_inputs.synthetic_group_map(dev.nsm, G, seed=3, inactive_frac=0.05)
    windows, cov = rr.rr_make_windows(region, W, region // 4, G, policy=2)
    assert cov == 1.0 and int(windows[-1].sum()) == region // (128 * W)
    covered, dmin, dmax = rr.rr_window_cover(windows, region // (128 * W))
    assert covered == region // (128 * W) and dmin >= 1 and dmax >= 2
    out = _out(dev, dev.nsm * 8)
    p = rr.ReadParams(dev.buf, region, W=W, warps_per_sm=8, reads_per_warp=77, seed=23,
                      group_of_sm=groups, windows=windows, variant=rr.RR_VARIANT_PACKED, unroll=2)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_per_sm(region, W, dev.nsm, 8, 77, 23,
                                                       group_of_sm=groups, windows=windows))


@pytest.mark.parametrize("sizes,drop", [
    ([8] * 12 + [6] * 2, 0.10),                 # the paper's A100 shape
    ([18] * 6 + [20] * 2, 0.06),                # 148 SMs
    ([16] * 16, 0.15),                          # 256 SMs: the table limit
    ([4, 6, 4], 0.2),
    ([2, 2, 2], 0.3),                           # 6 SMs: smallest with a group level
    ([2, 2], 0.3),                              # 4 SMs: no group level
    ([20] * 7, 0.0),                            # null matrix
])
def test_cluster_matches_oracle(dev, sizes, drop):
    for seed in range(4):
        T, truth = rr_inputs.planted_matrix(sizes, drop, seed=seed)
        g, G, conf, h = rr.rr_cluster(T, dev.scratch)
        og, oG, oconf, oh = oracle.cluster(T)
        assert G == oG and np.array_equal(g, og)
        assert np.array_equal(h, oh)                       # same divisions, same doubles
        assert conf == oconf or (np.isinf(conf) and np.isinf(oconf))
        T2, _ = rr_inputs.planted_matrix(sizes, drop, seed=seed, solo_spread=0.15)
        g, G, conf, h = rr.rr_cluster(T2, dev.scratch, flags=rr.RR_CLUSTER_SOLO_NORMALISE)
        og, oG, oconf, oh = oracle.cluster(T2, solo_normalise=True)
        assert G == oG and np.array_equal(g, og) and np.array_equal(h, oh)
        assert conf == oconf or (np.isinf(conf) and np.isinf(oconf))
        if drop >= 0.06 and len(sizes) >= 6 and sum(sizes) // 3 >= len(sizes):
            assert G == len(sizes) and np.array_equal(g, truth)


def test_cluster_two_sms_and_ties(dev):
    g, G, conf, h = rr.rr_cluster(np.array([[1, 2], [3, 1]], np.float32), dev.scratch)
    assert G == 1 and list(g) == [0, 0]
    T = np.full((9, 9), 50.0, np.float32)
    g, G, conf, h = rr.rr_cluster(T, dev.scratch)
    og, oG, oconf, oh = oracle.cluster(T)
    assert G == oG == 1 and np.array_equal(h, oh)


def test_gpc_map_from_cluster_placement(dev):
    g, n_gpcs = rr.rr_gpc_map(dev.scratch, dev.nsm)
    assert g.shape == (dev.nsm,) and g.min() == 0 and g.max() == n_gpcs - 1
    assert 2 <= n_gpcs <= dev.nsm // 2
    assert np.array_equal(g[0::2], g[1::2])            # the two SMs of a TPC share a GPC
    firsts = [int(np.argmax(g == k)) for k in range(n_gpcs)]
    assert firsts == sorted(firsts)                    # canonical labels
    g2, n2 = rr.rr_gpc_map(dev.scratch, dev.nsm)
    assert n2 == n_gpcs and np.array_equal(g, g2)      # placement facts, not timing: repeatable
    with pytest.raises(rr.RRError):
        rr.rr_gpc_map(dev.scratch, dev.nsm + 1)


@pytest.mark.parametrize("W,block", [(1, 0), (1, 64), (2, 100), (4, 1000)])
def test_pooled_mode_matches_oracle(dev, W, block):
    region = 900 * MiB + 128
    G = 7
    groups = rr_inputs.synthetic_group_map(dev.nsm, G, seed=9, inactive_frac=0.1)
    weights = [5, 1, 3, 3, 2, 8, 4]
    n_warps = 1500
    win, ws = rr.rr_make_weighted_windows(region, W, weights, n_warps)
    reads, first = 333, 17                       # not a multiple of the block: ragged last item
    out = _out(dev, n_warps)                     # poisoned: the call must clear it
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_POOLED, n_warps=n_warps,
                      warps_per_sm=16, nsm=dev.nsm, reads_per_warp=reads, first_read=first, seed=23,
                      group_of_sm=groups, windows=win, warp_start=ws, pool_block_reads=block)
    res = rr.rr_random_read(p, out, dev.scratch)
    expect = oracle.read_pooled(region, W, win, ws, reads, 23, first_read=first)
    assert np.array_equal(_np(out), expect)
    assert res.bytes == n_warps * reads * 128 * W
    assert res.sms_covered == int((groups != 0xFFFF).sum())
    # twice in a row: counters and outputs are cleared by the call
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), expect)


def test_pooled_mode_empty_group_and_zero_reads(dev):
    region = 64 * MiB
    groups = np.zeros(dev.nsm, np.uint16)
    groups[1::2] = 2                                # group 1 owns no warps and has no SM
    win = np.array([[0, 1000], [1000, 1000], [5000, 777]], np.uint32)
    ws = [0, 40, 40, 100]
    out = _out(dev, 100)
    p = rr.ReadParams(dev.buf, region, mode=rr.RR_MODE_POOLED, n_warps=100, warps_per_sm=4,
                      nsm=dev.nsm, reads_per_warp=50, seed=3, group_of_sm=groups, windows=win,
                      warp_start=ws)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_pooled(region, 1, win, ws, 50, 3))
    p0 = rr.ReadParams(dev.buf, region, mode=rr.RR_MODE_POOLED, n_warps=100, warps_per_sm=4,
                       nsm=dev.nsm, reads_per_warp=0, seed=3, group_of_sm=groups, windows=win,
                       warp_start=ws)
    rr.rr_random_read(p0, out, dev.scratch)
    assert not _np(out).any()


@pytest.mark.parametrize("wps", [32, 24, 5])
@pytest.mark.parametrize("variant", ["ldg", "packed", "sorted"])
def test_pooled_mode_one_sm_per_group_equal_shares(dev, variant, wps):
    """A pool that a single SM serves is cut into equal shares, one per warp (no guided grabs):
    shares that are not whole logical warps, a last share that is short, pools with fewer
    reads than warps."""
    region = 600 * MiB + 256
    owners = np.random.default_rng(5).permutation(dev.nsm).astype(np.uint16)
    weights = [3 + (g * 7) % 3 for g in range(dev.nsm)]
    kw = {"ldg": dict(variant=rr.RR_VARIANT_LDG),
          "packed": dict(variant=rr.RR_VARIANT_PACKED, unroll=1),
          "sorted": dict(variant=rr.RR_VARIANT_SORTED, unroll=1, sort_parts=16, sort_reads=64)}[variant]
    for n_warps, reads, first in [(dev.nsm * 3 + 1, 333, 5), (dev.nsm * 2, 1, 0),
                                  (dev.nsm * 4 + 9, 4099, 64)]:
        win, ws = rr.rr_make_weighted_windows(region, 1, weights, n_warps)
        out = _out(dev, n_warps)
        p = rr.ReadParams(dev.buf, region, W=1, mode=rr.RR_MODE_POOLED, n_warps=n_warps,
                          warps_per_sm=wps, nsm=dev.nsm, reads_per_warp=reads, first_read=first,
                          seed=23, group_of_sm=owners, windows=win, warp_start=ws, **kw)
        res = rr.rr_random_read(p, out, dev.scratch)
        expect = oracle.read_pooled(region, 1, win, ws, reads, 23, first_read=first)
        assert np.array_equal(_np(out), expect), (variant, wps, n_warps, reads)
        assert res.bytes == n_warps * reads * 128 and res.sms_covered == dev.nsm


@pytest.mark.parametrize("W", [1, 2, 4])
@pytest.mark.parametrize("unroll", [0, 2, 4, 8, 16])
def test_packed_variant_logical_ragged_reads(dev, W, unroll):
    region = 777 * MiB + 384
    for reads, first in [(0, 0), (1, 0), (2, 5), (3, 0), (7, 3), (31, 0), (32, 1), (33, 0),
                         (40, 100), (61, 7), (64, 0), (100, 9), (257, 2)]:
        n_warps = 200
        out = _out(dev, n_warps)
        p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=n_warps,
                          reads_per_warp=reads, first_read=first, seed=11, unroll=unroll,
                          variant=rr.RR_VARIANT_PACKED)
        rr.rr_random_read(p, out, dev.scratch)
        expect = oracle.read_logical(region, W, n_warps, reads, 11, first_read=first)
        assert np.array_equal(_np(out), expect), (W, unroll, reads, first)


@pytest.mark.parametrize("W", [1, 2])
def test_packed_variant_grouped_pooled_and_stride(dev, W):
    region = dev.buf_bytes
    G = 6
    groups = rr_inputs.synthetic_group_map(dev.nsm, G, seed=2, inactive_frac=0.05)
    windows, _ = rr.rr_make_windows(region, W, region // 4, G)
    windows[2] = (123, 1001)
    out = _out(dev, dev.nsm * 32)
    p = rr.ReadParams(dev.buf, region, W=W, warps_per_sm=32, reads_per_warp=133, seed=23,
                      group_of_sm=groups, windows=windows, variant=rr.RR_VARIANT_PACKED)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_per_sm(region, W, dev.nsm, 32, 133, 23,
                                                       group_of_sm=groups, windows=windows))
    win, ws = rr.rr_make_weighted_windows(region, W, [3, 1, 2, 2, 5, 1], 999)
    out = _out(dev, 999)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_POOLED, n_warps=999, warps_per_sm=32,
                      nsm=dev.nsm, reads_per_warp=301, seed=5, group_of_sm=groups, windows=win,
                      warp_start=ws, variant=rr.RR_VARIANT_PACKED)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_pooled(region, W, win, ws, 301, 5))
    V, R = 64, 96
    small = V * R * 128 * W
    out = _out(dev, V)
    p = rr.ReadParams(dev.buf, small, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=V, reads_per_warp=R,
                      index_mode=rr.RR_INDEX_STRIDE, variant=rr.RR_VARIANT_PACKED)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_logical(small, W, V, R, 0,
                                                        index_mode=oracle.INDEX_STRIDE))


@pytest.mark.parametrize("W", [1, 2, 4])
@pytest.mark.parametrize("variant", [rr.RR_VARIANT_LDG, rr.RR_VARIANT_PACKED,
                                     rr.RR_VARIANT_LDG_CHECKED])
def test_phased_index_mode_matches_oracle(dev, W, variant):
    region = dev.buf_bytes
    G = 5
    groups = rr_inputs.synthetic_group_map(dev.nsm, G, seed=6, inactive_frac=0.05)
    windows, _ = rr.rr_make_windows(region, W, region // 5, G)
    windows[1] = (777, 10007)                       # sub-windows of unequal size
    for B, sub_bytes, reads, first in [(32, 1000 * 128 * W, 300, 0), (64, 3000 * 128 * W, 129, 64),
                                       (256, 8 << 20, 1000, 32 * 9), (1024, 1 << 40, 100, 0)]:
        out = _out(dev, dev.nsm * 8)
        p = rr.ReadParams(dev.buf, region, W=W, warps_per_sm=8, reads_per_warp=reads,
                          first_read=first, seed=23, group_of_sm=groups, windows=windows,
                          variant=variant, index_mode=rr.RR_INDEX_PHASED, phase_reads=B,
                          phase_window_bytes=sub_bytes)
        res = rr.rr_random_read(p, out, dev.scratch)
        assert res.violations == 0
        expect = oracle.read_per_sm_phased(region, W, dev.nsm, 8, reads, 23, B, sub_bytes,
                                           group_of_sm=groups, windows=windows, first_read=first)
        assert np.array_equal(_np(out), expect), (W, variant, B, sub_bytes, reads, first)
    # logical mode: one window = the region (compare through a one-group per-SM oracle call)
    L = region // (128 * W)
    out = _out(dev, 64)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=64, reads_per_warp=200,
                      seed=3, variant=variant, index_mode=rr.RR_INDEX_PHASED, phase_reads=32,
                      phase_window_bytes=64 << 20)
    rr.rr_random_read(p, out, dev.scratch)
    got = _np(out)
    sub = (64 << 20) // (128 * W)
    for v in range(64):                              # logical warps: no SM, so no stagger
        assert tuple(got[v]) == oracle.warp_checksum_phased(3, v, 0, 200, W, 0, L, 32, sub, 0)
    # every SM on the whole region: the SMs start their cycles at staggered sub-windows
    out = _out(dev, dev.nsm * 4)
    p = rr.ReadParams(dev.buf, region, W=W, warps_per_sm=4, reads_per_warp=160, seed=3,
                      variant=variant, index_mode=rr.RR_INDEX_PHASED, phase_reads=32,
                      phase_window_bytes=8 << 20)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_per_sm_phased(region, W, dev.nsm, 4, 160, 3, 32,
                                                              8 << 20))


def test_launch_configuration_is_cached(dev):
    """A repeated call asks the runtime for no occupancy figure, attribute, event or device fact."""
    out = _out(dev, dev.nsm * 32)
    p = rr.ReadParams(dev.buf, 64 * MiB, warps_per_sm=32, reads_per_warp=40, seed=1,
                      variant=rr.RR_VARIANT_PACKED, unroll=2)
    rr.rr_random_read(p, out, dev.scratch)                     # may search and create
    before = rr.rr_host_counters()
    for _ in range(3):
        rr.rr_random_read(p, out, dev.scratch)
        rr.rr_random_read(p, out, dev.scratch, timed=False)
    rr.rr_probe_pair(dev.buf, 64 * MiB, 0, 1, 2 * 32 * 8, 32, 5, _out(dev, 64), dev.scratch)
    mid = rr.rr_host_counters()
    rr.rr_probe_pair(dev.buf, 64 * MiB, 0, 1, 2 * 32 * 8, 32, 5, _out(dev, 64), dev.scratch)
    after = rr.rr_host_counters()
    assert before["occupancy_queries"] > 0 and before["device_fact_queries"] == 1
    assert {k: mid[k] for k in ("event_creates", "device_fact_queries")} == \
           {k: before[k] for k in ("event_creates", "device_fact_queries")}
    assert after == mid


@pytest.mark.parametrize("W", [1, 2, 4])
@pytest.mark.parametrize("variant", [rr.RR_VARIANT_LDG, rr.RR_VARIANT_PACKED])
def test_mixed_index_mode_matches_oracle(dev, W, variant):
    region = dev.buf_bytes
    G = 5
    groups = rr_inputs.synthetic_group_map(dev.nsm, G, seed=8, inactive_frac=0.05)
    windows, _ = rr.rr_make_windows(region, W, region // 5, G)
    windows[1] = (777, 10007)
    for k, reads, first in [(1, 70, 0), (2, 133, 5), (8, 300, 64), (64, 257, 1000)]:
        out = _out(dev, dev.nsm * 8)
        p = rr.ReadParams(dev.buf, region, W=W, warps_per_sm=8, reads_per_warp=reads,
                          first_read=first, seed=23, group_of_sm=groups, windows=windows,
                          variant=variant, index_mode=rr.RR_INDEX_MIXED, mix_period=k)
        rr.rr_random_read(p, out, dev.scratch)
        expect = oracle.read_per_sm_mixed(region, W, dev.nsm, 8, reads, 23, k, group_of_sm=groups,
                                          windows=windows, first_read=first)
        assert np.array_equal(_np(out), expect), (W, variant, k, reads, first)
    L = region // (128 * W)
    out = _out(dev, 100)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=100, reads_per_warp=90,
                      seed=3, variant=variant, index_mode=rr.RR_INDEX_MIXED, mix_period=4)
    rr.rr_random_read(p, out, dev.scratch)
    got = _np(out)
    for v in range(0, 100, 7):
        assert tuple(got[v]) == oracle.warp_checksum_mixed(3, v, 0, 90, W, 0, L, 4, n_warps_total=100)


@pytest.mark.parametrize("W", [1, 2])
@pytest.mark.parametrize("unroll", [0, 2, 4])
@pytest.mark.parametrize("parts,sreads", [(2, 32), (4, 64), (8, 512), (16, 256), (16, 32), (2, 2048)])
def test_sorted_variant_reads_the_same_lines_in_another_order(dev, W, unroll, parts, sreads):
    """RR_VARIANT_SORTED only reorders a warp's reads (part by part of its window, epoch by epoch):
    the checksums must be those of the plain definition, for every ragged length."""
    region = 777 * MiB + 384
    for reads, first in [(0, 0), (1, 0), (5, 3), (31, 0), (32, 1), (33, 0), (64, 0), (100, 7),
                         (parts * sreads, 0), (parts * sreads + 1, 2), (3 * parts * sreads - 7, 5),
                         (257, 2)]:
        n_warps = 150
        out = _out(dev, n_warps)
        p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=n_warps,
                          reads_per_warp=reads, first_read=first, seed=11, unroll=unroll,
                          variant=rr.RR_VARIANT_SORTED, sort_parts=parts, sort_reads=sreads)
        rr.rr_random_read(p, out, dev.scratch)
        expect = oracle.read_logical(region, W, n_warps, reads, 11, first_read=first)
        assert np.array_equal(_np(out), expect), (W, unroll, parts, sreads, reads, first)


@pytest.mark.parametrize("W", [1, 2])
def test_sorted_variant_grouped_and_pooled(dev, W):
    region = dev.buf_bytes
    G = 6
    groups = rr_inputs.synthetic_group_map(dev.nsm, G, seed=2, inactive_frac=0.05)
    windows, _ = rr.rr_make_windows(region, W, region // 4, G)
    windows[2] = (123, 3)                           # fewer lines than parts: some parts are empty
    windows[4] = (5000, 1001)
    kw = dict(variant=rr.RR_VARIANT_SORTED, sort_parts=4, sort_reads=64)
    out = _out(dev, dev.nsm * 32)
    p = rr.ReadParams(dev.buf, region, W=W, warps_per_sm=32, reads_per_warp=700, first_read=96,
                      seed=23, group_of_sm=groups, windows=windows, **kw)
    res = rr.rr_random_read(p, out, dev.scratch)
    assert res.sms_covered == int((groups != 0xFFFF).sum())
    assert np.array_equal(_np(out), oracle.read_per_sm(region, W, dev.nsm, 32, 700, 23,
                                                       group_of_sm=groups, windows=windows,
                                                       first_read=96))
    win, ws = rr.rr_make_weighted_windows(region, W, [3, 1, 2, 2, 5, 1], 999)
    out = _out(dev, 999)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_POOLED, n_warps=999, warps_per_sm=32,
                      nsm=dev.nsm, reads_per_warp=901, seed=5, group_of_sm=groups, windows=win,
                      warp_start=ws, **kw)
    rr.rr_random_read(p, out, dev.scratch)
    assert np.array_equal(_np(out), oracle.read_pooled(region, W, win, ws, 901, 5))


@pytest.mark.parametrize("W", [1, 2, 4])
@pytest.mark.parametrize("variant", [rr.RR_VARIANT_LDG, rr.RR_VARIANT_PACKED,
                                     rr.RR_VARIANT_SORTED])
def test_logical_mode_with_a_window_per_warp(dev, W, variant):
    if variant == rr.RR_VARIANT_SORTED and W == 4:
        pytest.skip("16-byte lanes already cover a 512-byte line: no packed or sorted shape")
    kw = dict(sort_parts=8, sort_reads=32) if variant == rr.RR_VARIANT_SORTED else {}
    region = dev.buf_bytes
    win, cov = rr.rr_make_windows(region, W, region // 7, 37, policy=1, seed=23)   # hashed chunks
    win[5] = (321, 3)
    n_warps = 777
    out = _out(dev, n_warps)
    p = rr.ReadParams(dev.buf, region, W=W, mode=rr.RR_MODE_LOGICAL, n_warps=n_warps,
                      reads_per_warp=45, first_read=7, seed=23, windows=win, variant=variant, **kw)
    res = rr.rr_random_read(p, out, dev.scratch)
    assert res.bytes == n_warps * 45 * 128 * W
    assert np.array_equal(_np(out), oracle.read_logical_windows(region, W, n_warps, 45, 23, win,
                                                                first_read=7))
