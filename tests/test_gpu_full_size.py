"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times: one
buffer of ~90 % of free HBM, 32 warps on every SM, 2^8 x 64 reads per warp; outputs the oracle can
compute one by one are sampled (every 37th warp, the first and the last)."""
import numpy as np
import pytest

import oracle
import rr_inputs
from paper_2405_11425_b200 import binding as rr
from paper_2405_11425_b200 import build as rr_build
from paper_2405_11425_b200.pipeline import Session

pytestmark = pytest.mark.gpu
GiB = 1 << 30
WPS = 32


@pytest.fixture(scope="module")
def ses():
    import torch
    rr_build.build()
    torch.cuda.set_device(0)
    torch.cuda.empty_cache()
    s = Session(frac_of_free=0.90)
    assert s.region_bytes > 100 * GiB, "these tests are meant for a GPU with its HBM free"
    rate = s.fill()
    assert rate > 100
    yield s
    del s.buf
    torch.cuda.empty_cache()


def _sample(n):
    return sorted(set(list(range(0, n, 37)) + [0, n - 1]))


def _check_sampled(ses, got, region, W, reads, seed, groups=None, windows=None, first=0):
    V = ses.nsm * WPS
    L = region // (128 * W)
    for v in _sample(V):
        sm = v // WPS
        base, n = 0, L
        if groups is not None:
            if groups[sm] == 0xFFFF:
                assert tuple(got[v]) == (0, 0)
                continue
            base, n = map(int, windows[groups[sm]])
        assert tuple(got[v]) == oracle.warp_checksum(seed, v, first, reads, W, base, n), (v, W)


def test_fill_of_the_whole_buffer_sampled_beyond_32_bit_indices(ses):
    words = ses.buf.view(ses.torch.int32)
    n = ses.region_bytes // 4
    assert n > 1 << 32                                     # word indices need 64 bits
    rng = np.random.default_rng(1)
    starts = [0, (1 << 32) - 2048, (1 << 32), (1 << 33) + 5, n - 4096]
    starts += [int(x) for x in rng.integers(0, n - 4096, 24)]
    for s in starts:
        got = words[s:s + 4096].cpu().numpy().view(np.uint32)
        assert np.array_equal(got, oracle.fill(s, 4096)), s


@pytest.mark.parametrize("size_gib", list(rr_inputs.CFG1_SIZES_GIB) + [None])
def test_cfg1_unrestricted_sizes_sampled(ses, size_gib):
    region = ses.region_bytes if size_gib is None else size_gib * GiB
    if region > ses.region_bytes:
        pytest.skip("buffer smaller than this sweep point")
    reads = rr_inputs.CFG1_READS_PER_ITER * 4
    p = ses.params(region, W=1, warps_per_sm=WPS, reads_per_warp=reads, seed=rr_inputs.CFG1_SEED)
    res = rr.rr_random_read(p, ses.out, ses.scratch)
    assert res.sms_covered == ses.nsm and res.bytes == ses.nsm * WPS * reads * 128
    _check_sampled(ses, ses.checksums(ses.nsm * WPS), region, 1, reads, rr_inputs.CFG1_SEED)


@pytest.mark.parametrize("W", [1, 2, 4])
def test_cfg2_widths_at_32_gib_sampled(ses, W):
    reads = 1024
    p = ses.params(rr_inputs.CFG2_REGION, W=W, warps_per_sm=WPS, reads_per_warp=reads,
                   seed=rr_inputs.CFG2_SEED)
    rr.rr_random_read(p, ses.out, ses.scratch)
    _check_sampled(ses, ses.checksums(ses.nsm * WPS), rr_inputs.CFG2_REGION, W, reads,
                   rr_inputs.CFG2_SEED)


@pytest.mark.parametrize("W", [1, 2])
def test_cfg4_bench_launch_configuration_sampled(ses, W):
    # what bench.py times: whole buffer, 24 SM groups, windows of 35 GiB, 16384 reads per warp,
    # continuing the stream at a later first_read
    region = ses.region_bytes
    groups = rr_inputs.synthetic_group_map(ses.nsm, 24, seed=7)
    windows, cov = rr.rr_make_windows(region, W, 35 * GiB, 24)
    assert cov == 1.0
    reads, first = 256 * 64, 256 * 64 * 3
    p = ses.params(region, W=W, warps_per_sm=WPS, reads_per_warp=reads, first_read=first,
                   seed=rr_inputs.CFG4_SEED, group_of_sm=groups, windows=windows)
    assert rr.rr_random_read(p, ses.out, ses.scratch, timed=False) is None   # as bench launches it
    rep = rr.rr_read_report(p, ses.scratch)
    assert rep.sms_covered == ses.nsm and rep.bytes == ses.nsm * WPS * reads * 128 * W
    _check_sampled(ses, ses.checksums(ses.nsm * WPS), region, W, reads, rr_inputs.CFG4_SEED,
                   groups, windows, first)


def test_cfg4_naive_control_and_inactive_sms_sampled(ses):
    region = ses.region_bytes
    win, cov = rr.rr_make_windows(region, 1, region // 2, ses.nsm, policy=1, seed=23)
    groups = np.arange(ses.nsm, dtype=np.uint16)
    groups[5::11] = 0xFFFF
    p = ses.params(region, W=1, warps_per_sm=WPS, reads_per_warp=512, seed=23,
                   group_of_sm=groups, windows=win)
    res = rr.rr_random_read(p, ses.out, ses.scratch)
    assert res.sms_covered == int((groups != 0xFFFF).sum())
    _check_sampled(ses, ses.checksums(ses.nsm * WPS), region, 1, 512, 23, groups, win)


def test_cfg3_probe_over_the_whole_buffer(ses):
    total = 1 << 18
    per_warp = total // 2 // WPS
    a, b = 2, ses.nsm - 3
    res = rr.rr_probe_pair(ses.buf, ses.region_bytes, a, b, total, WPS, rr_inputs.CFG3_SEED,
                           ses.probe_out, ses.scratch)
    got = ses.probe_out.cpu().numpy().view(np.uint32)
    L = ses.region_bytes // 128
    for w in (0, 7, 31):
        assert tuple(got[w]) == oracle.warp_checksum(rr_inputs.CFG3_SEED, a * WPS + w, 0, per_warp,
                                                     1, 0, L)
        assert tuple(got[WPS + w]) == oracle.warp_checksum(rr_inputs.CFG3_SEED, b * WPS + w, 0,
                                                           per_warp, 1, 0, L)
    assert total * 128 <= res.bytes <= 2 * total * 128 and res.gbps > 1


def test_stride_mode_covers_every_line_of_a_large_prefix_once(ses):
    # property that holds at any size: with V*R == L every line is read once, so the per-warp
    # sums add up to the sum of the region's words, which the oracle can fold in chunks
    V = ses.nsm * WPS
    R = 2048
    region = V * R * 128                                     # ~1.2 GiB
    p = ses.params(region, W=1, warps_per_sm=WPS, reads_per_warp=R,
                   index_mode=rr.RR_INDEX_STRIDE)
    rr.rr_random_read(p, ses.out, ses.scratch)
    got = ses.checksums(V)
    x, s = 0, 0
    step = 1 << 24
    for first in range(0, region // 4, step):
        w = oracle.fill(first, min(step, region // 4 - first))
        x ^= int(np.bitwise_xor.reduce(w))
        s = (s + int(w.astype(np.uint64).sum())) & 0xFFFFFFFF
    assert int(np.bitwise_xor.reduce(got[:, 0])) == x
    assert int(got[:, 1].astype(np.uint64).sum() & 0xFFFFFFFF) == s


def test_contention_groups_nest_inside_gpcs(ses):
    # two independent views of the layout: timing (pair probe beyond the reach + clustering) and
    # cluster placement (no timing).  Every contention group must lie inside one GPC; TPCs that
    # the cluster scheduler never places a multi-block cluster on (components of one TPC) carry
    # no GPC information and are left out of the comparison.
    groups = ses.discover_groups(total_reads=1 << 16, repeats=3)
    assert groups.n_groups >= 2 and groups.confidence > 4.0
    assert np.array_equal(groups.group_of_sm[0::2], groups.group_of_sm[1::2])   # TPC mates together
    gpc, n_gpcs = rr.rr_gpc_map(ses.scratch, ses.nsm)
    informative = np.bincount(gpc)[gpc] > 2
    for k in range(groups.n_groups):
        members = (groups.group_of_sm == k) & informative
        assert len(set(gpc[members].tolist())) <= 1, (k, np.where(groups.group_of_sm == k)[0])
    # and the partition is finer than the GPCs, as the paper found on its card
    assert groups.n_groups > int((np.bincount(gpc) > 2).sum())


def test_pooled_bench_launch_configuration_sampled(ses):
    # the launch bench.py times: 148 x 32 logical warps owned by 24 SM groups in proportion to
    # their weights, windows tiling the whole buffer, 16384 reads per warp
    region = ses.region_bytes
    groups = rr_inputs.synthetic_group_map(ses.nsm, 24, seed=7)
    weights = [30000 if g % 8 == 0 else 43000 + 100 * g for g in range(24)]
    n_warps = ses.nsm * WPS
    win, ws = rr.rr_make_weighted_windows(region, 1, weights, n_warps, max_window_bytes=64 * GiB)
    assert int(win[-1, 0]) + int(win[-1, 1]) == region // 128 and ws[-1] == n_warps
    reads, first = 256 * 64, 256 * 64 * 5
    p = ses.params(region, W=1, mode=rr.RR_MODE_POOLED, n_warps=n_warps, warps_per_sm=WPS,
                   reads_per_warp=reads, first_read=first, seed=rr_inputs.CFG4_SEED,
                   group_of_sm=groups, windows=win, warp_start=ws)
    assert rr.rr_random_read(p, ses.out, ses.scratch, timed=False) is None
    rep = rr.rr_read_report(p, ses.scratch)
    assert rep.sms_covered == ses.nsm and rep.bytes == n_warps * reads * 128
    got = ses.checksums(n_warps)
    for v in _sample(n_warps):
        g = int(np.searchsorted(ws, v, side="right") - 1)
        base, n = map(int, win[g])
        assert tuple(got[v]) == oracle.warp_checksum(rr_inputs.CFG4_SEED, v, first, reads, 1, base,
                                                     n), v
    t0, t1 = rr.rr_read_block_times(ses.scratch, ses.nsm)
    assert (t1 > t0).all() and t0.min() > 0


def test_pooled_one_window_per_sm_sampled(ses):
    # bench.py's timed step: one window per SM (148 "groups"), weights differing per SM, 2^19
    # reads per warp continuing the stream at a late first_read, one warp load in flight per warp
    region = ses.region_bytes
    rng = np.random.default_rng(3)
    owners = rng.permutation(ses.nsm).astype(np.uint16)
    weights = rng.integers(5000, 8000, ses.nsm)
    n_warps = ses.nsm * WPS
    win, ws = rr.rr_make_weighted_windows(region, 1, weights, n_warps, max_window_bytes=64 * GiB)
    reads, first = 1 << 19, 24 << 19
    p = ses.params(region, W=1, mode=rr.RR_MODE_POOLED, n_warps=n_warps, warps_per_sm=WPS,
                   reads_per_warp=reads, first_read=first, seed=rr_inputs.CFG4_SEED,
                   group_of_sm=owners, windows=win, warp_start=ws, variant=rr.RR_VARIANT_PACKED,
                   unroll=1)
    assert rr.rr_random_read(p, ses.out, ses.scratch, timed=False) is None   # as bench launches it
    res = rr.rr_read_report(p, ses.scratch)
    assert res.sms_covered == ses.nsm and res.bytes == n_warps * reads * 128
    got = ses.checksums(n_warps)
    for v in _sample(n_warps)[::3]:
        g = int(np.searchsorted(ws, v, side="right") - 1)
        base, n = map(int, win[g])
        assert tuple(got[v]) == oracle.warp_checksum(rr_inputs.CFG4_SEED, v, first, reads, 1, base,
                                                     n), v


@pytest.mark.parametrize("reads,first", [(256 * 64 + 77, 4096 * 3), (1 << 19, 24 << 19)])
def test_sorted_execution_over_the_whole_buffer_sampled(ses, reads, first):
    # bench.py's arm g and, where it is the faster plan, its timed step: one static slice per SM,
    # equal work, each warp's reads taken in epochs of 16 x 256, part by part of its 1.1 GiB
    # window, one warp load in flight; once with a ragged last epoch, once a whole step of 2^19
    # reads continuing the stream at a late first_read
    region = ses.region_bytes
    owners = np.arange(ses.nsm, dtype=np.uint16)[::-1].copy()
    win, _ = rr.rr_make_weighted_windows(region, 1, [1] * ses.nsm, ses.nsm * WPS)
    p = ses.params(region, W=1, warps_per_sm=WPS, reads_per_warp=reads, first_read=first,
                   seed=rr_inputs.CFG4_SEED, group_of_sm=owners, windows=win,
                   variant=rr.RR_VARIANT_SORTED, unroll=1, sort_parts=16, sort_reads=256)
    assert rr.rr_random_read(p, ses.out, ses.scratch, timed=False) is None   # as bench launches it
    res = rr.rr_read_report(p, ses.scratch)
    assert res.sms_covered == ses.nsm and res.bytes == ses.nsm * WPS * reads * 128
    got = ses.checksums(ses.nsm * WPS)
    if reads > 1 << 16:                              # the oracle needs ~1 s per warp of 2^19 reads
        for v in _sample(ses.nsm * WPS)[::3]:
            base, n = map(int, win[owners[v // WPS]])
            assert tuple(got[v]) == oracle.warp_checksum(rr_inputs.CFG4_SEED, v, first, reads, 1,
                                                         base, n), v
    else:
        _check_sampled(ses, got, region, 1, reads, rr_inputs.CFG4_SEED, owners, win, first)


def test_balancing_loop_yields_a_valid_plan_and_exact_checksums(ses):
    # Session.balance on the card's real groups: whatever weights the timers lead to, the plan
    # must tile the buffer, hand out every logical warp once, and the read must stay bit exact
    groups = ses.discover_groups(total_reads=1 << 16, repeats=3)
    owners = ses.singleton_groups(groups)
    assert sorted(owners.group_of_sm.tolist()) == list(range(ses.nsm))
    order = np.argsort(owners.group_of_sm)          # SMs in window order: resource groups contiguous
    assert (np.diff(groups.group_of_sm[order].astype(np.int64)) >= 0).all()
    n_warps = ses.nsm * WPS
    win, ws, weights, history = ses.balance(owners, n_warps=n_warps, reads_per_warp=4096,
                                            rounds=3, launches_per_round=3,
                                            variant=rr.RR_VARIANT_PACKED, unroll=2)
    L = ses.region_bytes // 128
    assert win[0, 0] == 0 and int(win[-1, 0]) + int(win[-1, 1]) == L
    assert np.array_equal(win[1:, 0], win[:-1, 0] + win[:-1, 1])
    assert ws[0] == 0 and ws[-1] == n_warps and (np.diff(ws.astype(np.int64)) > 0).all()
    assert len(history) >= 1 and all(h > 100 for h in history) and weights.min() >= 1
    rate, res = ses.read_pooled(owners, win, ws, reads_per_warp=4096, seed=23,
                                variant=rr.RR_VARIANT_PACKED, unroll=2)
    assert res.sms_covered == ses.nsm and rate > 100
    got = ses.checksums(n_warps)
    for v in _sample(n_warps):
        g = int(np.searchsorted(ws, v, side="right") - 1)
        base, n = map(int, win[g])
        assert tuple(got[v]) == oracle.warp_checksum(23, v, 0, 4096, 1, base, n), v


def test_moving_windows_over_the_whole_buffer_sampled(ses):
    # one slice of the buffer per SM, eight sub-windows per slice, 1024 reads per phase
    region = ses.region_bytes
    rng = np.random.default_rng(5)
    owners = rng.permutation(ses.nsm).astype(np.uint16)
    win, _ = rr.rr_make_weighted_windows(region, 1, [1] * ses.nsm, ses.nsm * WPS)
    sub_bytes = (int(win[:, 1].max()) * 128 + 7) // 8
    reads, first = 256 * 64, 256 * 64 * 2
    p = ses.params(region, W=1, warps_per_sm=WPS, reads_per_warp=reads, first_read=first,
                   seed=rr_inputs.CFG4_SEED, group_of_sm=owners, windows=win,
                   variant=rr.RR_VARIANT_PACKED, unroll=2, index_mode=rr.RR_INDEX_PHASED,
                   phase_reads=1024, phase_window_bytes=sub_bytes)
    res = rr.rr_random_read(p, ses.out, ses.scratch)
    assert res.sms_covered == ses.nsm and res.bytes == ses.nsm * WPS * reads * 128
    got = ses.checksums(ses.nsm * WPS)
    for v in _sample(ses.nsm * WPS):
        base, n = map(int, win[owners[v // WPS]])
        st = oracle.stagger_of_sm(v // WPS, ses.nsm, n, sub_bytes // 128)
        assert tuple(got[v]) == oracle.warp_checksum_phased(rr_inputs.CFG4_SEED, v, first, reads, 1,
                                                            base, n, 1024, sub_bytes // 128, st), v


def test_moving_window_over_all_of_memory_from_every_sm_sampled(ses):
    # no partition at all: every SM's window is the whole buffer, cut into 128 MiB sub-windows,
    # SMs staggered over them
    region = ses.region_bytes
    reads = 256 * 64
    sub_bytes = 128 << 20
    p = ses.params(region, W=1, warps_per_sm=WPS, reads_per_warp=reads, seed=7,
                   variant=rr.RR_VARIANT_PACKED, unroll=2, index_mode=rr.RR_INDEX_PHASED,
                   phase_reads=1024, phase_window_bytes=sub_bytes)
    res = rr.rr_random_read(p, ses.out, ses.scratch)
    assert res.sms_covered == ses.nsm
    got = ses.checksums(ses.nsm * WPS)
    L = region // 128
    for v in _sample(ses.nsm * WPS):
        st = oracle.stagger_of_sm(v // WPS, ses.nsm, L, sub_bytes // 128)
        assert tuple(got[v]) == oracle.warp_checksum_phased(7, v, 0, reads, 1, 0, L, 1024,
                                                            sub_bytes // 128, st), v


def test_session_helpers_run_the_plans_they_describe(ses):
    """measure_group_rates, naive_control and windows(): the launches they make are the oracle's
    (checksums, not rates)."""
    groups = rr_inputs.synthetic_group_map(ses.nsm, 12, seed=5)
    from paper_2405_11425_b200.pipeline import Groups
    G = Groups(groups, 12, 10.0)
    S = 16 * GiB
    rates = ses.measure_group_rates(G, S, reads_per_warp=256)
    assert len(rates) == 12 and all(r > 1 for r in rates)
    # the last launch of measure_group_rates: group 11 alone inside [0, S)
    only = np.where(groups == 11, 0, 0xFFFF).astype(np.uint16)
    _check_sampled(ses, ses.checksums(ses.nsm * WPS), ses.region_bytes, 1, 256, 23, only,
                   np.array([[0, S // 128]], np.uint32))
    cg, cw, cov = ses.naive_control(S, 23)
    assert 0 < cov <= 1 and cg.tolist() == list(range(ses.nsm))
    ow, ocov = oracle.make_windows(ses.region_bytes, 1, S, ses.nsm, policy=1, seed=23)
    assert np.array_equal(cw, ow) and cov == ocov
    rate, res = ses.read(ses.region_bytes, seed=23, reads_per_warp=300, group_of_sm=cg, windows=cw)
    assert res.sms_covered == ses.nsm
    _check_sampled(ses, ses.checksums(ses.nsm * WPS), ses.region_bytes, 1, 300, 23, cg, cw)
    win, cov = ses.windows(G, S)
    ow, ocov = oracle.make_windows(ses.region_bytes, 1, S, 12)
    assert np.array_equal(win, ow) and cov == ocov


def test_sustained_protocol_reports_what_it_ran(ses):
    p = ses.params(8 * GiB, seed=7, reads_per_warp=1024, variant=rr.RR_VARIANT_PACKED, unroll=2)
    d = ses.sustained(p, settle=10, min_ms=20.0, reps=3)
    assert d["regions"] == 3 and d["launches_per_region"] >= 1
    assert d["bytes_per_launch"] == ses.nsm * WPS * 1024 * 128
    assert d["gbps_min"] <= d["gbps"] <= d["gbps_max"] and d["gbps"] > 100
    assert d["ms_per_region"] >= 15.0
    _check_sampled(ses, ses.checksums(ses.nsm * WPS), 8 * GiB, 1, 1024, 7)


def test_reach_measurement_refines_between_sweep_points(ses):
    r = ses.measure_reach(sizes_gib=(4, 16, 32, 64, 96, 128), sustained=False)
    sizes = [s for s, _ in r.sweep]
    assert sizes == sorted(sizes) and len(set(sizes)) == len(sizes)
    import oracle as orc
    assert (r.cliff, r.plateau_gbps, r.reach_bytes) == orc.reach(sizes, [g for _, g in r.sweep])
    if r.cliff:                                       # refined to the 2 GiB grid
        above = min(s for s in sizes if s > r.reach_bytes)
        assert above - r.reach_bytes <= 2 * GiB


def test_probe_rows_and_checkpoint_resume(ses, tmp_path):
    # rows probed block by block equal... not bit for bit (rates are measurements), but they fill
    # exactly the rows asked for, and a resumed run keeps the finished rows untouched
    reads = 2 * WPS * 64
    T = np.zeros((ses.nsm, ses.nsm), np.float32)
    st = rr.rr_probe_rows(ses.buf, 1 * GiB, reads, WPS, 5, 1, 10, 13, T, ses.probe_out,
                          ses.probe_scratch)
    touched = np.zeros_like(T, dtype=bool)
    touched[10:13, 10:] = True
    touched |= touched.T
    assert (T[touched] > 0).all() and not T[~touched].any()
    assert np.array_equal(T, T.T) and st["overlap_min"] <= 1.0
    with pytest.raises(rr.RRError):
        rr.rr_probe_rows(ses.buf, 1 * GiB, reads, WPS, 5, 1, 13, 13, T, ses.probe_out,
                         ses.probe_scratch)
    path = tmp_path / "probe.npz"
    g1 = ses.discover_groups(probe_region_bytes=1 * GiB, total_reads=reads, repeats=1,
                             checkpoint=path, rows_per_block=64)
    with np.load(path) as z:
        assert int(z["rows_done"]) == ses.nsm
        saved = z["T"].copy()
        meta, stats = str(z["meta"]), str(z["stats"])
    assert np.array_equal(saved, g1.matrix) and (saved > 0).all()
    # an interrupted run: only the first 64 rows done, marked with a value no probe produces
    half = saved.copy()
    half[64:, 64:] = 0
    half[:64, :] = 12345.0
    half[:, :64] = 12345.0
    np.savez(path, T=half, rows_done=64, meta=meta, stats=stats)
    g2 = ses.discover_groups(probe_region_bytes=1 * GiB, total_reads=reads, repeats=1,
                             checkpoint=path, rows_per_block=64)
    assert (g2.matrix[:64, :] == 12345.0).all() and (g2.matrix[:, :64] == 12345.0).all()
    assert (g2.matrix[64:, 64:] > 0).all() and not (g2.matrix[64:, 64:] == 12345.0).any()
    # other probe settings: the file is ignored and everything is probed afresh
    g3 = ses.discover_groups(probe_region_bytes=1 * GiB, total_reads=reads, repeats=1, seed=6,
                             checkpoint=path, rows_per_block=64)
    assert not (g3.matrix == 12345.0).any()
