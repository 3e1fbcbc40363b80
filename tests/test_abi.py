"""CPU-side checks of the C-ABI library: it builds and loads without a GPU, exports every
symbol the header declares, rejects bad arguments before touching CUDA, and its host-only
policies (windows, reach) agree with the oracle."""
import ctypes
import itertools
import random
import re
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2405_11425_b200 import binding as rr
from paper_2405_11425_b200 import build as rr_build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def built_library():
    rr_build.build()
    return rr._load()


def test_exports_match_header(built_library):
    header = (ROOT / "include" / "rr.h").read_text()
    declared = set(re.findall(r"^\s*(?:const\s+char\s*\*|int32_t|size_t)\s*\*?\s*(rr_\w+)\s*\(",
                              header, flags=re.M))
    assert declared == set(rr.EXPORTS)
    for name in declared:
        assert hasattr(built_library, name), name


def test_strerror_covers_all_codes():
    texts = {rr.rr_strerror(c) for c in range(0, -10, -1)}
    assert len(texts) == 10 and "unknown status" not in texts
    assert rr.rr_strerror(-99) == "unknown status"


FAKE = 0x7F0000000000  # a 512-byte aligned fake device address: validation never dereferences it


def _call(**kw):
    base = dict(W=1, mode=rr.RR_MODE_LOGICAL, n_warps=4, reads_per_warp=4, seed=1)
    base.update(kw)
    buf = base.pop("buf", FAKE)
    region = base.pop("region_bytes", 1 << 20)
    out = base.pop("out", FAKE)
    scratch = base.pop("scratch", FAKE)
    p = rr.ReadParams(buf, region, **base)
    return rr._load().rr_random_read(ctypes.byref(p.c), out, scratch, None, 0)


def test_read_argument_errors_come_before_any_cuda_call():
    assert _call(W=3) == rr.RR_ERR_ARG
    assert _call(mode=7) == rr.RR_ERR_ARG
    assert _call(index_mode=2) == rr.RR_ERR_ARG
    assert _call(index_mode=4) == rr.RR_ERR_ARG
    assert _call(index_mode=rr.RR_INDEX_MIXED) == rr.RR_ERR_ARG              # needs a period
    assert _call(index_mode=rr.RR_INDEX_MIXED, mix_period=6) == rr.RR_ERR_ARG  # a power of two
    assert _call(mix_period=4) == rr.RR_ERR_ARG                              # only with MIXED
    srt = dict(variant=rr.RR_VARIANT_SORTED, sort_parts=4, sort_reads=64)
    assert _call(**{**srt, "sort_parts": 3}) == rr.RR_ERR_ARG
    assert _call(**{**srt, "sort_parts": 32}) == rr.RR_ERR_ARG
    assert _call(**{**srt, "sort_parts": 8, "sort_reads": 544}) == rr.RR_ERR_ARG    # 4096 per epoch
    assert _call(**{**srt, "sort_reads": 48}) == rr.RR_ERR_ARG
    assert _call(**{**srt, "sort_reads": 0}) == rr.RR_ERR_ARG
    assert _call(**{**srt, "W": 4}) == rr.RR_ERR_ARG
    assert _call(**{**srt, "index_mode": rr.RR_INDEX_STRIDE}) == rr.RR_ERR_ARG
    assert _call(**{**srt, "unroll": 8}) == rr.RR_ERR_ARG
    assert _call(sort_parts=4) == rr.RR_ERR_ARG                              # only with SORTED
    assert _call(variant=9) == rr.RR_ERR_ARG
    assert _call(unroll=3) == rr.RR_ERR_ARG
    assert _call(n_warps=0) == rr.RR_ERR_ARG
    assert _call(buf=0) == rr.RR_ERR_ARG
    assert _call(out=0) == rr.RR_ERR_ARG
    assert _call(scratch=0) == rr.RR_ERR_ARG
    assert _call(buf=FAKE + 128) == rr.RR_ERR_ALIGN
    assert _call(out=FAKE + 4) == rr.RR_ERR_ALIGN
    assert _call(region_bytes=100) == rr.RR_ERR_RANGE
    assert _call(region_bytes=128 << 32) == rr.RR_ERR_RANGE         # 2^32 lines: one too many
    assert _call(reads_per_warp=1 << 63) == rr.RR_ERR_RANGE
    # logical mode takes no SM grouping; windows alone mean a window per warp
    assert _call(group_of_sm=np.zeros(4, np.uint16), windows=[[0, 8]]) == rr.RR_ERR_ARG
    assert _call(windows=[[0, 8], [8, 9000]]) == rr.RR_ERR_RANGE
    assert _call(windows=[[0, 8], [8, 0]]) == rr.RR_ERR_RANGE
    per_sm = dict(mode=rr.RR_MODE_PER_SM, n_warps=0, nsm=4)
    assert _call(warps_per_sm=0, **per_sm) == rr.RR_ERR_ARG
    assert _call(warps_per_sm=65, **per_sm) == rr.RR_ERR_ARG
    assert _call(warps_per_sm=33, **per_sm) == rr.RR_ERR_ARG
    assert _call(windows=[[0, 8]], **per_sm) == rr.RR_ERR_ARG       # windows without a map
    g = np.array([0, 1, 0, 1], np.uint16)
    assert _call(group_of_sm=g, windows=[[0, 8], [8, 9000]], **per_sm) == rr.RR_ERR_RANGE
    assert _call(group_of_sm=g, windows=[[0, 8], [8, 0]], **per_sm) == rr.RR_ERR_RANGE
    assert _call(group_of_sm=g, windows=[[0, 8]], **per_sm) == rr.RR_ERR_MAP
    dead = np.full(4, 0xFFFF, np.uint16)
    assert _call(group_of_sm=dead, windows=[[0, 8]], **per_sm) == rr.RR_ERR_MAP


def test_other_entry_points_reject_bad_arguments():
    lib = rr._load()
    assert lib.rr_fill(0, 16, 0) == rr.RR_ERR_ARG
    assert lib.rr_fill(FAKE + 64, 16, 0) == rr.RR_ERR_ALIGN
    assert lib.rr_fill(FAKE, 0, 0) == rr.RR_OK                      # empty fill is a no-op
    res = rr._Result()
    args = (FAKE, 1 << 30, 0, 1)
    assert lib.rr_probe_pair(*args, 1 << 10, 0, 5, FAKE, FAKE, ctypes.byref(res), 0) == rr.RR_ERR_ARG
    assert lib.rr_probe_pair(*args, 1000, 32, 5, FAKE, FAKE, ctypes.byref(res), 0) == rr.RR_ERR_ARG
    assert lib.rr_probe_pair(*args, 1 << 10, 33, 5, FAKE, FAKE, ctypes.byref(res), 0) == rr.RR_ERR_ARG
    assert lib.rr_probe_pair(FAKE, 64, 0, 1, 1 << 10, 8, 5, FAKE, FAKE, ctypes.byref(res), 0) == rr.RR_ERR_RANGE
    T = np.ones((8, 8), np.float32)
    T[2, 3] = np.nan
    g = np.zeros(8, np.int32)
    ng = ctypes.c_uint32()
    assert lib.rr_cluster(T.ctypes.data, 8, 0, FAKE, g.ctypes.data, ctypes.byref(ng), None, None, 0) == rr.RR_ERR_ARG
    T[2, 3] = -1
    assert lib.rr_cluster(T.ctypes.data, 8, 0, FAKE, g.ctypes.data, ctypes.byref(ng), None, None, 0) == rr.RR_ERR_ARG
    T[2, 3] = 1
    assert lib.rr_cluster(T.ctypes.data, 8, 2, FAKE, g.ctypes.data, ctypes.byref(ng), None, None, 0) == rr.RR_ERR_ARG
    T[4, 4] = 0   # solo normalisation needs a valid diagonal
    assert lib.rr_cluster(T.ctypes.data, 8, 1, FAKE, g.ctypes.data, ctypes.byref(ng), None, None, 0) == rr.RR_ERR_ARG
    T[4, 4] = 1
    assert lib.rr_cluster(T.ctypes.data, 1, 0, FAKE, g.ctypes.data, ctypes.byref(ng), None, None, 0) == rr.RR_ERR_ARG
    assert lib.rr_cluster(T.ctypes.data, 8, 0, FAKE + 4, g.ctypes.data, ctypes.byref(ng), None, None, 0) == rr.RR_ERR_ALIGN


def test_make_windows_matches_oracle():
    for L, S, G, W, policy in itertools.product((1, 2, 7, 40, 1000, 12345), (1, 3, 64, 999, 10 ** 6),
                                                (1, 2, 5, 14, 148), (1, 2, 4), (0, 1, 2)):
        lb = 128 * W
        a, ca = rr.rr_make_windows(L * lb + 5, W, S * lb, G, policy, seed=23)
        b, cb = oracle.make_windows(L * lb + 5, W, S * lb, G, policy, seed=23)
        assert np.array_equal(a, b) and ca == cb
    big = int(0.95 * 178 * (1 << 30)) // 512 * 512
    for S in (big // 8, big // 4, big // 2, big, 64 << 30, 37 << 30):
        for policy in (0, 2):
            a, ca = rr.rr_make_windows(big, 1, S, 16, policy)
            b, cb = oracle.make_windows(big, 1, S, 16, policy)
            assert np.array_equal(a, b) and ca == cb
    with pytest.raises(rr.RRError):
        rr.rr_make_windows(1 << 20, 1, 1 << 10, 2, policy=3)
    with pytest.raises(rr.RRError):
        rr.rr_make_windows(1 << 20, 3, 1 << 10, 2)
    with pytest.raises(rr.RRError):
        rr.rr_make_windows(1 << 20, 1, 1 << 10, 0)
    with pytest.raises(rr.RRError):
        rr.rr_make_windows(64, 1, 1 << 10, 2)


def test_weighted_windows_match_oracle():
    rng = np.random.default_rng(5)
    for _ in range(200):
        G = int(rng.integers(1, 40))
        w = rng.integers(1, 5000, G).astype(np.uint32)
        W = int(rng.choice([1, 2, 4]))
        region = int(rng.integers(G * 2000, 10 ** 8)) * 128 * W + 9
        V = int(rng.integers(G * 50, 10 ** 5))
        try:
            b_win, b_ws = oracle.make_weighted_windows(region, W, w, V)
        except oracle.OracleError:                   # a tiny weight left a group without warps
            with pytest.raises(rr.RRError):
                rr.rr_make_weighted_windows(region, W, w, V)
            continue
        a_win, a_ws = rr.rr_make_weighted_windows(region, W, w, V)
        assert np.array_equal(a_win, b_win) and np.array_equal(a_ws, b_ws)
    big = int(0.95 * 178 * (1 << 30)) // 512 * 512
    w = [249, 249, 250, 251, 138, 248] * 4
    a = rr.rr_make_weighted_windows(big, 1, w, 4736, max_window_bytes=70 << 30)
    b = oracle.make_weighted_windows(big, 1, w, 4736, max_window_bytes=70 << 30)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    for bad in (dict(weights=[1, 0, 1], n_warps=100), dict(weights=[1, 1, 1], n_warps=2),
                dict(weights=[2 ** 31, 2 ** 31], n_warps=100)):
        with pytest.raises(rr.RRError):
            rr.rr_make_weighted_windows(1 << 30, 1, bad["weights"], bad["n_warps"])
    with pytest.raises(rr.RRError):
        rr.rr_make_weighted_windows(1 << 30, 1, [1, 3], 100, max_window_bytes=600 << 20)


def test_pooled_mode_argument_errors():
    g = np.array([0, 1, 0, 1], np.uint16)
    ok = dict(mode=rr.RR_MODE_POOLED, n_warps=10, nsm=4, warps_per_sm=8, group_of_sm=g,
              windows=[[0, 100], [100, 100]], warp_start=[0, 4, 10])
    assert _call(**{**ok, "warp_start": None}) == rr.RR_ERR_ARG
    assert _call(**{**ok, "warp_start": [1, 4, 10]}) == rr.RR_ERR_ARG
    assert _call(**{**ok, "warp_start": [0, 4, 9]}) == rr.RR_ERR_ARG
    assert _call(**{**ok, "warp_start": [0, 11, 10]}) == rr.RR_ERR_ARG
    assert _call(**{**ok, "index_mode": rr.RR_INDEX_STRIDE}) == rr.RR_ERR_ARG
    assert _call(**{**ok, "windows": [[0, 100], [100, 90000]]}) == rr.RR_ERR_RANGE
    assert _call(**{**ok, "group_of_sm": np.array([0, 0, 0, 0], np.uint16)}) == rr.RR_ERR_MAP
    assert _call(**{**ok, "group_of_sm": np.array([0, 2, 0, 1], np.uint16)}) == rr.RR_ERR_MAP
    # other modes take no pool arguments
    assert _call(pool_block_reads=256) == rr.RR_ERR_ARG
    assert _call(warp_start=[0, 4]) == rr.RR_ERR_ARG


def test_phased_index_argument_errors():
    ok = dict(index_mode=rr.RR_INDEX_PHASED, phase_reads=256, phase_window_bytes=1 << 16)
    assert _call(**{**ok, "phase_reads": 0}) == rr.RR_ERR_ARG
    assert _call(**{**ok, "phase_reads": 16}) == rr.RR_ERR_ARG
    assert _call(**{**ok, "phase_reads": 96}) == rr.RR_ERR_ARG            # not a power of two
    assert _call(**{**ok, "first_read": 5}) == rr.RR_ERR_ARG              # streams start at x32
    assert _call(**{**ok, "phase_window_bytes": 64}) == rr.RR_ERR_RANGE
    assert _call(phase_reads=256) == rr.RR_ERR_ARG                        # only with PHASED
    assert _call(phase_window_bytes=1 << 20) == rr.RR_ERR_ARG
    g = np.array([0, 1, 0, 1], np.uint16)
    assert _call(mode=rr.RR_MODE_POOLED, n_warps=10, nsm=4, warps_per_sm=8, group_of_sm=g,
                 windows=[[0, 100], [100, 100]], warp_start=[0, 4, 10], **ok) == rr.RR_ERR_ARG


def test_reach_matches_oracle():
    rng = np.random.default_rng(3)
    sizes = [s << 30 for s in (1, 4, 16, 32, 48, 64, 96, 128, 160, 169)]
    for _ in range(200):
        g = rng.uniform(500, 4000, len(sizes))
        if rng.random() < 0.5:
            g[rng.integers(4, len(sizes)):] *= 0.3
        assert rr.rr_reach(sizes, g) == oracle.reach(sizes, g)
    with pytest.raises(rr.RRError):
        rr.rr_reach([2 << 30, 1 << 30], [1.0, 1.0])
    with pytest.raises(rr.RRError):
        rr.rr_reach([1 << 30], [1.0])


def test_reach_next_and_sm_reach_match_oracle():
    rng = np.random.default_rng(7)
    GiB = 1 << 30
    for _ in range(300):
        sizes = sorted({int(x) * 2 * GiB for x in rng.integers(1, 85, int(rng.integers(3, 14)))})
        if sizes[0] > 32 * GiB:
            sizes = [4 * GiB] + sizes
        g = rng.uniform(3000, 4600, len(sizes))
        cut = int(rng.integers(1, len(sizes) + 1))
        g[cut:] *= rng.choice([0.3, 0.85, 0.5])
        step = int(rng.choice([1, 2, 4])) * GiB
        try:
            expect = oracle.reach_next(sizes, g, step)
        except oracle.OracleError:
            with pytest.raises(rr.RRError):
                rr.rr_reach_next(sizes, g, step)
            continue
        assert rr.rr_reach_next(sizes, g, step) == expect
    with pytest.raises(rr.RRError):
        rr.rr_reach_next([4 * GiB, 8 * GiB], [1.0, 1.0], 0)
    for _ in range(300):
        n = int(rng.integers(1, 12))
        sizes = np.cumsum(rng.integers(1, 300, n)).astype(np.uint64) << 20
        rates = rng.uniform(4500, 6000, n)
        keep = float(rng.choice([1.0, 0.99, 0.97, 0.9, 0.6]))
        assert rr.rr_sm_reach(sizes, rates, keep) == oracle.sm_reach(sizes, rates, keep)
    with pytest.raises(rr.RRError):
        rr.rr_sm_reach([2, 2], [1.0, 1.0])
    with pytest.raises(rr.RRError):
        rr.rr_sm_reach([1, 2], [1.0, 1.0], keep=0.0)


def test_owner_map_phase_window_and_cover_match_oracle():
    rng = np.random.default_rng(8)
    for _ in range(200):
        nsm = int(rng.integers(1, 257))
        g = rng.integers(0, int(rng.integers(1, 40)), nsm).astype(np.uint16)
        g[rng.random(nsm) < 0.1] = 0xFFFF
        a, na = rr.rr_owner_map(g)
        b, nb = oracle.owner_map(g)
        assert na == nb and np.array_equal(a, b)
    for _ in range(500):
        sl, reach = int(rng.integers(1, 1 << 36)), int(rng.integers(1, 1 << 32))
        mp = int(rng.choice([1, 8, 64, 1000]))
        assert rr.rr_phase_window(sl, reach, mp) == oracle.phase_window(sl, reach, mp)
    with pytest.raises(rr.RRError):
        rr.rr_phase_window(0, 1 << 20)
    for _ in range(300):
        L = int(rng.integers(1, 10 ** 6))
        G = int(rng.integers(1, 60))
        base = rng.integers(0, L, G)
        n = np.minimum(rng.integers(1, L + 1, G), L - base)
        win = np.stack([base, np.maximum(n, 1)], axis=1).astype(np.uint32)
        win[:, 1] = np.minimum(win[:, 1], L - win[:, 0])
        assert rr.rr_window_cover(win, L) == oracle.window_cover(win, L)
    with pytest.raises(rr.RRError):
        rr.rr_window_cover([[5, 10]], 12)


def test_rebalance_and_spread_match_oracle():
    rng = np.random.default_rng(9)
    for _ in range(400):
        G = int(rng.integers(1, 150))
        work = rng.integers(0, 1 << int(rng.integers(1, 31)), G).astype(np.uint32)
        fin = rng.integers(1, 1 << int(rng.integers(8, 45)), G).astype(np.uint64)
        fin[rng.random(G) < 0.1] = 0
        scale = int(rng.integers(1, 1 << 31))
        assert rr.rr_finish_spread_ppm(fin) == oracle.finish_spread_ppm(fin)
        try:
            expect = oracle.rebalance_weights(work, fin, scale)
        except oracle.OracleError:
            with pytest.raises(rr.RRError):
                rr.rr_rebalance_weights(work, fin, scale)
            continue
        assert np.array_equal(rr.rr_rebalance_weights(work, fin, scale), expect)


def test_group_finish_matches_oracle():
    rng = np.random.default_rng(11)
    for _ in range(300):
        nsm = int(rng.integers(1, 257))
        G = int(rng.integers(1, 40))
        g = rng.integers(0, G, nsm).astype(np.uint16)
        g[rng.random(nsm) < 0.1] = 0xFFFF
        t0 = rng.integers(1 << 40, (1 << 40) + 5000, nsm).astype(np.uint64)
        t1 = t0 + rng.integers(1, 1 << 22, nsm).astype(np.uint64)
        t1[rng.random(nsm) < 0.1] = 0
        a, sa = rr.rr_group_finish(t0, t1, g, G)
        b, sb = oracle.group_finish(t0, t1, g, G)
        assert np.array_equal(a, b) and sa == sb
    with pytest.raises(rr.RRError):
        rr.rr_group_finish([1], [2], [3], 2)


def test_probe_rate_matches_oracle():
    rng = np.random.default_rng(10)
    for _ in range(500):
        t0 = rng.integers(1 << 40, 1 << 41, 2).astype(np.uint64)
        t1 = t0 + rng.integers(0, 1 << 22, 2).astype(np.uint64)
        claim = rng.integers(0, 3, 2).astype(np.uint32)
        if rng.random() < 0.1:
            t1[int(rng.integers(0, 2))] = 0
        solo = bool(rng.random() < 0.3)
        reads = int(rng.integers(1, 1 << 24)) * 2
        extra = rng.integers(0, 1 << 20, 2).astype(np.uint64) * 64
        try:
            expect = oracle.probe_rate(t0, t1, claim, solo, reads, extra)
        except oracle.OracleError as e:
            with pytest.raises(rr.RRError) as r:
                rr.rr_probe_rate(t0, t1, claim, solo, reads, extra)
            assert r.value.code == e.code == rr.RR_ERR_SM_UNCOVERED
            continue
        assert rr.rr_probe_rate(t0, t1, claim, solo, reads, extra) == expect


def test_exact_remainder_identity():
    # The kernels take r mod n as r - floor(r*m / 2^64)*n with m = floor((2^64-1)/n), corrected
    # by at most one subtraction of n.  Check that claim with big integers on edge cases.
    rnd = random.Random(1)
    ns = [1, 2, 3, 5, 777, 2 ** 23, 2 ** 23 + 1, 402653184, 2 ** 31 - 1, 2 ** 31, 2 ** 32 - 1]
    ns += [rnd.randrange(1, 2 ** 32) for _ in range(200)]
    for n in ns:
        m = (2 ** 64 - 1) // n
        rs = [0, 1, n - 1, n, n + 1, 2 ** 64 - 1, 2 ** 64 - n, 2 ** 63, m * n, m * n - 1,
              (m * n + n - 1) % 2 ** 64]
        rs += [rnd.randrange(0, 2 ** 64) for _ in range(50)]
        for r in rs:
            q = (r * m) >> 64
            rem = r - q * n
            assert 0 <= rem < 2 * n
            if rem >= n:
                rem -= n
            assert rem == r % n
