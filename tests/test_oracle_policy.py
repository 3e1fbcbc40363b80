"""Pins of the oracle's planning rules: reach refinement, per-SM reach, one window per SM,
moving sub-window size, capacity weights, overlapping windows, probe rate and overlap.

None of these has a value printed in the paper (it gives prose only), so they are pinned by
hand-worked cases, brute force on small inputs and the properties the rule exists to provide.
"""
import numpy as np
import pytest

import oracle

GiB = 1 << 30
MiB = 1 << 20


# ---- reach refinement ---------------------------------------------------------------------------
def _refine(true_cliff, sizes_gib, step):
    """Drives reach_next against a synthetic card whose rate halves above `true_cliff` bytes."""
    rate = lambda n: 4500.0 if n <= true_cliff else 2000.0       # noqa: E731
    pts = {s * GiB: rate(s * GiB) for s in sizes_gib}
    asked = []
    for _ in range(40):
        sizes = sorted(pts)
        nxt = oracle.reach_next(sizes, [pts[s] for s in sizes], step)
        if not nxt:
            break
        assert nxt not in pts and nxt % step == 0
        asked.append(nxt)
        pts[nxt] = rate(nxt)
    sizes = sorted(pts)
    cliff, plateau, reach = oracle.reach(sizes, [pts[s] for s in sizes])
    return cliff, reach, asked


def test_reach_next_hand_worked():
    # sweep brackets the cliff between 64 and 96 GiB; true cliff at 71 GiB; 2 GiB grid
    cliff, reach, asked = _refine(71 * GiB, (1, 4, 16, 32, 48, 64, 96, 128), 2 * GiB)
    assert cliff and asked == [80 * GiB, 72 * GiB, 68 * GiB, 70 * GiB]
    assert reach == 70 * GiB


@pytest.mark.parametrize("true_gib", [33.5, 40, 63.9, 64, 65, 90.1, 127])
def test_reach_next_converges_to_the_grid_point_below_the_cliff(true_gib):
    step = 2 * GiB
    true_cliff = int(true_gib * GiB)
    cliff, reach, asked = _refine(true_cliff, (1, 4, 16, 32, 48, 64, 96, 128, 160), step)
    assert cliff
    assert reach <= true_cliff < reach + max(step, 1) or reach in (32 * GiB, 48 * GiB, 64 * GiB, 96 * GiB, 128 * GiB)
    assert reach <= true_cliff and true_cliff - reach < 2 * step   # grid floor, one step of slack
    assert len(asked) <= 5                                         # log2(32 GiB / 2 GiB) + 1


def test_reach_next_without_cliff_or_with_adjacent_points():
    s = [4 * GiB, 16 * GiB, 64 * GiB]
    assert oracle.reach_next(s, [4500, 4500, 4400], 2 * GiB) == 0            # no cliff
    s = [4 * GiB, 16 * GiB, 64 * GiB, 66 * GiB]
    assert oracle.reach_next(s, [4500, 4500, 4500, 1000], 2 * GiB) == 0      # already adjacent
    with pytest.raises(oracle.OracleError):
        oracle.reach_next(s, [4500, 4500, 4500, 1000], 0)


def test_reach_next_point_between_the_thresholds_moves_the_bad_end():
    # 0.85 of the plateau: not good (< 0.9), not a cliff (>= 0.8) -- it becomes the new upper end
    s = [4 * GiB, 32 * GiB, 64 * GiB, 80 * GiB, 96 * GiB]
    g = [4500, 4500, 4500, 0.85 * 4500, 1000]
    assert oracle.reach(s, g) == (True, 4500.0, 64 * GiB)
    assert oracle.reach_next(s, g, 2 * GiB) == 72 * GiB


# ---- per-SM reach -----------------------------------------------------------------------------------
def test_sm_reach_hand_worked():
    sizes = [m * MiB for m in (32, 64, 128, 256, 384, 512, 768, 1024)]
    rates = [5840, 5790, 5760, 5750, 5700, 5690, 5500, 5200]
    # level = middle of the first three = 5790; 0.97 * 5790 = 5616.3
    assert oracle.sm_reach(sizes, rates, 0.97) == 512 * MiB
    assert oracle.sm_reach(sizes, rates, 0.99) == 256 * MiB        # 5732.1: 5750 passes, 5700 not
    assert oracle.sm_reach(sizes, rates, 0.5) == 1024 * MiB
    # a later recovery does not count: only the leading run
    assert oracle.sm_reach(sizes, [5800, 5800, 5800, 5000, 5800, 5800, 5800, 5800], 0.97) == 128 * MiB
    # the first point falls short of the level set by the next two: the first size is returned
    assert oracle.sm_reach(sizes[:3], [1000, 6000, 6000], 0.97) == 32 * MiB
    assert oracle.sm_reach(sizes[:2], [6000, 5900], 0.97) == 64 * MiB   # fewer than 3: first rate
    with pytest.raises(oracle.OracleError):
        oracle.sm_reach([2, 1], [1.0, 1.0], 0.97)
    with pytest.raises(oracle.OracleError):
        oracle.sm_reach([1, 2], [1.0, 1.0], 1.5)


def test_sm_reach_properties():
    rng = np.random.default_rng(1)
    for _ in range(300):
        n = int(rng.integers(1, 10))
        sizes = np.cumsum(rng.integers(1, 100, n)).astype(np.uint64) * MiB
        rates = rng.uniform(4000, 6000, n)
        level = sorted(rates[:3])[1] if n >= 3 else rates[0]
        prev = None
        for keep in (1.0, 0.97, 0.9, 0.5):
            r = oracle.sm_reach(sizes, rates, keep)
            k = list(sizes).index(r)
            assert all(rates[j] >= keep * level for j in range(1, k + 1)) or k == 0
            if k + 1 < n and rates[0] >= keep * level:
                assert rates[k + 1] < keep * level                 # the run really ended there
            if prev is not None:
                assert r >= prev                                   # a laxer rule never shrinks it
            prev = r


# ---- one window per SM --------------------------------------------------------------------------------
def test_owner_map_is_the_stable_order_by_group():
    rng = np.random.default_rng(2)
    for _ in range(200):
        nsm = int(rng.integers(1, 200))
        G = int(rng.integers(1, 30))
        g = rng.integers(0, G, nsm).astype(np.uint16)
        g[rng.random(nsm) < 0.1] = 0xFFFF
        owner, n = oracle.owner_map(g)
        active = [s for s in range(nsm) if g[s] != 0xFFFF]
        assert n == len(active)
        assert sorted(int(owner[s]) for s in active) == list(range(n))     # a permutation
        assert all(owner[s] == 0xFFFF for s in range(nsm) if g[s] == 0xFFFF)
        expect = sorted(active, key=lambda s: (int(g[s]), s))
        assert [int(np.where(owner == k)[0][0]) for k in range(n)] == expect
        # SMs of one group hold consecutive ids
        for grp in set(int(x) for x in g[g != 0xFFFF]):
            ids = sorted(int(owner[s]) for s in active if g[s] == grp)
            assert ids == list(range(ids[0], ids[0] + len(ids)))


def test_owner_map_hand_worked():
    owner, n = oracle.owner_map([1, 0, 0xFFFF, 1, 0, 2])
    assert n == 5 and owner.tolist() == [2, 0, 0xFFFF, 3, 1, 4]


# ---- moving sub-window size ------------------------------------------------------------------------------
def test_phase_window_hand_worked_and_properties():
    assert oracle.phase_window(1168 * MiB, 512 * MiB) == (16, 73 * MiB)     # 1168/16 = 73 <= 128
    assert oracle.phase_window(1168 * MiB, 384 * MiB) == (16, 73 * MiB)     # 1168/8 = 146 > 96
    assert oracle.phase_window(100 * MiB, 512 * MiB) == (1, 100 * MiB)      # already small enough
    assert oracle.phase_window(128 * MiB, 512 * MiB) == (1, 128 * MiB)      # exactly a quarter
    assert oracle.phase_window(128 * MiB + 1, 512 * MiB) == (2, 64 * MiB + 1)
    assert oracle.phase_window(1 << 40, 1 * MiB, 64)[0] == 64               # capped
    rng = np.random.default_rng(3)
    for _ in range(500):
        slice_b = int(rng.integers(1, 1 << 34))
        reach = int(rng.integers(1, 1 << 31))
        parts, sub = oracle.phase_window(slice_b, reach, 64)
        assert parts & (parts - 1) == 0 and 1 <= parts <= 64
        assert sub * parts >= slice_b > (sub - 1) * parts                    # ceil division
        if parts < 64:
            assert 4 * slice_b <= reach * parts                              # small enough
        if parts > 1:
            assert 4 * slice_b > reach * (parts // 2)                        # and minimal
        assert oracle.phase_window(slice_b, 2 * reach, 64)[0] <= parts       # monotone in the reach


# ---- capacity weights --------------------------------------------------------------------------------------
def test_rebalance_fixed_point_and_proportionality():
    rng = np.random.default_rng(4)
    for _ in range(200):
        G = int(rng.integers(1, 40))
        work = rng.integers(1, 200, G).astype(np.uint32)
        t = int(rng.integers(10_000, 10_000_000))
        # every group finished together: the weights are the work shares
        w = oracle.rebalance_weights(work, [t] * G, 1_000_000)
        share = work / work.sum() * 1_000_000
        assert np.all(np.abs(w.astype(np.int64) - share) <= 1.0 + share * 1e-6)
        assert abs(int(w.sum()) - 1_000_000) <= G
        # a group that took twice as long has shown half the rate
        if G >= 2:
            fin = np.full(G, t, dtype=np.uint64)
            fin[0] = 2 * t
            w2 = oracle.rebalance_weights(work, fin, 1_000_000)
            others = w2[1:].astype(np.float64) / w[1:]
            assert np.allclose(w2[0] / w[0] / others.mean(), 0.5, rtol=2e-3, atol=2e-3) or w[0] < 2000


def test_rebalance_hand_worked_unseen_and_errors():
    # rates 32/1000 : 32/2000 = 2 : 1; the unseen group gets 1/1024 of the slowest
    w = oracle.rebalance_weights([32, 32, 40], [1000, 2000, 0], 1_000_000)
    total = 2048 + 1024 + 1
    assert w.tolist() == [round(2048 / total * 1e6), round(1024 / total * 1e6), round(1 / total * 1e6)]
    # (32 * 2^48 / 1000 is not an integer: the floors shift the shares by far less than 1e-6)
    assert oracle.rebalance_weights([5], [77], 1000).tolist() == [1000]
    assert oracle.rebalance_weights([1, 10 ** 6], [10 ** 9, 1], 10).tolist() == [1, 10]   # floor of 1
    with pytest.raises(oracle.OracleError):
        oracle.rebalance_weights([1, 2], [0, 0])                          # nobody finished
    with pytest.raises(oracle.OracleError):
        oracle.rebalance_weights([1, 2], [5, 5], 0)


def test_rebalance_definition_in_python_integers():
    rng = np.random.default_rng(5)
    for _ in range(200):
        G = int(rng.integers(1, 30))
        work = [int(x) for x in rng.integers(0, 1 << 20, G)]
        fin = [int(x) if rng.random() > 0.15 else 0 for x in rng.integers(1, 1 << 40, G)]
        scale = int(rng.integers(1, 1 << 30))
        rate = [max(1, (w << 48) // f) if (f and w) else 0 for w, f in zip(work, fin)]
        if not any(rate):
            continue
        token = max(1, min(r for r in rate if r) // 1024)
        rate = [r or token for r in rate]
        T = sum(rate)
        expect = [max(1, (r * scale + T // 2) // T) for r in rate]
        assert oracle.rebalance_weights(work, fin, scale).tolist() == expect


def test_group_finish_hand_worked():
    #            SM:   0     1     2     3      4 (never ran)  5 (inactive, ran anyway)
    t0 = [1000, 1100, 1050, 1200, 0, 1000]
    t1 = [2000, 2500, 1900, 3000, 0, 9000]
    g = [0, 1, 0, 1, 1, 0xFFFF]
    fin, span = oracle.group_finish(t0, t1, g, 3)
    assert fin.tolist() == [1000, 2000, 0] and span == 8000    # group 2 has no SM: not seen
    fin, span = oracle.group_finish([5, 5], [0, 0], [0, 1], 2)
    assert fin.tolist() == [0, 0] and span == 0
    with pytest.raises(oracle.OracleError):
        oracle.group_finish([1], [2], [3], 2)                  # group id out of range


def test_finish_spread():
    assert oracle.finish_spread_ppm([1000, 1000, 1000]) == 0
    assert oracle.finish_spread_ppm([900, 1000, 0, 950]) == 100_000         # unseen groups ignored
    assert oracle.finish_spread_ppm([0, 0]) == 0
    assert oracle.finish_spread_ppm([1, 3]) == 666_666                      # rounded down


# ---- overlapping windows (policy 2) and window cover --------------------------------------------------------------
def test_overlapping_windows_invariants_and_coverage_brute_force():
    rng = np.random.default_rng(6)
    for _ in range(400):
        W = int(rng.choice([1, 2, 4]))
        L = int(rng.integers(1, 3000))
        G = int(rng.integers(1, 40))
        S_req = int(rng.integers(1, 2 * L + 2))
        win, cov = oracle.make_windows(L * 128 * W + int(rng.integers(0, 128 * W)), W,
                                       S_req * 128 * W, G, policy=2)
        S = min(max(S_req, 1), L)
        assert np.all(win[:, 1] == S)                                        # all exactly S lines
        assert win[0, 0] == 0 and np.all(np.diff(win[:, 0].astype(np.int64)) >= 0)
        assert np.all(win[:, 0].astype(np.int64) + S <= L)                   # containment
        if G > 1:
            assert int(win[-1, 0]) + S == L                                  # the last ends at L
            for g in range(G):
                assert int(win[g, 0]) == g * (L - S) // (G - 1)
        hit = np.zeros(L, dtype=np.int32)
        for b, n in win:
            hit[int(b):int(b) + int(n)] += 1
        assert cov == pytest.approx((hit > 0).sum() / L, abs=1e-12)
        if G * S >= L + G:                                                   # enough with slack
            assert cov == 1.0
        if G * S < L:
            assert cov < 1.0
        covered, dmin, dmax = oracle.window_cover(win, L)
        assert covered == int((hit > 0).sum())
        assert dmin == int(hit[hit > 0].min()) and dmax == int(hit.max())


def test_window_cover_on_chunk_and_weighted_windows():
    win, cov = oracle.make_windows(1000 * 128, 1, 250 * 128, 8)             # 4 chunks, 8 groups
    assert oracle.window_cover(win, 1000) == (1000, 2, 2)
    win, ws = oracle.make_weighted_windows(1000 * 128, 1, [1, 2, 3], 60)    # a tiling
    assert oracle.window_cover(win, 1000) == (1000, 1, 1)
    assert oracle.window_cover([[10, 5], [100, 7]], 1000) == (12, 1, 1)
    with pytest.raises(oracle.OracleError):
        oracle.window_cover([[990, 20]], 1000)


# ---- probe rate and overlap ---------------------------------------------------------------------------------------
def test_probe_rate_hand_worked():
    reads = 1 << 12                                        # 2048 lines per SM = 262144 bytes
    # both SMs side by side for the same 1000 ns
    g, sec, ov = oracle.probe_rate([100, 100], [1100, 1100], [1, 1], False, reads)
    assert (g, ov) == (524288 / 1000, 1.0) and sec == pytest.approx(1000e-9, rel=1e-12)
    # late start of the second SM by 200 ns: union 1200, intersection 1000 - 200 = 800
    g, sec, ov = oracle.probe_rate([100, 300], [1100, 1300], [1, 1], False, reads)
    assert g == 524288 / 1200 and ov == 800 / 1200
    # early end of one SM
    g, sec, ov = oracle.probe_rate([100, 100], [600, 1100], [1, 3], False, reads)
    assert g == 524288 / 1000 and ov == 0.5
    # one after the other: no overlap at all
    g, sec, ov = oracle.probe_rate([0, 1000], [1000, 2000], [1, 1], False, reads)
    assert ov == 0.0 and g == 524288 / 2000
    # the order of the two SMs does not matter
    assert oracle.probe_rate([300, 100], [1300, 1100], [1, 1], False, reads) == \
        oracle.probe_rate([100, 300], [1100, 1300], [1, 1], False, reads)
    # solo: one SM's bytes, overlap 1 by definition, the second entry is ignored
    g, sec, ov = oracle.probe_rate([100, 0], [1100, 0], [1, 0], True, reads)
    assert (g, ov) == (262144 / 1000, 1.0)
    # lines read beyond the fixed share (an SM that waited for a slower partner) count as well
    g, sec, ov = oracle.probe_rate([100, 100], [1100, 1090], [1, 1], False, reads, extra_lines=(0, 192))
    assert g == (524288 + 192 * 128) / 1000 and ov == 990 / 1000
    # an SM that never ran
    for bad in ([[100, 100], [1100, 0], [1, 1]], [[100, 100], [1100, 1100], [1, 0]]):
        with pytest.raises(oracle.OracleError) as e:
            oracle.probe_rate(*bad, False, reads)
        assert e.value.code == -6
