"""Window-policy invariants (Section 1.3 / 2.4: every SM group is held to one chunk):
containment, union coverage, the half-memory special case, and the naive per-SM control."""
import itertools

import numpy as np
import pytest

import oracle


def test_exhaustive_small_cases():
    for L, S, G, W in itertools.product(range(1, 41), range(1, 45), (1, 2, 3, 5, 8), (1, 2)):
        lb = 128 * W
        win, cov = oracle.make_windows(L * lb + 17, W, S * lb, G)
        S_eff = min(max(S, 1), L)
        K = -(-L // S_eff)
        chunk = L // K
        assert win.shape == (G, 2)
        covered = np.zeros(L, dtype=bool)
        for g in range(G):
            base, n = int(win[g, 0]), int(win[g, 1])
            assert n >= 1 and base + n <= L                    # inside the region
            assert base == (g % K) * chunk                     # group g -> chunk g mod K
            assert n == (L - base if g % K == K - 1 else chunk)
            assert n < chunk + K                               # only the last chunk is longer
            covered[base:base + n] = True
        assert cov == pytest.approx(min(G, K) / K)
        if K <= G:
            assert covered.all()                               # union of windows = region
        else:
            assert covered.sum() < L


def test_half_memory_is_the_papers_scheme():
    # "half the memory for simplicity": two chunks, groups alternate between them
    region = 170 * (1 << 30)
    win, cov = oracle.make_windows(region, 1, region // 2, 14)
    L = region // 128
    assert cov == 1.0
    for g in range(14):
        assert tuple(win[g]) == ((0, L // 2) if g % 2 == 0 else (L // 2, L - L // 2))


def test_window_larger_than_region_is_whole_region():
    win, cov = oracle.make_windows(1 << 30, 4, 1 << 40, 3)
    assert cov == 1.0 and all(tuple(w) == (0, (1 << 30) // 512) for w in win)


def test_naive_control_picks_a_hashed_chunk_per_sm():
    # the paper's "SM-to-chunk" control: every SM on its own picks a pseudo-random half
    region = 1 << 32
    nsm = 148
    win, cov = oracle.make_windows(region, 1, region // 2, nsm, policy=1, seed=23)
    L = region // 128
    halves = {(0, L // 2), (L // 2, L // 2)}
    picks = [tuple(w) for w in win]
    assert set(picks) == halves and cov == 1.0
    frac = sum(p[0] == 0 for p in picks) / nsm
    assert 0.3 < frac < 0.7
    for s in range(nsm):
        assert picks[s][0] == (oracle.sm64(23 ^ s) % 2) * (L // 2)


def test_errors():
    with pytest.raises(oracle.OracleError):
        oracle.make_windows(1 << 20, 3, 1 << 10, 2)
    with pytest.raises(oracle.OracleError):
        oracle.make_windows(100, 1, 1 << 10, 2)
    with pytest.raises(oracle.OracleError):
        oracle.make_windows(1 << 20, 1, 1 << 10, 0)


def test_per_warp_windows_equal_the_per_warp_definition():
    region = 5000 * 128
    win, cov = oracle.make_windows(region, 1, 700 * 128, 37, policy=1, seed=23)   # hashed chunks
    out = oracle.read_logical_windows(region, 1, 100, 9, 23, win, first_read=4)
    for v in range(100):
        base, n = map(int, win[v % 37])
        assert tuple(out[v]) == oracle.warp_checksum(23, v, 4, 9, 1, base, n, n_warps_total=100)
        for i in range(4, 13):
            assert base <= oracle.line(23, v, i, base, n) < base + n
    # one window covering everything: the plain logical mode
    whole = oracle.read_logical_windows(region, 1, 50, 7, 3, [[0, 5000]])
    assert np.array_equal(whole, oracle.read_logical(region, 1, 50, 7, 3))
    with pytest.raises(oracle.OracleError):
        oracle.read_logical_windows(region, 1, 10, 1, 1, [[4990, 20]])
