"""Pins of the capacity-weighted windows and the pooled read mode (Section 2.3: a group's
throughput is a property of the group, so work and window size follow the group's weight)."""
import itertools

import numpy as np
import pytest

import oracle


def test_weighted_windows_tile_the_region_exactly():
    rng = np.random.default_rng(0)
    for trial in range(300):
        G = int(rng.integers(1, 30))
        w = rng.integers(1, 1000, G).astype(np.uint32)
        W = int(rng.choice([1, 2, 4]))
        L = int(rng.integers(G * 1000, 10 ** 7))
        V = int(rng.integers(G * 1000, 10 ** 5 + G * 1000))
        win, ws = oracle.make_weighted_windows(L * 128 * W + 77, W, w, V)
        assert win[0, 0] == 0 and int(win[-1, 0]) + int(win[-1, 1]) == L
        assert np.array_equal(win[1:, 0], win[:-1, 0] + win[:-1, 1])      # no gap, no overlap
        assert ws[0] == 0 and ws[-1] == V and np.all(np.diff(ws.astype(np.int64)) > 0)
        T = int(w.sum())
        share = w.astype(np.float64) / T
        assert np.all(np.abs(win[:, 1] - share * L) < 1.0001)             # proportional +-1 line
        assert np.all(np.abs(np.diff(ws.astype(np.int64)) - share * V) < 1.0001)
        # the defining formula, retyped with Python integers
        P = 0
        for g in range(G):
            assert int(win[g, 0]) == L * P // T and int(ws[g]) == V * P // T
            P += int(w[g])


def test_equal_weights_give_equal_windows():
    win, ws = oracle.make_weighted_windows(24 * 1000 * 128, 1, [7] * 24, 24 * 32)
    assert set(win[:, 1].tolist()) == {1000} and set(np.diff(ws).tolist()) == {32}


def test_weighted_windows_errors():
    with pytest.raises(oracle.OracleError):
        oracle.make_weighted_windows(1 << 20, 1, [1, 0, 1], 100)          # zero weight
    with pytest.raises(oracle.OracleError):
        oracle.make_weighted_windows(1 << 20, 1, [1, 1, 1], 2)            # a group without warps
    with pytest.raises(oracle.OracleError):
        oracle.make_weighted_windows(256, 1, [1, 1, 1], 100)              # a group without lines
    with pytest.raises(oracle.OracleError):
        oracle.make_weighted_windows(1 << 30, 1, [1, 3], 100, max_window_bytes=600 << 20)
    oracle.make_weighted_windows(1 << 30, 1, [1, 3], 100, max_window_bytes=800 << 20)


def test_pooled_equals_per_warp_definition():
    region = (1 << 22) + 300
    win, ws = oracle.make_weighted_windows(region, 2, [3, 1, 5, 2], 37)
    out = oracle.read_pooled(region, 2, win, ws, reads=21, seed=23, first_read=4)
    assert out.shape == (37, 2)
    for v in range(37):
        g = int(np.searchsorted(ws, v, side="right") - 1)
        base, n = map(int, win[g])
        assert tuple(out[v]) == oracle.warp_checksum(23, v, 4, 21, 2, base, n)
        for i in range(4, 25):
            assert base <= oracle.line(23, v, i, base, n) < base + n      # inside the window


def test_pooled_with_148_groups_and_empty_groups_equals_per_warp_definition():
    """One window per SM (148 groups of ~32 warps) and groups that own no warps: the single loop
    over all warps must find each warp's owner, skipping empty ranges."""
    region = 148 * 5000 * 128
    win, ws = oracle.make_weighted_windows(region, 1, [900 + 7 * (g % 11) for g in range(148)], 4736)
    out = oracle.read_pooled(region, 1, win, ws, reads=5, seed=23, first_read=2)
    for v in list(range(0, 4736, 97)) + [4735]:
        g = int(np.searchsorted(ws, v, side="right") - 1)
        assert tuple(out[v]) == oracle.warp_checksum(23, v, 2, 5, 1, int(win[g, 0]), int(win[g, 1]))
    win = np.array([[0, 100], [100, 50], [150, 70], [300, 10]], np.uint32)
    ws = [0, 0, 6, 6, 9]                                   # groups 0 and 2 own nothing
    out = oracle.read_pooled(1 << 20, 1, win, ws, reads=7, seed=3)
    for v in range(9):
        g = 1 if v < 6 else 3
        assert tuple(out[v]) == oracle.warp_checksum(3, v, 0, 7, 1, int(win[g, 0]), int(win[g, 1]))


def test_pooled_with_one_group_is_the_logical_mode():
    region = 3 << 20
    L = region // 128
    out = oracle.read_pooled(region, 1, [[0, L]], [0, 50], reads=13, seed=9)
    assert np.array_equal(out, oracle.read_logical(region, 1, 50, 13, seed=9))


def test_pooled_errors():
    with pytest.raises(oracle.OracleError):
        oracle.read_pooled(1 << 20, 1, [[0, 10], [10, 10]], [0, 5, 3], 4, 1)     # decreasing starts
    with pytest.raises(oracle.OracleError):
        oracle.read_pooled(1 << 20, 1, [[0, 10], [10, 9000]], [0, 5, 8], 4, 1)   # window past end
    with pytest.raises(oracle.OracleError):
        oracle.read_pooled(1 << 20, 1, [[0, 10]], [1, 5], 4, 1)                  # must start at 0
