"""Pins of the moving-window (phased) index mode: sub-windows tile the window, every read of a
phase lies in that phase's sub-window, one sub-window is the plain random mode, a big-integer
restatement, and uniform coverage over a full cycle."""
import numpy as np
import pytest

import oracle

M64 = (1 << 64) - 1


def _py_sm64(x):
    z = (x + 0x9E3779B97F4A7C15) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def test_lines_stay_in_the_sub_window_of_their_phase_and_sub_windows_tile():
    base, n, B, sub = 5000, 10007, 64, 3000           # Q = 4 sub-windows of 2501/2502 lines
    Q = -(-n // sub)
    bounds = [n * q // Q for q in range(Q + 1)]
    assert bounds[0] == 0 and bounds[-1] == n and all(b > a for a, b in zip(bounds, bounds[1:]))
    for v in (0, 7):
        for i in range(0, 64 * 9, 5):
            q = (i // B) % Q
            line = oracle.line_phased(3, v, i, base, n, B, sub)
            assert base + bounds[q] <= line < base + bounds[q + 1], (v, i)
            kv = _py_sm64(_py_sm64(3) ^ v)
            r = _py_sm64((kv + i * 0x9E3779B97F4A7C15) & M64)
            assert line == base + bounds[q] + r % (bounds[q + 1] - bounds[q])


def test_one_sub_window_is_the_plain_random_mode():
    for sub in (777, 10 ** 6):
        for i in range(0, 500, 7):
            assert oracle.line_phased(23, 42, i, 1000, 777, 32, sub) == oracle.line(23, 42, i, 1000, 777)
    a = oracle.read_per_sm_phased(1 << 22, 2, 5, 3, 50, 9, phase_reads=32, phase_window_bytes=1 << 40)
    b = oracle.read_per_sm(1 << 22, 2, 5, 3, 50, 9)
    assert np.array_equal(a, b)


def test_checksums_follow_the_lines():
    n_bytes = 1 << 20
    L = n_bytes // 128
    groups = np.array([0, 1, 0xFFFF, 1], np.uint16)
    windows = np.array([[0, 3000], [3000, L - 3000]], np.uint32)
    out = oracle.read_per_sm_phased(n_bytes, 1, 4, 2, 100, 5, phase_reads=32,
                                    phase_window_bytes=1000 * 128, group_of_sm=groups,
                                    windows=windows, first_read=64)
    for v in range(8):
        sm = v // 2
        if groups[sm] == 0xFFFF:
            assert tuple(out[v]) == (0, 0)
            continue
        base, n = map(int, windows[groups[sm]])
        x = s = 0
        st = oracle.stagger_of_sm(sm, 4, n, 1000)
        for i in range(64, 164):
            w = oracle.fill(oracle.line_phased(5, v, i, base, n, 32, 1000, st) * 32, 32)
            x ^= int(np.bitwise_xor.reduce(w))
            s = (s + int(w.astype(np.uint64).sum())) & 0xFFFFFFFF
        assert tuple(out[v]) == (x, s)
        assert tuple(out[v]) == oracle.warp_checksum_phased(5, v, 64, 100, 1, base, n, 32, 1000, st)


def test_a_full_cycle_covers_the_window_uniformly():
    n, B, sub = 4096, 256, 1024                      # Q = 4
    lines = np.array([oracle.line_phased(1, v, i, 0, n, B, sub) for v in range(40)
                      for i in range(4 * B)])
    counts = np.bincount(lines * 16 // n, minlength=16)
    expect = len(lines) / 16
    assert np.all(np.abs(counts - expect) < 5 * np.sqrt(expect))


def test_errors():
    with pytest.raises(oracle.OracleError):
        oracle.read_per_sm_phased(1 << 20, 1, 2, 2, 4, 1, phase_reads=0, phase_window_bytes=1 << 16)
    with pytest.raises(oracle.OracleError):
        oracle.read_per_sm_phased(1 << 20, 1, 2, 2, 4, 1, phase_reads=32, phase_window_bytes=64)


def test_stagger_spreads_sms_that_share_one_window():
    # 8 SMs, one window cut into 4 sub-windows: in any phase the SMs sit two per sub-window,
    # and each SM still cycles through all four
    n, B, sub, nsm = 4000, 32, 1000, 8
    for phase in range(6):
        seen = []
        for sm in range(nsm):
            st = oracle.stagger_of_sm(sm, nsm, n, sub)
            assert st == sm * 4 // nsm
            seen.append(oracle.line_phased(1, sm * 2, phase * B, 0, n, B, sub, st) * 4 // n)
        assert sorted(seen) == [0, 0, 1, 1, 2, 2, 3, 3]
    cycle = [oracle.line_phased(1, 6, p * B, 0, n, B, sub, oracle.stagger_of_sm(3, nsm, n, sub)) * 4 // n
             for p in range(4)]
    assert sorted(cycle) == [0, 1, 2, 3]
