"""Structural pins of the read oracle: a big-integer brute force over tiny materialised buffers,
the width identity, grouped == ungrouped for one whole-region window, the sequential mode folding
the whole buffer, first_read continuation, and draw statistics."""
import math

import numpy as np
import pytest

import oracle

M64 = (1 << 64) - 1


# --- an independent, literal restatement in Python integers (materialise, then index) ---------
def py_sm64(x):
    z = (x + 0x9E3779B97F4A7C15) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def py_buffer(n_words):
    return [py_sm64(i) & 0xFFFFFFFF for i in range(n_words)]


def py_checksum(buf, seed, v, first, reads, W, base, n):
    kv = py_sm64(py_sm64(seed) ^ v)
    x = s = 0
    lines = []
    for i in range(first, first + reads):
        r = py_sm64((kv + i * 0x9E3779B97F4A7C15) & M64)
        line = base + r % n
        lines.append(line)
        chunk = buf[line * 32 * W:(line + 1) * 32 * W]   # the literal coalesced line
        assert len(chunk) == 32 * W
        for w in chunk:
            x ^= w
            s = (s + w) & 0xFFFFFFFF
    return x, s, lines


@pytest.mark.parametrize("n_bytes", [4096, 65536, 1 << 20])
@pytest.mark.parametrize("W", [1, 2, 4])
def test_brute_force_tiny_buffers(n_bytes, W):
    buf = py_buffer(n_bytes // 4)
    assert np.array_equal(oracle.fill(0, n_bytes // 4), np.array(buf, dtype=np.uint32))
    L = n_bytes // (128 * W)
    n_warps, reads = 12, 9
    got = oracle.read_logical(n_bytes, W, n_warps, reads, seed=3, first_read=5)
    for v in range(n_warps):
        x, s, lines = py_checksum(buf, 3, v, 5, reads, W, 0, L)
        assert tuple(got[v]) == (x, s)
        assert all(0 <= l < L for l in lines)


def test_brute_force_windows_per_sm():
    n_bytes = 1 << 18
    buf = py_buffer(n_bytes // 4)
    nsm, wps, W = 6, 3, 1
    L = n_bytes // 128
    groups = np.array([0, 1, 0xFFFF, 2, 1, 0], dtype=np.uint16)
    windows = np.array([[0, 100], [100, 777], [1500, L - 1500]], dtype=np.uint32)
    got = oracle.read_per_sm(n_bytes, W, nsm, wps, 7, seed=23, group_of_sm=groups, windows=windows)
    for sm in range(nsm):
        for w in range(wps):
            v = sm * wps + w
            if groups[sm] == 0xFFFF:
                assert tuple(got[v]) == (0, 0)
                continue
            base, n = map(int, windows[groups[sm]])
            x, s, lines = py_checksum(buf, 23, v, 0, 7, W, base, n)
            assert tuple(got[v]) == (x, s)
            assert all(base <= l < base + n for l in lines)   # invariant: inside the window


def test_width_identity():
    # a W=2 read of line l folds the words of W=1 lines 2l, 2l+1; W=4 <-> 4l..4l+3
    n_bytes = 1 << 22
    for W in (2, 4):
        L = n_bytes // (128 * W)
        for v in range(5):
            x = s = 0
            for i in range(6):
                l = oracle.line(11, v, i, 0, L)
                words = oracle.fill(l * 32 * W, 32 * W)
                x ^= int(np.bitwise_xor.reduce(words))
                s = (s + int(words.astype(np.uint64).sum())) & 0xFFFFFFFF
                # the same words through W=1 reads of the covering narrow lines
                xs = [oracle.fill((l * W + k) * 32, 32) for k in range(W)]
                assert np.array_equal(np.concatenate(xs), words)
            assert oracle.warp_checksum(11, v, 0, 6, W, 0, L) == (x, s)


def test_single_whole_window_equals_ungrouped():
    n_bytes = 3 * (1 << 20) + 640          # ragged tail shorter than a line is never read
    nsm, wps = 5, 4
    L = n_bytes // 128
    a = oracle.read_per_sm(n_bytes, 1, nsm, wps, 10, seed=7)
    b = oracle.read_per_sm(n_bytes, 1, nsm, wps, 10, seed=7,
                           group_of_sm=np.zeros(nsm, dtype=np.uint16),
                           windows=np.array([[0, L]], dtype=np.uint32))
    assert np.array_equal(a, b)


def test_first_read_continues_the_stream():
    a = oracle.warp_checksum(7, 9, 0, 40, 1, 0, 1000)
    b = oracle.warp_checksum(7, 9, 0, 25, 1, 0, 1000)
    c = oracle.warp_checksum(7, 9, 25, 15, 1, 0, 1000)
    assert a == (b[0] ^ c[0], (b[1] + c[1]) & 0xFFFFFFFF)


@pytest.mark.parametrize("W", [1, 2, 4])
def test_stride_mode_folds_the_whole_buffer(W):
    # sequential mode visits line (i*V + v) mod n: with V*R == n every line exactly once, so the
    # checksums combined over warps equal the fold of the whole region
    V, R = 16, 8
    n_bytes = V * R * 128 * W
    out = oracle.read_logical(n_bytes, W, V, R, seed=99, index_mode=oracle.INDEX_STRIDE)
    words = oracle.fill(0, n_bytes // 4)
    assert int(np.bitwise_xor.reduce(out[:, 0])) == int(np.bitwise_xor.reduce(words))
    assert int(out[:, 1].astype(np.uint64).sum() & 0xFFFFFFFF) == int(
        words.astype(np.uint64).sum() & 0xFFFFFFFF)


def test_draws_are_uniform_and_mostly_distinct():
    # chi-square of idx over 256 equal buckets, and the birthday fraction of distinct lines
    n = 1 << 20
    m = 200_000
    idx = np.array([oracle.line(7, v, i, 0, n) for v in range(200) for i in range(m // 200)])
    counts = np.bincount(idx * 256 // n, minlength=256)
    chi2 = float(((counts - m / 256) ** 2 / (m / 256)).sum())
    assert 170 < chi2 < 350          # 255 dof: mean 255, sd ~22.6
    distinct = len(np.unique(idx)) / m
    expect = n * (1 - math.exp(-m / n)) / m
    assert abs(distinct - expect) < 0.005


def test_argument_errors():
    with pytest.raises(oracle.OracleError):
        oracle.read_logical(1 << 20, 3, 4, 4, seed=1)            # width
    with pytest.raises(oracle.OracleError):
        oracle.read_logical(64, 1, 4, 4, seed=1)                 # region shorter than a line
    with pytest.raises(oracle.OracleError):
        oracle.read_per_sm(1 << 20, 1, 2, 2, 4, seed=1, group_of_sm=np.array([0, 1], np.uint16),
                           windows=np.array([[0, 10]], np.uint32))        # group id >= n_groups
    with pytest.raises(oracle.OracleError):
        oracle.read_per_sm(1 << 20, 1, 2, 2, 4, seed=1, group_of_sm=np.array([0, 0], np.uint16),
                           windows=np.array([[8000, 1000]], np.uint32))   # window past the region


@pytest.mark.parametrize("W", [1, 2, 4])
def test_materialised_buffer_read_equals_regenerating_read(W):
    # 64 MiB really filled and really indexed, against the oracle that regenerates every word
    n_bytes = (64 << 20) + 256
    buf = oracle.fill(0, n_bytes // 4)
    a = oracle.read_logical_materialised(buf, W, 300, 50, seed=11, first_read=3)
    b = oracle.read_logical(n_bytes, W, 300, 50, seed=11, first_read=3)
    assert np.array_equal(a, b)
