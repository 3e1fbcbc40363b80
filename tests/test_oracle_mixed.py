"""Pins of the mixed sequential/random stream: it is a blend of two streams that are pinned on
their own (the random draws by the known answers, the sequential walk by the stride mode's
whole-buffer fold), so it is pinned by taking it apart again."""
import numpy as np
import pytest

import oracle


def test_mixed_lines_are_the_two_pinned_rules_interleaved():
    seed, v, V, base, n = 23, 5, 64, 1000, 777
    for k in (1, 2, 4, 7, 64):
        for i in range(0, 200):
            got = oracle.line_mixed(seed, v, i, base, n, k, n_warps_total=V)
            if i % k == 0:
                assert got == oracle.line(seed, v, i // k, base, n, oracle.INDEX_STRIDE, V)
            else:
                assert got == oracle.line(seed, v, i, base, n)
            assert base <= got < base + n


def test_period_one_is_the_sequential_mode():
    region = 64 * 96 * 128
    a = oracle.read_per_sm_mixed(region, 1, 8, 8, 96, 3, 1)
    b = oracle.read_per_sm(region, 1, 8, 8, 96, 3, index_mode=oracle.INDEX_STRIDE)
    assert np.array_equal(a, b)
    # and so it folds the whole buffer exactly once (V * R == L)
    words = oracle.fill(0, region // 4)
    assert int(np.bitwise_xor.reduce(a[:, 0])) == int(np.bitwise_xor.reduce(words))


@pytest.mark.parametrize("W", [1, 2, 4])
def test_mixed_checksum_splits_into_its_sequential_and_random_parts(W):
    seed, v, V, base, n, k, R = 7, 11, 40, 50, 5000, 4, 64
    x, s = oracle.warp_checksum_mixed(seed, v, 0, R, W, base, n, k, n_warps_total=V)
    # sequential part: reads 0 .. R/k - 1 of the warp's stride walk
    xs, ss = oracle.warp_checksum(seed, v, 0, R // k, W, base, n, oracle.INDEX_STRIDE, V)
    # random part: the random stream minus the reads whose place the sequential ones took
    xr, sr = oracle.warp_checksum(seed, v, 0, R, W, base, n)
    for i in range(0, R, k):
        xi, si = oracle.warp_checksum(seed, v, i, 1, W, base, n)
        xr ^= xi
        sr = (sr - si) & 0xFFFFFFFF
    assert (x, s) == (xs ^ xr, (ss + sr) & 0xFFFFFFFF)


def test_mixed_stream_continues_across_calls_and_share_is_one_in_k():
    seed, v, V, n, k = 1, 0, 16, 1 << 20, 8
    x1, s1 = oracle.warp_checksum_mixed(seed, v, 0, 40, 1, 0, n, k, V)
    x2, s2 = oracle.warp_checksum_mixed(seed, v, 40, 24, 1, 0, n, k, V)
    x, s = oracle.warp_checksum_mixed(seed, v, 0, 64, 1, 0, n, k, V)
    assert (x, s) == (x1 ^ x2, (s1 + s2) & 0xFFFFFFFF)
    seq = [oracle.line_mixed(seed, v, i, 0, n, k, V) for i in range(0, 800, k)]
    assert seq == [(j * V + v) % n for j in range(100)]            # a walk with stride V
    with pytest.raises(oracle.OracleError):
        oracle.read_per_sm_mixed(1 << 20, 1, 4, 4, 8, 1, 0)
