"""Bookkeeping of the plateau / cliff / reach rule applied to a size sweep (Section 2.1, Fig. 1).
The thresholds themselves are a reading with no external truth (parity unpinned); these tests
only fix what the rule does on synthetic curves."""
import numpy as np
import pytest

import oracle

GiB = 1 << 30
SIZES = [s * GiB for s in (1, 4, 16, 32, 48, 64, 96, 128, 160)]


def test_a100_like_cliff():
    gbps = [1500, 1000, 1000, 1010, 1000, 990, 300, 250, 240]
    cliff, plateau, reach = oracle.reach(SIZES, gbps)
    assert cliff and plateau == 1000 and reach == 64 * GiB


def test_no_cliff():
    gbps = [4000, 3500, 3400, 3450, 3400, 3390, 3300, 3200, 3150]
    cliff, plateau, reach = oracle.reach(SIZES, gbps)
    assert not cliff and plateau == 3450 and reach == 160 * GiB


def test_gradual_decline_reach_is_last_point_above_90_percent():
    gbps = [4000, 1000, 1000, 1000, 950, 880, 790, 500, 400]
    cliff, plateau, reach = oracle.reach(SIZES, gbps)
    assert cliff and reach == 48 * GiB


def test_errors():
    with pytest.raises(oracle.OracleError):
        oracle.reach([1 * GiB, 2 * GiB], [1.0, 1.0])          # no point on the plateau range
    with pytest.raises(oracle.OracleError):
        oracle.reach([8 * GiB, 4 * GiB], [1.0, 1.0])          # sizes must increase
