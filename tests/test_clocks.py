"""The nvidia-smi sample parser and the window summary (no GPU, no nvidia-smi needed)."""
import datetime

from paper_2405_11425_b200 import clocks


def _row(t, mhz, watts, power_cap="Not Active", thermal="Not Active"):
    ts = datetime.datetime.fromtimestamp(t).strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
    return (f"{ts}, {mhz}, 1965, {watts}, 0x0000000000000004, Not Active, {thermal}, Not Active, "
            f"{power_cap}")


def test_parse_and_summarise_a_window():
    t0 = 1_700_000_000.0
    rows = [_row(t0 + 0.05 * k, 1965 if k < 10 else 1650 + k, 400 + 30 * k,
                 "Active" if k >= 10 else "Not Active") for k in range(30)]
    rows.insert(3, "garbage line")
    rows.append("2023/11/14 22:13:20.000, [N/A], 1965, 1.0, 0, a, b, c, d")   # unparsable clock
    s = clocks.parse_rows(rows)
    assert len(s) == 30 and s[0][1] == 1965.0 and s[-1][4]["sw_power_cap"]
    w = clocks.summarise(s, t0 + 0.5, t0 + 1.0)
    assert w["during_timed_region"] and w["samples"] == 11        # samples 10..20 (+- slack)
    assert w["sm_mhz"] == 1665.0 and w["sm_mhz_min"] == 1660.0 and w["sm_max_mhz"] == 1965.0
    assert w["reasons"] == ["sw_power_cap"] and not w["rejected"]
    # too few samples inside: all samples are used and the summary says so
    w = clocks.summarise(s, t0 + 100, t0 + 101)
    assert not w["during_timed_region"] and w["samples"] == 30
    assert clocks.summarise([], 0, 1)["reasons"] == ["no samples"]


def test_thermal_slowdown_rejects_the_window():
    t0 = 1_700_000_000.0
    rows = [_row(t0 + 0.05 * k, 1200, 900, thermal="Active" if k == 4 else "Not Active")
            for k in range(8)]
    w = clocks.summarise(clocks.parse_rows(rows), t0, t0 + 0.4)
    assert w["rejected"] and "hw_thermal_slowdown" in w["reasons"]
