"""The report's formatting code on a synthetic result dictionary (no GPU involved)."""
from paper_2405_11425_b200 import alloc_study, report


def _s(x):
    return {"median": float(x), "min": float(x) - 1, "max": float(x) + 1}


def test_markdown_renders_every_section():
    widths = {"128B": _s(4600), "256B": _s(6900), "512B": _s(6950)}
    win = {"window_gib": 35.0, "coverage": 1.0, "grouped": _s(4630),
           "unrestricted_inside_one_window": _s(4630), "naive_per_sm_control": _s(1138),
           "overlapping": dict(_s(4626), coverage=1.0, depth_min=4, depth_max=6)}
    R = {
        "device": {"name": "test GPU", "nsm_prop": 148, "theoretical_gbps": 7672.0},
        "region_gib": 168.7, "fill_gbps": 6246.0, "seconds": 123.0,
        "cfg1_size_sweep": [{"gib": 1.0, "wps16": _s(5300), "wps32": _s(5330)}],
        "reach": {"cliff": True, "plateau_gbps": 4560.0, "reach_gib": 70.0, "points": []},
        "cfg2_widths_32gib": widths, "stride_full": widths,
        "mixed_32gib": {"1": _s(6700), "4": _s(5000)},
        "cfg3_probe": {"inside_reach_16gib": {"n_groups": 1, "pair_min_med_max": [147, 148, 149]},
                       "whole_buffer": {"n_groups": 24, "confidence": 950.0, "sizes": [6] * 24,
                                        "seconds": 15.4}},
        "gpc_map": {"sizes": [18] * 8, "gpcs_of_group": [[0]] * 24},
        "single_groups": [{"group": 0, "sms": 6, "gbps": 250.0}],
        "group_pairs_distinct_windows": [{"a": 0, "b": 1, "gbps": 499.0,
                                          "ratio_to_sum_of_singles": 0.998}],
        "cfg4_grouped": {"128B": {"unrestricted_full": _s(1016), "windows": {"reach/2": win}}},
        "per_sm_window_sweep": [{"window_mib": 512.0, "gbps": 5787.0}],
        "moving_windows": [{"sub_windows": 16, "sub_window_mib": 73.0, "phase_reads": 1024,
                            "sustained_gbps": 5870.0}],
        "moving_windows_no_partition": [{"sub_window_mib": 128, "phase_reads": 1024,
                                         "sustained_gbps": 5850.0}],
        "sorted_execution": [dict(_s(5600), parts=4, unroll=1)],
        "balanced_pooled": {"128B packed, one window per SM": {
            "burst_gbps": 5800.0, "sustained_gbps": 5548.0, "window_gib_min_max": [0.95, 1.24]}},
        "alloc_study": {"device": "test GPU", "bytes": 160 << 30, "granularity_minimum": 2 << 20,
                        "granularity_recommended": 2 << 20,
                        "paths": {"cudaMalloc (torch)": {
                            "plateau_gbps": 4560.0, "cliff": True, "reach_gib": 64.0,
                            "sweep": [[s, 4500.0] for s in alloc_study.SIZES_GIB] + [[160.0, 1000.0]]}}},
    }
    text = report.markdown(R)
    for needle in ("Unrestricted size sweep", "one read in k sequential", "24 groups",
                   "overlapping windows", "4626 [4625-4627] (1.00, 4-6)", "Sorted execution",
                   "Moving windows", "Allocation paths", "cudaMalloc (torch)", "total 123 s"):
        assert needle in text, needle
