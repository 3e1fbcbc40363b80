"""Small, self-contained runs of single kernels, sized for profiling captures.

    python -m paper_2405_11425_b200.cases read  [--region-gib 4] [--W 1] [--reads 4096]
                                                [--launches 3] [--groups 0] [--unroll 0]
                                                [--stride] [--warps-per-sm 32] [--packed] [--pooled]
                                                [--sorted-parts 8] [--sorted-reads 512]
    python -m paper_2405_11425_b200.cases fill  [--region-gib 4] [--launches 3]
    python -m paper_2405_11425_b200.cases probe [--region-gib 4] [--reads 65536] [--pairs 4]
    python -m paper_2405_11425_b200.cases cluster [--n 148]

Each prints one JSON line with the event-timed rate of the last launch.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding as rr

GiB = 1 << 30


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["read", "fill", "probe", "cluster"])
    ap.add_argument("--region-gib", type=float, default=4.0)
    ap.add_argument("--W", type=int, default=1)
    ap.add_argument("--reads", type=int, default=4096)
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--groups", type=int, default=0, help="synthetic SM groups, one window each")
    ap.add_argument("--unroll", type=int, default=0)
    ap.add_argument("--stride", action="store_true")
    ap.add_argument("--packed", action="store_true", help="16-byte lanes, 4/W lines per warp load")
    ap.add_argument("--pooled", action="store_true",
                    help="logical warps owned by the synthetic groups, work shared inside a group")
    ap.add_argument("--sorted-parts", type=int, default=0,
                    help="sorted execution: one window per SM, reads taken part by part")
    ap.add_argument("--sorted-reads", type=int, default=0,
                    help="reads per part and epoch (default 4096 / parts)")
    ap.add_argument("--warps-per-sm", type=int, default=32)
    ap.add_argument("--pairs", type=int, default=4)
    ap.add_argument("--n", type=int, default=148)
    a = ap.parse_args(argv)

    import torch
    torch.cuda.set_device(0)
    info = rr.rr_device_info()
    nsm = info["nsm_prop"]
    scratch = torch.zeros(rr.rr_scratch_bytes(), dtype=torch.uint8, device="cuda")
    region = (int(a.region_gib * GiB) // 512) * 512
    out = {"case": a.case, "device": info["name"]}

    if a.case == "cluster":
        import rr_inputs
        sizes = [6] * (a.n // 6 - 1) + [a.n - 6 * (a.n // 6 - 1)]
        T, _ = rr_inputs.planted_matrix(sizes, 0.3, seed=0, solo_spread=0.1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g, G, conf, _ = rr.rr_cluster(T, scratch, rr.RR_CLUSTER_SOLO_NORMALISE)
        e1.record()
        torch.cuda.synchronize()
        out.update(n=a.n, n_groups=G, confidence=conf, ms=e0.elapsed_time(e1))
        print(json.dumps(out))
        return 0

    buf = torch.empty(region, dtype=torch.uint8, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(a.launches if a.case == "fill" else 1):
        e0.record()
        rr.rr_fill(buf, region // 4)
        e1.record()
        torch.cuda.synchronize()
    if a.case == "fill":
        out.update(region_bytes=region, gbps=region / e0.elapsed_time(e1) * 1e-6)
        print(json.dumps(out))
        return 0

    if a.case == "probe":
        o = torch.zeros((64, 2), dtype=torch.int32, device="cuda")
        rates = []
        for k in range(a.pairs):
            r = rr.rr_probe_pair(buf, region, 2 * k, 2 * k + 1, a.reads, 32, 5, o, scratch)
            rates.append(r.gbps)
        out.update(region_bytes=region, pair_gbps=rates)
        print(json.dumps(out))
        return 0

    groups = windows = None
    if a.groups:
        import rr_inputs
        groups = rr_inputs.synthetic_group_map(nsm, a.groups, seed=1)
        windows, _ = rr.rr_make_windows(region, a.W, -(-region // a.groups), a.groups)
    o = torch.zeros((nsm * a.warps_per_sm, 2), dtype=torch.int32, device="cuda")
    variant = rr.RR_VARIANT_PACKED if a.packed else rr.RR_VARIANT_LDG
    if a.sorted_parts:  # one window per SM, equal work; with --pooled each SM's warps share it
        groups = np.arange(nsm, dtype=np.uint16)
        n_warps = nsm * a.warps_per_sm
        windows, warp_start = rr.rr_make_weighted_windows(region, a.W, [1] * nsm, n_warps)
        kw = dict(mode=rr.RR_MODE_POOLED, n_warps=n_warps, nsm=nsm,
                  warp_start=warp_start) if a.pooled else {}
        p = rr.ReadParams(buf, region, W=a.W, warps_per_sm=a.warps_per_sm, reads_per_warp=a.reads,
                          seed=7, unroll=a.unroll, group_of_sm=groups, windows=windows,
                          variant=rr.RR_VARIANT_SORTED, sort_parts=a.sorted_parts,
                          sort_reads=a.sorted_reads or 4096 // a.sorted_parts, **kw)
    elif a.pooled:
        import rr_inputs
        n_groups = a.groups or 24
        groups = rr_inputs.synthetic_group_map(nsm, n_groups, seed=1)
        n_warps = nsm * a.warps_per_sm
        windows, warp_start = rr.rr_make_weighted_windows(region, a.W, [1] * n_groups, n_warps)
        p = rr.ReadParams(buf, region, W=a.W, mode=rr.RR_MODE_POOLED, n_warps=n_warps,
                          warps_per_sm=a.warps_per_sm, nsm=nsm, reads_per_warp=a.reads, seed=7,
                          unroll=a.unroll, group_of_sm=groups, windows=windows,
                          warp_start=warp_start, variant=variant)
    else:
        p = rr.ReadParams(buf, region, W=a.W, warps_per_sm=a.warps_per_sm, reads_per_warp=a.reads,
                          seed=7, unroll=a.unroll, group_of_sm=groups, windows=windows,
                          variant=variant,
                          index_mode=rr.RR_INDEX_STRIDE if a.stride else rr.RR_INDEX_RANDOM)
    for _ in range(a.launches):
        res = rr.rr_random_read(p, o, scratch)
    out.update(region_bytes=region, W=a.W, reads=a.reads, bytes=res.bytes, gbps=res.gbps,
               seconds=res.seconds_event)
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
