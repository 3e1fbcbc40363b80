"""Runs the paper's experiments on the current GPU and writes report.json / report.md.

    python -m paper_2405_11425_b200.report --out DIR [--quick]

Experiments (paper section -> workload configuration):
  size sweep, unrestricted            Section 2.1, Fig. 1            configs[1]
  line widths at 32 GiB               Section 2.1                    configs[2]
  pair probe + clustering             Section 2.2, Fig. 2-3          configs[3]
  single groups, group pairs          Section 2.3, Fig. 4-5
  grouped windows over all memory     Section 2.4, Fig. 6            configs[4]
  sequential reads of the same kernel Section 2.1 (last paragraph)
  allocation paths (--alloc-study)    Section 1.2 (reach = translations x page size)
All numbers are event-timed GB/s (10^9 B/s) by the sustained protocol of Session.sustained (settling
launches, then regions of back-to-back launches; median [min-max] of the regions); nothing is
computed here beyond bookkeeping.
"""
from __future__ import annotations

import argparse
import json
import time
from pathlib import Path

import numpy as np

from . import binding as rr
from .pipeline import GiB, Session


def _stats(ses, region, reps=5, *, settle=30, min_ms=50.0, **kw):
    """One figure of the report: Session.sustained (settling launches, then `reps` regions of at
    least `min_ms` of back-to-back launches), median / min / max GB/s."""
    if "variant" not in kw:          # the packed shape wherever it exists (W = 1, 2), as bench.py
        packed = kw.get("W", 1) < 4
        kw["variant"] = rr.RR_VARIANT_PACKED if packed else rr.RR_VARIANT_LDG
        kw.setdefault("unroll", 2 if packed else 8)
    d = ses.sustained(ses.params(region, **kw), settle=settle, min_ms=min_ms, reps=reps)
    return {"median": d["gbps"], "min": d["gbps_min"], "max": d["gbps_max"]}


def run(out_dir: Path, quick: bool = False, alloc_study: bool = False) -> dict:
    import torch
    torch.cuda.set_device(0)
    out_dir.mkdir(parents=True, exist_ok=True)
    t_start = time.time()
    ses = Session()
    N = ses.region_bytes
    R = {"device": ses.info, "region_bytes": N, "region_gib": N / GiB,
         "alloc_conf": __import__("os").environ.get("PYTORCH_CUDA_ALLOC_CONF", "")}
    R["fill_gbps"] = max(ses.fill(), ses.fill())
    reads = 256 * (16 if quick else 64)
    reps = 3 if quick else 5

    # configs[0]: correctness case, rate informational
    out0 = torch.zeros((1 << 16, 2), dtype=torch.int32, device="cuda")
    p0 = rr.ReadParams(ses.buf, 1 * GiB, W=1, mode=rr.RR_MODE_LOGICAL, n_warps=1 << 16,
                       reads_per_warp=16, seed=1)
    rr.rr_random_read(p0, out0, ses.scratch)
    R["cfg0_gbps_informational"] = rr.rr_random_read(p0, out0, ses.scratch).gbps

    # configs[1]: size sweep, two occupancies
    sizes = [s * GiB for s in (1, 4, 16, 32, 48, 64, 96, 128, 160) if s * GiB < N] + [N]
    sweep = []
    for n in sizes:
        row = {"gib": n / GiB}
        for wps in (16, 32):
            row[f"wps{wps}"] = _stats(ses, n, reps, seed=7, reads_per_warp=reads, warps_per_sm=wps)
        row["best"] = max(row["wps16"]["median"], row["wps32"]["median"])
        sweep.append(row)
    R["cfg1_size_sweep"] = sweep
    reach = ses.measure_reach()
    R["reach"] = {"cliff": reach.cliff, "plateau_gbps": reach.plateau_gbps,
                  "reach_gib": reach.reach_bytes / GiB,
                  "points": [[s / GiB, g] for s, g in reach.sweep]}

    # configs[2]: widths
    R["cfg2_widths_32gib"] = {f"{128 * W}B": _stats(ses, 32 * GiB, reps, W=W, seed=11,
                                                    reads_per_warp=reads) for W in (1, 2, 4)}
    # sequential control of the same kernel
    R["stride_full"] = {f"{128 * W}B": _stats(ses, N, reps, W=W, reads_per_warp=reads,
                                              index_mode=rr.RR_INDEX_STRIDE) for W in (1, 2, 4)}

    # between the two: one read in k sequential, the rest random (32 GiB, inside the reach)
    R["mixed_32gib"] = {str(k): _stats(ses, 32 * GiB, reps, W=1, seed=11, reads_per_warp=reads,
                                       index_mode=rr.RR_INDEX_MIXED, mix_period=k)
                        for k in (1, 2, 4, 16, 64)}

    # configs[3]: probe inside the reach (as the config says) and over everything
    t0 = time.time()
    g16 = ses.discover_groups(probe_region_bytes=16 * GiB,
                              total_reads=(1 << 18) if quick else (1 << 20),
                              repeats=3, seed=5)
    np.save(out_dir / "probe_matrix_16gib.npy", g16.matrix)
    gf = ses.discover_groups(total_reads=1 << 18, repeats=3, seed=5)
    np.save(out_dir / "probe_matrix_full.npy", gf.matrix)
    R["cfg3_probe"] = {
        "inside_reach_16gib": {"n_groups": g16.n_groups, "confidence": g16.confidence,
                               "seconds": g16.probe_seconds,
                               "pair_min_med_max": _offdiag(g16.matrix)},
        "whole_buffer": {"n_groups": gf.n_groups, "confidence": gf.confidence,
                         "seconds": gf.probe_seconds, "sizes": gf.sizes,
                         "group_of_sm": gf.group_of_sm.tolist(),
                         "pair_min_med_max": _offdiag(gf.matrix),
                         "solo_min_med_max": _mmm(np.diag(gf.matrix))},
        "total_seconds": time.time() - t0,
    }
    groups = gf
    gpc, n_gpcs = rr.rr_gpc_map(ses.scratch, ses.nsm)
    R["gpc_map"] = {"n_components": n_gpcs, "sizes": np.bincount(gpc).tolist(),
                    "gpc_of_sm": gpc.tolist(),
                    "gpcs_of_group": [sorted(set(gpc[gf.group_of_sm == k].tolist()))
                                      for k in range(gf.n_groups)]}

    # Section 2.3: every group alone inside the reach, and pairs of groups in distinct windows
    S = (reach.reach_bytes // 2) if reach.cliff else N // 4
    L_S = S // 128
    singles = []
    for g in range(groups.n_groups):
        gm = np.where(groups.group_of_sm == g, 0, 0xFFFF).astype(np.uint16)
        rate = _stats(ses, N, 3, settle=5, min_ms=20.0, seed=23, reads_per_warp=reads,
                      group_of_sm=gm, windows=[[0, L_S]])["median"]
        singles.append({"group": g, "sms": int((gm == 0).sum()), "gbps": rate})
    R["single_groups"] = singles
    pairs = []
    ids = list(range(groups.n_groups))
    chosen = [(a, b) for a in ids for b in ids if a < b]
    if quick:
        chosen = chosen[:: max(1, len(chosen) // 12)]
    for a, b in chosen:
        gm = np.full(ses.nsm, 0xFFFF, np.uint16)
        gm[groups.group_of_sm == a] = 0
        gm[groups.group_of_sm == b] = 1
        rate = _stats(ses, N, 3, settle=5, min_ms=20.0, seed=23, reads_per_warp=reads,
                      group_of_sm=gm, windows=[[0, L_S], [2 * L_S, L_S]])["median"]
        pairs.append({"a": a, "b": b, "gbps": rate,
                      "ratio_to_sum_of_singles": rate / (singles[a]["gbps"] + singles[b]["gbps"])})
    R["group_pairs_distinct_windows"] = pairs

    # configs[4]: window sweep, both widths, and the naive control
    if reach.cliff:
        wsizes = {"reach/4": reach.reach_bytes // 4, "reach/2": reach.reach_bytes // 2,
                  "reach": reach.reach_bytes, "2*reach": 2 * reach.reach_bytes, "N/2": N // 2}
    else:
        wsizes = {"N/8": N // 8, "N/4": N // 4, "N/2": N // 2, "N": N}
    cfg4 = {}
    for W in (1, 2):
        rows = {}
        for name, S_w in wsizes.items():
            win, cov = ses.windows(groups, S_w, W=W)
            rows[name] = {"window_gib": S_w / GiB, "coverage": cov,
                          "grouped": _stats(ses, N, reps, W=W, seed=23, reads_per_warp=reads,
                                            group_of_sm=groups.group_of_sm, windows=win),
                          "unrestricted_inside_one_window": _stats(
                              ses, min(S_w, N), reps, W=W, seed=23, reads_per_warp=reads)}
            cg, cw, ccov = ses.naive_control(S_w, 23, W=W)
            rows[name]["naive_per_sm_control"] = _stats(ses, N, reps, W=W, seed=23,
                                                        reads_per_warp=reads, group_of_sm=cg,
                                                        windows=cw)
            # the same control one level finer: a hashed chunk per warp, whatever SM runs it
            pw, _ = rr.rr_make_windows(N, W, S_w, 256, policy=1, seed=23)
            rows[name]["naive_per_warp_control"] = _stats(
                ses, N, reps, W=W, seed=23, reads_per_warp=reads, mode=rr.RR_MODE_LOGICAL,
                n_warps=ses.nsm * 32, windows=pw)
            # windows of the same size, evenly spaced and overlapping (policy 2)
            ow, ocov = rr.rr_make_windows(N, W, S_w, groups.n_groups, policy=2)
            covered, dmin, dmax = rr.rr_window_cover(ow, N // (128 * W))
            rows[name]["overlapping"] = dict(
                _stats(ses, N, reps, W=W, seed=23, reads_per_warp=reads,
                       group_of_sm=groups.group_of_sm, windows=ow),
                coverage=ocov, depth_min=dmin, depth_max=dmax)
        cfg4[f"{128 * W}B"] = {"unrestricted_full": _stats(ses, N, reps, W=W, seed=23,
                                                           reads_per_warp=reads),
                               "windows": rows}
    R["cfg4_grouped"] = cfg4

    # one window per SM, spread over the buffer: how far does an SM's own translation cache reach?
    MiB = 1 << 20
    per_sm = []
    ids = np.arange(ses.nsm, dtype=np.uint16)
    stride = (N // 128) // ses.nsm
    for S_sm in (8 * MiB, 32 * MiB, 128 * MiB, 256 * MiB, 512 * MiB, 768 * MiB, 1024 * MiB,
                 stride * 128):
        win = np.array([[k * stride, min(S_sm // 128, stride)] for k in range(ses.nsm)], np.uint32)
        per_sm.append({"window_mib": float(win[0, 1]) * 128 / MiB,
                       "gbps": _stats(ses, N, 3, seed=23, reads_per_warp=reads, group_of_sm=ids,
                                      windows=win)["median"]})
    R["per_sm_window_sweep"] = per_sm

    # moving windows: every SM owns 1/148 of the buffer and works through it in sub-windows
    owners_eq = ses.singleton_groups(groups)
    eq_win, _ = rr.rr_make_weighted_windows(N, 1, [1] * ses.nsm, ses.nsm * 32)
    slice_bytes = int(eq_win[:, 1].max()) * 128
    moving = []
    for parts in (2, 4, 8, 16):
        for B in (256, 1024, 4096):
            p = ses.params(N, seed=23, reads_per_warp=reads, group_of_sm=owners_eq.group_of_sm,
                           windows=eq_win, variant=rr.RR_VARIANT_PACKED, unroll=2,
                           index_mode=rr.RR_INDEX_PHASED, phase_reads=B,
                           phase_window_bytes=(slice_bytes + parts - 1) // parts)
            n = 30 if quick else 200
            for _ in range(10 if quick else 100):
                rr.rr_random_read(p, ses.out, ses.scratch, timed=False)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                rr.rr_random_read(p, ses.out, ses.scratch, timed=False)
            e1.record()
            torch.cuda.synchronize()
            rep = rr.rr_read_report(p, ses.scratch)
            moving.append({"sub_windows": parts, "sub_window_mib": slice_bytes / parts / MiB,
                           "phase_reads": B,
                           "sustained_gbps": rep.bytes * n / e0.elapsed_time(e1) * 1e-6})
    R["moving_windows"] = moving
    # no partition: every SM's window is the whole buffer, SM cycles staggered
    moving_all = []
    for sub_mib in (64, 128, 256, 512):
        for B in (1024, 4096):
            p = ses.params(N, seed=23, reads_per_warp=reads, variant=rr.RR_VARIANT_PACKED, unroll=2,
                           index_mode=rr.RR_INDEX_PHASED, phase_reads=B,
                           phase_window_bytes=sub_mib * MiB)
            n = 30 if quick else 200
            for _ in range(10 if quick else 100):
                rr.rr_random_read(p, ses.out, ses.scratch, timed=False)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                rr.rr_random_read(p, ses.out, ses.scratch, timed=False)
            e1.record()
            torch.cuda.synchronize()
            rep = rr.rr_read_report(p, ses.scratch)
            moving_all.append({"sub_window_mib": sub_mib, "phase_reads": B,
                               "sustained_gbps": rep.bytes * n / e0.elapsed_time(e1) * 1e-6})
    R["moving_windows_no_partition"] = moving_all

    # sorted execution: the same static per-SM slices, equal work, each warp's reads taken part by
    # part of its window (epochs of 4096 reads), in launches of the benchmark's step size: the
    # warps of an SM start every launch on the same part and stay together through it
    sorted_rows = []
    for parts in (4, 8, 16):
        for U in (1, 2):
            d = _stats(ses, N, 3, settle=20, min_ms=500.0, seed=23, reads_per_warp=1 << 19,
                       group_of_sm=owners_eq.group_of_sm, windows=eq_win,
                       variant=rr.RR_VARIANT_SORTED, unroll=U, sort_parts=parts,
                       sort_reads=4096 // parts)
            sorted_rows.append({"parts": parts, "unroll": U, **d})
    R["sorted_execution"] = sorted_rows

    # work in proportion to group capacity (pooled mode), balanced under sustained load
    balanced = {}
    n_warps = ses.nsm * 32
    max_window = reach.reach_bytes if reach.cliff else 0
    singles_map = ses.singleton_groups(groups)
    for W, variant, unroll, owners, name in (
            (1, rr.RR_VARIANT_PACKED, 2, singles_map, "128B packed, one window per SM"),
            (1, rr.RR_VARIANT_PACKED, 2, groups, "128B packed, one window per group"),
            (1, rr.RR_VARIANT_LDG, 8, groups, "128B 32-lane, one window per group"),
            (2, rr.RR_VARIANT_LDG, 8, groups, "256B 32-lane, one window per group")):
        win, ws, weights, hist = ses.balance(owners, W=W, n_warps=n_warps, reads_per_warp=reads,
                                             seed=23, max_window_bytes=max_window,
                                             launches_per_round=20 if quick else 150, rounds=8,
                                             variant=variant, unroll=unroll)
        p = ses.params(N, W=W, mode=rr.RR_MODE_POOLED, n_warps=n_warps, reads_per_warp=reads,
                       seed=23, group_of_sm=owners.group_of_sm, windows=win, warp_start=ws,
                       variant=variant, unroll=unroll)
        torch.cuda.synchronize()
        time.sleep(1.0)
        burst = rr.rr_random_read(p, ses.out, ses.scratch).gbps      # first launch after a pause
        n = 50 if quick else 500
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(20 if quick else 150):
            rr.rr_random_read(p, ses.out, ses.scratch, timed=False)
        e0.record()
        for _ in range(n):
            rr.rr_random_read(p, ses.out, ses.scratch, timed=False)
        e1.record()
        torch.cuda.synchronize()
        rep = rr.rr_read_report(p, ses.scratch)
        balanced[name] = {"burst_gbps": burst,
                          "sustained_gbps": rep.bytes * n / e0.elapsed_time(e1) * 1e-6,
                          "gbps_by_balancing_round": hist, "weights": weights.tolist(),
                          "window_gib_min_max": [float(win[:, 1].min()) * 128 * W / GiB,
                                                 float(win[:, 1].max()) * 128 * W / GiB]}
    R["balanced_pooled"] = balanced
    R["seconds"] = time.time() - t_start
    if alloc_study:
        # the study maps the same amount of memory four ways: give the big buffer back first
        del ses.buf
        torch.cuda.empty_cache()
        from . import alloc_study as study
        R["alloc_study"] = study.run()
    (out_dir / "report.json").write_text(json.dumps(R, indent=1))
    (out_dir / "report.md").write_text(markdown(R))
    return R


def _mmm(a):
    a = np.asarray(a, dtype=np.float64)
    return [float(a.min()), float(np.median(a)), float(a.max())]


def _offdiag(T):
    n = T.shape[0]
    return _mmm(T[~np.eye(n, dtype=bool)])


def markdown(R: dict) -> str:
    peak = R["device"]["theoretical_gbps"]
    L = [f"# Random line reads on {R['device']['name']} ({R['device']['nsm_prop']} SMs, "
         f"region {R['region_gib']:.1f} GiB, theoretical {peak:.0f} GB/s)", "",
         f"fill: {R['fill_gbps']:.0f} GB/s", "",
         "## Unrestricted size sweep (random 128-B lines, GB/s median [min-max])", "",
         "| GiB | 16 warps/SM | 32 warps/SM |", "|---|---|---|"]
    f = lambda s: f"{s['median']:.0f} [{s['min']:.0f}-{s['max']:.0f}]"  # noqa: E731
    for r in R["cfg1_size_sweep"]:
        L.append(f"| {r['gib']:.1f} | {f(r['wps16'])} | {f(r['wps32'])} |")
    rc = R["reach"]
    L += ["", f"plateau {rc['plateau_gbps']:.0f} GB/s, cliff {rc['cliff']}, reach "
              f"{rc['reach_gib']:.0f} GiB", "", "## Line widths at 32 GiB / sequential over everything",
          "", "| line | random 32 GiB | sequential whole buffer |", "|---|---|---|"]
    for k in ("128B", "256B", "512B"):
        L.append(f"| {k} | {f(R['cfg2_widths_32gib'][k])} | {f(R['stride_full'][k])} |")
    if "mixed_32gib" in R:
        L += ["", "one read in k sequential, the others random (128-B lines, 32 GiB): "
              + ", ".join(f"k={k}: {f(v)}" for k, v in R["mixed_32gib"].items())]
    p = R["cfg3_probe"]
    L += ["", "## Pair probe and clustering", "",
          f"inside the reach (16 GiB): {p['inside_reach_16gib']['n_groups']} group(s), pair GB/s "
          f"min/med/max {p['inside_reach_16gib']['pair_min_med_max']}",
          f"whole buffer: {p['whole_buffer']['n_groups']} groups, confidence "
          f"{p['whole_buffer']['confidence']:.1f}, sizes {p['whole_buffer']['sizes']}, "
          f"{p['whole_buffer']['seconds']:.1f} s",
          f"cluster-placement components (GPCs, plus TPCs never used for clusters): sizes "
          f"{R['gpc_map']['sizes']}; components touched by each group: "
          f"{R['gpc_map']['gpcs_of_group']}", "",
          "## Single groups (inside one sub-reach window)", "", "| group | SMs | GB/s |", "|---|---|---|"]
    for s in R["single_groups"]:
        L.append(f"| {s['group']} | {s['sms']} | {s['gbps']:.0f} |")
    ratios = [x["ratio_to_sum_of_singles"] for x in R["group_pairs_distinct_windows"]]
    if ratios:
        L += ["", f"group pairs in distinct windows / sum of the two singles: min {min(ratios):.3f} "
                  f"median {float(np.median(ratios)):.3f} max {max(ratios):.3f} "
                  f"({len(ratios)} pairs)"]
    L += ["", "## Grouped windows over the whole buffer", ""]
    for width, d in R["cfg4_grouped"].items():
        L += [f"### {width} lines: unrestricted over everything {f(d['unrestricted_full'])}", "",
              "| window | GiB | coverage | grouped | unrestricted inside one window | naive per-SM "
              "| naive per-warp | overlapping windows (coverage, depth min-max) |",
              "|---|---|---|---|---|---|---|---|"]
        for name, r in d["windows"].items():
            o = r.get("overlapping")
            ov = (f"{f(o)} ({o['coverage']:.2f}, {o['depth_min']}-{o['depth_max']})" if o else "")
            L.append(f"| {name} | {r['window_gib']:.1f} | {r['coverage']:.2f} | {f(r['grouped'])} | "
                     f"{f(r['unrestricted_inside_one_window'])} | {f(r['naive_per_sm_control'])} "
                     f"| {f(r['naive_per_warp_control']) if 'naive_per_warp_control' in r else ''} "
                     f"| {ov} |")
        L.append("")
    L += ["## One window per SM, windows spread over the buffer (equal work per SM)", "",
          "| window MiB | GB/s |", "|---|---|"]
    for r in R.get("per_sm_window_sweep", []):
        L.append(f"| {r['window_mib']:.0f} | {r['gbps']:.0f} |")
    L.append("")
    L += ["## Moving windows: one slice per SM, read one sub-window at a time (sustained GB/s)", "",
          "| sub-windows per slice | sub-window MiB | reads per phase | GB/s |", "|---|---|---|---|"]
    for r in R.get("moving_windows", []):
        L.append(f"| {r['sub_windows']} | {r['sub_window_mib']:.0f} | {r['phase_reads']} | "
                 f"{r['sustained_gbps']:.0f} |")
    L.append("")
    L += ["## Moving windows with no partition: every SM's window is the whole buffer", "",
          "| sub-window MiB | reads per phase | GB/s |", "|---|---|---|"]
    for r in R.get("moving_windows_no_partition", []):
        L.append(f"| {r['sub_window_mib']} | {r['phase_reads']} | {r['sustained_gbps']:.0f} |")
    L.append("")
    if "sorted_execution" in R:
        L += ["## Sorted execution: static per-SM slices, equal work, reads taken part by part "
              "(2^19 reads per warp and launch)", "",
              "| parts | reads per part and epoch | warp loads in flight | GB/s |",
              "|---|---|---|---|"]
        for r in R["sorted_execution"]:
            L.append(f"| {r['parts']} | {4096 // r['parts']} | {r['unroll']} | {f(r)} |")
        L.append("")
    L += ["## Work in proportion to group capacity (pooled mode, windows tile the buffer)", "",
          "| workload | first launch after 1 s idle, GB/s | sustained GB/s (500 launches) | windows GiB |", "|---|---|---|---|"]
    for name, b in R.get("balanced_pooled", {}).items():
        L.append(f"| {name} | {b['burst_gbps']:.0f} | {b['sustained_gbps']:.0f} | "
                 f"{b['window_gib_min_max'][0]:.1f}-{b['window_gib_min_max'][1]:.1f} |")
    L.append("")
    if "alloc_study" in R:
        from . import alloc_study as study
        L.append(study.markdown(R["alloc_study"]))
    L.append(f"total {R['seconds']:.0f} s")
    return "\n".join(L) + "\n"


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="report_out")
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--alloc-study", action="store_true",
                    help="also map the same memory through four allocation paths and locate the "
                         "cliff for each (Section 1.2: reach = translations x page size)")
    a = ap.parse_args(argv)
    R = run(Path(a.out), a.quick, a.alloc_study)
    print(markdown(R))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
