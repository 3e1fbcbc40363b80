"""The paper's experiments strung together over the C-ABI entry points.

Nothing here computes on the data path or decides a plan: every read, probe and clustering step,
and every rule that turns measurements into windows, weights or sizes, is a call into librr (see
binding.py).  This module only owns device buffers (torch), loops over sizes, and keeps the
bookkeeping of a run:

  Session.fill()            Section 2.1 needs a region with known contents       (rr_fill)
  Session.read()            one random-read launch, grouped or not               (rr_random_read)
  Session.size_sweep()      Section 2.1 / Fig. 1: GB/s versus region size
  Session.measure_reach()   plateau, cliff, reach; bisection between sweep points (rr_reach)
  Session.discover_groups() Section 2.2 / Fig. 2-3: pair probe + clustering      (rr_probe_matrix,
                                                                                  rr_cluster)
  Session.windows()         Section 2.4: one chunk per SM group                  (rr_make_windows)
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import binding as rr

GiB = 1 << 30


@dataclass
class Groups:
    group_of_sm: np.ndarray        # uint16[nsm]
    n_groups: int
    confidence: float
    matrix: np.ndarray | None = None
    overlap_min: float = 1.0
    probe_seconds: float = 0.0
    sizes: list = field(default_factory=list)
    probe_stats: dict = field(default_factory=dict)


@dataclass
class Reach:
    cliff: bool
    plateau_gbps: float
    reach_bytes: int
    sweep: list                    # [(size_bytes, gbps)], increasing size


def aggregate_throughput(local_bytes: float, local_seconds: float, group=None) -> tuple:
    """Whole-job (bytes, seconds) of independent replicas: bytes add up, the slowest rank sets
    the time.  `group` is a torch.distributed process group (None = not distributed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(local_bytes), float(local_seconds)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    b = torch.tensor([float(local_bytes)], dtype=torch.float64, device=dev)
    s = torch.tensor([float(local_seconds)], dtype=torch.float64, device=dev)
    dist.all_reduce(b, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(s, op=dist.ReduceOp.MAX, group=group)
    return float(b.item()), float(s.item())


def save_calibration(path, uuid: str, groups: "Groups", reach: "Reach | None" = None,
                     weights=None, extra: dict | None = None) -> None:
    """Writes what was measured on one card (SM groups, reach, capacity weights, and whatever
    else the caller adds under `extra`) as JSON, keyed by the GPU's UUID: the layout is a
    property of the card (Section 1.1), so it can be reused."""
    import json
    doc = {"uuid": uuid, "n_groups": int(groups.n_groups), "confidence": float(groups.confidence),
           "group_of_sm": [int(g) for g in groups.group_of_sm],
           "probe_stats": groups.probe_stats, "probe_seconds": float(groups.probe_seconds),
           "reach": None if reach is None else {"cliff": bool(reach.cliff),
                                                "plateau_gbps": float(reach.plateau_gbps),
                                                "reach_bytes": int(reach.reach_bytes),
                                                "sweep": [[int(s), float(g)] for s, g in reach.sweep]},
           "weights": None if weights is None else [int(w) for w in weights],
           "extra": extra or {}}
    with open(path, "w") as f:
        json.dump(doc, f)


def load_calibration(path, uuid: str, nsm: int, with_extra: bool = False):
    """Reads a calibration written by save_calibration; refuses one taken on another card or with
    another SM count.  Returns (Groups, Reach or None, weights or None[, extra])."""
    import json
    with open(path) as f:
        doc = json.load(f)
    if doc.get("uuid") != uuid:
        raise ValueError(f"calibration belongs to GPU {doc.get('uuid')}, this is {uuid}")
    g = np.asarray(doc["group_of_sm"], dtype=np.uint16)
    if g.shape != (nsm,) or int(g.max()) + 1 != doc["n_groups"]:
        raise ValueError("calibration does not describe this SM count")
    stats = doc.get("probe_stats") or {}
    groups = Groups(g, int(doc["n_groups"]), float(doc["confidence"]), None,
                    float(stats.get("overlap_min", 1.0)), float(doc.get("probe_seconds", 0.0)),
                    np.bincount(g, minlength=doc["n_groups"]).tolist(), stats)
    r = doc.get("reach")
    reach = None if r is None else Reach(bool(r["cliff"]), float(r["plateau_gbps"]),
                                         int(r["reach_bytes"]),
                                         [(int(s), float(x)) for s, x in r.get("sweep", [])])
    w = doc.get("weights")
    out = (groups, reach, None if w is None else np.asarray(w, dtype=np.uint32))
    return out + (doc.get("extra") or {},) if with_extra else out


class Session:
    """Device buffers of one GPU plus the calls of the path."""

    def __init__(self, region_bytes: int | None = None, frac_of_free: float = 0.95,
                 max_warps_per_sm: int = 32):
        import torch
        self.torch = torch
        # small buffers first, so the region can take what is left
        self.scratch = torch.zeros(rr.rr_scratch_bytes(), dtype=torch.uint8, device="cuda")
        self.info = rr.rr_device_info(self.scratch)
        self.nsm = int(self.info["nsm_prop"])
        if self.info["nsm_reg"] != self.nsm:
            raise RuntimeError(f"%nsmid = {self.info['nsm_reg']} but the device reports "
                               f"{self.nsm} SMs")
        self.probe_scratch = torch.zeros(rr.rr_probe_matrix_scratch_bytes(self.nsm),
                                         dtype=torch.uint8, device="cuda")
        self.out = torch.zeros((self.nsm * max_warps_per_sm, 2), dtype=torch.int32, device="cuda")
        self.probe_out = torch.zeros((2 * 32, 2), dtype=torch.int32, device="cuda")
        if region_bytes is None:
            free, _ = torch.cuda.mem_get_info()
            region_bytes = (int(free * frac_of_free) // 512) * 512
        self.region_bytes = int(region_bytes)
        self.buf = torch.empty(self.region_bytes, dtype=torch.uint8, device="cuda")
        if self.buf.data_ptr() % 512:
            raise RuntimeError("allocator returned a buffer that is not 512-byte aligned")
        self.filled = False

    # -- fill --------------------------------------------------------------------------------
    def fill(self) -> float:
        """Fills the whole buffer; returns the write rate in GB/s (CUDA events)."""
        t = self.torch
        e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        e0.record()
        rr.rr_fill(self.buf, self.region_bytes // 4)
        e1.record()
        t.cuda.synchronize()
        self.filled = True
        return self.region_bytes / (e0.elapsed_time(e1) * 1e-3) * 1e-9

    # -- reads -------------------------------------------------------------------------------
    def params(self, region_bytes=None, **kw) -> rr.ReadParams:
        kw.setdefault("warps_per_sm", 32)
        kw.setdefault("nsm", self.nsm)
        return rr.ReadParams(self.buf, region_bytes or self.region_bytes, **kw)

    def read(self, region_bytes=None, *, reps: int = 3, warm: int = 1, **kw):
        """Median GB/s of `reps` timed launches (after `warm` untimed ones) and the last result."""
        p = self.params(region_bytes, **kw)
        for _ in range(warm):
            rr.rr_random_read(p, self.out, self.scratch)
        res = [rr.rr_random_read(p, self.out, self.scratch) for _ in range(reps)]
        rates = sorted(r.gbps for r in res)
        return rates[(len(rates) - 1) // 2], res[-1]

    def sustained(self, p: rr.ReadParams, out=None, *, settle: int = 150, min_ms: float = 50.0,
                  reps: int = 5, sampler=None) -> dict:
        """The one measurement protocol every arm of a comparison goes through: `settle` untimed
        launches of the very same call (clocks and caches reach their sustained state), then
        `reps` timed regions, each a run of back-to-back asynchronous launches long enough to
        hold at least `min_ms` of kernel time, bracketed by CUDA events on the launching stream.
        Returns median / min / max GB/s over the regions, the launches per region and, with a
        clocks.ClockSampler, the SM clock and power seen while the regions ran."""
        import time
        t = self.torch
        out = self.out if out is None else out
        e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)

        def region(n):
            e0.record()
            for _ in range(n):
                rr.rr_random_read(p, out, self.scratch, timed=False)
            e1.record()
            t.cuda.synchronize()
            return e0.elapsed_time(e1)

        region(max(1, settle))
        probe_n = 4
        per_launch_ms = max(region(probe_n) / probe_n, 1e-3)
        n = max(1, int(np.ceil(min_ms / per_launch_ms)))
        rep = rr.rr_read_report(p, self.scratch)          # also checks coverage and status
        t_begin = time.time()
        ms = [region(n) for _ in range(max(1, reps))]
        t_end = time.time()
        rates = sorted(rep.bytes * n / m * 1e-6 for m in ms)
        res = {"gbps": rates[(len(rates) - 1) // 2], "gbps_min": rates[0], "gbps_max": rates[-1],
               "launches_per_region": n, "regions": len(ms), "ms_per_region": float(np.median(ms)),
               "bytes_per_launch": int(rep.bytes), "settle_launches": settle}
        if sampler is not None:
            c = sampler.window(t_begin, t_end)
            res["sm_mhz"], res["power_w"], res["clock_reasons"] = (c["sm_mhz"], c["power_w"],
                                                                   c["reasons"])
            if c["sm_mhz"]:
                res["gbps_per_sm_ghz"] = res["gbps"] / (c["sm_mhz"] * 1e-3)
        return res

    def checksums(self, n: int) -> np.ndarray:
        return self.out[:n].cpu().numpy().view(np.uint32)

    # -- reach-------------------------------------------------------------------------------
    def size_sweep(self, sizes_bytes, *, seed: int = 7, reads_per_warp: int = 256 * 16, **kw):
        pts = []
        for n in sizes_bytes:
            if n > self.region_bytes:
                continue
            g, _ = self.read(n, seed=seed, reads_per_warp=reads_per_warp, **kw)
            pts.append((int(n), g))
        return pts

    def measure_reach(self, sizes_gib=(1, 4, 16, 32, 48, 64, 96, 128, 160), *, seed: int = 7,
                      refine_gib: int = 2, sustained: bool = True, **kw) -> Reach:
        """Size sweep, then refinement at `refine_gib` granularity: rr_reach_next names the next
        size to measure until it has none left.  With `sustained` every point is measured by the
        settle-then-time protocol (>= 50 ms of kernel time, 5 regions), else by short bursts."""
        sizes = [s * GiB for s in sizes_gib if s * GiB < self.region_bytes] + [self.region_bytes]

        def rate(n):
            if not sustained:
                return self.read(n, seed=seed, reads_per_warp=256 * 16, **kw)[0]
            p = self.params(n, seed=seed, reads_per_warp=256 * 16, **kw)
            return self.sustained(p, settle=20, min_ms=50.0, reps=5)["gbps"]

        pts = {int(n): rate(n) for n in sizes}
        for _ in range(64):
            xs = sorted(pts)
            nxt = rr.rr_reach_next(xs, [pts[x] for x in xs], refine_gib * GiB)
            if not nxt or nxt in pts:
                break
            pts[nxt] = rate(nxt)
        xs = sorted(pts)
        cliff, plateau, reach = rr.rr_reach(xs, [pts[x] for x in xs])
        return Reach(cliff, plateau, reach, [(x, pts[x]) for x in xs])

    def measure_sm_reach(self, sizes_mib=(32, 64, 128, 256, 384, 512, 768, 1024), *,
                         keep: float = 0.97, seed: int = 23, reads_per_warp: int = 256 * 16):
        """How large a window can one SM read at random before its own translation cache stops
        covering it?  Every SM gets a window of the given size (windows spread over the buffer,
        equal work); rr_sm_reach turns the rates into the answer.
        Returns (reach_bytes, [(size_bytes, GB/s)])."""
        ids = np.arange(self.nsm, dtype=np.uint16)
        stride = (self.region_bytes // 128) // self.nsm
        pts = []
        for mib in sizes_mib:
            n = min((mib << 20) // 128, stride)
            if pts and int(n) * 128 <= pts[-1][0]:
                continue
            win = np.array([[k * stride, n] for k in range(self.nsm)], np.uint32)
            g, _ = self.read(self.region_bytes, seed=seed, reads_per_warp=reads_per_warp,
                             group_of_sm=ids, windows=win)
            pts.append((int(n) * 128, g))
        reach = rr.rr_sm_reach([p[0] for p in pts], [p[1] for p in pts], keep)
        return reach, pts

    # -- groups -----------------------------------------------------------------------------
    def discover_groups(self, *, probe_region_bytes=None, total_reads: int = 1 << 18,
                        warps_per_sm: int = 32, seed: int = 5, repeats: int = 3,
                        solo_normalise: bool = True, checkpoint=None,
                        rows_per_block: int = 16) -> Groups:
        """Pair-probe matrix, then clustering.  With `checkpoint` (a path) the matrix is probed in
        blocks of rows and saved after each block; a later call with the same card and probe
        settings picks up after the last finished block instead of starting over."""
        import time
        region = probe_region_bytes or self.region_bytes
        t0 = time.time()
        if checkpoint is None:
            T, stats = rr.rr_probe_matrix(self.buf, region, total_reads, warps_per_sm, seed,
                                          repeats, self.nsm, self.probe_out, self.probe_scratch)
        else:
            T, stats = self._probe_with_checkpoint(checkpoint, region, total_reads, warps_per_sm,
                                                   seed, repeats, rows_per_block)
        dt = time.time() - t0
        flags = rr.RR_CLUSTER_SOLO_NORMALISE if solo_normalise else 0
        g, n_groups, conf, _ = rr.rr_cluster(T, self.scratch, flags)
        return Groups(g.astype(np.uint16), n_groups, conf, T, stats["overlap_min"], dt,
                      np.bincount(g, minlength=n_groups).tolist(), stats)

    def _probe_with_checkpoint(self, path, region, total_reads, wps, seed, repeats, rows_per_block):
        import json
        from pathlib import Path
        path = Path(path)
        meta = {"uuid": self.info["uuid"], "nsm": self.nsm, "region_bytes": int(region),
                "total_reads": int(total_reads), "warps_per_sm": int(wps), "seed": int(seed),
                "repeats": int(repeats)}
        T = np.zeros((self.nsm, self.nsm), dtype=np.float32)
        done = 0
        stats = {"overlap_min": 1.0, "pairs_below_goal": 0, "reruns": 0, "relaunched": 0}
        if path.exists():
            with np.load(path, allow_pickle=False) as z:
                if json.loads(str(z["meta"])) == meta:          # same card, same probe settings
                    T = np.ascontiguousarray(z["T"], dtype=np.float32)
                    done = int(z["rows_done"])
                    stats = json.loads(str(z["stats"]))
        while done < self.nsm:
            end = min(self.nsm, done + max(1, rows_per_block))
            st = rr.rr_probe_rows(self.buf, region, total_reads, wps, seed, repeats, done, end, T,
                                  self.probe_out, self.probe_scratch)
            stats = {"overlap_min": min(stats["overlap_min"], st["overlap_min"]),
                     **{k: stats[k] + st[k] for k in ("pairs_below_goal", "reruns", "relaunched")}}
            done = end
            tmp = path.with_suffix(".tmp.npz")
            np.savez(tmp, T=T, rows_done=done, meta=json.dumps(meta), stats=json.dumps(stats))
            tmp.replace(path)
        return T, stats

    # -- windows-------------------------------------------------------------------------------
    def windows(self, groups: Groups, window_bytes: int, W: int = 1, region_bytes=None):
        return rr.rr_make_windows(region_bytes or self.region_bytes, W, window_bytes,
                                  groups.n_groups)

    # -- Section 2.3: every group on its own; work in proportion to capacity ---------------------
    def measure_group_rates(self, groups: Groups, window_bytes: int, *, W: int = 1,
                            reads_per_warp: int = 256 * 8, seed: int = 23) -> list:
        """GB/s of each group running alone inside one window of `window_bytes` (below the reach)."""
        n_lines = max(1, min(window_bytes, self.region_bytes) // (128 * W))
        rates = []
        for g in range(groups.n_groups):
            only = np.where(groups.group_of_sm == g, 0, rr.RR_SM_INACTIVE).astype(np.uint16)
            rate, _ = self.read(self.region_bytes, W=W, seed=seed, reads_per_warp=reads_per_warp,
                                group_of_sm=only, windows=[[0, n_lines]], reps=3, warm=1)
            rates.append(rate)
        return rates

    def balance(self, groups: Groups, *, W: int = 1, n_warps: int | None = None,
                reads_per_warp: int = 256 * 64, seed: int = 23, max_window_bytes: int = 0,
                rounds: int = 6, spread_goal: float = 0.02, start_rates=None,
                launches_per_round: int = 1, **kw):
        """Closed loop: run the pooled workload, see from the per-SM
        timers when each group finished, move work (and window size) towards the groups that
        finished early, repeat.  Needed because a group's capacity with every other group
        running differs from its capacity alone.  Stops after `rounds` rounds or once the
        groups' finish times lie within `spread_goal` of each other.  Each round queues
        `launches_per_round` launches back to back and reads the timers of the last one: under
        sustained load the clocks settle lower than in a single burst, and the groups whose
        limit follows the clock lose capacity while the others do not.  Returns (windows,
        warp_start, weights, [GB/s of each round, from the device timers])."""
        n_warps = n_warps or self.nsm * 32
        G = groups.n_groups
        if start_rates is None:
            weights = np.full(G, 1000, dtype=np.uint32)
        else:
            weights = np.maximum(1, np.rint(np.asarray(start_rates, np.float64) * 1000)).astype(
                np.uint32)
        history = []
        for _ in range(rounds):
            win, ws = rr.rr_make_weighted_windows(self.region_bytes, W, weights, n_warps,
                                                  max_window_bytes)
            p = self.params(None, mode=rr.RR_MODE_POOLED, n_warps=n_warps, W=W,
                            reads_per_warp=reads_per_warp, seed=seed,
                            group_of_sm=groups.group_of_sm, windows=win, warp_start=ws, **kw)
            for _ in range(max(1, launches_per_round)):
                rr.rr_random_read(p, self.out, self.scratch, timed=False)
            t0, t1 = rr.rr_read_block_times(self.scratch, self.nsm)
            finish, span_ns = rr.rr_group_finish(t0, t1, groups.group_of_sm, G)
            history.append(n_warps * reads_per_warp * 128 * W / max(span_ns, 1))
            work = np.diff(ws.astype(np.int64)).astype(np.uint32)
            if rr.rr_finish_spread_ppm(finish) <= int(spread_goal * 1e6):
                break
            weights = rr.rr_rebalance_weights(work, finish)
        win, ws = rr.rr_make_weighted_windows(self.region_bytes, W, weights, n_warps,
                                              max_window_bytes)
        return win, ws, weights, history

    def read_pooled(self, groups: Groups, windows, warp_start, *, region_bytes=None,
                    reps: int = 3, warm: int = 1, out=None, **kw):
        """Median GB/s of pooled-mode launches; `out` must hold warp_start[-1] checksum pairs."""
        n_warps = int(warp_start[-1])
        if out is None:
            out = self.out
        if out.shape[0] < n_warps:
            raise ValueError("output buffer smaller than the number of logical warps")
        p = self.params(region_bytes, mode=rr.RR_MODE_POOLED, n_warps=n_warps,
                        group_of_sm=groups.group_of_sm, windows=windows, warp_start=warp_start,
                        **kw)
        for _ in range(warm):
            rr.rr_random_read(p, out, self.scratch)
        res = [rr.rr_random_read(p, out, self.scratch) for _ in range(reps)]
        rates = sorted(r.gbps for r in res)
        return rates[(len(rates) - 1) // 2], res[-1]

    def singleton_groups(self, groups: Groups) -> Groups:
        """One "group" per SM, numbered so that the SMs of one resource group are neighbours:
        their windows then lie side by side inside what would be the resource group's window.
        A window per SM is still a window per group in the paper's sense (every group's
        footprint stays below its reach), and it lets each SM's own small translation cache
        catch a share of the lookups before they reach the group's shared path."""
        ids, n = rr.rr_owner_map(groups.group_of_sm)
        return Groups(ids, n, groups.confidence, None, groups.overlap_min, 0.0, [1] * n)

    def naive_control(self, window_bytes: int, seed: int, W: int = 1, region_bytes=None):
        """The paper's per-SM control: every SM on its own picks a pseudo-random chunk."""
        win, cov = rr.rr_make_windows(region_bytes or self.region_bytes, W, window_bytes, self.nsm,
                                      policy=1, seed=seed)
        return np.arange(self.nsm, dtype=np.uint16), win, cov
