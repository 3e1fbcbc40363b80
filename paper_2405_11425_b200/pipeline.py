"""The paper's experiments strung together over the C-ABI entry points.

Nothing here computes on the data path: every read, probe and clustering step is a call into
librr (see binding.py).  This module only owns device buffers (torch), picks sizes, and keeps
the bookkeeping of a run:

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


class Session:
    """Device buffers of one GPU plus the calls of the path."""

    def __init__(self, region_bytes: int | None = None, frac_of_free: float = 0.95,
                 max_warps_per_sm: int = 32):
        import torch
        self.torch = torch
        self.info = rr.rr_device_info()
        self.nsm = int(self.info["nsm_prop"])
        if self.info["nsm_reg"] != self.nsm:
            raise RuntimeError(f"%nsmid = {self.info['nsm_reg']} but the device reports "
                               f"{self.nsm} SMs")
        # small buffers first, so the region can take what is left
        self.scratch = torch.zeros(rr.rr_scratch_bytes(), dtype=torch.uint8, device="cuda")
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

    # -- A1 ----------------------------------------------------------------------------------
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

    # -- A2-A5, A9 ---------------------------------------------------------------------------
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

    def checksums(self, n: int) -> np.ndarray:
        return self.out[:n].cpu().numpy().view(np.uint32)

    # -- A8 ----------------------------------------------------------------------------------
    def size_sweep(self, sizes_bytes, *, seed: int = 7, reads_per_warp: int = 256 * 16, **kw):
        pts = []
        for n in sizes_bytes:
            if n > self.region_bytes:
                continue
            g, _ = self.read(n, seed=seed, reads_per_warp=reads_per_warp, **kw)
            pts.append((int(n), g))
        return pts

    def measure_reach(self, sizes_gib=(1, 4, 16, 32, 48, 64, 96, 128, 160), *, seed: int = 7,
                      refine_gib: int = 2, **kw) -> Reach:
        """Size sweep, then bisection at `refine_gib` granularity between the last size at or
        above 0.9 plateau and the first below it."""
        sizes = [s * GiB for s in sizes_gib if s * GiB < self.region_bytes] + [self.region_bytes]
        pts = self.size_sweep(sizes, seed=seed, **kw)
        cliff, plateau, reach = rr.rr_reach([p[0] for p in pts], [p[1] for p in pts])
        if cliff:
            good = reach
            bad = min(p[0] for p in pts if p[0] > reach)
            step = refine_gib * GiB
            while bad - good > step:
                mid = ((good + bad) // 2 // step) * step
                if mid <= good or mid >= bad:
                    break
                g, _ = self.read(mid, seed=seed, reads_per_warp=256 * 16, **kw)
                pts.append((mid, g))
                if g >= 0.9 * plateau:
                    good = mid
                else:
                    bad = mid
            pts.sort()
            cliff, plateau, reach = rr.rr_reach([p[0] for p in pts], [p[1] for p in pts])
        return Reach(cliff, plateau, reach, pts)

    # -- A6, A7 ------------------------------------------------------------------------------
    def discover_groups(self, *, probe_region_bytes=None, total_reads: int = 1 << 18,
                        warps_per_sm: int = 32, seed: int = 5, repeats: int = 3,
                        solo_normalise: bool = True) -> Groups:
        import time
        region = probe_region_bytes or self.region_bytes
        t0 = time.time()
        T, overlap = rr.rr_probe_matrix(self.buf, region, total_reads, warps_per_sm, seed, repeats,
                                        self.nsm, self.probe_out, self.probe_scratch)
        dt = time.time() - t0
        flags = rr.RR_CLUSTER_SOLO_NORMALISE if solo_normalise else 0
        g, n_groups, conf, _ = rr.rr_cluster(T, self.scratch, flags)
        return Groups(g.astype(np.uint16), n_groups, conf, T, overlap, dt,
                      np.bincount(g, minlength=n_groups).tolist())

    # -- A9 ----------------------------------------------------------------------------------
    def windows(self, groups: Groups, window_bytes: int, W: int = 1, region_bytes=None):
        return rr.rr_make_windows(region_bytes or self.region_bytes, W, window_bytes,
                                  groups.n_groups)

    def naive_control(self, window_bytes: int, seed: int, W: int = 1, region_bytes=None):
        """The paper's per-SM control: every SM on its own picks a pseudo-random chunk."""
        win, cov = rr.rr_make_windows(region_bytes or self.region_bytes, W, window_bytes, self.nsm,
                                      policy=1, seed=seed)
        return np.arange(self.nsm, dtype=np.uint16), win, cov
