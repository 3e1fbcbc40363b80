"""Seeded synthetic inputs shared by the tests, the oracle-side checks and the benchmark.

This module holds none of the method's arithmetic (no hash, no index generation, no
checksum, no clustering): only workload shapes and random test matrices, so that the CPU
oracle and the CUDA library can be fed the same inputs without sharing any code.

The paper's workloads are synthetic uniform random line reads (Section 2.1), so these
shapes *are* its workloads, rescaled from an 80 GB card to B200 memory.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

GiB = 1 << 30


@dataclass(frozen=True)
class ReadCase:
    """One call of the random-read path."""
    name: str
    region_bytes: int
    W: int                 # 32-bit words per lane: line = 128*W bytes
    seed: int
    reads_per_warp: int
    mode: str              # "logical" | "per_sm"
    n_warps: int = 0       # logical mode
    warps_per_sm: int = 32  # per_sm mode


# configs[0]: 1 GiB, 2^16 logical warps x 16 reads of a 128-B line, seed 1, no grouping.
CFG0 = ReadCase("cfg0", 1 * GiB, 1, 1, 16, "logical", n_warps=1 << 16)
# configs[1]: unrestricted region sweep, seed 7, 2^8 reads per warp per iteration.
CFG1_SIZES_GIB = (1, 4, 16, 32, 48, 64, 96, 128, 160)
CFG1_SEED = 7
CFG1_READS_PER_ITER = 1 << 8
# configs[2]: width sweep at 32 GiB, seed 11.
CFG2_REGION = 32 * GiB
CFG2_SEED = 11
# configs[3]: pair probe over 16 GiB, 2^22 reads per pair; the seed is left open (5 here).
CFG3_REGION = 16 * GiB
CFG3_TOTAL_READS = 1 << 22
CFG3_SEED = 5
# configs[4]: grouped full-memory access, seed 23.
CFG4_SEED = 23


def usable_region_bytes(free_bytes: int, frac: float = 0.95) -> int:
    """~95 % of free device memory, rounded down to 512 B (one widest line)."""
    return (int(free_bytes * frac) // 512) * 512


def planted_matrix(group_sizes, drop: float, seed: int, tpc_drop: float = 0.10,
                   background: float = 0.02, sigma: float = 0.02, shuffle: bool = True,
                   base_gbps: float = 100.0, solo_spread: float = 0.0):
    """A synthetic SM x SM pair-throughput matrix with a planted partition.

    SMs come in TPC pairs (ids 2k, 2k+1).  SM i alone runs at solo_i = base/2 * (1 + solo_spread
    * U(-1,1)) (the diagonal).  Entry (i, j):
      (solo_i + solo_j) * (1 - drop [same group]) * (1 - tpc_drop [same TPC])
           * (1 - background [the two SMs lie in different halves of the chip])
           * (1 + sigma * N(0,1)),   drawn independently for (i,j) and (j,i).
    Group sizes must be even.  With ``shuffle`` the TPCs are permuted at random so groups are
    not contiguous in SM id.  Returns (T float32 [n,n], truth int32[n]) with truth labelled
    canonically (groups numbered by their smallest SM id).
    """
    rng = np.random.default_rng(seed)
    sizes = [int(s) for s in group_sizes]
    assert all(s % 2 == 0 and s > 0 for s in sizes)
    n = sum(sizes)
    grp = np.concatenate([np.full(s, g) for g, s in enumerate(sizes)])
    half = (np.arange(n) >= n // 2).astype(np.int64)  # two dies
    if shuffle:
        perm_tpc = rng.permutation(n // 2)
        order = np.empty(n, dtype=np.int64)
        order[0::2] = 2 * perm_tpc
        order[1::2] = 2 * perm_tpc + 1
        grp = grp[order]
        half = half[order]
    tpc = np.arange(n) // 2
    same_g = grp[:, None] == grp[None, :]
    same_t = tpc[:, None] == tpc[None, :]
    diff_h = half[:, None] != half[None, :]
    solo = 0.5 * base_gbps * (1.0 + solo_spread * rng.uniform(-1.0, 1.0, n))
    if solo_spread == 0.0:
        solo = np.full(n, 0.5 * base_gbps)
    T = solo[:, None] + solo[None, :]
    T *= np.where(same_g, 1.0 - drop, 1.0)
    T *= np.where(same_t, 1.0 - tpc_drop, 1.0)
    T *= np.where(diff_h, 1.0 - background, 1.0)
    T *= 1.0 + sigma * rng.standard_normal((n, n))
    T[np.arange(n), np.arange(n)] = solo * (1.0 + 0.25 * sigma * rng.standard_normal(n))
    # canonical truth labels
    truth = np.empty(n, dtype=np.int32)
    seen = {}
    for i in range(n):
        g = int(grp[i])
        if g not in seen:
            seen[g] = len(seen)
        truth[i] = seen[g]
    return T.astype(np.float32), truth


def random_group_sizes(seed: int, lo_groups: int = 8, hi_groups: int = 16, lo: int = 8,
                       hi: int = 20, n_max: int = 256):
    """8-16 groups of 8-20 SMs (even sizes), as the contention-probe config describes."""
    rng = np.random.default_rng(seed)
    while True:
        g = int(rng.integers(lo_groups, hi_groups + 1))
        sizes = [int(2 * rng.integers(lo // 2, hi // 2 + 1)) for _ in range(g)]
        if sum(sizes) <= n_max:
            return sizes


def synthetic_group_map(nsm: int, n_groups: int, seed: int, inactive_frac: float = 0.0):
    """A random SM -> group map (uint16) that uses every group at least once."""
    rng = np.random.default_rng(seed)
    g = rng.integers(0, n_groups, size=nsm).astype(np.uint16)
    g[rng.permutation(nsm)[:n_groups]] = np.arange(n_groups, dtype=np.uint16)
    if inactive_frac > 0:
        k = int(nsm * inactive_frac)
        g[rng.permutation(nsm)[:k]] = 0xFFFF
    return g
