"""CPU oracle for the random-line-read path -- TEST INFRASTRUCTURE.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / reference legs of
``bench.py`` may import this package.  It shares no code with the CUDA library and the
product never routes through it.

The arithmetic lives in ``rr_oracle.c`` (plain C, one word at a time); this module only
compiles that file with gcc and marshals numpy arrays into it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "rr_oracle.c"
_LIB = _HERE / "librr_oracle.so"

INDEX_RANDOM = 0
INDEX_STRIDE = 1
SM_INACTIVE = 0xFFFF


def build(force: bool = False) -> Path:
    """Compile rr_oracle.c into a shared object next to it (gcc, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
             str(_SRC), "-o", str(tmp), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        u64, u32, i32 = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int32
        p = ctypes.c_void_p
        lib.orc_sm64.restype = u64
        lib.orc_sm64.argtypes = [u64]
        lib.orc_word.restype = u32
        lib.orc_word.argtypes = [u64]
        lib.orc_fill.restype = None
        lib.orc_fill.argtypes = [p, u64, u64]
        lib.orc_warp_key.restype = u64
        lib.orc_warp_key.argtypes = [u64, u64]
        lib.orc_draw.restype = u64
        lib.orc_draw.argtypes = [u64, u64, u64]
        lib.orc_line.restype = u64
        lib.orc_line.argtypes = [u32, u64, u64, u64, u64, u64, u64]
        lib.orc_warp_checksum.restype = None
        lib.orc_warp_checksum.argtypes = [u32, u64, u64, u64, u64, u64, u32, u64, u64, p, p]
        lib.orc_line_phased.restype = u64
        lib.orc_line_phased.argtypes = [u64, u64, u64, u64, u64, u64, u64, u64]
        lib.orc_warp_checksum_phased.restype = None
        lib.orc_warp_checksum_phased.argtypes = [u64, u64, u64, u64, u32, u64, u64, u64, u64, u64, p, p]
        lib.orc_read_per_sm_phased.restype = i32
        lib.orc_read_per_sm_phased.argtypes = [u64, u32, u32, u32, u64, u64, u64, p, p, p, u32, u64,
                                               u64, p]
        lib.orc_line_mixed.restype = u64
        lib.orc_line_mixed.argtypes = [u64, u64, u64, u64, u64, u64, u64]
        lib.orc_warp_checksum_mixed.restype = None
        lib.orc_warp_checksum_mixed.argtypes = [u64, u64, u64, u64, u64, u32, u64, u64, u64, p, p]
        lib.orc_read_per_sm_mixed.restype = i32
        lib.orc_read_per_sm_mixed.argtypes = [u64, u32, u32, u32, u64, u64, u64, p, p, p, u32, u64, p]
        lib.orc_read_logical_windows.restype = i32
        lib.orc_read_logical_windows.argtypes = [u64, u32, u64, u64, u64, u64, p, p, u32, p]
        lib.orc_read_logical.restype = i32
        lib.orc_read_logical.argtypes = [u64, u32, u32, u64, u64, u64, u64, p]
        lib.orc_read_logical_materialised.restype = i32
        lib.orc_read_logical_materialised.argtypes = [p, u64, u32, u64, u64, u64, u64, p]
        lib.orc_read_per_sm.restype = i32
        lib.orc_read_per_sm.argtypes = [u64, u32, u32, u32, u32, u64, u64, u64, p, p, p, u32, p]
        lib.orc_make_windows.restype = i32
        lib.orc_make_windows.argtypes = [u64, u32, u64, u32, u32, u64, p, p, p]
        lib.orc_make_weighted_windows.restype = i32
        lib.orc_make_weighted_windows.argtypes = [u64, u32, u32, p, u64, u64, p, p, p]
        lib.orc_read_pooled.restype = i32
        lib.orc_read_pooled.argtypes = [u64, u32, u32, p, p, p, u64, u64, u64, p]
        lib.orc_cluster.restype = i32
        lib.orc_cluster.argtypes = [p, u32, u32, p, p, p, p]
        lib.orc_reach.restype = i32
        lib.orc_reach.argtypes = [p, p, u32, p, p]
        lib.orc_reach_next.restype = i32
        lib.orc_reach_next.argtypes = [p, p, u32, u64, p]
        lib.orc_sm_reach.restype = i32
        lib.orc_sm_reach.argtypes = [p, p, u32, ctypes.c_double, p]
        lib.orc_owner_map.restype = i32
        lib.orc_owner_map.argtypes = [p, u32, p, p]
        lib.orc_phase_window.restype = i32
        lib.orc_phase_window.argtypes = [u64, u64, u32, p, p]
        lib.orc_rebalance_weights.restype = i32
        lib.orc_rebalance_weights.argtypes = [p, p, u32, u32, p]
        lib.orc_finish_spread_ppm.restype = i32
        lib.orc_finish_spread_ppm.argtypes = [p, u32, p]
        lib.orc_group_finish.restype = i32
        lib.orc_group_finish.argtypes = [p, p, p, u32, u32, p, p]
        lib.orc_window_cover.restype = i32
        lib.orc_window_cover.argtypes = [p, p, u32, u64, p, p, p]
        lib.orc_probe_rate.restype = i32
        lib.orc_probe_rate.argtypes = [p, p, p, p, u32, u64, p, p, p]
        _lib = lib
    return _lib


class OracleError(ValueError):
    def __init__(self, code: int):
        super().__init__(f"oracle rejected its arguments (code {code})")
        self.code = code


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def sm64(x: int) -> int:
    return int(_load().orc_sm64(x & 0xFFFFFFFFFFFFFFFF))


def word(i: int) -> int:
    return int(_load().orc_word(i))


def fill(first_word: int, n_words: int) -> np.ndarray:
    out = np.empty(n_words, dtype=np.uint32)
    _load().orc_fill(_ptr(out), first_word, n_words)
    return out


def warp_key(seed: int, v: int) -> int:
    return int(_load().orc_warp_key(seed, v))


def draw(seed: int, v: int, i: int) -> int:
    return int(_load().orc_draw(seed, v, i))


def line(seed: int, v: int, i: int, base: int, n: int, index_mode: int = INDEX_RANDOM,
         n_warps_total: int = 1) -> int:
    return int(_load().orc_line(index_mode, seed, v, n_warps_total, i, base, n))


def warp_checksum(seed: int, v: int, first_read: int, reads: int, W: int, base: int, n: int,
                  index_mode: int = INDEX_RANDOM, n_warps_total: int = 1):
    x = ctypes.c_uint32()
    s = ctypes.c_uint32()
    _load().orc_warp_checksum(index_mode, seed, v, n_warps_total, first_read, reads, W, base, n,
                              ctypes.byref(x), ctypes.byref(s))
    return int(x.value), int(s.value)


def read_logical(region_bytes: int, W: int, n_warps: int, reads: int, seed: int,
                 first_read: int = 0, index_mode: int = INDEX_RANDOM) -> np.ndarray:
    """Checksums {X, S} of logical warps 0..n_warps-1 over the whole region: (n_warps, 2) uint32."""
    out = np.zeros((n_warps, 2), dtype=np.uint32)
    rc = _load().orc_read_logical(region_bytes, W, index_mode, n_warps, first_read, reads, seed,
                                  _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def read_logical_windows(region_bytes: int, W: int, n_warps: int, reads: int, seed: int, windows,
                         first_read: int = 0) -> np.ndarray:
    """Logical warps 0..n_warps-1, warp v inside window v mod len(windows)."""
    w = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
    wb = np.ascontiguousarray(w[:, 0])
    wn = np.ascontiguousarray(w[:, 1])
    out = np.zeros((n_warps, 2), dtype=np.uint32)
    rc = _load().orc_read_logical_windows(region_bytes, W, n_warps, first_read, reads, seed,
                                          _ptr(wb), _ptr(wn), w.shape[0], _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def read_logical_materialised(buf: np.ndarray, W: int, n_warps: int, reads: int, seed: int,
                              first_read: int = 0) -> np.ndarray:
    """Logical-mode checksums read from a real host buffer (uint32 words, see fill())."""
    buf = np.ascontiguousarray(buf, dtype=np.uint32)
    out = np.zeros((n_warps, 2), dtype=np.uint32)
    rc = _load().orc_read_logical_materialised(_ptr(buf), buf.size * 4, W, n_warps, first_read,
                                               reads, seed, _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def read_per_sm(region_bytes: int, W: int, nsm: int, wps: int, reads: int, seed: int,
                group_of_sm=None, windows=None, first_read: int = 0,
                index_mode: int = INDEX_RANDOM) -> np.ndarray:
    """Checksums of warps v = smid*wps + warp: (nsm*wps, 2) uint32.

    ``windows`` is an (n_groups, 2) array of {base_line, n_lines}."""
    out = np.zeros((nsm * wps, 2), dtype=np.uint32)
    g = wb = wn = None
    ng = 0
    if group_of_sm is not None:
        g = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
        if g.shape != (nsm,):
            raise OracleError(-1)
        w = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
        wb = np.ascontiguousarray(w[:, 0])
        wn = np.ascontiguousarray(w[:, 1])
        ng = w.shape[0]
    rc = _load().orc_read_per_sm(region_bytes, W, index_mode, nsm, wps, first_read, reads, seed,
                                 _ptr(g), _ptr(wb), _ptr(wn), ng, _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def line_phased(seed: int, v: int, i: int, base: int, n: int, phase_reads: int,
                sub_lines: int, stagger: int = 0) -> int:
    return int(_load().orc_line_phased(seed, v, i, base, n, phase_reads, sub_lines, stagger))


def stagger_of_sm(sm: int, nsm: int, n: int, sub_lines: int) -> int:
    """Shift of SM `sm`'s phase cycle in per-SM mode: floor(sm * Q / nsm), Q = ceil(n/sub_lines)."""
    return sm * (-(-n // sub_lines)) // nsm


def warp_checksum_phased(seed: int, v: int, first_read: int, reads: int, W: int, base: int, n: int,
                         phase_reads: int, sub_lines: int, stagger: int = 0):
    x = ctypes.c_uint32()
    s = ctypes.c_uint32()
    _load().orc_warp_checksum_phased(seed, v, first_read, reads, W, base, n, phase_reads, sub_lines,
                                     stagger, ctypes.byref(x), ctypes.byref(s))
    return int(x.value), int(s.value)


def read_per_sm_phased(region_bytes: int, W: int, nsm: int, wps: int, reads: int, seed: int,
                       phase_reads: int, phase_window_bytes: int, group_of_sm=None, windows=None,
                       first_read: int = 0) -> np.ndarray:
    """Per-SM mode with windows that move: phase p of a warp's stream reads inside sub-window
    p mod Q of the warp's window."""
    out = np.zeros((nsm * wps, 2), dtype=np.uint32)
    g = wb = wn = None
    ng = 0
    if group_of_sm is not None:
        g = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
        w = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
        wb = np.ascontiguousarray(w[:, 0])
        wn = np.ascontiguousarray(w[:, 1])
        ng = w.shape[0]
    rc = _load().orc_read_per_sm_phased(region_bytes, W, nsm, wps, first_read, reads, seed, _ptr(g),
                                        _ptr(wb), _ptr(wn), ng, phase_reads, phase_window_bytes,
                                        _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def line_mixed(seed: int, v: int, i: int, base: int, n: int, mix_period: int,
               n_warps_total: int = 1) -> int:
    return int(_load().orc_line_mixed(seed, v, n_warps_total, i, base, n, mix_period))


def warp_checksum_mixed(seed: int, v: int, first_read: int, reads: int, W: int, base: int, n: int,
                        mix_period: int, n_warps_total: int = 1):
    x = ctypes.c_uint32()
    s = ctypes.c_uint32()
    _load().orc_warp_checksum_mixed(seed, v, n_warps_total, first_read, reads, W, base, n,
                                    mix_period, ctypes.byref(x), ctypes.byref(s))
    return int(x.value), int(s.value)


def read_per_sm_mixed(region_bytes: int, W: int, nsm: int, wps: int, reads: int, seed: int,
                      mix_period: int, group_of_sm=None, windows=None,
                      first_read: int = 0) -> np.ndarray:
    """Per-SM mode where every mix_period-th read of a warp's stream is sequential."""
    out = np.zeros((nsm * wps, 2), dtype=np.uint32)
    g = wb = wn = None
    ng = 0
    if group_of_sm is not None:
        g = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
        w = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
        wb = np.ascontiguousarray(w[:, 0])
        wn = np.ascontiguousarray(w[:, 1])
        ng = w.shape[0]
    rc = _load().orc_read_per_sm_mixed(region_bytes, W, nsm, wps, first_read, reads, seed, _ptr(g),
                                       _ptr(wb), _ptr(wn), ng, mix_period, _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def make_windows(region_bytes: int, W: int, window_bytes: int, n_groups: int, policy: int = 0,
                 seed: int = 0):
    """Windows per group as (n_groups, 2) uint32 {base_line, n_lines}, and the coverage fraction."""
    wb = np.zeros(n_groups, dtype=np.uint32)
    wn = np.zeros(n_groups, dtype=np.uint32)
    cov = ctypes.c_double()
    rc = _load().orc_make_windows(region_bytes, W, window_bytes, n_groups, policy, seed, _ptr(wb),
                                  _ptr(wn), ctypes.byref(cov))
    if rc != 0:
        raise OracleError(rc)
    return np.stack([wb, wn], axis=1), float(cov.value)


def make_weighted_windows(region_bytes: int, W: int, weights, n_warps: int,
                          max_window_bytes: int = 0):
    """Windows and logical-warp ranges in proportion to integer group weights.

    Returns ((G, 2) uint32 {base_line, n_lines}, warp_start uint32[G+1])."""
    w = np.ascontiguousarray(weights, dtype=np.uint32)
    G = int(w.shape[0])
    wb = np.zeros(G, dtype=np.uint32)
    wn = np.zeros(G, dtype=np.uint32)
    ws = np.zeros(G + 1, dtype=np.uint32)
    rc = _load().orc_make_weighted_windows(region_bytes, W, G, _ptr(w), n_warps, max_window_bytes,
                                           _ptr(wb), _ptr(wn), _ptr(ws))
    if rc != 0:
        raise OracleError(rc)
    return np.stack([wb, wn], axis=1), ws


def read_pooled(region_bytes: int, W: int, windows, warp_start, reads: int, seed: int,
                first_read: int = 0) -> np.ndarray:
    """Checksums of logical warps 0..warp_start[-1]-1, each inside its group's window."""
    w = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
    wb = np.ascontiguousarray(w[:, 0])
    wn = np.ascontiguousarray(w[:, 1])
    ws = np.ascontiguousarray(warp_start, dtype=np.uint32)
    if ws.shape != (w.shape[0] + 1,):
        raise OracleError(-1)
    out = np.zeros((int(ws[-1]), 2), dtype=np.uint32)
    rc = _load().orc_read_pooled(region_bytes, W, w.shape[0], _ptr(wb), _ptr(wn), _ptr(ws),
                                 first_read, reads, seed, _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def cluster(T, solo_normalise: bool = False):
    """SM x SM throughput matrix -> (group_of_sm int32[n], n_groups, confidence, heights[n-1]).

    ``solo_normalise`` divides every pair entry by the sum of the two solo rates on the diagonal."""
    T = np.ascontiguousarray(T, dtype=np.float32)
    n = T.shape[0]
    if T.shape != (n, n):
        raise OracleError(-1)
    groups = np.zeros(n, dtype=np.int32)
    heights = np.zeros(max(n - 1, 1), dtype=np.float64)
    ng = ctypes.c_uint32()
    conf = ctypes.c_double()
    rc = _load().orc_cluster(_ptr(T), n, 1 if solo_normalise else 0, _ptr(groups), ctypes.byref(ng), ctypes.byref(conf),
                             _ptr(heights))
    if rc != 0:
        raise OracleError(rc)
    return groups, int(ng.value), float(conf.value), heights[: n - 1]


def reach(size_bytes, gbps):
    """(cliff_exists, plateau GB/s, reach bytes) from an increasing size sweep."""
    s = np.ascontiguousarray(size_bytes, dtype=np.uint64)
    g = np.ascontiguousarray(gbps, dtype=np.float64)
    plateau = ctypes.c_double()
    r = ctypes.c_uint64()
    rc = _load().orc_reach(_ptr(s), _ptr(g), len(s), ctypes.byref(plateau), ctypes.byref(r))
    if rc < 0:
        raise OracleError(rc)
    return bool(rc), float(plateau.value), int(r.value)


def reach_next(size_bytes, gbps, step_bytes: int) -> int:
    """Next size to measure while refining the reach, or 0 when done."""
    s = np.ascontiguousarray(size_bytes, dtype=np.uint64)
    g = np.ascontiguousarray(gbps, dtype=np.float64)
    nxt = ctypes.c_uint64()
    rc = _load().orc_reach_next(_ptr(s), _ptr(g), len(s), step_bytes, ctypes.byref(nxt))
    if rc < 0:
        raise OracleError(rc)
    return int(nxt.value) if rc else 0


def sm_reach(size_bytes, gbps, keep: float = 0.97) -> int:
    s = np.ascontiguousarray(size_bytes, dtype=np.uint64)
    g = np.ascontiguousarray(gbps, dtype=np.float64)
    r = ctypes.c_uint64()
    rc = _load().orc_sm_reach(_ptr(s), _ptr(g), len(s), keep, ctypes.byref(r))
    if rc != 0:
        raise OracleError(rc)
    return int(r.value)


def owner_map(group_of_sm):
    """(owner_of_sm uint16[nsm], n_owners): one window id per active SM, group by group."""
    g = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
    out = np.zeros(g.shape[0], dtype=np.uint16)
    n = ctypes.c_uint32()
    rc = _load().orc_owner_map(_ptr(g), g.shape[0], _ptr(out), ctypes.byref(n))
    if rc != 0:
        raise OracleError(rc)
    return out, int(n.value)


def phase_window(slice_bytes: int, sm_reach_bytes: int, max_parts: int = 64):
    """(parts, sub_bytes) of the moving sub-windows."""
    parts = ctypes.c_uint32()
    sub = ctypes.c_uint64()
    rc = _load().orc_phase_window(slice_bytes, sm_reach_bytes, max_parts, ctypes.byref(parts),
                                  ctypes.byref(sub))
    if rc != 0:
        raise OracleError(rc)
    return int(parts.value), int(sub.value)


def rebalance_weights(work, finish_ns, scale: int = 1_000_000) -> np.ndarray:
    w = np.ascontiguousarray(work, dtype=np.uint32)
    f = np.ascontiguousarray(finish_ns, dtype=np.uint64)
    if w.shape != f.shape:
        raise OracleError(-1)
    out = np.zeros(w.shape[0], dtype=np.uint32)
    rc = _load().orc_rebalance_weights(_ptr(w), _ptr(f), w.shape[0], scale, _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


def group_finish(t_start, t_end, group_of_sm, n_groups: int):
    """(finish_ns uint64[n_groups], span_ns) from the per-SM block timers of one run."""
    a = np.ascontiguousarray(t_start, dtype=np.uint64)
    b = np.ascontiguousarray(t_end, dtype=np.uint64)
    g = np.ascontiguousarray(group_of_sm, dtype=np.uint16)
    out = np.zeros(n_groups, dtype=np.uint64)
    span = ctypes.c_uint64()
    rc = _load().orc_group_finish(_ptr(a), _ptr(b), _ptr(g), g.shape[0], n_groups, _ptr(out),
                                  ctypes.byref(span))
    if rc != 0:
        raise OracleError(rc)
    return out, int(span.value)


def finish_spread_ppm(finish_ns) -> int:
    f = np.ascontiguousarray(finish_ns, dtype=np.uint64)
    ppm = ctypes.c_uint32()
    rc = _load().orc_finish_spread_ppm(_ptr(f), f.shape[0], ctypes.byref(ppm))
    if rc != 0:
        raise OracleError(rc)
    return int(ppm.value)


def window_cover(windows, n_lines: int):
    """(covered lines, smallest depth, largest depth) of a set of windows."""
    w = np.ascontiguousarray(windows, dtype=np.uint32).reshape(-1, 2)
    wb = np.ascontiguousarray(w[:, 0])
    wn = np.ascontiguousarray(w[:, 1])
    cov = ctypes.c_uint64()
    lo = ctypes.c_uint32()
    hi = ctypes.c_uint32()
    rc = _load().orc_window_cover(_ptr(wb), _ptr(wn), w.shape[0], n_lines, ctypes.byref(cov),
                                  ctypes.byref(lo), ctypes.byref(hi))
    if rc != 0:
        raise OracleError(rc)
    return int(cov.value), int(lo.value), int(hi.value)


def probe_rate(t_start, t_end, claim, solo: bool, total_reads: int, extra_lines=(0, 0)):
    """(GB/s, seconds, overlap) of one probe from its timers; OracleError(-6) if an SM never ran."""
    a = np.ascontiguousarray(t_start, dtype=np.uint64)
    b = np.ascontiguousarray(t_end, dtype=np.uint64)
    c = np.ascontiguousarray(claim, dtype=np.uint32)
    x = np.ascontiguousarray(extra_lines, dtype=np.uint64)
    g = ctypes.c_double()
    sec = ctypes.c_double()
    ov = ctypes.c_double()
    rc = _load().orc_probe_rate(_ptr(a), _ptr(b), _ptr(c), _ptr(x), 1 if solo else 0, total_reads,
                                ctypes.byref(g), ctypes.byref(sec), ctypes.byref(ov))
    if rc != 0:
        raise OracleError(rc)
    return float(g.value), float(sec.value), float(ov.value)


def n_threads() -> int:
    """Threads the OpenMP loops will use (host cores available to this process)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))
